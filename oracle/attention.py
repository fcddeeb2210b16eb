"""Oracle: block-restricted and dense causal attention rows (Algorithm 2; Eq. 2), fp64.

TEST INFRASTRUCTURE -- loads the plain-C row routine in attention_oracle.c (built with gcc by
oracle/build.py) through ctypes.  Not part of the product path.

Pins (tests/test_oracle_attention.py): dense rows against torch's fp64
scaled_dot_product_attention(is_causal=True) and against an explicit numpy masked softmax;
a budget that covers every block reproduces dense attention; sparse rows against a numpy
mask-matrix brute force built from the block list; exp(lse) row normalisation; constant V;
causality; GQA = MHA with replicated KV heads; a single-block list in closed form.

Readings: softmax runs over the selected keys only (Algorithm 2, line 10, as written), with
token-level causality u <= t applied inside the selected blocks (the paper's decoder setting).
The arithmetic is pinned (tests above); the causal reading inside Algorithm 2 is parity unpinned against
the authors' code.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import sys

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


def _lib():
    global _LIB
    if _LIB is None:
        path = os.path.join(_HERE, "liboracle_attention.so")
        src = os.path.join(_HERE, "attention_oracle.c")
        if not os.path.exists(path) or os.path.getmtime(path) < os.path.getmtime(src):
            subprocess.check_call([sys.executable, os.path.join(_HERE, "build.py")])
        _LIB = ctypes.CDLL(path)
        _LIB.oracle_attention_rows.restype = ctypes.c_int
    return _LIB


def _f32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().cpu().float().numpy()
    x = np.asarray(x)
    assert x.dtype in (np.float32, np.float64)
    y = np.ascontiguousarray(x, dtype=np.float32)
    assert x.dtype == np.float32 or np.array_equal(y.astype(np.float64), x), "inputs must be fp32-representable"
    return y


def _rows(Q, K, V, idx, cnt, seg, blk, k, sm_scale, rows):
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    B, Hq, n, d = Q.shape
    Hkv = K.shape[1]
    rows = np.ascontiguousarray(rows, dtype=np.int64).reshape(-1, 3)
    O = np.empty((rows.shape[0], d), dtype=np.float64)
    lse = np.empty((rows.shape[0],), dtype=np.float64)
    P = ctypes.c_void_p
    if idx is not None:
        idx = np.ascontiguousarray(idx, dtype=np.int32)
        cnt = np.ascontiguousarray(cnt, dtype=np.int32)
        assert idx.shape == (B, Hq, -(-n // seg), k) and cnt.shape == (B, Hq, -(-n // seg))
    err = _lib().oracle_attention_rows(
        P(Q.ctypes.data), P(K.ctypes.data), P(V.ctypes.data),
        P(idx.ctypes.data) if idx is not None else P(0), P(cnt.ctypes.data) if idx is not None else P(0),
        ctypes.c_int(B), ctypes.c_int(Hq), ctypes.c_int(Hkv), ctypes.c_int64(n), ctypes.c_int(d),
        ctypes.c_int(seg), ctypes.c_int(blk), ctypes.c_int(k), ctypes.c_double(sm_scale),
        P(rows.ctypes.data), ctypes.c_int64(rows.shape[0]), P(O.ctypes.data), P(lse.ctypes.data))
    if err:
        raise ValueError("block list holds an index outside [0, n2)")
    return O, lse


def _all_rows(B, H, n):
    b, h, t = np.meshgrid(np.arange(B), np.arange(H), np.arange(n), indexing="ij")
    return np.stack([b.ravel(), h.ravel(), t.ravel()], axis=1)


def sparse_attention_rows(Q, K, V, idx, cnt, segment_size, block_size, sm_scale, rows):
    """Rows (b, h, t) of Algorithm 2's output -> (O [n_rows,d], lse [n_rows]) fp64."""
    return _rows(Q, K, V, idx, cnt, segment_size, block_size, idx.shape[-1], sm_scale, rows)


def dense_attention_rows(Q, K, V, sm_scale, rows):
    """Rows (b, h, t) of causal Eq. 2 -> (O [n_rows,d], lse [n_rows]) fp64."""
    return _rows(Q, K, V, None, None, 1, 1, 0, sm_scale, rows)


def sparse_attention(Q, K, V, idx, cnt, segment_size, block_size, sm_scale):
    """Algorithm 2 for every row -> (O [B,Hq,n,d], lse [B,Hq,n]) fp64."""
    B, Hq, n, d = Q.shape
    O, lse = sparse_attention_rows(Q, K, V, idx, cnt, segment_size, block_size, sm_scale, _all_rows(B, Hq, n))
    return O.reshape(B, Hq, n, d), lse.reshape(B, Hq, n)


def dense_attention(Q, K, V, sm_scale):
    """Causal Eq. 2 for every row -> (O [B,Hq,n,d], lse [B,Hq,n]) fp64."""
    B, Hq, n, d = Q.shape
    O, lse = dense_attention_rows(Q, K, V, sm_scale, _all_rows(B, Hq, n))
    return O.reshape(B, Hq, n, d), lse.reshape(B, Hq, n)
