"""Thin ctypes binding of the C ABI declared in include/critiprefill.h.

Argument marshalling only: every step of the path runs in the CUDA library.  PyTorch is
used for device memory and streams.  There is no CPU fallback: if the library cannot be
loaded, or a call returns a non-zero status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import math
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcritiprefill.so")

CP_OK = 0
CP_ERR_NULL, CP_ERR_SHAPE = 1, 2
CP_BF16, CP_F32, CP_F16 = 0, 1, 2
FLAG_MASK_BEFORE_SOFTMAX = 1
FLAG_FORCE_SIMT = 2
FLAG_TEST_WITHHOLD_V = 4
FLAG_SHARED_GROUP_LISTS = 8
FLAG_FORCE_SPLIT_SCORE = 16
FLAG_SUMMARIES_READY = 32

EXPORTS = (
    "critiprefill_workspace_bytes", "critiprefill_estimate", "critiprefill_select",
    "critiprefill_attention", "critiprefill_dense_attention", "critiprefill_device_status",
    "critiprefill_estimate_static", "critiprefill_static_scratch_bytes",
    "critiprefill_decode_estimate", "critiprefill_decode_select", "critiprefill_project_qk",
    "critiprefill_prefill_varlen", "critiprefill_varlen_sizes", "critiprefill_project_qkv",
    "critiprefill_status_string",
)


class CpParams(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("seq_len", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("segment_size", ctypes.c_int32), ("block_size", ctypes.c_int32), ("budget_blocks", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("flags", ctypes.c_int32),
        ("q_stride", ctypes.c_int64 * 3), ("k_stride", ctypes.c_int64 * 3),
        ("v_stride", ctypes.c_int64 * 3), ("o_stride", ctypes.c_int64 * 3),
        ("est_scale", ctypes.c_float), ("sm_scale", ctypes.c_float), ("alpha", ctypes.c_float),
        ("forced_blocks", ctypes.c_int32),
    ]


class CritiPrefillError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


_lib = None


def load_library() -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2409_12490_b200.build` "
                              "(or __graft_entry__.build()) first; there is no CPU fallback")
        lib = ctypes.CDLL(LIB_PATH)
        P, SZ = ctypes.c_void_p, ctypes.c_size_t
        PP = ctypes.POINTER(CpParams)
        lib.critiprefill_workspace_bytes.argtypes = [PP, ctypes.POINTER(SZ)]
        lib.critiprefill_estimate.argtypes = [PP, P, P, P, P, P, SZ, P]
        lib.critiprefill_select.argtypes = [PP, P, P, P, P, SZ, P]
        lib.critiprefill_attention.argtypes = [PP, P, P, P, P, P, P, P, P, SZ, P]
        lib.critiprefill_dense_attention.argtypes = [PP, P, P, P, P, P, P, SZ, P]
        lib.critiprefill_device_status.argtypes = [P, ctypes.POINTER(ctypes.c_int32), P]
        lib.critiprefill_estimate_static.argtypes = [PP, P, P, P, P, P]
        lib.critiprefill_decode_estimate.argtypes = [PP, P, P, P, P, SZ, P]
        lib.critiprefill_decode_select.argtypes = [PP, P, P, P, P, SZ, P]
        lib.critiprefill_project_qk.argtypes = [PP, P, P, P, P, P, ctypes.c_int32, P, P, P, SZ, P]
        lib.critiprefill_project_qkv.argtypes = [PP, P, P, P, P, P, P, ctypes.c_int32, P, P, P, P, SZ, P]
        lib.critiprefill_prefill_varlen.argtypes = [PP, P, ctypes.c_int32, P, P, P, P, P, P, P, P, P, P, SZ, P]
        I64P = ctypes.POINTER(ctypes.c_int64)
        lib.critiprefill_varlen_sizes.argtypes = [PP, P, ctypes.c_int32, I64P, I64P, I64P]
        lib.critiprefill_static_scratch_bytes.argtypes = []
        lib.critiprefill_status_string.argtypes = [ctypes.c_int]
        lib.critiprefill_status_string.restype = ctypes.c_char_p
        for name in EXPORTS[:-1]:
            getattr(lib, name).restype = ctypes.c_int
        lib.critiprefill_static_scratch_bytes.restype = ctypes.c_size_t
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load_library().critiprefill_status_string(int(status)).decode()


def _check(rc: int, where: str):
    if rc != CP_OK:
        raise CritiPrefillError(rc, where)


def _strides(t: torch.Tensor):
    assert t.dim() == 4 and t.stride(3) == 1, "tensors are [batch, heads, tokens, head_dim] with head_dim contiguous"
    return (ctypes.c_int64 * 3)(t.stride(0), t.stride(1), t.stride(2))


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t) -> ctypes.c_void_p:
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


@dataclass
class Problem:
    """Sizes and hyper-parameters of one layer; builds cp_params for given tensors."""
    batch: int
    n_q_heads: int
    n_kv_heads: int
    seq_len: int
    head_dim: int
    segment_size: int
    block_size: int
    budget_blocks: int
    dtype: torch.dtype = torch.bfloat16
    est_scale: float = 1.0
    sm_scale: float | None = None
    alpha: float = 0.25
    flags: int = 0
    n_sink: int = 0      # always-kept first blocks of the sequence (variant; counts against the budget)
    n_local: int = 0     # always-kept blocks right before each segment (variant; counts against the budget)

    @classmethod
    def from_config(cls, cfg, **kw) -> "Problem":
        return cls(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq_len, cfg.head_dim, cfg.segment_size,
                   cfg.block_size, cfg.budget_blocks,
                   {"bf16": torch.bfloat16, "f32": torch.float32, "f16": torch.float16}[cfg.dtype],
                   est_scale=cfg.est_scale, alpha=cfg.alpha, **kw)

    @property
    def n1(self):
        return -(-self.seq_len // self.segment_size)

    @property
    def n2(self):
        return -(-self.seq_len // self.block_size)

    def _contig(self, heads):
        n, d = self.seq_len, self.head_dim
        return (ctypes.c_int64 * 3)(heads * n * d, n * d, d)

    def params(self, Q=None, K=None, V=None, O=None) -> CpParams:
        p = CpParams()
        p.batch, p.n_q_heads, p.n_kv_heads = self.batch, self.n_q_heads, self.n_kv_heads
        p.seq_len, p.head_dim = self.seq_len, self.head_dim
        p.segment_size, p.block_size, p.budget_blocks = self.segment_size, self.block_size, self.budget_blocks
        p.dtype = {torch.bfloat16: CP_BF16, torch.float32: CP_F32, torch.float16: CP_F16}[self.dtype]
        p.flags = self.flags
        p.q_stride = _strides(Q) if Q is not None else self._contig(self.n_q_heads)
        p.k_stride = _strides(K) if K is not None else self._contig(self.n_kv_heads)
        p.v_stride = _strides(V) if V is not None else self._contig(self.n_kv_heads)
        p.o_stride = _strides(O) if O is not None else self._contig(self.n_q_heads)
        p.est_scale = self.est_scale
        p.sm_scale = self.sm_scale if self.sm_scale is not None else 1.0 / math.sqrt(self.head_dim)
        p.alpha = self.alpha
        p.forced_blocks = self.n_sink | (self.n_local << 16)
        return p


def workspace_bytes(prob: Problem) -> int:
    out = ctypes.c_size_t(0)
    p = prob.params()
    _check(load_library().critiprefill_workspace_bytes(ctypes.byref(p), ctypes.byref(out)), "critiprefill_workspace_bytes")
    return int(out.value)


def alloc_workspace(prob: Problem, device="cuda") -> torch.Tensor:
    """Zeroed scratch buffer (its head is the device status block)."""
    return torch.zeros(workspace_bytes(prob), dtype=torch.uint8, device=device)


def estimate(prob: Problem, Q, K, ws, S_prev=None, S_out=None) -> torch.Tensor:
    """critiprefill_estimate: ln S [B,Hq,n1,n2] fp64 (Algorithm 1)."""
    if S_out is None:
        S_out = torch.empty((prob.batch, prob.n_q_heads, prob.n1, prob.n2), dtype=torch.float64, device=Q.device)
    p = prob.params(Q=Q, K=K)
    _check(load_library().critiprefill_estimate(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(S_prev), _ptr(S_out),
                                                _ptr(ws), ws.numel(), _stream()), "critiprefill_estimate")
    return S_out


def estimate_static(prob: Problem, Q, K, S_prev=None, S_out=None) -> torch.Tensor:
    """critiprefill_estimate_static: critiprefill_estimate without a caller workspace, for callers
    that cannot allocate device memory (the scratch is a fixed array inside the library)."""
    if S_out is None:
        S_out = torch.empty((prob.batch, prob.n_q_heads, prob.n1, prob.n2), dtype=torch.float64, device=Q.device)
    p = prob.params(Q=Q, K=K)
    _check(load_library().critiprefill_estimate_static(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(S_prev), _ptr(S_out),
                                                       _stream()), "critiprefill_estimate_static")
    return S_out


def static_scratch_bytes() -> int:
    return int(load_library().critiprefill_static_scratch_bytes())


def select(prob: Problem, S, ws, idx=None, cnt=None):
    """critiprefill_select: (idx [B,Hq,n1,k] int32, cnt [B,Hq,n1] int32) (Algorithm 2, line 8)."""
    if idx is None:
        idx = torch.empty((prob.batch, prob.n_q_heads, prob.n1, prob.budget_blocks), dtype=torch.int32, device=S.device)
    if cnt is None:
        cnt = torch.empty((prob.batch, prob.n_q_heads, prob.n1), dtype=torch.int32, device=S.device)
    p = prob.params()
    _check(load_library().critiprefill_select(ctypes.byref(p), _ptr(S), _ptr(idx), _ptr(cnt), _ptr(ws), ws.numel(),
                                              _stream()), "critiprefill_select")
    return idx, cnt


def project_qk(prob: Problem, X, Wq, Wk, ws, rope_cos=None, rope_sin=None, Q_out=None, K_out=None):
    """critiprefill_project_qk: Q = W_Q X, K = W_K X (Eq. 1) with rotary embedding; also leaves the representatives of
    Algorithm 1 in `ws` (follow with estimate(..., flags |= FLAG_SUMMARIES_READY)).  Returns (Q [B,Hq,n,d], K [B,Hkv,n,d])."""
    B, n, d_model = X.shape
    assert X.is_contiguous() and Wq.is_contiguous() and Wk.is_contiguous()
    if Q_out is None:
        Q_out = torch.empty((B, prob.n_q_heads, n, prob.head_dim), dtype=X.dtype, device=X.device)
    if K_out is None:
        K_out = torch.empty((B, prob.n_kv_heads, n, prob.head_dim), dtype=X.dtype, device=X.device)
    p = prob.params(Q=Q_out, K=K_out)
    _check(load_library().critiprefill_project_qk(ctypes.byref(p), _ptr(X), _ptr(Wq), _ptr(Wk), _ptr(rope_cos), _ptr(rope_sin),
                                                  int(d_model), _ptr(Q_out), _ptr(K_out), _ptr(ws), ws.numel(), _stream()),
           "critiprefill_project_qk")
    return Q_out, K_out


def project_qkv(prob: Problem, X, Wq, Wk, Wv, ws, rope_cos=None, rope_sin=None, Q_out=None, K_out=None, V_out=None):
    """critiprefill_project_qkv: project_qk plus V = W_V X (no rotation) in the same launch.  Returns (Q, K, V)."""
    B, n, d_model = X.shape
    assert X.is_contiguous() and Wq.is_contiguous() and Wk.is_contiguous() and Wv.is_contiguous()
    mk = lambda h: torch.empty((B, h, n, prob.head_dim), dtype=X.dtype, device=X.device)
    Q_out = mk(prob.n_q_heads) if Q_out is None else Q_out
    K_out = mk(prob.n_kv_heads) if K_out is None else K_out
    V_out = mk(prob.n_kv_heads) if V_out is None else V_out
    p = prob.params(Q=Q_out, K=K_out, V=V_out)
    _check(load_library().critiprefill_project_qkv(ctypes.byref(p), _ptr(X), _ptr(Wq), _ptr(Wk), _ptr(Wv), _ptr(rope_cos),
                                                   _ptr(rope_sin), int(d_model), _ptr(Q_out), _ptr(K_out), _ptr(V_out), _ptr(ws),
                                                   ws.numel(), _stream()),
           "critiprefill_project_qkv")
    return Q_out, K_out, V_out


def decode_estimate(prob: Problem, q_last, K, ws, S_out=None) -> torch.Tensor:
    """critiprefill_decode_estimate: ln S [B,Hq,n2] fp64 of the last query token (Section 2.1)."""
    assert q_last.is_contiguous() and q_last.shape == (prob.batch, prob.n_q_heads, prob.head_dim)
    if S_out is None:
        S_out = torch.empty((prob.batch, prob.n_q_heads, prob.n2), dtype=torch.float64, device=K.device)
    p = prob.params(K=K)
    _check(load_library().critiprefill_decode_estimate(ctypes.byref(p), _ptr(q_last), _ptr(K), _ptr(S_out), _ptr(ws),
                                                       ws.numel(), _stream()), "critiprefill_decode_estimate")
    return S_out


def decode_select(prob: Problem, S, ws):
    """critiprefill_decode_select: (idx [B,Hq,k] int32, cnt [B,Hq] int32) for the last query token."""
    idx = torch.empty((prob.batch, prob.n_q_heads, prob.budget_blocks), dtype=torch.int32, device=S.device)
    cnt = torch.empty((prob.batch, prob.n_q_heads), dtype=torch.int32, device=S.device)
    p = prob.params()
    _check(load_library().critiprefill_decode_select(ctypes.byref(p), _ptr(S), _ptr(idx), _ptr(cnt), _ptr(ws), ws.numel(),
                                                     _stream()), "critiprefill_decode_select")
    return idx, cnt


def attention(prob: Problem, Q, K, V, idx, cnt, ws, O=None, lse=None, want_lse=False):
    """critiprefill_attention: O (and optionally lse) over the listed blocks (Algorithm 2)."""
    if O is None:
        O = torch.empty_like(Q)
    if lse is None and want_lse:
        lse = torch.empty((prob.batch, prob.n_q_heads, prob.seq_len), dtype=torch.float32, device=Q.device)
    p = prob.params(Q=Q, K=K, V=V, O=O)
    _check(load_library().critiprefill_attention(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(idx), _ptr(cnt),
                                                 _ptr(O), _ptr(lse), _ptr(ws), ws.numel(), _stream()),
           "critiprefill_attention")
    return (O, lse) if want_lse else O


def dense_attention(prob: Problem, Q, K, V, ws, O=None, lse=None, want_lse=False):
    """critiprefill_dense_attention: causal Eq. 2."""
    if O is None:
        O = torch.empty_like(Q)
    if lse is None and want_lse:
        lse = torch.empty((prob.batch, prob.n_q_heads, prob.seq_len), dtype=torch.float32, device=Q.device)
    p = prob.params(Q=Q, K=K, V=V, O=O)
    _check(load_library().critiprefill_dense_attention(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(lse),
                                                       _ptr(ws), ws.numel(), _stream()), "critiprefill_dense_attention")
    return (O, lse) if want_lse else O


def device_status(ws) -> int:
    """critiprefill_device_status: synchronises the current stream, returns the device status word."""
    out = ctypes.c_int32(0)
    _check(load_library().critiprefill_device_status(_ptr(ws), ctypes.byref(out), _stream()), "critiprefill_device_status")
    return int(out.value)


def _packed_strides(t: torch.Tensor):
    """Strides of a packed [heads, total_tokens, d] view as (batch: unused, head, token)."""
    assert t.dim() == 3 and t.stride(2) == 1
    return (ctypes.c_int64 * 3)(0, t.stride(0), t.stride(1))


def prefill_varlen(prob: Problem, cu_seqlens, Q, K, V, ws, S_prev=None, want_lse=False):
    """critiprefill_prefill_varlen: one layer for every sequence of a packed batch.

    Q [Hq, total, d], K and V [Hkv, total, d] (any head / token strides, e.g. views of [total, H, d] storage);
    cu_seqlens: host integers 0, len_0, len_0 + len_1, ...; prob.batch = 1 and prob.seq_len = the longest sequence.
    Returns (O, S, idx, cnt, S_flat[, lse]): O like Q; S, idx, cnt are lists of per-sequence views ([Hq,n1_i,n2_i]
    fp64, [Hq,n1_i,k] int32, [Hq,n1_i] int32) of the packed arrays the call fills; S_flat is the packed score array
    itself, which is what the next layer's call takes as S_prev; lse is [Hq * total] fp32, sequence i's [Hq, len_i]
    part starting at Hq * cu_seqlens[i]."""
    lib = load_library()
    cu = (ctypes.c_int32 * len(cu_seqlens))(*[int(c) for c in cu_seqlens])
    n_seqs = len(cu_seqlens) - 1
    p = prob.params()
    p.q_stride, p.k_stride, p.v_stride = _packed_strides(Q), _packed_strides(K), _packed_strides(V)
    O = torch.empty_like(Q)
    p.o_stride = _packed_strides(O)
    sizes = [ctypes.c_int64(0) for _ in range(3)]
    _check(lib.critiprefill_varlen_sizes(ctypes.byref(p), cu, n_seqs, *[ctypes.byref(s) for s in sizes]),
           "critiprefill_varlen_sizes")
    S_flat = torch.empty(sizes[0].value, dtype=torch.float64, device=Q.device)
    idx_flat = torch.empty(sizes[1].value, dtype=torch.int32, device=Q.device)
    cnt_flat = torch.empty(sizes[2].value, dtype=torch.int32, device=Q.device)
    lse = torch.empty((prob.n_q_heads * Q.shape[1],), dtype=torch.float32, device=Q.device) if want_lse else None
    _check(lib.critiprefill_prefill_varlen(ctypes.byref(p), cu, n_seqs, _ptr(Q), _ptr(K), _ptr(V), _ptr(S_prev), _ptr(S_flat),
                                           _ptr(idx_flat), _ptr(cnt_flat), _ptr(O), _ptr(lse), _ptr(ws), ws.numel(), _stream()),
           "critiprefill_prefill_varlen")
    S, idx, cnt = [], [], []
    so = io = co = 0
    H, k = prob.n_q_heads, prob.budget_blocks
    for a, b in zip(cu_seqlens[:-1], cu_seqlens[1:]):
        n = int(b) - int(a)
        n1, n2 = -(-n // prob.segment_size), -(-n // prob.block_size)
        S.append(S_flat[so:so + H * n1 * n2].view(H, n1, n2)); so += H * n1 * n2
        idx.append(idx_flat[io:io + H * n1 * k].view(H, n1, k)); io += H * n1 * k
        cnt.append(cnt_flat[co:co + H * n1].view(H, n1)); co += H * n1
    out = (O, S, idx, cnt, S_flat)
    return out + (lse,) if want_lse else out


def prefill_layer(prob: Problem, Q, K, V, ws, S_prev=None):
    """One layer of the hot path: estimate -> select -> attention.  Returns (O, S, idx, cnt)."""
    S = estimate(prob, Q, K, ws, S_prev=S_prev)
    idx, cnt = select(prob, S, ws)
    O = attention(prob, Q, K, V, idx, cnt, ws)
    return O, S, idx, cnt
