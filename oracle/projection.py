"""Oracle: the query / key / value projections of Eq. 1, rotary position embedding on Q and K, fp64, plain numpy.

TEST INFRASTRUCTURE -- checks the fused projection kernel; not part of the product path.

    Q[b,h,t,:] = rope_t( W_Q[h] X[b,t,:] ),   K[b,h,t,:] = rope_t( W_K[h] X[b,t,:] )        (Eq. 1: Q = W_Q X, K = W_K X)

with W_Q [Hq*d, d_model], W_K [Hkv*d, d_model] (row c of head h is row h*d + c) and X [B, n, d_model].
The rotation is the rotate-half form: channel i < d/2 pairs with channel i + d/2 and the pair is turned by the
angle whose cosine / sine the caller tabulates per token, cos[t,i], sin[t,i]:
    out[i]       = x[i] cos - x[i+d/2] sin,      out[i+d/2] = x[i+d/2] cos + x[i] sin.
The paper does not mention position embeddings; the models it evaluates (Llama3, Yi) apply this rotation to Q and K
right after the projection, which is why the fused kernel carries it.  (cos = 1, sin = 0 gives Eq. 1 as printed.)

V = W_V X is the plain product.
Pins (tests/test_oracle_projection.py): the matrix products against explicit loops; the rotation against complex
multiplication (x[i] + 1j x[i+d/2]) * exp(1j theta), norm preservation, and the identity for theta = 0.
"""
from __future__ import annotations

import numpy as np


def _f64(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().cpu()
        x = x.float().numpy() if x.dtype.is_floating_point and x.element_size() < 4 else x.numpy()
    return np.asarray(x, dtype=np.float64)


def rope(x: np.ndarray, cos: np.ndarray, sin: np.ndarray) -> np.ndarray:
    """x [..., n, d], cos / sin [n, d/2] -> rotated x (rotate-half pairing)."""
    d = x.shape[-1]
    lo, hi = x[..., : d // 2], x[..., d // 2:]
    return np.concatenate([lo * cos - hi * sin, hi * cos + lo * sin], axis=-1)


def project_qk(X, Wq, Wk, head_dim: int, cos=None, sin=None):
    """X [B,n,d_model], Wq [Hq*d, d_model], Wk [Hkv*d, d_model] -> Q [B,Hq,n,d], K [B,Hkv,n,d] in fp64 (not rounded)."""
    X, Wq, Wk = _f64(X), _f64(Wq), _f64(Wk)
    B, n, dm = X.shape
    out = []
    for W in (Wq, Wk):
        H = W.shape[0] // head_dim
        P = np.empty((B, H, n, head_dim), dtype=np.float64)
        for b in range(B):
            for h in range(H):
                P[b, h] = X[b] @ W[h * head_dim:(h + 1) * head_dim].T
        if cos is not None:
            P = rope(P, _f64(cos), _f64(sin))
        out.append(P)
    return out[0], out[1]


def project_v(X, Wv, head_dim: int):
    """V = W_V X of Eq. 1: X [B,n,d_model], Wv [Hkv*d, d_model] -> V [B,Hkv,n,d] in fp64 (not rounded).  Values carry no
    position embedding and Algorithm 1 takes nothing from them, so this is the matrix product alone."""
    X, Wv = _f64(X), _f64(Wv)
    B, n, _ = X.shape
    H = Wv.shape[0] // head_dim
    V = np.empty((B, H, n, head_dim), dtype=np.float64)
    for b in range(B):
        for h in range(H):
            V[b, h] = X[b] @ Wv[h * head_dim:(h + 1) * head_dim].T
    return V


def rope_tables(n: int, head_dim: int, theta: float = 500000.0):
    """cos / sin [n, d/2] in fp32 for angles t * theta^(-2i/d) (the usual rotary schedule; an input generator, the
    method itself takes the tables as given)."""
    inv = theta ** (-np.arange(0, head_dim, 2, dtype=np.float64) / head_dim)
    ang = np.arange(n, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)
