"""Oracle: segment-wise criticality estimation (Algorithm 1), fp64, plain numpy.

TEST INFRASTRUCTURE -- a slow, literal restatement of Algorithm 1 used to check the CUDA
kernels.  Not part of the product path.

Pins (tests/test_oracle_estimation.py): bit-exact summaries against an explicit token
loop; row sums of the four softmax maps; agreement of the log-domain result with the
probability-domain formulas of Algorithm 1 (lines 9-14) evaluated in long double on
small inputs; the segment = block = 1 special case (a plain library softmax of q K^T,
i.e. Eq. 3 without the top-k); alpha = 1 and S' = S identities of the fusion step;
brute-force mask.

Readings of the paper taken here (the paper prints no worked example, so the choice
among them is "parity unpinned" with respect to the authors' implementation):
  * scores are kept as natural logarithms ln S in fp64 (the probabilities of Algorithm 1
    underflow at 128K tokens; ordering and the fusion are unchanged);
  * the estimation logits carry no 1/sqrt(d) unless est_scale says so (Algorithm 1,
    lines 9-10, as written);
  * softmax over all n2 blocks first, causal mask afterwards (lines 9-13 in order);
    ``mask_before_softmax`` gives the other order;
  * a block is masked iff it starts at or after the end of the segment;
  * every query head has its own score map, using the key summaries of its KV group;
  * S' = None means no fusion; the fused S is what the next layer receives;
  * a sequence length that is not a multiple of the segment / block size leaves a shorter last
    segment / block (n1 = ceil(n/seg), n2 = ceil(n/blk)); the paper writes the divisions as exact.
"""
from __future__ import annotations

import numpy as np

LN2 = float(np.log(2.0))


def _f64(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().cpu()
        x = x.float().numpy() if x.dtype.is_floating_point and x.element_size() < 4 else x.numpy()
    return np.asarray(x, dtype=np.float64)


def summaries(Q, K, segment_size: int, block_size: int):
    """Algorithm 1, lines 3-8: element-wise max / min over the tokens of each query
    segment and of each key block.  Q [B,Hq,n,d], K [B,Hkv,n,d] ->
    Qmax,Qmin [B,Hq,n1,d]; Kmax,Kmin [B,Hkv,n2,d]."""
    Q = _f64(Q)
    K = _f64(K)
    B, Hq, n, d = Q.shape
    Hkv = K.shape[1]
    def grouped(X, size):
        """max / min over consecutive groups of `size` tokens; the last group may be shorter."""
        groups = -(-n // size)
        mx = np.stack([X[:, :, i * size:(i + 1) * size].max(axis=2) for i in range(groups)], axis=2)
        mn = np.stack([X[:, :, i * size:(i + 1) * size].min(axis=2) for i in range(groups)], axis=2)
        return mx, mn

    Qmax, Qmin = grouped(Q, segment_size)
    Kmax, Kmin = grouped(K, block_size)
    return Qmax, Qmin, Kmax, Kmin


def logits(Qrep: np.ndarray, Krep: np.ndarray, est_scale: float = 1.0) -> np.ndarray:
    """Algorithm 1, lines 9-10 (argument of the softmax): whole-vector dot products of a
    query representative with every key representative of its KV group.
    Qrep [B,Hq,n1,d], Krep [B,Hkv,n2,d] -> [B,Hq,n1,n2]."""
    B, Hq, n1, d = Qrep.shape
    Hkv = Krep.shape[1]
    g = Hq // Hkv
    out = np.empty((B, Hq, n1, Krep.shape[2]), dtype=np.float64)
    for b in range(B):
        for h in range(Hq):
            out[b, h] = est_scale * (Qrep[b, h] @ Krep[b, h // g].T)
    return out


def _logsumexp(x: np.ndarray, axis: int = -1) -> np.ndarray:
    m = np.max(x, axis=axis, keepdims=True)
    m = np.where(np.isfinite(m), m, 0.0)
    with np.errstate(divide="ignore"):
        return m + np.log(np.sum(np.exp(x - m), axis=axis, keepdims=True))


def _logaddexp(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    with np.errstate(invalid="ignore"):
        return np.logaddexp(a, b)  # (-inf, -inf) -> -inf


def causal_block_mask(n1: int, n2: int, segment_size: int, block_size: int) -> np.ndarray:
    """True where block b lies entirely in the future of segment j (Algorithm 1, line 13):
    its first token b*blk is not before the segment's end (j+1)*seg."""
    j = np.arange(n1)[:, None]
    b = np.arange(n2)[None, :]
    return b * block_size >= (j + 1) * segment_size


def estimate(Q, K, segment_size: int, block_size: int, *, est_scale: float = 1.0,
             alpha: float = 0.25, S_prev: np.ndarray | None = None,
             mask_before_softmax: bool = False) -> np.ndarray:
    """Algorithm 1 in full.  Returns ln S, shape [B,Hq,n1,n2], fp64; masked entries -inf.

    ``S_prev`` is the ln S returned for the previous layer (None: first layer, no fusion).
    """
    Qmax, Qmin, Kmax, Kmin = summaries(Q, K, segment_size, block_size)          # lines 3-8
    n1, n2 = Qmax.shape[2], Kmax.shape[2]
    masked = causal_block_mask(n1, n2, segment_size, block_size)
    L = []
    for qrep, krep in ((Qmax, Kmax), (Qmax, Kmin), (Qmin, Kmax), (Qmin, Kmin)):   # S1..S4, lines 9-10
        l = logits(qrep, krep, est_scale)
        if mask_before_softmax:
            l = np.where(masked, -np.inf, l)
        L.append(l - _logsumexp(l, axis=-1))                                     # ln softmax over blocks
    Lmax = _logaddexp(L[0], L[2]) - LN2                                          # line 11: (S1+S3)/2
    Lmin = _logaddexp(L[1], L[3]) - LN2                                          #          (S2+S4)/2
    Lg = np.maximum(Lmax, Lmin)                                                  # line 12
    Lg = np.where(masked, -np.inf, Lg)                                           # line 13
    if S_prev is not None:                                                       # line 14
        Lprev = np.asarray(S_prev, dtype=np.float64)
        with np.errstate(divide="ignore"):                                       # alpha = 0 or 1: one weight is ln 0 = -inf
            ln_a, ln_1ma = np.log(np.float64(alpha)), np.log1p(-np.float64(alpha))
        Lg = _logaddexp(ln_a + Lg, ln_1ma + Lprev)                               # ln(a*S + (1-a)*S')
    return Lg


def decode_estimate(q_last, K, block_size: int, *, est_scale: float = 1.0) -> np.ndarray:
    """Criticality of every key block for the LAST query token (the decoding-phase use of query criticality that
    Section 2.1 describes: the query of the last token against the cached keys).  Algorithm 1 with the one-token
    segment {q}: Qmax = Qmin = q, no block lies in the token's future, no previous layer.
    q_last [B,Hq,d], K [B,Hkv,n,d] -> ln S [B,Hq,n2] fp64.

    Reading (the paper gives no formula for the decoding phase): the segment-wise estimator applied to a segment of
    one token.  Pins (tests/test_oracle_estimation.py): with block_size = 1 it is the last row of `estimate` run with
    segment_size = block_size = 1 (Algorithm 1 itself); for any block size, max(softmax(q Kmax^T), softmax(q Kmin^T))
    written out with loops."""
    q = _f64(q_last)
    K = _f64(K)
    B, Hq, d = q.shape
    n = K.shape[2]
    _, _, Kmax, Kmin = summaries(np.zeros((B, Hq, n, d)), K, n, block_size)      # key-block summaries (lines 5-8)
    qrep = q[:, :, None, :]                                                      # the segment's two representatives coincide
    L = []
    for krep in (Kmax, Kmin, Kmax, Kmin):                                        # S1..S4 with Qmax = Qmin
        l = logits(qrep, krep, est_scale)
        L.append(l - _logsumexp(l, axis=-1))
    Lmax = _logaddexp(L[0], L[2]) - LN2
    Lmin = _logaddexp(L[1], L[3]) - LN2
    return np.maximum(Lmax, Lmin)[:, :, 0, :]
