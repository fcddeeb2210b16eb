"""Batches of sequences of different lengths, packed one after another along the token axis (fp64 CPU oracle).

TEST INFRASTRUCTURE ONLY (see the package docstring).

The paper describes one sequence (Algorithms 1 and 2 partition "the" sequence of n tokens).  Reading taken here for a
packed batch: every sequence is a problem of its own -- its segments and blocks are counted from ITS first token, its
score map is [n1_i, n2_i] with n1_i = ceil(len_i / segment_size), n2_i = ceil(len_i / block_size), its lists hold block
indices relative to its first token, and no query ever sees a key of another sequence.  So the definition is a loop over
the sequences that calls the single-sequence functions of this package on slices; nothing else is computed here.

Pins (tests/test_oracle_varlen.py): equal lengths reproduce the batched functions on the reshaped tensors; a sequence's
results do not move when the other sequences' tokens are replaced; a one-sequence batch is the plain call; the slices
are checked against explicit token loops over `cu_seqlens`.
"""
from __future__ import annotations

import numpy as np

from .attention import sparse_attention
from .estimation import estimate
from .selection import select


def _np(x) -> np.ndarray:
    return x.detach().cpu().float().numpy() if hasattr(x, "detach") else np.asarray(x)


def sequence_bounds(cu_seqlens) -> list[tuple[int, int]]:
    """[(first token, one past the last token)] of every sequence; cu_seqlens = [0, len_0, len_0+len_1, ...]."""
    cu = [int(c) for c in cu_seqlens]
    if len(cu) < 2 or cu[0] != 0 or any(b <= a for a, b in zip(cu, cu[1:])):
        raise ValueError("cu_seqlens must start at 0 and increase strictly")
    return list(zip(cu[:-1], cu[1:]))


def prefill_varlen(Q, K, V, cu_seqlens, segment_size: int, block_size: int, budget_blocks: int, sm_scale: float, *,
                   est_scale: float = 1.0, alpha: float = 0.25, S_prev=None):
    """One layer of the hot path (Algorithm 1, Algorithm 2) for every sequence of a packed batch.

    Q [Hq, total, d], K and V [Hkv, total, d]; S_prev: None or the list of ln S this function returned for the previous
    layer.  Returns (S, idx, cnt, O, lse): S, idx, cnt are lists with one entry per sequence ([Hq,n1_i,n2_i] fp64,
    [Hq,n1_i,k] int32, [Hq,n1_i] int32), O is [Hq, total, d] fp64; lse [Hq, total] is returned as a fifth value.
    """
    Q, K, V = (_np(t) for t in (Q, K, V))
    total = Q.shape[1]
    bounds = sequence_bounds(cu_seqlens)
    if bounds[-1][1] != total:
        raise ValueError("cu_seqlens does not cover the packed tensors")
    S_all, idx_all, cnt_all = [], [], []
    O = np.zeros(Q.shape, dtype=np.float64)
    lse = np.zeros(Q.shape[:2], dtype=np.float64)
    for i, (lo, hi) in enumerate(bounds):
        q, k, v = Q[None, :, lo:hi], K[None, :, lo:hi], V[None, :, lo:hi]
        prev = None if S_prev is None else np.asarray(S_prev[i])[None]
        S = estimate(q, k, segment_size, block_size, est_scale=est_scale, alpha=alpha, S_prev=prev)
        idx, cnt = select(S, segment_size, block_size, budget_blocks)
        o, l = sparse_attention(q, k, v, idx, cnt, segment_size, block_size, sm_scale)
        O[:, lo:hi], lse[:, lo:hi] = o[0], l[0]
        S_all.append(S[0]); idx_all.append(idx[0]); cnt_all.append(cnt[0])
    return S_all, idx_all, cnt_all, O, lse
