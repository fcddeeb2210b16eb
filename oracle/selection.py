"""Oracle: per-segment critical block selection (Algorithm 2, line 8), plain numpy / Python.

TEST INFRASTRUCTURE -- not part of the product path.

Pins (tests/test_oracle_selection.py): full-sort brute force on small inputs; budget >=
visible blocks returns every visible block; the diagonal blocks are always present and no
future block ever is; cnt = min(k, (j+1)*r); consistent permutation of the past scores.

Readings: the r = seg/blk blocks that overlap the segment are always selected and count
against the budget of k = B/blk blocks; the other k - r slots go to the strictly past
blocks with the largest score, ties to the larger block index; segments that see fewer
than k blocks take all of them (cnt < k, list padded with -1); lists are ascending.  With a
sequence length that is not a multiple of the segment size the last segment overlaps fewer than r
blocks and the slots it does not need go to past blocks.
The selection itself is pinned (tests above); which reading the authors' code takes is parity unpinned.

Variants the paper's text does not fix (readings of this build, each pinned against brute force and against the
plain selection as their special case):
  * shared lists per KV group (``group``): the g query heads that share a KV head use ONE list per segment, taken
    from the element-wise maximum of their scores (the maximum of the probabilities S, i.e. of ln S) -- a block
    that is critical for any head of the group is kept for all of them;
  * forced sink / local blocks (``n_sink``, ``n_local``): the first n_sink blocks of the sequence and the n_local
    blocks right before the segment are always kept, like the diagonal blocks, and count against the budget;
    n_sink + n_local <= k - r is required, so they always fit.
"""
from __future__ import annotations

import numpy as np


def pool_group_scores(S: np.ndarray, group: int) -> np.ndarray:
    """Element-wise maximum of ln S over the `group` consecutive query heads that share a KV head, written back to
    every head of the group: [B,Hq,n1,n2] -> [B,Hq,n1,n2]."""
    S = np.asarray(S, dtype=np.float64)
    B, H, n1, n2 = S.shape
    assert H % group == 0
    out = np.empty_like(S)
    for b in range(B):
        for kv in range(H // group):
            pooled = S[b, kv * group]
            for h in range(kv * group + 1, (kv + 1) * group):
                pooled = np.maximum(pooled, S[b, h])
            for h in range(kv * group, (kv + 1) * group):
                out[b, h] = pooled
    return out


def select(S: np.ndarray, segment_size: int, block_size: int, budget_blocks: int, *, group: int = 1,
           n_sink: int = 0, n_local: int = 0):
    """S: ln-scores [B,Hq,n1,n2] -> (idx int32 [B,Hq,n1,k], cnt int32 [B,Hq,n1]).
    group > 1: one list per KV group (see the module text); n_sink / n_local: forced past blocks."""
    S = np.asarray(S, dtype=np.float64)
    if group > 1:
        S = pool_group_scores(S, group)
    B, H, n1, n2 = S.shape
    r = segment_size // block_size
    k = budget_blocks
    assert segment_size % block_size == 0 and r <= k
    assert n_sink >= 0 and n_local >= 0 and n_sink + n_local <= k - r
    idx = np.full((B, H, n1, k), -1, dtype=np.int32)
    cnt = np.zeros((B, H, n1), dtype=np.int32)
    for b in range(B):
        for h in range(H):
            for j in range(n1):
                past = j * r                               # blocks strictly before the segment
                diag = list(range(j * r, min(n2, (j + 1) * r)))   # blocks overlapping the segment (fewer in a short last one)
                m = k - len(diag)
                if past <= m:
                    chosen = list(range(past))
                else:
                    row = S[b, h, j, :past].copy()
                    forced = [x for x in range(past) if x < n_sink or x >= past - n_local]
                    row[forced] = np.inf                   # forced blocks come before every scored block
                    # descending by (score, index): stable ascending argsort of the reversed row
                    order = np.argsort(-row[::-1], kind="stable")
                    chosen = sorted(int(past - 1 - o) for o in order[:m])
                sel = chosen + diag
                cnt[b, h, j] = len(sel)
                idx[b, h, j, :len(sel)] = sel
    return idx, cnt


def decode_select(S: np.ndarray, budget_blocks: int):
    """Critical blocks of the last query token: S ln-scores [B,Hq,n2] -> (idx int32 [B,Hq,k] ascending, -1 padded;
    cnt int32 [B,Hq]).  The block that holds the token itself (the last one) is always kept and counts against the
    budget; the other k-1 slots go to the blocks with the largest score, ties to the larger index."""
    S = np.asarray(S, dtype=np.float64)
    B, H, n2 = S.shape
    k = budget_blocks
    idx = np.full((B, H, k), -1, dtype=np.int32)
    cnt = np.zeros((B, H), dtype=np.int32)
    for b in range(B):
        for h in range(H):
            past = n2 - 1
            if past <= k - 1:
                chosen = list(range(past))
            else:
                order = np.argsort(-S[b, h, :past][::-1], kind="stable")
                chosen = sorted(int(past - 1 - o) for o in order[:k - 1])
            sel = chosen + [n2 - 1]
            cnt[b, h] = len(sel)
            idx[b, h, :len(sel)] = sel
    return idx, cnt
