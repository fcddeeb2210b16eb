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
"""
from __future__ import annotations

import numpy as np


def select(S: np.ndarray, segment_size: int, block_size: int, budget_blocks: int):
    """S: ln-scores [B,Hq,n1,n2] -> (idx int32 [B,Hq,n1,k], cnt int32 [B,Hq,n1])."""
    S = np.asarray(S, dtype=np.float64)
    B, H, n1, n2 = S.shape
    r = segment_size // block_size
    k = budget_blocks
    assert segment_size % block_size == 0 and r <= k
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
                    row = S[b, h, j, :past]
                    # descending by (score, index): stable ascending argsort of the reversed row
                    order = np.argsort(-row[::-1], kind="stable")
                    chosen = sorted(int(past - 1 - o) for o in order[:m])
                sel = chosen + diag
                cnt[b, h, j] = len(sel)
                idx[b, h, j, :len(sel)] = sel
    return idx, cnt
