"""Pins for oracle/selection.py (Algorithm 2, line 8 + forced diagonal blocks).  CPU only."""
import numpy as np
import pytest

from oracle.selection import select


def scores(n1, n2, seed, ties=False):
    rng = np.random.default_rng(seed)
    S = rng.standard_normal((1, 2, n1, n2))
    if ties:
        S = np.round(S * 2) / 2            # many equal scores
    return S


@pytest.mark.parametrize("seg,blk,k,ties", [(8, 2, 6, False), (8, 2, 6, True), (4, 4, 3, True),
                                            (16, 2, 8, False), (6, 3, 5, True)])
def test_against_full_sort(seg, blk, k, ties):
    n = 96
    n1, n2, r = n // seg, n // blk, seg // blk
    S = scores(n1, n2, 3, ties)
    idx, cnt = select(S, seg, blk, k)
    for h in range(2):
        for j in range(n1):
            past = list(range(j * r))
            diag = list(range(j * r, (j + 1) * r))
            ranked = sorted(past, key=lambda b: (S[0, h, j, b], b), reverse=True)   # ties: larger index first
            want = sorted(ranked[:k - r] + diag)
            got = idx[0, h, j, :cnt[0, h, j]].tolist()
            assert got == want
            assert cnt[0, h, j] == min(k, (j + 1) * r)
            assert (idx[0, h, j, cnt[0, h, j]:] == -1).all()
            assert set(diag) <= set(got) and max(got) < (j + 1) * r


def test_budget_covering_everything_returns_all_visible_blocks():
    seg, blk, n = 8, 4, 64
    n1, n2, r = n // seg, n // blk, seg // blk
    idx, cnt = select(scores(n1, n2, 4), seg, blk, n2)
    for j in range(n1):
        assert idx[0, 0, j, :cnt[0, 0, j]].tolist() == list(range((j + 1) * r))


def test_consistent_permutation_of_past_blocks():
    seg, blk, n, k = 8, 2, 64, 10
    n1, n2, r = n // seg, n // blk, seg // blk
    S = scores(n1, n2, 5)
    j = n1 - 1
    perm = np.random.default_rng(6).permutation(j * r)
    S2 = S.copy()
    S2[0, 0, j, :j * r] = S[0, 0, j, perm]        # new position p holds the score of old block perm[p]
    a, ca = select(S, seg, blk, k)
    b, cb = select(S2, seg, blk, k)
    past_a = {x for x in a[0, 0, j, :ca[0, 0, j]].tolist() if x < j * r}
    past_b = {int(perm[x]) for x in b[0, 0, j, :cb[0, 0, j]].tolist() if x < j * r}
    assert past_a == past_b


def test_future_scores_are_ignored_even_if_huge():
    seg, blk, n, k = 8, 2, 32, 6
    n1, n2, r = n // seg, n // blk, seg // blk
    S = scores(n1, n2, 7)
    S2 = S.copy()
    for j in range(n1):
        S2[0, :, j, (j + 1) * r:] = 1e9
    assert np.array_equal(select(S, seg, blk, k)[0], select(S2, seg, blk, k)[0])


@pytest.mark.parametrize("n,seg,blk,k", [(90, 8, 2, 6), (50, 16, 4, 5), (7, 8, 2, 4)])
def test_short_last_segment(n, seg, blk, k):
    """n not a multiple of the segment: the last segment overlaps fewer than r blocks and its spare
    slots go to past blocks; a budget larger than the number of blocks selects everything."""
    n1, n2, r = -(-n // seg), -(-n // blk), seg // blk
    S = scores(n1, n2, 11, ties=True)
    idx, cnt = select(S, seg, blk, k)
    for h in range(2):
        for j in range(n1):
            past = list(range(j * r))
            diag = list(range(j * r, min(n2, (j + 1) * r)))
            ranked = sorted(past, key=lambda b: (S[0, h, j, b], b), reverse=True)
            want = sorted(ranked[:k - len(diag)] + diag)
            assert idx[0, h, j, :cnt[0, h, j]].tolist() == want
            assert cnt[0, h, j] == min(k, len(past) + len(diag))
