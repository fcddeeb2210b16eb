"""Pins for oracle/selection.py (Algorithm 2, line 8 + forced diagonal blocks).  CPU only."""
import numpy as np
import pytest

from oracle.selection import pool_group_scores, select


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


def test_group_pooling_is_the_elementwise_maximum_and_group_one_changes_nothing():
    rng = np.random.default_rng(8)
    S = rng.standard_normal((2, 6, 5, 20))
    S[:, :, :, 15:] = -np.inf
    P = pool_group_scores(S, 3)
    for b in range(2):
        for h in range(6):
            for j in range(5):
                for x in range(20):
                    kv = h // 3
                    assert P[b, h, j, x] == max(S[b, kv * 3 + u, j, x] for u in range(3))
    assert np.array_equal(pool_group_scores(S, 1), S)
    seg, blk, k = 8, 2, 6
    S = scores(12, 48, 9)
    a = select(S, seg, blk, k)
    b = select(S, seg, blk, k, group=1)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


@pytest.mark.parametrize("ties", [False, True])
def test_shared_group_lists_against_brute_force(ties):
    seg, blk, k, n, g = 8, 2, 7, 96, 2
    n1, n2, r = n // seg, n // blk, seg // blk
    rng = np.random.default_rng(10)
    S = rng.standard_normal((1, 4, n1, n2))
    if ties:
        S = np.round(S * 2) / 2
    idx, cnt = select(S, seg, blk, k, group=g)
    for kv in range(2):
        for j in range(n1):
            past = list(range(j * r))
            pooled = {x: max(S[0, kv * g + u, j, x] for u in range(g)) for x in past}
            ranked = sorted(past, key=lambda x: (pooled[x], x), reverse=True)
            want = sorted(ranked[:k - r] + list(range(j * r, (j + 1) * r)))
            for u in range(g):                                   # every head of the group gets the same list
                assert idx[0, kv * g + u, j, :cnt[0, kv * g + u, j]].tolist() == want


@pytest.mark.parametrize("n_sink,n_local,ties", [(1, 0, False), (0, 2, False), (2, 1, True), (1, 1, True)])
def test_forced_sink_and_local_blocks_against_brute_force(n_sink, n_local, ties):
    seg, blk, k, n = 8, 2, 9, 128
    n1, n2, r = n // seg, n // blk, seg // blk
    S = scores(n1, n2, 11, ties)
    idx, cnt = select(S, seg, blk, k, n_sink=n_sink, n_local=n_local)
    plain = select(S, seg, blk, k)
    for h in range(2):
        for j in range(n1):
            past = list(range(j * r))
            forced = [x for x in past if x < n_sink or x >= j * r - n_local]
            free = [x for x in past if x not in forced]
            ranked = sorted(free, key=lambda x: (S[0, h, j, x], x), reverse=True)
            m = k - r
            want = sorted(past) if len(past) <= m else sorted(forced + ranked[:m - len(forced)])
            want = want + list(range(j * r, (j + 1) * r))
            got = idx[0, h, j, :cnt[0, h, j]].tolist()
            assert got == want and set(forced) <= set(got)
            assert cnt[0, h, j] == plain[1][0, h, j]            # forced blocks count against the same budget
    z = select(S, seg, blk, k, n_sink=0, n_local=0)
    assert np.array_equal(z[0], plain[0])
