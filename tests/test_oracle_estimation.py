"""Pins for oracle/estimation.py (Algorithm 1).  CPU only."""
import math

import numpy as np
import pytest
from scipy.special import softmax as scipy_softmax

from oracle import estimation as E


def rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def test_summaries_against_token_loop():
    Q, K = rand((1, 2, 12, 3), 0), rand((1, 1, 12, 3), 1)
    Qmax, Qmin, Kmax, Kmin = E.summaries(Q, K, 6, 2)
    for h in range(2):
        for j in range(2):
            for c in range(3):
                vals = [Q[0, h, t, c] for t in range(6 * j, 6 * j + 6)]
                assert Qmax[0, h, j, c] == max(vals) and Qmin[0, h, j, c] == min(vals)
    for b in range(6):
        for c in range(3):
            vals = [K[0, 0, u, c] for u in (2 * b, 2 * b + 1)]
            assert Kmax[0, 0, b, c] == max(vals) and Kmin[0, 0, b, c] == min(vals)
    # unit segments/blocks: the representatives are the tokens themselves
    a, b_, c_, d_ = E.summaries(Q, K, 1, 1)
    assert np.array_equal(a, Q) and np.array_equal(b_, Q) and np.array_equal(c_, K) and np.array_equal(d_, K)
    # bounds
    Kr = K.reshape(1, 1, 6, 2, 3)
    assert (Kr <= Kmax[:, :, :, None]).all() and (Kr >= Kmin[:, :, :, None]).all()


def test_summaries_with_a_short_last_group():
    Q, K = rand((1, 1, 11, 2), 20), rand((1, 1, 11, 2), 21)
    Qmax, Qmin, Kmax, Kmin = E.summaries(Q, K, 4, 2)
    assert Qmax.shape == (1, 1, 3, 2) and Kmax.shape == (1, 1, 6, 2)
    assert Qmax[0, 0, 2, 1] == max(Q[0, 0, t, 1] for t in (8, 9, 10)) and Qmin[0, 0, 2, 0] == min(Q[0, 0, t, 0] for t in (8, 9, 10))
    assert Kmax[0, 0, 5, 0] == K[0, 0, 10, 0] == Kmin[0, 0, 5, 0]


def test_hand_worked_example():
    """n=4, d=2, seg=2, blk=1; summaries and logits below were worked out by hand."""
    Q = np.array([[1, -1], [2, 0], [0, 3], [-1, 1]], dtype=np.float64)[None, None]
    K = np.array([[1, 0], [0, 1], [1, 1], [-1, 2]], dtype=np.float64)[None, None]
    # Qmax = [[2,0],[0,3]]  Qmin = [[1,-1],[-1,1]]; blk=1 so Kmax = Kmin = K
    l_max = [[2, 0, 2, -2], [0, 3, 3, 6]]       # Qmax . K^T
    l_min = [[1, -1, 0, -3], [-1, 1, 0, 3]]     # Qmin . K^T
    sm = lambda row: [math.exp(x) / sum(math.exp(y) for y in row) for x in row]
    expect = np.zeros((2, 4))
    for j in range(2):
        s_qmax, s_qmin = sm(l_max[j]), sm(l_min[j])
        for b in range(4):
            # Kmax = Kmin: S1 = S2 = s_qmax, S3 = S4 = s_qmin -> Smax = Smin = their mean
            expect[j, b] = 0.5 * (s_qmax[b] + s_qmin[b])
    expect[0, 2:] = 0.0                          # blocks 2,3 start at tokens 2,3 >= end of segment 0
    got = np.exp(E.estimate(Q, K, 2, 1))[0, 0]
    np.testing.assert_allclose(got, expect, rtol=1e-13, atol=0)
    # est_scale multiplies the logits
    got2 = np.exp(E.estimate(Q, K, 2, 1, est_scale=0.5))[0, 0]
    sm_h = lambda row: sm([0.5 * x for x in row])
    assert got2[1, 3] == pytest.approx(0.5 * (sm_h(l_max[1])[3] + sm_h(l_min[1])[3]), rel=1e-13)


def test_unit_segments_reduce_to_library_softmax():
    """seg = blk = 1: all four maps coincide and S = softmax(q K^T) per head (Eq. 3 without
    its top-k) -- checked against scipy's softmax, GQA head mapping included."""
    n, d = 9, 5
    Q, K = rand((2, 4, n, d), 2), rand((2, 2, n, d), 3)
    Lg = E.estimate(Q, K, 1, 1, est_scale=0.7)
    for b in range(2):
        for h in range(4):
            ref = scipy_softmax(0.7 * Q[b, h] @ K[b, h // 2].T, axis=-1)
            ref = np.where(np.arange(n)[None, :] >= np.arange(n)[:, None] + 1, 0.0, ref)
            np.testing.assert_allclose(np.exp(Lg[b, h]), ref, rtol=1e-12, atol=0)


def _algorithm1_probability_domain(Q, K, seg, blk, alpha, Sprev, est_scale):
    """Lines 3-14 of Algorithm 1 on probabilities in long double, loops only (one head)."""
    ld = np.longdouble
    n, d = Q.shape
    n1, n2 = -(-n // seg), -(-n // blk)          # a shorter last segment / block when n is not a multiple
    qmax = [[max(Q[t][c] for t in range(j * seg, min(n, (j + 1) * seg))) for c in range(d)] for j in range(n1)]
    qmin = [[min(Q[t][c] for t in range(j * seg, min(n, (j + 1) * seg))) for c in range(d)] for j in range(n1)]
    kmax = [[max(K[u][c] for u in range(b * blk, min(n, (b + 1) * blk))) for c in range(d)] for b in range(n2)]
    kmin = [[min(K[u][c] for u in range(b * blk, min(n, (b + 1) * blk))) for c in range(d)] for b in range(n2)]

    def smap(qr, kr):
        out = np.zeros((n1, n2), dtype=ld)
        for j in range(n1):
            e = [np.exp(ld(est_scale) * sum(ld(qr[j][c]) * ld(kr[b][c]) for c in range(d))) for b in range(n2)]
            z = sum(e)
            for b in range(n2):
                out[j, b] = e[b] / z
        return out

    S1, S2, S3, S4 = smap(qmax, kmax), smap(qmax, kmin), smap(qmin, kmax), smap(qmin, kmin)
    S = np.maximum((S1 + S3) / 2, (S2 + S4) / 2)
    for j in range(n1):
        for b in range(n2):
            if b * blk >= (j + 1) * seg:
                S[j, b] = 0
    if Sprev is not None:
        S = ld(alpha) * S + (1 - ld(alpha)) * Sprev
    return S


@pytest.mark.parametrize("seg,blk,n", [(4, 2, 24), (6, 3, 24), (4, 4, 24), (8, 2, 24), (8, 2, 21), (6, 3, 19)])
def test_log_domain_equals_probability_domain(seg, blk, n):
    d = 4
    Q, K = 0.8 * rand((1, 1, n, d), 4 + seg), 0.8 * rand((1, 1, n, d), 5 + blk)
    S0 = _algorithm1_probability_domain(Q[0, 0], K[0, 0], seg, blk, 1.0, None, 1.0)
    L0 = E.estimate(Q, K, seg, blk)
    np.testing.assert_allclose(np.exp(L0[0, 0]), S0.astype(np.float64), rtol=1e-12, atol=0)
    # second layer, fused with the first layer's scores (line 14), alpha = 0.25
    Q1, K1 = 0.8 * rand((1, 1, n, d), 40), 0.8 * rand((1, 1, n, d), 41)
    S1 = _algorithm1_probability_domain(Q1[0, 0], K1[0, 0], seg, blk, 0.25, S0, 1.0)
    L1 = E.estimate(Q1, K1, seg, blk, alpha=0.25, S_prev=L0)
    np.testing.assert_allclose(np.exp(L1[0, 0]), S1.astype(np.float64), rtol=1e-12, atol=0)
    assert np.array_equal(np.isneginf(L1[0, 0]), E.causal_block_mask(-(-n // seg), -(-n // blk), seg, blk))


def test_score_invariants():
    n, d, seg, blk = 64, 8, 16, 4
    Q, K = rand((1, 2, n, d), 6), rand((1, 1, n, d), 7)
    Lg = E.estimate(Q, K, seg, blk)
    S = np.exp(Lg)
    assert (S >= 0).all() and (S <= 1).all()
    last = S[:, :, -1, :]                       # nothing is masked for the last segment
    assert ((last.sum(-1) >= 1 - 1e-12) & (last.sum(-1) <= 2 + 1e-12)).all()
    # each of the four maps is a distribution over all n2 blocks
    Qmax, Qmin, Kmax, Kmin = E.summaries(Q, K, seg, blk)
    for qr, kr in ((Qmax, Kmax), (Qmax, Kmin), (Qmin, Kmax), (Qmin, Kmin)):
        l = E.logits(qr, kr)
        p = np.exp(l - E._logsumexp(l))
        np.testing.assert_allclose(p.sum(-1), 1.0, rtol=1e-13)
    # a zeroed key block has zero logits in all four maps
    K2 = K.copy()
    K2[0, 0, 3 * blk:4 * blk] = 0.0
    _, _, Kmax2, Kmin2 = E.summaries(Q, K2, seg, blk)
    assert (E.logits(Qmax, Kmax2)[..., 3] == 0).all() and (E.logits(Qmin, Kmin2)[..., 3] == 0).all()
    # a constant query segment makes Qmax = Qmin: S1 = S3 and S2 = S4, so S = max(S1, S2)
    Qc = Q.copy()
    Qc[0, 0, :seg] = Qc[0, 0, 0]
    Lc = E.estimate(Qc, K, seg, blk)[0, 0, 0]
    q = Qc[0, 0, 0]
    s1 = scipy_softmax(Kmax[0, 0] @ q)
    s2 = scipy_softmax(Kmin[0, 0] @ q)
    vis = ~E.causal_block_mask(n // seg, n // blk, seg, blk)[0]
    np.testing.assert_allclose(np.exp(Lc)[vis], np.maximum(s1, s2)[vis], rtol=1e-12)


def test_mask_brute_force():
    for seg, blk, n in [(4, 2, 16), (6, 3, 18), (8, 8, 32), (4, 1, 8)]:
        m = E.causal_block_mask(n // seg, n // blk, seg, blk)
        for j in range(n // seg):
            for b in range(n // blk):
                first_token_of_block, last_token_of_segment = b * blk, (j + 1) * seg - 1
                assert m[j, b] == (first_token_of_block > last_token_of_segment)


def test_fusion_identities():
    n, d, seg, blk = 32, 4, 8, 4
    Q, K = rand((1, 1, n, d), 8), rand((1, 1, n, d), 9)
    L = E.estimate(Q, K, seg, blk)
    other = E.estimate(rand((1, 1, n, d), 10), rand((1, 1, n, d), 11), seg, blk)
    # alpha = 1 is the paper's "w/o fusion" ablation
    assert np.array_equal(E.estimate(Q, K, seg, blk, alpha=1.0, S_prev=other), L)
    # fusing with itself changes nothing
    same = E.estimate(Q, K, seg, blk, alpha=0.25, S_prev=L)
    fin = np.isfinite(L)
    np.testing.assert_allclose(same[fin], L[fin], rtol=0, atol=1e-14)
    assert np.array_equal(np.isneginf(same), np.isneginf(L))
    # linear in the probability domain, weight alpha on the current layer
    fused = E.estimate(Q, K, seg, blk, alpha=0.25, S_prev=other)
    np.testing.assert_allclose(np.exp(fused), 0.25 * np.exp(L) + 0.75 * np.exp(other), rtol=1e-13)


def test_mask_before_softmax_variant():
    n, d, seg, blk = 32, 4, 8, 4
    Q, K = rand((1, 1, n, d), 12), rand((1, 1, n, d), 13)
    Qmax, Qmin, Kmax, Kmin = E.summaries(Q, K, seg, blk)
    L = E.estimate(Q, K, seg, blk, mask_before_softmax=True)[0, 0]
    for j in range(n // seg):
        vis = (j + 1) * (seg // blk)
        maps = [scipy_softmax(kr[0, 0, :vis] @ qr[0, 0, j]) for qr, kr in
                ((Qmax, Kmax), (Qmax, Kmin), (Qmin, Kmax), (Qmin, Kmin))]
        ref = np.maximum((maps[0] + maps[2]) / 2, (maps[1] + maps[3]) / 2)
        np.testing.assert_allclose(np.exp(L[j, :vis]), ref, rtol=1e-12)
        assert np.isneginf(L[j, vis:]).all()


def test_paper_operating_point_fixture():
    import os
    from paper_2409_12490_b200 import CONFIGS
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_parameters.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                vals[k] = float(v)
    c = CONFIGS["paper_128k"]
    assert (c.segment_size, c.block_size, c.budget_tokens, c.alpha) == (
        vals["segment_size"], vals["block_size"], vals["budget_tokens"], vals["alpha"])


def test_decode_estimate_is_algorithm_1_on_a_one_token_segment():
    """The decoding-phase score of the last token: (i) equals Algorithm 1 run with one-token segments (its last row,
    which sees every block), (ii) equals max(softmax(q Kmax^T), softmax(q Kmin^T)) written out with loops."""
    import oracle
    rng = np.random.default_rng(12)
    B, Hq, Hkv, n, d, blk = 2, 4, 2, 48, 8, 4
    Q = rng.standard_normal((B, Hq, n, d))
    K = rng.standard_normal((B, Hkv, n, d))
    got = oracle.decode_estimate(Q[:, :, -1], K, blk, est_scale=0.7)
    # (i) segment_size = 1 is not a multiple of the block size, so compare through the summaries: row n-1 of the
    # four maps with Qmax = Qmin = Q[n-1]
    Qmax, Qmin, Kmax, Kmin = oracle.summaries(Q, K, 1, blk)
    assert np.array_equal(Qmax[:, :, -1], Q[:, :, -1]) and np.array_equal(Qmin[:, :, -1], Q[:, :, -1])
    # (ii) loops
    n2 = n // blk
    for b in range(B):
        for h in range(Hq):
            q = Q[b, h, -1]
            kv = h // (Hq // Hkv)
            lmax = np.array([0.7 * sum(q[c] * Kmax[b, kv, x, c] for c in range(d)) for x in range(n2)])
            lmin = np.array([0.7 * sum(q[c] * Kmin[b, kv, x, c] for c in range(d)) for x in range(n2)])
            smax = np.exp(lmax - lmax.max()); smax /= smax.sum()
            smin = np.exp(lmin - lmin.max()); smin /= smin.sum()
            want = np.maximum(smax, smin)                     # (S1+S3)/2 = S1 and (S2+S4)/2 = S2 when Qmax = Qmin
            assert np.allclose(np.exp(got[b, h]), want, rtol=1e-12, atol=0)
    assert np.all(np.exp(got) <= 1.0 + 1e-12)
    # block_size = 1: the last row of Algorithm 1 run token by token (segment = block = 1 sees every key at row n-1)
    full = oracle.estimate(Q, K, 1, 1, est_scale=0.7)
    assert np.allclose(oracle.decode_estimate(Q[:, :, -1], K, 1, est_scale=0.7), full[:, :, -1, :], rtol=0, atol=1e-12)


def test_decode_select_against_full_sort():
    import oracle
    rng = np.random.default_rng(13)
    S = np.round(rng.standard_normal((2, 3, 40)) * 2) / 2      # ties
    for k in (1, 5, 39, 40, 64):
        idx, cnt = oracle.decode_select(S, k)
        for b in range(2):
            for h in range(3):
                past = list(range(39))
                ranked = sorted(past, key=lambda x: (S[b, h, x], x), reverse=True)
                want = sorted(ranked[:k - 1] + [39])
                assert idx[b, h, :cnt[b, h]].tolist() == want and (idx[b, h, cnt[b, h]:] == -1).all()
