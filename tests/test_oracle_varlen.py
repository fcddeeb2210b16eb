"""Pins for oracle/varlen.py: a packed batch of sequences of different lengths is a set of independent
single-sequence problems (Algorithms 1 and 2 per sequence).  CPU only."""
import numpy as np
import pytest

from oracle import estimate, prefill_varlen, select, sequence_bounds, sparse_attention

SEG, BLK, K, D = 8, 2, 6, 8
SM = 1.0 / np.sqrt(D)


def packed(lens, seed, hq=4, hkv=2):
    rng = np.random.default_rng(seed)
    total = sum(lens)
    mk = lambda h: rng.standard_normal((h, total, D)).astype(np.float32)
    return mk(hq), mk(hkv), mk(hkv), np.concatenate([[0], np.cumsum(lens)])


def test_bounds_follow_the_prefix_sums():
    assert sequence_bounds([0, 5, 7, 20]) == [(0, 5), (5, 7), (7, 20)]
    for bad in ([1, 5], [0, 5, 5], [0], [0, 7, 3]):
        with pytest.raises(ValueError):
            sequence_bounds(bad)


def test_equal_lengths_reproduce_the_batched_functions():
    lens = [24, 24, 24]
    Q, Kt, V, cu = packed(lens, 0)
    S, idx, cnt, O, lse = prefill_varlen(Q, Kt, V, cu, SEG, BLK, K, SM)
    # the same tokens as a [B, H, n, d] batch
    Qb = Q.reshape(4, 3, 24, D).transpose(1, 0, 2, 3)
    Kb = Kt.reshape(2, 3, 24, D).transpose(1, 0, 2, 3)
    Vb = V.reshape(2, 3, 24, D).transpose(1, 0, 2, 3)
    Sb = estimate(Qb, Kb, SEG, BLK)
    ib, cb = select(Sb, SEG, BLK, K)
    Ob, lb = sparse_attention(Qb, Kb, Vb, ib, cb, SEG, BLK, SM)
    for i in range(3):
        np.testing.assert_array_equal(S[i], Sb[i])
        np.testing.assert_array_equal(idx[i], ib[i])
        np.testing.assert_array_equal(cnt[i], cb[i])
        np.testing.assert_array_equal(O[:, 24 * i:24 * (i + 1)], Ob[i])
        np.testing.assert_array_equal(lse[:, 24 * i:24 * (i + 1)], lb[i])


def test_a_sequence_does_not_see_its_neighbours():
    lens = [19, 40, 7, 33]            # ragged last segments and blocks
    Q, Kt, V, cu = packed(lens, 1)
    ref = prefill_varlen(Q, Kt, V, cu, SEG, BLK, K, SM)
    Q2, K2, V2 = Q.copy(), Kt.copy(), V.copy()
    rng = np.random.default_rng(9)
    lo, hi = int(cu[1]), int(cu[2])     # keep sequence 1, replace everything else
    for t in (Q2, K2, V2):
        keep = t[:, lo:hi].copy()
        t[...] = (rng.standard_normal(t.shape) * 3).astype(np.float32)
        t[:, lo:hi] = keep
    out = prefill_varlen(Q2, K2, V2, cu, SEG, BLK, K, SM)
    np.testing.assert_array_equal(out[0][1], ref[0][1])
    np.testing.assert_array_equal(out[1][1], ref[1][1])
    np.testing.assert_array_equal(out[3][:, lo:hi], ref[3][:, lo:hi])
    assert not np.array_equal(out[3][:, :lo], ref[3][:, :lo])


def test_shapes_and_single_sequence_and_explicit_rows():
    lens = [19, 40, 7]
    Q, Kt, V, cu = packed(lens, 2)
    S, idx, cnt, O, lse = prefill_varlen(Q, Kt, V, cu, SEG, BLK, K, SM)
    for i, n in enumerate(lens):
        n1, n2 = -(-n // SEG), -(-n // BLK)
        assert S[i].shape == (4, n1, n2) and idx[i].shape == (4, n1, K) and cnt[i].shape == (4, n1)
        assert idx[i].max() < n2            # block indices are relative to the sequence's first token
    # a one-sequence batch is the plain call
    one = prefill_varlen(Q[:, :19], Kt[:, :19], V[:, :19], [0, 19], SEG, BLK, K, SM)
    np.testing.assert_array_equal(one[3], O[:, :19])
    # rows of the second sequence from their definition: softmax over the listed blocks' keys up to the row, keys
    # taken at packed position first_token + block*BLK + offset
    first = int(cu[1])
    g = 2
    for h, t in ((0, 0), (1, 17), (3, 39), (2, 24)):
        j = t // SEG
        blocks = idx[1][h, j, :cnt[1][h, j]]
        keys = [b * BLK + o for b in blocks for o in range(BLK) if b * BLK + o <= t and b * BLK + o < 40]
        kk = Kt[h // g, [first + u for u in keys]]
        vv = V[h // g, [first + u for u in keys]]
        w = np.exp(SM * kk @ Q[h, first + t] - np.max(SM * kk @ Q[h, first + t]))
        np.testing.assert_allclose(O[h, first + t], (w / w.sum()) @ vv, rtol=1e-12, atol=1e-12)


def test_layer_fusion_uses_each_sequences_own_previous_scores():
    lens = [16, 24]
    Q, Kt, V, cu = packed(lens, 3)
    Q1, K1, V1, _ = packed(lens, 4)
    S0 = prefill_varlen(Q, Kt, V, cu, SEG, BLK, K, SM)[0]
    S1 = prefill_varlen(Q1, K1, V1, cu, SEG, BLK, K, SM, alpha=0.25, S_prev=S0)[0]
    for i, (lo, hi) in enumerate(sequence_bounds(cu)):
        want = estimate(Q1[None, :, lo:hi], K1[None, :, lo:hi], SEG, BLK, alpha=0.25, S_prev=S0[i][None])[0]
        np.testing.assert_array_equal(S1[i], want)
