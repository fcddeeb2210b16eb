"""Pins for oracle/attention.py (Algorithm 2, lines 6-13; Eq. 2).  CPU only."""
import numpy as np
import pytest
import torch

from oracle import attention as A
from oracle.selection import select


def rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


def qkv(B=1, Hq=4, Hkv=2, n=48, d=8, seed=0):
    return rand((B, Hq, n, d), seed), rand((B, Hkv, n, d), seed + 1), rand((B, Hkv, n, d), seed + 2)


def numpy_masked_attention(Q, K, V, allowed, scale):
    """Explicit n x n masked softmax for one head (allowed[t,u] boolean)."""
    s = (Q.astype(np.float64) @ K.astype(np.float64).T) * scale
    s = np.where(allowed, s, -np.inf)
    p = np.exp(s - s.max(-1, keepdims=True))
    z = p.sum(-1, keepdims=True)
    return (p / z) @ V.astype(np.float64), (np.log(z) + s.max(-1, keepdims=True))[:, 0]


def test_dense_equals_library_sdpa():
    Q, K, V = qkv()
    O, lse = A.dense_attention(Q, K, V, 0.3)
    tq, tk, tv = (torch.from_numpy(x).double() for x in (Q, K, V))
    ref = torch.nn.functional.scaled_dot_product_attention(
        tq, tk.repeat_interleave(2, dim=1), tv.repeat_interleave(2, dim=1), is_causal=True, scale=0.3)
    np.testing.assert_allclose(O, ref.numpy(), rtol=1e-12, atol=1e-14)
    # and the normaliser against the explicit matrix form
    n = Q.shape[2]
    causal = np.tril(np.ones((n, n), dtype=bool))
    for h in range(4):
        o2, l2 = numpy_masked_attention(Q[0, h], K[0, h // 2], V[0, h // 2], causal, 0.3)
        np.testing.assert_allclose(O[0, h], o2, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(lse[0, h], l2, rtol=1e-12)


def test_full_budget_equals_dense():
    seg, blk = 16, 4
    Q, K, V = qkv(n=64)
    n2 = 64 // blk
    S = np.random.default_rng(5).standard_normal((1, 4, 64 // seg, n2))
    idx, cnt = select(S, seg, blk, n2)
    Os, ls = A.sparse_attention(Q, K, V, idx, cnt, seg, blk, 0.35)
    Od, ld = A.dense_attention(Q, K, V, 0.35)
    np.testing.assert_allclose(Os, Od, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(ls, ld, rtol=1e-13)


@pytest.mark.parametrize("seg,blk,k,n", [(16, 4, 6, 96), (8, 8, 2, 96), (12, 3, 5, 96), (16, 4, 6, 90), (12, 3, 5, 67)])
def test_sparse_against_mask_matrix_brute_force(seg, blk, k, n):
    Q, K, V = qkv(n=n, seed=3)
    n1, n2 = -(-n // seg), -(-n // blk)
    S = np.random.default_rng(9).standard_normal((1, 4, n1, n2))
    idx, cnt = select(S, seg, blk, k)
    O, lse = A.sparse_attention(Q, K, V, idx, cnt, seg, blk, 0.4)
    for h in range(4):
        allowed = np.zeros((n, n), dtype=bool)
        for t in range(n):
            j = t // seg
            for b in idx[0, h, j, :cnt[0, h, j]]:
                for u in range(b * blk, min(n, (b + 1) * blk)):
                    allowed[t, u] = u <= t
        o2, l2 = numpy_masked_attention(Q[0, h], K[0, h // 2], V[0, h // 2], allowed, 0.4)
        np.testing.assert_allclose(O[0, h], o2, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(lse[0, h], l2, rtol=1e-12)


def test_constant_v_and_row_normalisation():
    seg, blk, k, n = 16, 4, 5, 64
    Q, K, V = qkv(n=n, seed=6)
    V[:] = 1.5
    S = np.random.default_rng(1).standard_normal((1, 4, n // seg, n // blk))
    idx, cnt = select(S, seg, blk, k)
    O, lse = A.sparse_attention(Q, K, V, idx, cnt, seg, blk, 0.5)
    np.testing.assert_allclose(O, 1.5, rtol=1e-13)
    # exp(score - lse) over the row's key set sums to one
    t, h = 37, 3
    j = t // seg
    keys = [u for b in idx[0, h, j, :cnt[0, h, j]] for u in range(b * blk, (b + 1) * blk) if u <= t]
    s = 0.5 * (K[0, h // 2, keys].astype(np.float64) @ Q[0, h, t].astype(np.float64))
    assert np.exp(s - lse[0, h, t]).sum() == pytest.approx(1.0, rel=1e-12)


def test_causality_with_fixed_list():
    seg, blk, k, n = 16, 4, 6, 64
    Q, K, V = qkv(n=n, seed=7)
    S = np.random.default_rng(2).standard_normal((1, 4, n // seg, n // blk))
    idx, cnt = select(S, seg, blk, k)
    t = 41
    O1, _ = A.sparse_attention(Q, K, V, idx, cnt, seg, blk, 0.5)
    Q2, K2, V2 = Q.copy(), K.copy(), V.copy()
    Q2[:, :, t + 1:] += 3.0
    K2[:, :, t + 1:] -= 2.0
    V2[:, :, t + 1:] *= -1.0
    O2, _ = A.sparse_attention(Q2, K2, V2, idx, cnt, seg, blk, 0.5)
    assert np.array_equal(O1[:, :, :t + 1], O2[:, :, :t + 1])


def test_gqa_equals_mha_with_replicated_kv():
    seg, blk, k, n = 16, 4, 6, 64
    Q, K, V = qkv(n=n, seed=8)
    S = np.random.default_rng(3).standard_normal((1, 4, n // seg, n // blk))
    idx, cnt = select(S, seg, blk, k)
    O1, l1 = A.sparse_attention(Q, K, V, idx, cnt, seg, blk, 0.5)
    O2, l2 = A.sparse_attention(Q, np.repeat(K, 2, axis=1), np.repeat(V, 2, axis=1), idx, cnt, seg, blk, 0.5)
    assert np.array_equal(O1, O2) and np.array_equal(l1, l2)


def test_single_block_closed_form():
    seg = blk = 8
    n = 32
    Q, K, V = qkv(Hq=1, Hkv=1, n=n, seed=9)
    idx = np.array([[j] for j in range(n // seg)], dtype=np.int32)[None, None]
    cnt = np.ones((1, 1, n // seg), dtype=np.int32)
    O, _ = A.sparse_attention(Q, K, V, idx, cnt, seg, blk, 1.0)
    # the first token of each segment sees exactly one key: O = that key's value
    for j in range(n // seg):
        np.testing.assert_allclose(O[0, 0, j * seg], V[0, 0, j * seg].astype(np.float64), rtol=1e-15)
    # the second token sees two keys: a logistic weight
    t = 17
    q, k0, k1 = (x.astype(np.float64) for x in (Q[0, 0, t], K[0, 0, 16], K[0, 0, 17]))
    w1 = 1.0 / (1.0 + np.exp(q @ k0 - q @ k1))
    np.testing.assert_allclose(O[0, 0, t], (1 - w1) * V[0, 0, 16] + w1 * V[0, 0, 17], rtol=1e-12)


def test_rows_interface_matches_full():
    seg, blk, k, n = 16, 4, 6, 64
    Q, K, V = qkv(n=n, seed=10)
    S = np.random.default_rng(4).standard_normal((1, 4, n // seg, n // blk))
    idx, cnt = select(S, seg, blk, k)
    O, lse = A.sparse_attention(Q, K, V, idx, cnt, seg, blk, 0.5)
    rows = np.array([[0, 3, 63], [0, 0, 0], [0, 2, 17]])
    o, l = A.sparse_attention_rows(Q, K, V, idx, cnt, seg, blk, 0.5, rows)
    for i, (b, h, t) in enumerate(rows):
        assert np.array_equal(o[i], O[b, h, t]) and l[i] == lse[b, h, t]
    od, _ = A.dense_attention_rows(Q, K, V, 0.5, rows)
    Od, _ = A.dense_attention(Q, K, V, 0.5)
    assert np.array_equal(od[2], Od[0, 2, 17])
