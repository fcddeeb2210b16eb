"""Seeded random shapes through the whole path (estimate -> select -> attention, C ABI) against the fp64 oracle:
dtype, head_dim, batch, GQA group, ragged length, segment / block size, budget, layer fusion, the score-path and
list-sharing flags all drawn at random.  Small problems, many of them."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_12490_b200 import binding as cp
from paper_2409_12490_b200.inputs import make_uniform_qkv

from helpers import compare_scores, compare_selection, f32

pytestmark = pytest.mark.gpu


def draw(seed):
    rng = np.random.default_rng(seed)
    c = {"dtype": str(rng.choice(["bf16", "bf16", "f16", "f32"])), "d": int(rng.choice([128, 128, 128, 64])),
         "blk": int(rng.choice([16, 32, 64, 128]))}
    r = int(rng.choice([1, 2, 4, 8]))
    r = min(r, 1024 // c["blk"])
    c["seg"], c["r"] = c["blk"] * r, r
    c["n"] = int(rng.integers(1, 2600))
    c["Hkv"], c["g"], c["B"] = int(rng.choice([1, 2, 3])), int(rng.choice([1, 2, 4])), int(rng.choice([1, 1, 2]))
    c["k"] = r + int(rng.integers(0, 24))
    c["fuse"] = bool(rng.integers(0, 2))
    flags = 0
    if rng.integers(0, 4) == 0:
        flags |= cp.FLAG_MASK_BEFORE_SOFTMAX
    if c["dtype"] != "f32" and c["d"] == 128 and rng.integers(0, 2) == 0:
        flags |= cp.FLAG_FORCE_SPLIT_SCORE
    c["shared"] = bool(rng.integers(0, 5) == 0)
    if c["shared"]:
        flags |= cp.FLAG_SHARED_GROUP_LISTS
    c["flags"] = flags
    return c


@pytest.mark.parametrize("seed", range(48))
def test_random_shape_matches_oracle(seed):
    c = draw(seed)
    dtype, d, B, n, seg, blk, k, r, g = c["dtype"], c["d"], c["B"], c["n"], c["seg"], c["blk"], c["k"], c["r"], c["g"]
    Hq, Hkv = c["Hkv"] * g, c["Hkv"]
    tdt = {"bf16": torch.bfloat16, "f16": torch.float16, "f32": torch.float32}[dtype]
    Q, K, V = make_uniform_qkv(B, Hq, Hkv, n, d, dtype=dtype, seed=seed)
    prob = cp.Problem(B, Hq, Hkv, n, d, seg, blk, k, tdt, alpha=0.25, flags=c["flags"])
    ws = cp.alloc_workspace(prob)
    mb = bool(c["flags"] & cp.FLAG_MASK_BEFORE_SOFTMAX)
    S_prev = S_prev_ref = None
    if c["fuse"]:
        Q0, K0, _ = make_uniform_qkv(B, Hq, Hkv, n, d, dtype=dtype, seed=seed + 1000)
        S_prev = cp.estimate(prob, Q0.cuda(), K0.cuda(), ws)
        S_prev_ref = oracle.estimate(Q0, K0, seg, blk, est_scale=1.0, mask_before_softmax=mb)
    O, S, idx, cnt = cp.prefill_layer(prob, Q.cuda(), K.cuda(), V.cuda(), ws, S_prev=S_prev)
    assert cp.device_status(ws) == 0, c
    S_ref = oracle.estimate(Q, K, seg, blk, est_scale=1.0, alpha=f32(0.25), S_prev=S_prev_ref, mask_before_softmax=mb)
    compare_scores(S, S_ref)                                                       # ln S within 1e-9
    idx_ref, cnt_ref = oracle.select(S_ref, seg, blk, k, group=g if c["shared"] else 1)
    S_sel = oracle.pool_group_scores(S_ref, g) if c["shared"] else S_ref
    assert compare_selection(idx, cnt, idx_ref, cnt_ref, S_sel, r)[1] == 0, c
    O_ref, _ = oracle.sparse_attention(Q, K, V, idx.cpu().numpy(), cnt.cpu().numpy(), seg, blk, f32(1.0 / np.sqrt(d)))
    err = np.abs(O.float().cpu().numpy().astype(np.float64) - O_ref)
    # 16-bit outputs: the stated absolute bound on unit-scale values, relative beyond |O| = 2 (output spacing)
    tol = {"f32": 1e-5, "f16": 2e-3, "bf16": 1e-2}[dtype]
    assert (err / np.maximum(1.0, np.abs(O_ref) / 2)).max() <= tol, (c, float(err.max()))


@pytest.mark.parametrize("seed", range(24))
def test_random_valid_lists_and_dense(seed):
    """critiprefill_attention on lists it did not get from critiprefill_select (Algorithm 2 takes any index set): empty
    lists, any visible blocks, a lone diagonal block, the usual form with fewer past blocks, every other diagonal block --
    drawn per (head, segment); and critiprefill_dense_attention on the same inputs."""
    rng = np.random.default_rng(10_000 + seed)
    dtype = str(rng.choice(["bf16", "bf16", "f16", "f32"]))
    d, blk = int(rng.choice([128, 128, 128, 64])), int(rng.choice([16, 32, 64, 128]))
    r = min(int(rng.choice([1, 2, 4, 8])), 1024 // blk)
    seg, n = blk * r, int(rng.integers(1, 2600))
    Hkv, g, B = int(rng.choice([1, 2])), int(rng.choice([1, 2, 4])), int(rng.choice([1, 2]))
    Hq, k = Hkv * g, r + int(rng.integers(0, 20))
    flags = cp.FLAG_FORCE_SIMT if rng.integers(0, 6) == 0 else 0
    n1, n2 = -(-n // seg), -(-n // blk)
    idx = np.full((B, Hq, n1, k), -1, dtype=np.int32)
    cnt = np.zeros((B, Hq, n1), dtype=np.int32)
    for b in range(B):
        for h in range(Hq):
            for j in range(n1):
                vis = min(n2, (j + 1) * r)
                rj = vis - j * r
                mode = int(rng.integers(0, 6))
                if mode == 0:
                    sel = []
                elif mode == 1:
                    sel = sorted(rng.choice(vis, size=min(k, vis, 1 + int(rng.integers(k))), replace=False).tolist())
                elif mode == 2:
                    sel = [j * r + int(rng.integers(rj))]
                elif mode in (3, 4):
                    m = min(k - rj, j * r)
                    past = sorted(rng.choice(j * r, size=int(rng.integers(0, m + 1)), replace=False).tolist()) if j and m > 0 else []
                    sel = past + list(range(j * r, vis))
                else:
                    sel = sorted(set(range(j * r, vis, 2)) | ({0} if j else set()))[:k]
                cnt[b, h, j] = len(sel)
                idx[b, h, j, :len(sel)] = sel
    tdt = {"bf16": torch.bfloat16, "f16": torch.float16, "f32": torch.float32}[dtype]
    Q, K, V = make_uniform_qkv(B, Hq, Hkv, n, d, dtype=dtype, seed=seed)
    prob = cp.Problem(B, Hq, Hkv, n, d, seg, blk, k, tdt, flags=flags)
    ws = cp.alloc_workspace(prob)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    O, lse = cp.attention(prob, Qd, Kd, Vd, torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda(), ws, want_lse=True)
    assert cp.device_status(ws) == 0
    sm = f32(1.0 / np.sqrt(d))
    tol = {"f32": 1e-5, "f16": 2e-3, "bf16": 1e-2}[dtype]
    O_ref, lse_ref = oracle.sparse_attention(Q, K, V, idx, cnt, seg, blk, sm)
    err = np.abs(O.float().cpu().numpy().astype(np.float64) - O_ref)
    assert (err / np.maximum(1.0, np.abs(O_ref) / 2)).max() <= tol
    none = np.isneginf(lse_ref)                                    # rows that see no key: zeros, lse = -inf
    lg = lse.cpu().numpy()
    assert np.array_equal(np.isneginf(lg), none) and (O.float().cpu().numpy()[none] == 0).all()
    if (~none).any():
        assert np.abs(lg[~none] - lse_ref[~none]).max() <= 2e-3
    Od = cp.dense_attention(prob, Qd, Kd, Vd, ws)
    assert cp.device_status(ws) == 0
    Od_ref, _ = oracle.dense_attention(Q, K, V, sm)
    errd = np.abs(Od.float().cpu().numpy().astype(np.float64) - Od_ref)
    assert (errd / np.maximum(1.0, np.abs(Od_ref) / 2)).max() <= tol
