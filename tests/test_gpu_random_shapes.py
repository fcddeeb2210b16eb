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
