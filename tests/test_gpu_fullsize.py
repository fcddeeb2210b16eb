"""Full-size parity at the benchmark workload (128K tokens, Llama3-8B shape), in the launch
configuration bench.py times.  The oracle cannot afford every output at this size, so: scores and
selection are checked in full for two KV groups (8 query heads, all 128 segments); attention is
checked on sampled rows of sampled (head, segment) units, the oracle running on the same block lists."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_12490_b200 import CONFIGS
from paper_2409_12490_b200 import binding as cp
from paper_2409_12490_b200.inputs import make_qkv

from helpers import assert_attention_close, compare_scores, compare_selection, f32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def c4():
    cfg = CONFIGS["C4"]
    Q, K, V = make_qkv(cfg)
    prob = cp.Problem.from_config(cfg)
    ws = cp.alloc_workspace(prob)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    O, S, idx, cnt = cp.prefill_layer(prob, Qd, Kd, Vd, ws)
    assert cp.device_status(ws) == 0
    return dict(cfg=cfg, Q=Q, K=K, V=V, prob=prob, ws=ws, Qd=Qd, Kd=Kd, Vd=Vd, O=O, S=S, idx=idx, cnt=cnt)


def test_scores_and_selection_two_kv_groups(c4):
    cfg = c4["cfg"]
    g = cfg.n_q_heads // cfg.n_kv_heads
    excused_total = 0
    for kvh in (1, 6):
        hs = slice(kvh * g, (kvh + 1) * g)
        S_ref = oracle.estimate(c4["Q"][:, hs], c4["K"][:, kvh:kvh + 1], cfg.segment_size, cfg.block_size,
                                est_scale=f32(cfg.est_scale), alpha=f32(cfg.alpha))
        compare_scores(c4["S"][:, hs], S_ref, atol=1e-9)
        idx_ref, cnt_ref = oracle.select(S_ref, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
        excused, unexcused = compare_selection(c4["idx"][:, hs], c4["cnt"][:, hs], idx_ref, cnt_ref, S_ref, cfg.r)
        assert unexcused == 0
        excused_total += excused
    print(f"selection: {excused_total} excused k-th-boundary swaps (gap < 1e-5), 0 unexcused")


def _sampled_rows(cfg, n_units, rows_per_unit, seed):
    rng = np.random.default_rng(seed)
    first_real = -(-(cfg.budget_blocks - cfg.r) // cfg.r)
    units = [(int(rng.integers(cfg.n_q_heads)), j) for j in (0, 1, first_real, first_real + 1, cfg.n1 - 1)]
    units += [(int(rng.integers(cfg.n_q_heads)), int(rng.integers(cfg.n1))) for _ in range(n_units - len(units))]
    rows = []
    for h, j in units:
        t0 = j * cfg.segment_size
        ts = {t0, t0 + 127, t0 + 128, t0 + cfg.segment_size - 1}
        ts |= {t0 + int(x) for x in rng.integers(0, cfg.segment_size, rows_per_unit - len(ts))}
        rows += [(0, h, t) for t in sorted(ts)]
    return np.array(rows, dtype=np.int64)


def test_sparse_attention_sampled_rows(c4):
    cfg = c4["cfg"]
    rows = _sampled_rows(cfg, 64, 32, seed=1)
    idx, cnt = c4["idx"].cpu().numpy(), c4["cnt"].cpu().numpy()
    O_ref, _ = oracle.sparse_attention_rows(c4["Q"], c4["K"], c4["V"], idx, cnt, cfg.segment_size, cfg.block_size,
                                            f32(1.0 / np.sqrt(cfg.head_dim)), rows)
    O = c4["O"][rows[:, 0], rows[:, 1], rows[:, 2]].float().cpu().numpy()
    mx, mean, n_big = assert_attention_close(O, O_ref)
    print(f"sparse attention, {len(rows)} rows: max abs err {mx:.2e}, mean {mean:.2e}, {n_big} outputs with |O| >= 2")


def test_dense_attention_sampled_rows(c4):
    cfg = c4["cfg"]
    Od = cp.dense_attention(c4["prob"], c4["Qd"], c4["Kd"], c4["Vd"], c4["ws"])
    assert cp.device_status(c4["ws"]) == 0
    rng = np.random.default_rng(2)
    ts = [0, 127, 128, 255, 256, cfg.seq_len - 1] + [int(x) for x in rng.integers(0, cfg.seq_len, 58)]
    rows = np.array([(0, int(rng.integers(cfg.n_q_heads)), t) for t in ts], dtype=np.int64)
    O_ref, _ = oracle.dense_attention_rows(c4["Q"], c4["K"], c4["V"], f32(1.0 / np.sqrt(cfg.head_dim)), rows)
    O = Od[rows[:, 0], rows[:, 1], rows[:, 2]].float().cpu().numpy()
    assert_attention_close(O, O_ref)


def test_properties_at_full_size(c4):
    """Properties that hold at any size: lists ascending with the diagonal suffix, cnt = min(k,(j+1)r),
    outputs finite, and row 0 of every head equals V[0] (its only visible key)."""
    cfg = c4["cfg"]
    idx, cnt = c4["idx"].cpu().numpy(), c4["cnt"].cpu().numpy()
    j = np.arange(cfg.n1)
    assert np.array_equal(cnt[0, 0], np.minimum(cfg.budget_blocks, (j + 1) * cfg.r))
    full = cnt == cfg.budget_blocks
    assert (np.diff(idx[full], axis=-1) > 0).all()
    diag = idx[full][:, -cfg.r:]
    jj = np.broadcast_to(j[None, None, :], cnt.shape)[full]
    assert np.array_equal(diag, jj[:, None] * cfg.r + np.arange(cfg.r)[None, :])
    assert torch.isfinite(c4["O"].float()).all()
    g = cfg.n_q_heads // cfg.n_kv_heads
    v0 = c4["V"][0, :, 0].repeat_interleave(g, dim=0)
    assert torch.equal(c4["O"][0, :, 0].cpu(), v0)


def test_yi_shape_two_layer_chain_at_full_size():
    """C5's shape (32 query / 4 KV heads, 128K tokens) with the score carried from layer 0 into layer 1
    (Algorithm 1, line 14): scores and selection of one KV group against the oracle for both layers, and
    layer 1's attention on sampled rows of that group."""
    cfg = CONFIGS["C5"]
    g = cfg.n_q_heads // cfg.n_kv_heads
    prob = cp.Problem.from_config(cfg)
    ws = cp.alloc_workspace(prob)
    kvh = 2
    hs = slice(kvh * g, (kvh + 1) * g)
    S_prev_gpu, S_prev_ref = None, None
    for layer in (0, 1):
        Q, K, V = make_qkv(cfg, layer=layer)
        Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
        S = cp.estimate(prob, Qd, Kd, ws, S_prev=S_prev_gpu)
        idx, cnt = cp.select(prob, S, ws)
        S_ref = oracle.estimate(Q[:, hs], K[:, kvh:kvh + 1], cfg.segment_size, cfg.block_size,
                                est_scale=f32(cfg.est_scale), alpha=f32(cfg.alpha), S_prev=S_prev_ref)
        compare_scores(S[:, hs], S_ref, atol=1e-9)
        idx_ref, cnt_ref = oracle.select(S_ref, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
        assert compare_selection(idx[:, hs], cnt[:, hs], idx_ref, cnt_ref, S_ref, cfg.r)[1] == 0
        S_prev_gpu, S_prev_ref = S, S_ref
    O = cp.attention(prob, Qd, Kd, Vd, idx, cnt, ws)
    assert cp.device_status(ws) == 0
    rng = np.random.default_rng(3)
    rows = np.array([(0, kvh * g + int(rng.integers(g)), int(t)) for t in rng.integers(0, cfg.seq_len, 512)], dtype=np.int64)
    O_ref, _ = oracle.sparse_attention_rows(Q, K, V, idx.cpu().numpy(), cnt.cpu().numpy(), cfg.segment_size,
                                            cfg.block_size, f32(1.0 / np.sqrt(cfg.head_dim)), rows)
    assert_attention_close(O[rows[:, 0], rows[:, 1], rows[:, 2]], O_ref)


def test_paper_operating_point_at_full_size():
    """The paper's own setting (Section 3.1.3: segment 512, block 32, budget 1024, alpha 0.25) at 128K tokens:
    n2 = 4096 key blocks, so the score kernel splits them over a thread-block cluster, a gathered K/V tile
    is four 32-token boxes and the list holds 16 diagonal + 16 past blocks.  Scores with layer fusion
    (Algorithm 1, line 14) and selection of one KV group against the oracle; attention on sampled rows."""
    cfg = CONFIGS["paper_128k"]
    g = cfg.n_q_heads // cfg.n_kv_heads
    prob = cp.Problem.from_config(cfg)
    ws = cp.alloc_workspace(prob)
    kvh = 5
    hs = slice(kvh * g, (kvh + 1) * g)
    Q, K, V = make_qkv(cfg)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    S0 = cp.estimate(prob, Qd, Kd, ws)
    S0_ref = oracle.estimate(Q[:, hs], K[:, kvh:kvh + 1], cfg.segment_size, cfg.block_size, est_scale=f32(cfg.est_scale))
    compare_scores(S0[:, hs], S0_ref, atol=1e-9)
    # a second layer on the same inputs, fused onto layer 0's score: the fusion path at this size
    S1 = cp.estimate(prob, Qd, Kd, ws, S_prev=S0)
    S1_ref = oracle.estimate(Q[:, hs], K[:, kvh:kvh + 1], cfg.segment_size, cfg.block_size, est_scale=f32(cfg.est_scale),
                             alpha=f32(cfg.alpha), S_prev=S0_ref)
    compare_scores(S1[:, hs], S1_ref, atol=1e-9)
    idx, cnt = cp.select(prob, S1, ws)
    idx_ref, cnt_ref = oracle.select(S1_ref, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
    excused, unexcused = compare_selection(idx[:, hs], cnt[:, hs], idx_ref, cnt_ref, S1_ref, cfg.r)
    assert unexcused == 0
    O = cp.attention(prob, Qd, Kd, Vd, idx, cnt, ws)
    assert cp.device_status(ws) == 0
    rng = np.random.default_rng(4)
    ts = [0, 31, 32, 511, 512, cfg.seq_len - 1] + [int(t) for t in rng.integers(0, cfg.seq_len, 506)]
    rows = np.array([(0, kvh * g + int(rng.integers(g)), t) for t in ts], dtype=np.int64)
    O_ref, _ = oracle.sparse_attention_rows(Q, K, V, idx.cpu().numpy(), cnt.cpu().numpy(), cfg.segment_size,
                                            cfg.block_size, f32(1.0 / np.sqrt(cfg.head_dim)), rows)
    mx, mean, _ = assert_attention_close(O[rows[:, 0], rows[:, 1], rows[:, 2]], O_ref)
    print(f"paper operating point: {excused} excused swaps, attention max abs err {mx:.2e}, mean {mean:.2e}")
