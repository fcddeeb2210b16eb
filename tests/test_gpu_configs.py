"""The benchmark configurations at their stated shapes, CUDA path (through the C ABI) against the fp64 oracle:
C2 in full, C3 with every (head, segment) unit of estimate/select and attention on sampled units plus the four
corners of its budget x block-size sweep, C4 scores and selection on all 32 heads and the dense kernel on 64 rows
of every head.  (C1 runs in full in test_gpu_parity.py, C5's shape and the paper's operating point in
test_gpu_fullsize.py.)"""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_12490_b200 import CONFIGS
from paper_2409_12490_b200 import binding as cp
from paper_2409_12490_b200.inputs import make_qkv

from helpers import assert_attention_close, compare_scores, compare_selection, f32

pytestmark = pytest.mark.gpu


def _estimate_select_all_units(cfg, Q, K, S, idx, cnt):
    """ln S and the block lists of every (head, segment) unit against the oracle, one KV group at a time.
    Returns the oracle's (idx, cnt) for the whole layer and the number of excused k-th-boundary swaps."""
    g = cfg.n_q_heads // cfg.n_kv_heads
    idx_all = np.empty((cfg.batch, cfg.n_q_heads, cfg.n1, cfg.budget_blocks), dtype=np.int32)
    cnt_all = np.empty((cfg.batch, cfg.n_q_heads, cfg.n1), dtype=np.int32)
    excused_total, worst = 0, 0.0
    for kvh in range(cfg.n_kv_heads):
        hs = slice(kvh * g, (kvh + 1) * g)
        S_ref = oracle.estimate(Q[:, hs], K[:, kvh:kvh + 1], cfg.segment_size, cfg.block_size,
                                est_scale=f32(cfg.est_scale), alpha=f32(cfg.alpha))
        worst = max(worst, compare_scores(S[:, hs], S_ref, atol=1e-9))
        idx_ref, cnt_ref = oracle.select(S_ref, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
        excused, unexcused = compare_selection(idx[:, hs], cnt[:, hs], idx_ref, cnt_ref, S_ref, cfg.r)
        assert unexcused == 0, f"KV head {kvh}: {unexcused} unexcused selection differences"
        excused_total += excused
        idx_all[:, hs], cnt_all[:, hs] = idx_ref, cnt_ref
    print(f"[parity] {cfg.name}: ln S max abs diff {worst:.2e} over all {cfg.n_q_heads * cfg.n1} units, "
          f"{excused_total} excused swaps, 0 unexcused")
    return idx_all, cnt_all, excused_total


def _unit_rows(cfg, n_units, rows_per_unit, seed):
    """Rows (b, h, t) of sampled (head, segment) units: always segments 0, 1, the first two with a real
    selection and the last, plus random ones; per unit the tile edges plus random rows."""
    rng = np.random.default_rng(seed)
    first_real = min(cfg.n1 - 1, -(-(cfg.budget_blocks - cfg.r) // cfg.r))
    fixed = sorted({0, min(1, cfg.n1 - 1), first_real, min(first_real + 1, cfg.n1 - 1), cfg.n1 - 1})
    units = [(int(rng.integers(cfg.n_q_heads)), j) for j in fixed]
    units += [(int(rng.integers(cfg.n_q_heads)), int(rng.integers(cfg.n1))) for _ in range(max(0, n_units - len(units)))]
    rows = []
    for h, j in units:
        t0 = j * cfg.segment_size
        ts = {t0, t0 + 127, t0 + 128, t0 + cfg.segment_size - 1}
        ts |= {t0 + int(x) for x in rng.integers(0, cfg.segment_size, max(0, rows_per_unit - len(ts)))}
        rows += [(0, h, t) for t in sorted(ts) if t < cfg.seq_len]
    return np.array(rows, dtype=np.int64)


def _run_layer(cfg, Q, K, V):
    prob = cp.Problem.from_config(cfg)
    ws = cp.alloc_workspace(prob)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    O, S, idx, cnt = cp.prefill_layer(prob, Qd, Kd, Vd, ws)
    assert cp.device_status(ws) == 0
    return prob, ws, (Qd, Kd, Vd), O, S, idx, cnt


def test_C2_at_its_stated_shape_every_row():
    cfg = CONFIGS["C2"]
    Q, K, V = make_qkv(cfg)
    prob, ws, (Qd, Kd, Vd), O, S, idx, cnt = _run_layer(cfg, Q, K, V)
    idx_ref, cnt_ref, _ = _estimate_select_all_units(cfg, Q, K, S, idx, cnt)
    sm = f32(1.0 / np.sqrt(cfg.head_dim))
    # attention on the oracle's lists, every row of every head
    O2 = cp.attention(prob, Qd, Kd, Vd, torch.from_numpy(idx_ref).cuda(), torch.from_numpy(cnt_ref).cuda(), ws)
    assert cp.device_status(ws) == 0
    O_ref, _ = oracle.sparse_attention(Q, K, V, idx_ref, cnt_ref, cfg.segment_size, cfg.block_size, sm)
    assert_attention_close(O2, O_ref, label="C2 sparse, all rows")
    Od = cp.dense_attention(prob, Qd, Kd, Vd, ws)
    assert cp.device_status(ws) == 0
    Od_ref, _ = oracle.dense_attention(Q, K, V, sm)
    assert_attention_close(Od, Od_ref, label="C2 dense, all rows")


@pytest.fixture(scope="module")
def c3_inputs():
    return make_qkv(CONFIGS["C3"])


def test_C3_at_its_stated_shape(c3_inputs):
    cfg = CONFIGS["C3"]
    Q, K, V = c3_inputs
    prob, ws, (Qd, Kd, Vd), O, S, idx, cnt = _run_layer(cfg, Q, K, V)
    idx_ref, cnt_ref, _ = _estimate_select_all_units(cfg, Q, K, S, idx, cnt)
    rows = _unit_rows(cfg, 96, 48, seed=11)
    sm = f32(1.0 / np.sqrt(cfg.head_dim))
    O2 = cp.attention(prob, Qd, Kd, Vd, torch.from_numpy(idx_ref).cuda(), torch.from_numpy(cnt_ref).cuda(), ws)
    assert cp.device_status(ws) == 0
    O_ref, _ = oracle.sparse_attention_rows(Q, K, V, idx_ref, cnt_ref, cfg.segment_size, cfg.block_size, sm, rows)
    assert_attention_close(O2[rows[:, 0], rows[:, 1], rows[:, 2]], O_ref, label=f"C3 sparse, {len(rows)} rows of 96 units")
    Od = cp.dense_attention(prob, Qd, Kd, Vd, ws)
    assert cp.device_status(ws) == 0
    Od_ref, _ = oracle.dense_attention_rows(Q, K, V, sm, rows[::4])
    r4 = rows[::4]
    assert_attention_close(Od[r4[:, 0], r4[:, 1], r4[:, 2]], Od_ref, label=f"C3 dense, {len(r4)} rows")


@pytest.mark.parametrize("blk,budget", [(32, 1024), (32, 8192), (128, 1024), (128, 8192)])
def test_C3_sweep_corners(c3_inputs, blk, budget):
    """The corners of the budget x block-size sweep whose accuracy-versus-speed trace the benchmark reports:
    every unit of estimate/select, attention on sampled rows."""
    cfg = CONFIGS["C3"].with_(name=f"C3 blk{blk} budget{budget}", block_size=blk, budget_tokens=budget)
    Q, K, V = c3_inputs
    prob, ws, (Qd, Kd, Vd), O, S, idx, cnt = _run_layer(cfg, Q, K, V)
    idx_ref, cnt_ref, _ = _estimate_select_all_units(cfg, Q, K, S, idx, cnt)
    rows = _unit_rows(cfg, 24, 24, seed=blk + budget)
    sm = f32(1.0 / np.sqrt(cfg.head_dim))
    O2 = cp.attention(prob, Qd, Kd, Vd, torch.from_numpy(idx_ref).cuda(), torch.from_numpy(cnt_ref).cuda(), ws)
    assert cp.device_status(ws) == 0
    O_ref, _ = oracle.sparse_attention_rows(Q, K, V, idx_ref, cnt_ref, cfg.segment_size, cfg.block_size, sm, rows)
    assert_attention_close(O2[rows[:, 0], rows[:, 1], rows[:, 2]], O_ref, label=f"{cfg.name} sparse, {len(rows)} rows")


def test_C4_scores_selection_all_heads_and_dense_rows_per_head():
    cfg = CONFIGS["C4"]
    Q, K, V = make_qkv(cfg)
    prob, ws, (Qd, Kd, Vd), O, S, idx, cnt = _run_layer(cfg, Q, K, V)
    _estimate_select_all_units(cfg, Q, K, S, idx, cnt)
    del O, S
    Od = cp.dense_attention(prob, Qd, Kd, Vd, ws)
    assert cp.device_status(ws) == 0
    rng = np.random.default_rng(21)
    rows = []
    for h in range(cfg.n_q_heads):
        ts = [0, 127, 128, cfg.seq_len - 1] + [int(x) for x in rng.integers(0, cfg.seq_len, 60)]
        rows += [(0, h, t) for t in ts]
    rows = np.array(rows, dtype=np.int64)
    Od_ref, _ = oracle.dense_attention_rows(Q, K, V, f32(1.0 / np.sqrt(cfg.head_dim)), rows)
    assert_attention_close(Od[rows[:, 0], rows[:, 1], rows[:, 2]], Od_ref, label=f"C4 dense, 64 rows of each of {cfg.n_q_heads} heads")


def test_mass_recall_from_the_kernels_lse_equals_the_oracles():
    """The accuracy diagnostic the benchmark reports -- the share of a row's dense softmax mass that the listed keys
    hold, exp(lse_sparse - lse_dense) from the two kernels -- against the same quantity from the oracle, on C3."""
    cfg = CONFIGS["C3"].with_(name="C3 recall", budget_tokens=1024)
    Q, K, V = make_qkv(cfg)
    prob, ws, (Qd, Kd, Vd), O, S, idx, cnt = _run_layer(cfg, Q, K, V)
    _, lse_s = cp.attention(prob, Qd, Kd, Vd, idx, cnt, ws, want_lse=True)
    _, lse_d = cp.dense_attention(prob, Qd, Kd, Vd, ws, want_lse=True)
    assert cp.device_status(ws) == 0
    rows = _unit_rows(cfg, 32, 16, seed=5)
    sm = f32(1.0 / np.sqrt(cfg.head_dim))
    _, ls_ref = oracle.sparse_attention_rows(Q, K, V, idx.cpu().numpy(), cnt.cpu().numpy(), cfg.segment_size, cfg.block_size, sm, rows)
    _, ld_ref = oracle.dense_attention_rows(Q, K, V, sm, rows)
    recall_ref = np.exp(ls_ref - ld_ref)
    sel = (rows[:, 0], rows[:, 1], rows[:, 2])
    recall_gpu = torch.exp(lse_s.double() - lse_d.double())[sel].cpu().numpy()
    assert ((recall_ref > 0) & (recall_ref <= 1 + 1e-12)).all()
    assert np.abs(recall_gpu - recall_ref).max() <= 5e-3, np.abs(recall_gpu - recall_ref).max()
    print(f"[parity] mass recall on {len(rows)} rows: max abs diff {np.abs(recall_gpu - recall_ref).max():.2e}, "
          f"median recall {np.median(recall_ref):.3f}")
