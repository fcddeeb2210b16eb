"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same bits."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_12490_b200 import CONFIGS
from paper_2409_12490_b200 import binding as cp
from paper_2409_12490_b200.inputs import make_qkv, make_uniform_qkv

from helpers import (TOL_BF16_MAX, TOL_BF16_MEAN, TOL_F32, assert_attention_close, attention_errors, compare_scores, compare_selection,
                     f32, oracle_scores, problem, to_dev)

pytestmark = pytest.mark.gpu

SMALL_BF16 = CONFIGS["C2"].with_(name="small_bf16", seq_len=2048, n_q_heads=4, n_kv_heads=2, segment_size=256,
                                 block_size=64, budget_tokens=512, n_clusters=16)


def run_estimate_select(cfg, Q, K, S_prev=None, **kw):
    prob = problem(cfg, **kw)
    ws = cp.alloc_workspace(prob)
    Qd, Kd = to_dev(Q, K)
    Sp = None if S_prev is None else torch.from_numpy(S_prev).cuda()
    S = cp.estimate(prob, Qd, Kd, ws, S_prev=Sp)
    idx, cnt = cp.select(prob, S, ws)
    assert cp.device_status(ws) == 0
    return prob, ws, S, idx, cnt


@pytest.mark.parametrize("name", ["C1", "small_bf16"])
def test_estimate_and_select_match_oracle(name):
    cfg = CONFIGS.get(name, SMALL_BF16)
    Q, K, V = make_qkv(cfg)
    prob, ws, S, idx, cnt = run_estimate_select(cfg, Q, K)
    S_ref = oracle_scores(cfg, Q, K)
    compare_scores(S, S_ref)
    idx_ref, cnt_ref = oracle.select(S_ref, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
    excused, unexcused = compare_selection(idx, cnt, idx_ref, cnt_ref, S_ref, cfg.r)
    assert unexcused == 0
    # second layer: fusion with the first layer's scores (Algorithm 1, line 14)
    Q1, K1, _ = make_qkv(cfg, layer=1)
    _, _, S1, idx1, cnt1 = run_estimate_select(cfg, Q1, K1, S_prev=S_ref)
    S1_ref = oracle_scores(cfg, Q1, K1, S_prev=S_ref)
    compare_scores(S1, S1_ref)
    i1, c1 = oracle.select(S1_ref, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
    assert compare_selection(idx1, cnt1, i1, c1, S1_ref, cfg.r)[1] == 0


@pytest.mark.parametrize("est_scale,flags", [(1.0 / np.sqrt(64.0), 0), (1.0, cp.FLAG_MASK_BEFORE_SOFTMAX)])
def test_estimate_variants(est_scale, flags):
    cfg = CONFIGS["C1"].with_(est_scale=f32(est_scale))
    Q, K, _ = make_qkv(cfg)
    _, _, S, _, _ = run_estimate_select(cfg, Q, K, flags=flags)
    compare_scores(S, oracle_scores(cfg, Q, K, mask_before_softmax=bool(flags)))


def test_alpha_one_with_previous_scores_is_the_unfused_score():
    """alpha = 1 with a non-NULL S_prev (the paper's "w/o fusion" setting run through the fusing call): the kernel
    must return the unfused ln S.  The oracle evaluates line 14 in full, logaddexp(ln 1 + ln S, ln 0 + ln S')."""
    cfg = SMALL_BF16.with_(alpha=1.0)
    Q, K, _ = make_qkv(cfg)
    rng = np.random.default_rng(3)
    S_prev = oracle_scores(cfg, *make_qkv(cfg, layer=1)[:2]) + rng.standard_normal((1, 4, cfg.n1, cfg.n2))
    _, _, S, idx, cnt = run_estimate_select(cfg, Q, K, S_prev=S_prev)
    S_ref = oracle_scores(cfg, Q, K, S_prev=S_prev)
    assert np.array_equal(S_ref, oracle_scores(cfg, Q, K))          # identity on the oracle side, through the formula
    compare_scores(S, S_ref)
    # alpha = 0 is the other end: the previous layer's score is returned
    cfg0 = SMALL_BF16.with_(alpha=0.0)
    _, _, S0, _, _ = run_estimate_select(cfg0, Q, K, S_prev=S_prev)
    compare_scores(S0, oracle_scores(cfg0, Q, K, S_prev=S_prev))


def test_attention_fp32_simt_matches_oracle():
    cfg = CONFIGS["C1"]
    Q, K, V = make_qkv(cfg)
    S_ref = oracle_scores(cfg, Q, K)
    idx_ref, cnt_ref = oracle.select(S_ref, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
    prob = problem(cfg)
    ws = cp.alloc_workspace(prob)
    Qd, Kd, Vd = to_dev(Q, K, V)
    O, lse = cp.attention(prob, Qd, Kd, Vd, torch.from_numpy(idx_ref).cuda(), torch.from_numpy(cnt_ref).cuda(), ws,
                          want_lse=True)
    assert cp.device_status(ws) == 0
    sm = f32(1.0 / np.sqrt(cfg.head_dim))
    O_ref, lse_ref = oracle.sparse_attention(Q, K, V, idx_ref, cnt_ref, cfg.segment_size, cfg.block_size, sm)
    mx, mean = attention_errors(O, O_ref)
    assert mx <= TOL_F32, (mx, mean)
    assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 1e-4
    Od = cp.dense_attention(prob, Qd, Kd, Vd, ws)
    Od_ref, _ = oracle.dense_attention(Q, K, V, sm)
    assert attention_errors(Od, Od_ref)[0] <= TOL_F32


def _sparse_case(cfg, Q, K, V, flags=0):
    S_ref = oracle_scores(cfg, Q, K)
    idx_ref, cnt_ref = oracle.select(S_ref, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
    prob = problem(cfg, flags=flags)
    ws = cp.alloc_workspace(prob)
    Qd, Kd, Vd = to_dev(Q, K, V)
    O, lse = cp.attention(prob, Qd, Kd, Vd, torch.from_numpy(idx_ref).cuda(), torch.from_numpy(cnt_ref).cuda(), ws,
                          want_lse=True)
    assert cp.device_status(ws) == 0
    sm = f32(1.0 / np.sqrt(cfg.head_dim))
    O_ref, lse_ref = oracle.sparse_attention(Q, K, V, idx_ref, cnt_ref, cfg.segment_size, cfg.block_size, sm)
    return O, lse, O_ref, lse_ref


@pytest.mark.parametrize("flags", [0, cp.FLAG_FORCE_SIMT])
@pytest.mark.parametrize("blk,budget", [(64, 512), (32, 416), (128, 768), (64, 2048)])
def test_attention_bf16_matches_oracle(blk, budget, flags):
    """blk 32 / budget 416 leaves a ragged last gathered tile; budget 2048 covers everything."""
    cfg = SMALL_BF16.with_(block_size=blk, budget_tokens=budget)
    Q, K, V = make_qkv(cfg)
    O, lse, O_ref, lse_ref = _sparse_case(cfg, Q, K, V, flags)
    assert_attention_close(O, O_ref)
    assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 2e-3


def test_dense_bf16_matches_oracle_and_full_budget_sparse():
    cfg = SMALL_BF16
    Q, K, V = make_qkv(cfg)
    prob = problem(cfg)
    ws = cp.alloc_workspace(prob)
    Qd, Kd, Vd = to_dev(Q, K, V)
    O, lse = cp.dense_attention(prob, Qd, Kd, Vd, ws, want_lse=True)
    assert cp.device_status(ws) == 0
    sm = f32(1.0 / np.sqrt(cfg.head_dim))
    O_ref, lse_ref = oracle.dense_attention(Q, K, V, sm)
    assert_attention_close(O, O_ref)
    assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 2e-3


def test_uniform_inputs_batch2_strided():
    """i.i.d. inputs, batch 2, and Q/K/V/O taken as strided views of a packed [B,n,H,d] buffer."""
    B, Hq, Hkv, n, d = 2, 4, 2, 1024, 128
    Q, K, V = make_uniform_qkv(B, Hq, Hkv, n, d, seed=5)
    cfg = SMALL_BF16.with_(batch=B, seq_len=n, budget_tokens=384)
    S_ref = oracle_scores(cfg, Q, K)
    idx_ref, cnt_ref = oracle.select(S_ref, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
    prob = problem(cfg)
    ws = cp.alloc_workspace(prob)
    packed = torch.empty((B, n, Hq + 2 * Hkv, d), dtype=torch.bfloat16, device="cuda")
    Qd = packed[:, :, :Hq].permute(0, 2, 1, 3)
    Kd = packed[:, :, Hq:Hq + Hkv].permute(0, 2, 1, 3)
    Vd = packed[:, :, Hq + Hkv:].permute(0, 2, 1, 3)
    Qd.copy_(Q); Kd.copy_(K); Vd.copy_(V)
    S = cp.estimate(prob, Qd, Kd, ws)
    compare_scores(S, S_ref)
    idx, cnt = cp.select(prob, S, ws)
    assert compare_selection(idx, cnt, idx_ref, cnt_ref, S_ref, cfg.r)[1] == 0
    O_buf = torch.zeros((B, n, Hq, d), dtype=torch.bfloat16, device="cuda")
    O = cp.attention(prob, Qd, Kd, Vd, torch.from_numpy(idx_ref).cuda(), torch.from_numpy(cnt_ref).cuda(), ws,
                     O=O_buf.permute(0, 2, 1, 3))
    assert cp.device_status(ws) == 0
    O_ref, _ = oracle.sparse_attention(Q, K, V, idx_ref, cnt_ref, cfg.segment_size, cfg.block_size,
                                       f32(1.0 / np.sqrt(d)))
    assert_attention_close(O, O_ref)


def test_select_with_ties_matches_oracle():
    cfg = SMALL_BF16
    prob = problem(cfg)
    ws = cp.alloc_workspace(prob)
    rng = np.random.default_rng(0)
    S = np.round(rng.standard_normal((1, 4, cfg.n1, cfg.n2)) * 2) / 2      # heavy ties
    idx, cnt = cp.select(prob, torch.from_numpy(S).cuda(), ws)
    idx_ref, cnt_ref = oracle.select(S, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
    assert np.array_equal(idx.cpu().numpy(), idx_ref) and np.array_equal(cnt.cpu().numpy(), cnt_ref)


@pytest.mark.parametrize("n_sink,n_local,shared", [(0, 0, True), (1, 2, False), (2, 1, True)])
def test_selection_variants_match_oracle(n_sink, n_local, shared):
    """One list per KV group (score = maximum over the group's heads) and forced sink / local blocks, alone and
    together; then attention on the GPU's lists against the oracle on the same lists."""
    cfg = SMALL_BF16.with_(block_size=32, budget_tokens=512)          # r = 8, k = 16: 8 free slots
    Q, K, V = make_qkv(cfg)
    g = cfg.n_q_heads // cfg.n_kv_heads
    flags = cp.FLAG_SHARED_GROUP_LISTS if shared else 0
    prob = problem(cfg, flags=flags, n_sink=n_sink, n_local=n_local)
    ws = cp.alloc_workspace(prob)
    Qd, Kd, Vd = to_dev(Q, K, V)
    S = cp.estimate(prob, Qd, Kd, ws)
    idx, cnt = cp.select(prob, S, ws)
    S_ref = oracle_scores(cfg, Q, K)
    compare_scores(S, S_ref)
    idx_ref, cnt_ref = oracle.select(S_ref, cfg.segment_size, cfg.block_size, cfg.budget_blocks, group=g if shared else 1,
                                     n_sink=n_sink, n_local=n_local)
    assert np.array_equal(idx.cpu().numpy(), idx_ref) and np.array_equal(cnt.cpu().numpy(), cnt_ref)
    if shared:
        assert torch.equal(idx[:, 0::2], idx[:, 1::2])                  # g = 2: both heads of a group share the list
    O = cp.attention(prob, Qd, Kd, Vd, idx, cnt, ws)
    assert cp.device_status(ws) == 0
    O_ref, _ = oracle.sparse_attention(Q, K, V, idx_ref, cnt_ref, cfg.segment_size, cfg.block_size, f32(1.0 / np.sqrt(cfg.head_dim)))
    assert_attention_close(O, O_ref)
    # heavy ties on top of the variants
    rng = np.random.default_rng(1)
    St = np.round(rng.standard_normal(S_ref.shape) * 2) / 2
    it, ct = cp.select(prob, torch.from_numpy(St).cuda(), ws)
    ir, cr = oracle.select(St, cfg.segment_size, cfg.block_size, cfg.budget_blocks, group=g if shared else 1, n_sink=n_sink, n_local=n_local)
    assert np.array_equal(it.cpu().numpy(), ir) and np.array_equal(ct.cpu().numpy(), cr)


@pytest.mark.parametrize("name,blk", [("small_bf16", 64), ("small_bf16", 32), ("C1", 32)])
def test_decode_phase_criticality_matches_oracle(name, blk):
    """The last token's block criticality (Section 2.1) and its block list: bf16 (tensor-core log-sum-exp path) and fp32."""
    cfg = CONFIGS.get(name, SMALL_BF16).with_(block_size=blk)
    Q, K, _ = make_qkv(cfg)
    prob = problem(cfg)
    ws = cp.alloc_workspace(prob)
    q_last = Q[:, :, -1].contiguous()
    S = cp.decode_estimate(prob, q_last.cuda(), K.cuda(), ws)
    idx, cnt = cp.decode_select(prob, S, ws)
    assert cp.device_status(ws) == 0
    S_ref = oracle.decode_estimate(q_last, K, cfg.block_size, est_scale=f32(cfg.est_scale))
    assert np.abs(S.cpu().numpy() - S_ref).max() <= 1e-9
    idx_ref, cnt_ref = oracle.decode_select(S_ref, cfg.budget_blocks)
    assert np.array_equal(idx.cpu().numpy(), idx_ref) and np.array_equal(cnt.cpu().numpy(), cnt_ref)


def test_bad_list_sets_bounds_status_without_faulting():
    cfg = SMALL_BF16
    Q, K, V = make_qkv(cfg)
    S_ref = oracle_scores(cfg, Q, K)
    idx_ref, cnt_ref = oracle.select(S_ref, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
    bad = idx_ref.copy()
    bad[0, 1, -1, 0] = 10 ** 6            # out of range
    for flags in (0, cp.FLAG_FORCE_SIMT):
        prob = problem(cfg, flags=flags)
        ws = cp.alloc_workspace(prob)
        Qd, Kd, Vd = to_dev(Q, K, V)
        cp.attention(prob, Qd, Kd, Vd, torch.from_numpy(bad).cuda(), torch.from_numpy(cnt_ref).cuda(), ws)
        assert cp.device_status(ws) == 7


def test_host_side_argument_errors():
    cfg = SMALL_BF16
    prob = problem(cfg)
    ws = cp.alloc_workspace(prob)
    Q, K, V = to_dev(*make_uniform_qkv(1, 4, 2, cfg.seq_len, 128, seed=1))
    with pytest.raises(cp.CritiPrefillError) as e:
        cp.estimate(prob, Q, K, ws[:1024])
    assert e.value.status == 4
    bad = cp.Problem.from_config(cfg.with_(segment_size=200))        # not a multiple of the block size
    with pytest.raises(cp.CritiPrefillError) as e:
        cp.workspace_bytes(bad)
    assert e.value.status == 2
    bad = cp.Problem.from_config(cfg.with_(budget_tokens=128))     # budget smaller than one segment
    with pytest.raises(cp.CritiPrefillError) as e:
        cp.workspace_bytes(bad)
    assert e.value.status == 2
    bad = cp.Problem.from_config(cfg, n_sink=3, n_local=2)         # k - r = 4 free slots cannot hold 5 forced blocks
    with pytest.raises(cp.CritiPrefillError) as e:
        cp.workspace_bytes(bad)
    assert e.value.status == 2
    S_prev = torch.zeros((1, 4, cfg.n1, cfg.n2), dtype=torch.float64, device="cuda")
    for alpha in (-0.1, 1.5, float("nan")):                        # line 14 is a convex combination
        with pytest.raises(cp.CritiPrefillError) as e:
            cp.estimate(cp.Problem.from_config(cfg.with_(alpha=alpha)), Q, K, ws, S_prev=S_prev)
        assert e.value.status == 2
