"""Edge cases of the CUDA path against the oracle: smallest shapes, budgets that hold only the
diagonal, large logits (rescale path), the SIMT fallback shapes, and the bounded-wait status."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_12490_b200 import CONFIGS
from paper_2409_12490_b200 import binding as cp
from paper_2409_12490_b200.inputs import make_qkv, make_uniform_qkv

from helpers import TOL_BF16_MAX, TOL_BF16_MEAN, assert_attention_close, attention_errors, compare_scores, compare_selection, f32, oracle_scores, problem, to_dev

pytestmark = pytest.mark.gpu

BASE = CONFIGS["C2"].with_(name="edge", seq_len=1024, n_q_heads=2, n_kv_heads=1, segment_size=256,
                           block_size=128, budget_tokens=256, n_clusters=8)


def full_path_vs_oracle(cfg, Q, K, V, flags=0, tol=(TOL_BF16_MAX, TOL_BF16_MEAN)):
    prob = problem(cfg, flags=flags)
    ws = cp.alloc_workspace(prob)
    Qd, Kd, Vd = to_dev(Q, K, V)
    O, S, idx, cnt = cp.prefill_layer(prob, Qd, Kd, Vd, ws)
    assert cp.device_status(ws) == 0
    S_ref = oracle_scores(cfg, Q, K)
    compare_scores(S, S_ref)
    idx_ref, cnt_ref = oracle.select(S_ref, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
    assert compare_selection(idx, cnt, idx_ref, cnt_ref, S_ref, cfg.r)[1] == 0
    O_ref, _ = oracle.sparse_attention(Q, K, V, idx.cpu().numpy(), cnt.cpu().numpy(), cfg.segment_size, cfg.block_size,
                                       f32(1.0 / np.sqrt(cfg.head_dim)))
    assert_attention_close(O, O_ref, *tol)
    return O


def test_budget_holds_only_the_diagonal_blocks():
    cfg = BASE                                   # k = r = 2: no past block is ever taken
    full_path_vs_oracle(cfg, *make_qkv(cfg))


def test_single_unit_sequence():
    cfg = BASE.with_(seq_len=256)                # one segment, one 256-row unit, two tiles
    full_path_vs_oracle(cfg, *make_qkv(cfg))


def test_many_small_units_batch3():
    cfg = BASE.with_(batch=3, n_q_heads=4, n_kv_heads=4, seq_len=2048, block_size=32, budget_tokens=352)
    full_path_vs_oracle(cfg, *make_qkv(cfg))     # 11 blocks of 32: ragged last gathered tile


def test_large_logits_exercise_the_rescale_path():
    cfg = BASE.with_(seq_len=2048, budget_tokens=1024)
    Q, K, V = make_uniform_qkv(1, 2, 1, 2048, 128, seed=11, scale=1.0)
    Q = (Q.float() * 6.0).to(torch.bfloat16)     # logits up to ~ +-60: row maxima jump between tiles
    prob = problem(cfg)
    ws = cp.alloc_workspace(prob)
    Qd, Kd, Vd = to_dev(Q, K, V)
    Od = cp.dense_attention(prob, Qd, Kd, Vd, ws)
    assert cp.device_status(ws) == 0
    O_ref, _ = oracle.dense_attention(Q, K, V, f32(1.0 / np.sqrt(128)))
    # Peaked rows put almost all weight on a few keys, so the unit-scale tolerance does not apply.
    # From the arithmetic: each probability is rounded to bf16 (unit roundoff 2^-8) while the row sum
    # is taken before rounding, and O is rounded to bf16 once more, so
    #   |O_gpu - O| <= 2^-8 * (sum_u p_u |v_u| + |O|) <= 2^-7 * max|V|.
    bound = 2.0 ** -7 * float(V.float().abs().max())
    mx, mean = attention_errors(Od, O_ref)
    assert mx <= bound and mean <= TOL_BF16_MEAN, (mx, mean, bound)


@pytest.mark.parametrize("n,seg,blk,d", [(768, 128, 32, 128), (768, 384, 64, 128), (1280, 640, 128, 128),
                                         (640, 128, 128, 128), (768, 256, 64, 64)])
def test_odd_tile_counts_and_simt_shapes(n, seg, blk, d):
    """Segments of 1, 3 or 5 query tiles (the last work unit of a segment then has a single tile), a
    sequence of 5 tiles for the dense kernel, and head_dim 64, which the SIMT kernel serves."""
    cfg = BASE.with_(seq_len=n, segment_size=seg, block_size=blk, budget_tokens=max(seg, 256), head_dim=d)
    Q, K, V = make_qkv(cfg)
    full_path_vs_oracle(cfg, Q, K, V)
    prob = problem(cfg)
    ws = cp.alloc_workspace(prob)
    Od = cp.dense_attention(prob, *to_dev(Q, K, V), ws)
    assert cp.device_status(ws) == 0
    O_ref, _ = oracle.dense_attention(Q, K, V, f32(1.0 / np.sqrt(cfg.head_dim)))
    assert_attention_close(Od, O_ref)


def test_fp32_path_with_strided_output():
    cfg = CONFIGS["C1"].with_(seq_len=512)
    Q, K, V = make_qkv(cfg)
    O = full_path_vs_oracle(cfg, Q, K, V, tol=(1e-5, 1e-6))
    assert O.dtype == torch.float32


def test_bounded_wait_reports_timeout_and_context_survives():
    """Failure detection without a fault: with the V loads withheld a pipeline wait runs out, the
    kernel drains, the status reads CP_ERR_TIMEOUT, and the next call on the same context works."""
    cfg = BASE.with_(seq_len=256)
    Q, K, V = make_qkv(cfg)
    S_ref = oracle_scores(cfg, Q, K)
    idx_ref, cnt_ref = oracle.select(S_ref, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
    Qd, Kd, Vd = to_dev(Q, K, V)
    idx, cnt = torch.from_numpy(idx_ref).cuda(), torch.from_numpy(cnt_ref).cuda()
    prob = problem(cfg, flags=cp.FLAG_TEST_WITHHOLD_V)
    ws = cp.alloc_workspace(prob)
    cp.attention(prob, Qd, Kd, Vd, idx, cnt, ws)
    assert cp.device_status(ws) == 6
    ws.zero_()
    prob = problem(cfg)
    O = cp.attention(prob, Qd, Kd, Vd, idx, cnt, ws)
    assert cp.device_status(ws) == 0
    O_ref, _ = oracle.sparse_attention(Q, K, V, idx_ref, cnt_ref, cfg.segment_size, cfg.block_size,
                                       f32(1.0 / np.sqrt(cfg.head_dim)))
    assert_attention_close(O, O_ref)


@pytest.mark.parametrize("n,seg,blk", [(8192, 64, 4), (16384, 128, 4), (8224, 8, 4)])
def test_many_key_blocks_split_over_a_cluster(n, seg, blk):
    """n2 = 2048 / 4096 / 2056 key blocks: the score kernel spreads them over 2 or 4 clustered CTAs
    (the last case with a ragged split); estimate and select must still match the oracle."""
    cfg = CONFIGS["C1"].with_(name="wide", seq_len=n, n_q_heads=4, n_kv_heads=1, head_dim=64, segment_size=seg,
                              block_size=blk, budget_tokens=max(2 * seg, 64 * blk), n_clusters=8)
    Q, K, _ = make_qkv(cfg)
    prob = problem(cfg)
    ws = cp.alloc_workspace(prob)
    Qd, Kd = to_dev(Q, K)
    S = cp.estimate(prob, Qd, Kd, ws)
    idx, cnt = cp.select(prob, S, ws)
    S_ref = oracle_scores(cfg, Q, K)
    compare_scores(S, S_ref)
    idx_ref, cnt_ref = oracle.select(S_ref, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
    assert compare_selection(idx, cnt, idx_ref, cnt_ref, S_ref, cfg.r)[1] == 0
    # a fused second layer through the same path
    Q1, K1, _ = make_qkv(cfg, layer=1)
    S1 = cp.estimate(prob, *to_dev(Q1, K1), ws, S_prev=S)
    compare_scores(S1, oracle_scores(cfg, Q1, K1, S_prev=S_ref))


def test_host_pipelined_layer_equals_resident_path():
    from paper_2409_12490_b200.pipeline import HostPipelinedLayer
    cfg = CONFIGS["C2"].with_(name="pipe", seq_len=2048, n_q_heads=8, n_kv_heads=4, segment_size=256, block_size=64,
                              budget_tokens=512, n_clusters=16)
    Q, K, V = make_qkv(cfg)
    prob = problem(cfg)
    ws = cp.alloc_workspace(prob)
    O_res, _, _, _ = cp.prefill_layer(prob, *to_dev(Q, K, V), ws)
    hQ, hK, hV = Q.pin_memory(), K.pin_memory(), V.pin_memory()
    hO = torch.empty_like(hQ).pin_memory()
    layer = HostPipelinedLayer(prob)
    layer(hQ, hK, hV, hO)
    torch.cuda.synchronize()
    assert layer.status() == 0 and cp.device_status(ws) == 0
    assert torch.equal(hO, O_res.cpu())


@pytest.mark.parametrize("flags", [0, cp.FLAG_FORCE_SIMT])
def test_fp16_inputs_whole_path(flags):
    """fp16 is the precision the paper ran in (Section 3.1.3): same path, same oracle, same bounds."""
    cfg = CONFIGS["C2"].with_(name="half", dtype="f16", seq_len=2048, n_q_heads=4, n_kv_heads=2, segment_size=256,
                              block_size=64, budget_tokens=512, n_clusters=16)
    Q, K, V = make_qkv(cfg)
    assert Q.dtype == torch.float16
    O = full_path_vs_oracle(cfg, Q, K, V, flags=flags)
    assert O.dtype == torch.float16
    prob = problem(cfg, flags=flags)
    ws = cp.alloc_workspace(prob)
    Od = cp.dense_attention(prob, *to_dev(Q, K, V), ws)
    assert cp.device_status(ws) == 0
    O_ref, _ = oracle.dense_attention(Q, K, V, f32(1.0 / np.sqrt(cfg.head_dim)))
    assert_attention_close(Od, O_ref)


@pytest.mark.parametrize("n,seg,blk,d,dtype", [(1000, 256, 64, 128, "bf16"), (1340, 256, 32, 128, "bf16"),
                                               (777, 128, 128, 128, "f16"), (200, 256, 64, 128, "bf16"),
                                               (1000, 128, 32, 64, "f32")])
def test_sequence_lengths_that_are_not_multiples(n, seg, blk, d, dtype):
    """A shorter last segment / block (n1 = ceil(n/seg), n2 = ceil(n/blk)): every step against the oracle,
    plus the dense kernel, and nothing is written past the end of O."""
    cfg = BASE.with_(seq_len=n, segment_size=seg, block_size=blk, budget_tokens=2 * seg, head_dim=d, dtype=dtype,
                     n_q_heads=4, n_kv_heads=2)
    Q, K, V = make_qkv(cfg)
    tol = (1e-5, 1e-6) if dtype == "f32" else (TOL_BF16_MAX, TOL_BF16_MEAN)
    full_path_vs_oracle(cfg, Q, K, V, tol=tol)
    prob = problem(cfg)
    ws = cp.alloc_workspace(prob)
    Qd, Kd, Vd = to_dev(Q, K, V)
    guard = torch.full((1, cfg.n_q_heads, n + 8, d), 7.0, dtype=Q.dtype, device="cuda")   # canary rows behind every head
    Od = cp.dense_attention(prob, Qd, Kd, Vd, ws, O=guard[:, :, :n])
    assert cp.device_status(ws) == 0
    assert (guard[:, :, n:] == 7.0).all()
    O_ref, _ = oracle.dense_attention(Q, K, V, f32(1.0 / np.sqrt(d)))
    assert_attention_close(Od, O_ref, *tol)


def test_repeated_runs_are_bit_identical_and_stay_inside_their_buffers():
    """No atomics touch the outputs, so two runs must agree bit for bit; every output buffer sits
    inside a poisoned allocation whose padding must come back untouched."""
    cfg = CONFIGS["C2"].with_(name="det", seq_len=4096, n_q_heads=8, n_kv_heads=2, segment_size=512, block_size=64,
                              budget_tokens=1024, n_clusters=16)
    Q, K, V = make_qkv(cfg)
    prob = problem(cfg)
    ws = cp.alloc_workspace(prob)
    Qd, Kd, Vd = to_dev(Q, K, V)
    pad = 64

    def padded(shape, dtype, fill):
        flat = torch.full((int(np.prod(shape)) + 2 * pad,), fill, dtype=dtype, device="cuda")
        return flat, flat[pad:-pad].view(shape)

    outs = []
    for _ in range(2):
        S_raw, S = padded((1, cfg.n_q_heads, cfg.n1, cfg.n2), torch.float64, float("nan"))
        i_raw, idx = padded((1, cfg.n_q_heads, cfg.n1, cfg.budget_blocks), torch.int32, -7)
        c_raw, cnt = padded((1, cfg.n_q_heads, cfg.n1), torch.int32, -7)
        O_raw, O = padded(tuple(Qd.shape), torch.bfloat16, float("nan"))
        l_raw, lse = padded((1, cfg.n_q_heads, cfg.seq_len), torch.float32, float("nan"))
        cp.estimate(prob, Qd, Kd, ws, S_out=S)
        cp.select(prob, S, ws, idx=idx, cnt=cnt)
        cp.attention(prob, Qd, Kd, Vd, idx, cnt, ws, O=O, lse=lse)
        assert cp.device_status(ws) == 0
        for raw in (S_raw, O_raw, l_raw):
            assert torch.isnan(raw[:pad]).all() and torch.isnan(raw[-pad:]).all()
        for raw in (i_raw, c_raw):
            assert (raw[:pad] == -7).all() and (raw[-pad:] == -7).all()
        assert not torch.isnan(O.float()).any() and not torch.isnan(lse).any()
        outs.append((S.clone(), idx.clone(), cnt.clone(), O.clone(), lse.clone()))
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_output_rows_that_are_only_16_byte_aligned():
    """The tensor-core kernel stores O with 32-byte stores when every row of O starts on a 32-byte boundary and
    with 16-byte stores otherwise (the interface only asks for 16): an O whose token stride is 136 elements and
    whose base is offset by 8 elements must receive exactly the bits of the contiguous case, and the padding
    between its rows must stay untouched."""
    cfg = BASE.with_(seq_len=768)
    Q, K, V = make_qkv(cfg)
    prob = problem(cfg)
    ws = cp.alloc_workspace(prob)
    Qd, Kd, Vd = to_dev(Q, K, V)
    O_ref, S, idx, cnt = cp.prefill_layer(prob, Qd, Kd, Vd, ws)
    canary = 12345.0
    buf = torch.full((cfg.batch, cfg.n_q_heads, cfg.seq_len, cfg.head_dim + 8), canary, dtype=Qd.dtype, device=Qd.device)
    O = buf[..., 8:]
    assert O.data_ptr() % 32 == 16 and O.stride(2) % 16 == 8
    cp.attention(prob, Qd, Kd, Vd, idx, cnt, ws, O=O)
    Od = cp.dense_attention(prob, Qd, Kd, Vd, ws)
    buf2 = torch.full_like(buf, canary)
    cp.dense_attention(prob, Qd, Kd, Vd, ws, O=buf2[..., 8:])
    assert cp.device_status(ws) == 0
    assert torch.equal(O, O_ref) and torch.equal(buf2[..., 8:], Od)
    assert (buf[..., :8] == canary).all() and (buf2[..., :8] == canary).all()


def test_single_token_segments_and_blocks_give_token_wise_critical_sets():
    """segment = block = 1: the four score maps coincide, S is softmax(q K^T) per token and the selection is the
    token-wise top-k of Eq. 3 (plus the token itself).  Scores, lists and attention over the lists against the oracle."""
    cfg = BASE.with_(seq_len=640, segment_size=1, block_size=1, budget_tokens=48)
    Q, K, V = make_qkv(cfg)
    full_path_vs_oracle(cfg, Q, K, V)


def test_layer_replays_from_a_cuda_graph():
    """estimate + select + attention captured once into a CUDA graph (the library only enqueues kernels and one
    memset on the caller's stream, and encodes its tensor maps on the host) and replayed on new inputs written
    into the same buffers: every replay must equal the eager result for those inputs."""
    cfg = BASE.with_(seq_len=1536)
    prob = problem(cfg)
    ws = cp.alloc_workspace(prob)
    Q0, K0, V0 = to_dev(*make_qkv(cfg))
    Q, K, V = Q0.clone(), K0.clone(), V0.clone()
    O_eager, S_eager, idx_eager, cnt_eager = cp.prefill_layer(prob, Q, K, V, ws)
    S, idx, cnt, O = torch.empty_like(S_eager), torch.empty_like(idx_eager), torch.empty_like(cnt_eager), torch.empty_like(O_eager)
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            cp.estimate(prob, Q, K, ws, S_out=S)
            cp.select(prob, S, ws, idx=idx, cnt=cnt)
            cp.attention(prob, Q, K, V, idx, cnt, ws, O=O)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(O, O_eager) and torch.equal(idx, idx_eager) and torch.equal(S, S_eager)
    Q1, K1, V1 = to_dev(*make_qkv(cfg, layer=1))
    O1_eager, _, idx1_eager, _ = cp.prefill_layer(prob, Q1, K1, V1, ws)
    Q.copy_(Q1); K.copy_(K1); V.copy_(V1)
    graph.replay()
    torch.cuda.synchronize()
    assert cp.device_status(ws) == 0
    assert torch.equal(O, O1_eager) and torch.equal(idx, idx1_eager)
    assert not torch.equal(O1_eager, O_eager)


@pytest.mark.parametrize("flags", [0, cp.FLAG_FORCE_SIMT])
@pytest.mark.parametrize("blk,k", [(32, 14), (64, 9), (128, 6)])
def test_any_ascending_list_of_visible_blocks_is_accepted(blk, k, flags):
    """Algorithm 2 takes any index set: lists with diagonal blocks missing, out of their usual place or alone, empty
    lists (rows of zeros, lse = -inf), and lists of the usual form, mixed over the segments of one call."""
    cfg = BASE.with_(seq_len=2048, n_q_heads=4, n_kv_heads=2, segment_size=256, block_size=blk, budget_tokens=k * blk)
    Q, K, V = make_qkv(cfg)
    r, n1 = cfg.r, cfg.n1
    rng = np.random.default_rng(blk + k)
    idx = np.full((1, 4, n1, k), -1, dtype=np.int32)
    cnt = np.zeros((1, 4, n1), dtype=np.int32)
    for h in range(4):
        for j in range(n1):
            vis = (j + 1) * r
            mode = (h + j) % 5
            if mode == 0:
                sel = []                                                     # nothing listed
            elif mode == 1:
                sel = sorted(rng.choice(vis, size=min(k, vis, 1 + int(rng.integers(k))), replace=False).tolist())   # any visible blocks
            elif mode == 2:
                sel = [j * r + int(rng.integers(r))]                         # a single diagonal block
            elif mode == 3:
                past = sorted(rng.choice(max(j * r, 1), size=min(max(k - r, 0), j * r), replace=False).tolist()) if j else []
                sel = past + list(range(j * r, (j + 1) * r))                 # the usual form
                sel = sel[-k:] if len(sel) > k else sel
                sel = sorted(set(sel))
            else:
                sel = sorted(set(range(j * r, (j + 1) * r, 2)) | ({0} if j else set()))[:k]   # every other diagonal block
            cnt[0, h, j] = len(sel)
            idx[0, h, j, :len(sel)] = sel
    prob = problem(cfg, flags=flags)
    ws = cp.alloc_workspace(prob)
    Qd, Kd, Vd = to_dev(Q, K, V)
    O, lse = cp.attention(prob, Qd, Kd, Vd, torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda(), ws, want_lse=True)
    assert cp.device_status(ws) == 0
    O_ref, lse_ref = oracle.sparse_attention(Q, K, V, idx, cnt, cfg.segment_size, cfg.block_size, f32(1.0 / np.sqrt(cfg.head_dim)))
    assert_attention_close(O, O_ref)
    lse_gpu = lse.cpu().numpy()
    none = np.isneginf(lse_ref)
    assert none.any() and np.array_equal(np.isneginf(lse_gpu), none)         # rows without any visible key
    assert (O.float().cpu().numpy()[none] == 0).all()
    assert np.abs(lse_gpu[~none] - lse_ref[~none]).max() <= 2e-3
    # a list that is not ascending, or reaches a block the segment cannot see, still sets CP_ERR_BOUNDS
    for bad_val, pos in ((10 ** 6, 0), (None, 1)):
        bad = idx.copy()
        jb = n1 - 1
        full = np.arange(k, dtype=np.int32)
        bad[0, 1, jb] = full
        bad_cnt = cnt.copy(); bad_cnt[0, 1, jb] = k
        if bad_val is None:
            bad[0, 1, jb, 1] = bad[0, 1, jb, 0]                                  # duplicate entry
        else:
            bad[0, 1, jb, k - 1] = bad_val
        ws.zero_()
        cp.attention(prob, Qd, Kd, Vd, torch.from_numpy(bad).cuda(), torch.from_numpy(bad_cnt).cuda(), ws)
        assert cp.device_status(ws) == 7


@pytest.mark.parametrize("case", ["gqa2_fused", "mha_batch3", "ragged", "mask_first", "fp16_scaled", "blk32_wide"])
def test_split_score_path_on_small_ragged_and_variant_shapes(case):
    """The two-kernel score path (tensor-core log-sum-exps + exact visible logits) is chosen by size; forced here on small
    shapes so that its corner cases run against the oracle: 1, 2 and 4 heads per CTA, batch > 1, lengths that are not
    multiples of the segment / block / tile sizes, the mask-first variant, fp16 with a logit scale, layer fusion."""
    f = cp.FLAG_FORCE_SPLIT_SCORE
    if case == "gqa2_fused":
        cfg, flags = BASE.with_(seq_len=2048, n_q_heads=4, n_kv_heads=2, block_size=64, budget_tokens=512), f
    elif case == "mha_batch3":
        cfg, flags = BASE.with_(batch=3, n_q_heads=3, n_kv_heads=3, seq_len=1536, block_size=32, budget_tokens=384), f
    elif case == "ragged":
        cfg, flags = BASE.with_(seq_len=1340, n_q_heads=8, n_kv_heads=2, block_size=32, budget_tokens=320), f
    elif case == "mask_first":
        cfg, flags = BASE.with_(seq_len=2304, n_q_heads=4, n_kv_heads=1, block_size=64, budget_tokens=512), f | cp.FLAG_MASK_BEFORE_SOFTMAX
    elif case == "fp16_scaled":
        cfg, flags = BASE.with_(seq_len=2048, n_q_heads=4, n_kv_heads=2, dtype="f16", est_scale=f32(1.0 / np.sqrt(128.0))), f
    else:
        cfg, flags = BASE.with_(seq_len=9000, n_q_heads=4, n_kv_heads=1, segment_size=128, block_size=32, budget_tokens=512), f
    Q, K, _ = make_qkv(cfg)
    prob = problem(cfg, flags=flags)
    ws = cp.alloc_workspace(prob)
    Qd, Kd = to_dev(Q, K)
    mf = bool(flags & cp.FLAG_MASK_BEFORE_SOFTMAX)
    S0 = cp.estimate(prob, Qd, Kd, ws)
    S0_ref = oracle_scores(cfg, Q, K, mask_before_softmax=mf)
    compare_scores(S0, S0_ref)
    # the general kernel must agree to the last bits it can (same representatives, fp64 on both sides)
    S0_gen = cp.estimate(problem(cfg, flags=flags & ~f), Qd, Kd, ws)
    fin = torch.isfinite(S0_gen)
    assert torch.equal(torch.isneginf(S0), torch.isneginf(S0_gen)) and (S0[fin] - S0_gen[fin]).abs().max().item() <= 1e-10
    # second layer fused onto the first
    Q1, K1, _ = make_qkv(cfg, layer=1)
    S1 = cp.estimate(prob, *to_dev(Q1, K1), ws, S_prev=S0)
    compare_scores(S1, oracle_scores(cfg, Q1, K1, S_prev=S0_ref, mask_before_softmax=mf))
    idx, cnt = cp.select(prob, S1, ws)
    assert cp.device_status(ws) == 0
