"""Packed batches of sequences of different lengths through the C ABI against the fp64 oracle (one problem per
sequence: Algorithms 1 and 2 counted from each sequence's first token)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_12490_b200 import binding as cp
from paper_2409_12490_b200.inputs import make_uniform_qkv

from helpers import assert_attention_close, compare_scores, compare_selection, f32

pytestmark = pytest.mark.gpu

HQ, HKV, D = 8, 2, 128


def packed_inputs(lens, dtype, seed):
    """Q [Hq,total,d], K, V [Hkv,total,d] as views of [total, heads, d] storage (the layout serving stacks pack in)."""
    total = sum(lens)
    Q, K, V = make_uniform_qkv(1, HQ, HKV, total, D, dtype=dtype, seed=seed)
    pack = lambda t: t[0].permute(1, 0, 2).contiguous().cuda().permute(1, 0, 2)
    return pack(Q), pack(K), pack(V), [0] + np.cumsum(lens).tolist()


@pytest.mark.parametrize("lens,seg,blk,k,dtype", [
    ([1536, 1000, 2304, 300, 128], 256, 32, 12, "bf16"),     # ragged tails, a sequence shorter than a segment
    ([2048, 700], 512, 64, 16, "f16"),
    ([640, 96, 1111], 128, 32, 8, "f32"),                     # SIMT path; a sequence shorter than a query tile
])
def test_varlen_matches_oracle_per_sequence(lens, seg, blk, k, dtype):
    Q, K, V, cu = packed_inputs(lens, dtype, seed=11)
    tdt = {"bf16": torch.bfloat16, "f16": torch.float16, "f32": torch.float32}[dtype]
    prob = cp.Problem(1, HQ, HKV, max(lens), D, seg, blk, k, tdt)
    ws = cp.alloc_workspace(prob)
    O, S, idx, cnt, S_flat, lse = cp.prefill_varlen(prob, cu, Q, K, V, ws, want_lse=True)
    assert cp.device_status(ws) == cp.CP_OK
    sm = f32(1.0 / np.sqrt(D))
    S_ref, idx_ref, cnt_ref, _, _ = oracle.prefill_varlen(Q, K, V, cu, seg, blk, k, sm, est_scale=f32(prob.est_scale))
    lse_all = lse.view(-1)
    for i, (lo, hi) in enumerate(zip(cu[:-1], cu[1:])):
        compare_scores(S[i][None], S_ref[i][None])
        excused, unexcused = compare_selection(idx[i][None], cnt[i][None], idx_ref[i][None], cnt_ref[i][None],
                                               S_ref[i][None], seg // blk)
        assert unexcused == 0
        # attention against the oracle on the lists the GPU selected (identical unless a near-tie was excused)
        q, kk, vv = Q[None, :, lo:hi], K[None, :, lo:hi], V[None, :, lo:hi]
        O_ref, lse_ref = oracle.sparse_attention(q, kk, vv, idx[i][None].cpu().numpy(), cnt[i][None].cpu().numpy(),
                                                 seg, blk, sm)
        if dtype == "f32":
            assert np.abs(O[:, lo:hi].float().cpu().numpy() - O_ref[0]).max() <= 1e-5
        else:
            assert_attention_close(O[None, :, lo:hi], O_ref, label="test_varlen_matches_oracle_per_sequence")
        got = lse_all[HQ * lo:HQ * hi].view(HQ, hi - lo).cpu().numpy()
        assert np.abs(got - lse_ref[0]).max() <= 2e-3


def test_varlen_equals_single_sequence_calls_bit_for_bit_and_chains_layers():
    lens, seg, blk, k = [1280, 900, 2048], 256, 32, 12
    Q, K, V, cu = packed_inputs(lens, "bf16", seed=5)
    Q1, K1, V1, _ = packed_inputs(lens, "bf16", seed=6)
    prob = cp.Problem(1, HQ, HKV, max(lens), D, seg, blk, k, torch.bfloat16, alpha=0.25)
    ws = cp.alloc_workspace(prob)
    O0, S0, idx0, cnt0, S0_flat = cp.prefill_varlen(prob, cu, Q, K, V, ws)
    O1, S1, idx1, cnt1, _ = cp.prefill_varlen(prob, cu, Q1, K1, V1, ws, S_prev=S0_flat)
    for i, (lo, hi) in enumerate(zip(cu[:-1], cu[1:])):
        one = cp.Problem(1, HQ, HKV, hi - lo, D, seg, blk, k, torch.bfloat16, alpha=0.25)
        ws1 = cp.alloc_workspace(one)
        q, kk, vv = (t[None, :, lo:hi].contiguous() for t in (Q, K, V))
        Oa, Sa, ia, ca = cp.prefill_layer(one, q, kk, vv, ws1)
        assert torch.equal(Sa[0], S0[i]) and torch.equal(ia[0], idx0[i]) and torch.equal(ca[0], cnt0[i])
        assert torch.equal(Oa[0], O0[:, lo:hi])
        q, kk, vv = (t[None, :, lo:hi].contiguous() for t in (Q1, K1, V1))
        Ob, Sb, ib, cb = cp.prefill_layer(one, q, kk, vv, ws1, S_prev=Sa)
        assert torch.equal(Sb[0], S1[i]) and torch.equal(ib[0], idx1[i]) and torch.equal(Ob[0], O1[:, lo:hi])
    assert cp.device_status(ws) == cp.CP_OK


def test_varlen_rejects_bad_arguments():
    lens = [512, 256]
    Q, K, V, cu = packed_inputs(lens, "bf16", seed=1)
    prob = cp.Problem(1, HQ, HKV, 512, D, 256, 32, 12, torch.bfloat16)
    ws = cp.alloc_workspace(prob)
    with pytest.raises(cp.CritiPrefillError):
        cp.prefill_varlen(prob, [0, 512, 512], Q, K, V, ws)                      # an empty sequence
    short = cp.Problem(1, HQ, HKV, 256, D, 256, 32, 12, torch.bfloat16)           # seq_len below the longest sequence
    with pytest.raises(cp.CritiPrefillError):
        cp.prefill_varlen(short, cu, Q, K, V, cp.alloc_workspace(short))
