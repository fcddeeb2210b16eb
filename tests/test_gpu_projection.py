"""The fused projection (Eq. 1 + rotary embedding + representatives of Algorithm 1 in its epilogue) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_12490_b200 import binding as cp

from helpers import compare_scores, f32

pytestmark = pytest.mark.gpu


def _inputs(B, n, d_model, Hq, Hkv, d, dtype, seed):
    rng = np.random.default_rng(seed)
    tdt = {"bf16": torch.bfloat16, "f16": torch.float16}[dtype]
    X = torch.from_numpy(rng.standard_normal((B, n, d_model), dtype=np.float32)).to(tdt)
    s = 1.0 / np.sqrt(d_model)                                   # unit-scale Q and K, as the attention inputs elsewhere
    Wq = torch.from_numpy((s * rng.standard_normal((Hq * d, d_model), dtype=np.float32))).to(tdt)
    Wk = torch.from_numpy((s * rng.standard_normal((Hkv * d, d_model), dtype=np.float32))).to(tdt)
    return X, Wq, Wk


@pytest.mark.parametrize("B,n,d_model,Hq,Hkv,seg,blk,dtype,rot", [
    (1, 1024, 256, 4, 2, 256, 64, "bf16", True),
    (2, 640, 192, 2, 1, 128, 32, "bf16", True),          # batch 2, a segment count that leaves CTAs with several units
    (1, 1000, 128, 4, 4, 256, 128, "bf16", True),        # ragged length: last tile, last block and last segment are short
    (1, 512, 320, 2, 2, 512, 64, "f16", False),          # fp16, no rotation (Eq. 1 as printed)
])
def test_projection_summaries_and_estimate(B, n, d_model, Hq, Hkv, seg, blk, dtype, rot):
    d = 128
    X, Wq, Wk = _inputs(B, n, d_model, Hq, Hkv, d, dtype, seed=n + d_model)
    cos, sin = oracle.rope_tables(n, d) if rot else (None, None)
    k = max(seg // blk, min(-(-n // blk), (seg + 256) // blk))
    tdt = X.dtype
    prob = cp.Problem(B, Hq, Hkv, n, d, seg, blk, k, dtype=tdt)
    ws = cp.alloc_workspace(prob)
    cd = torch.from_numpy(cos).cuda() if rot else None
    sd = torch.from_numpy(sin).cuda() if rot else None
    Q, K = cp.project_qk(prob, X.cuda(), Wq.cuda(), Wk.cuda(), ws, rope_cos=cd, rope_sin=sd)
    assert cp.device_status(ws) == 0
    # (1) the projection itself: fp64 reference on the same input bits; one rounding to the 16-bit type + fp32 accumulation
    Q_ref, K_ref = oracle.project_qk(X, Wq, Wk, d, cos, sin)
    ulp = 2.0 ** -8 if dtype == "bf16" else 2.0 ** -11
    for got, ref in ((Q, Q_ref), (K, K_ref)):
        err = np.abs(got.float().cpu().numpy().astype(np.float64) - ref)
        assert (err <= ulp * np.abs(ref) + 2e-5 * np.sqrt(d_model)).all(), err.max()
    # (2) the representatives left in the workspace are those of the stored bits: the estimate that trusts them equals
    #     the estimate that recomputes them from Q and K, bit for bit, and both match the oracle on those bits
    ready = cp.Problem(B, Hq, Hkv, n, d, seg, blk, k, dtype=tdt, flags=cp.FLAG_SUMMARIES_READY)
    S_fused = cp.estimate(ready, Q, K, ws)
    torch.cuda.synchronize()
    ws2 = cp.alloc_workspace(prob)
    S_plain = cp.estimate(prob, Q, K, ws2)
    assert torch.equal(S_fused, S_plain)
    S_ref = oracle.estimate(Q.cpu(), K.cpu(), seg, blk, est_scale=1.0)
    compare_scores(S_fused, S_ref)
    # (3) and the summaries themselves, read back from the workspace layout [status 256 B][Qmax][Qmin][Kmax][Kmin]
    Qmax, Qmin, Kmax, Kmin = oracle.summaries(Q.cpu(), K.cpu(), seg, blk)
    n1, n2 = -(-n // seg), -(-n // blk)
    up = lambda x: (x + 255) // 256 * 256
    qs, ks = up(B * Hq * n1 * d * 2), up(B * Hkv * n2 * d * 2)
    raw = ws.cpu()
    def view(off, count, shape):
        return raw[off:off + count * 2].view(tdt).float().numpy().reshape(shape).astype(np.float64)
    assert np.array_equal(view(256, B * Hq * n1 * d, (B, Hq, n1, d)), Qmax)
    assert np.array_equal(view(256 + qs, B * Hq * n1 * d, (B, Hq, n1, d)), Qmin)
    assert np.array_equal(view(256 + 2 * qs, B * Hkv * n2 * d, (B, Hkv, n2, d)), Kmax)
    assert np.array_equal(view(256 + 2 * qs + ks, B * Hkv * n2 * d, (B, Hkv, n2, d)), Kmin)


def test_projection_rejects_shapes_outside_its_envelope():
    prob = cp.Problem(1, 2, 1, 1024, 128, 256, 64, 8)
    ws = cp.alloc_workspace(prob)
    X = torch.zeros((1, 1024, 100), dtype=torch.bfloat16, device="cuda")          # d_model not a multiple of 64
    W = torch.zeros((256, 100), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(cp.CritiPrefillError) as e:
        cp.project_qk(prob, X, W, W[:128].contiguous(), ws)
    assert e.value.status == 3


@pytest.mark.parametrize("B,n,d_model,Hq,Hkv,seg,blk,dtype", [
    (1, 1024, 256, 4, 2, 256, 64, "bf16"),
    (2, 1000, 192, 2, 1, 128, 32, "f16"),                # batch 2, ragged length
])
def test_value_projection_in_the_same_launch(B, n, d_model, Hq, Hkv, seg, blk, dtype):
    d = 128
    X, Wq, Wk = _inputs(B, n, d_model, Hq, Hkv, d, dtype, seed=7)
    _, _, Wv = _inputs(B, n, d_model, Hq, Hkv, d, dtype, seed=8)
    cos, sin = oracle.rope_tables(n, d)
    prob = cp.Problem(B, Hq, Hkv, n, d, seg, blk, max(seg // blk, 8), dtype=X.dtype)
    ws, ws2 = cp.alloc_workspace(prob), cp.alloc_workspace(prob)
    cd, sd = torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda()
    Q, K, V = cp.project_qkv(prob, X.cuda(), Wq.cuda(), Wk.cuda(), Wv.cuda(), ws, rope_cos=cd, rope_sin=sd)
    assert cp.device_status(ws) == 0
    # V = W_V X (Eq. 1), unrotated: fp64 reference on the same bits, one rounding + fp32 accumulation
    V_ref = oracle.project_v(X, Wv, d)
    ulp = 2.0 ** -8 if dtype == "bf16" else 2.0 ** -11
    err = np.abs(V.float().cpu().numpy().astype(np.float64) - V_ref)
    assert (err <= ulp * np.abs(V_ref) + 2e-5 * np.sqrt(d_model)).all(), err.max()
    # Q, K and the representatives are what the two-matrix call produces, bit for bit
    Q2, K2 = cp.project_qk(prob, X.cuda(), Wq.cuda(), Wk.cuda(), ws2, rope_cos=cd, rope_sin=sd)
    assert torch.equal(Q, Q2) and torch.equal(K, K2)
    torch.cuda.synchronize()
    assert torch.equal(ws[256:], ws2[256:])
