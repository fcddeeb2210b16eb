"""critiprefill_estimate_static -- the entry point for callers that cannot allocate device memory
(its scratch is a fixed array inside the library) -- must give what critiprefill_estimate gives,
and what the fp64 oracle gives.

Collected last on purpose: the array is shared by every call in the process, so this runs after
all other tests and must also pass alone in a fresh process.
"""
import ctypes

import pytest
import torch

from paper_2409_12490_b200 import CONFIGS
from paper_2409_12490_b200 import binding as cp
from paper_2409_12490_b200.inputs import make_qkv

from helpers import compare_scores, oracle_scores

pytestmark = pytest.mark.gpu

BIG = CONFIGS["C2"].with_(name="no_alloc_big", seq_len=4096, n_q_heads=8, n_kv_heads=2, segment_size=256,
                          block_size=32, budget_tokens=512, n_clusters=16)
SMALL = CONFIGS["C2"].with_(name="no_alloc", seq_len=2048, n_q_heads=4, n_kv_heads=2, segment_size=256,
                            block_size=64, budget_tokens=512, n_clusters=16)


def test_static_scratch_estimate_matches_workspace_estimate_and_oracle():
    """Calls in a row on one device share the array: a larger problem first, so that the smaller ones after it
    find its leftovers beyond (and under) their own summaries; the second small call fuses the first one's score."""
    prev, prev_ref = None, None
    for cfg, layer in ((BIG, 0), (SMALL, 0), (SMALL, 1)):
        prob = cp.Problem.from_config(cfg)
        assert cp.workspace_bytes(prob) <= cp.static_scratch_bytes()
        ws = cp.alloc_workspace(prob)
        Q, K, _ = make_qkv(cfg, layer=layer)
        Qd, Kd = Q.cuda(), K.cuda()
        fuse = cfg is SMALL and layer == 1
        want = cp.estimate(prob, Qd, Kd, ws, S_prev=prev if fuse else None)
        S_out = torch.full_like(want, float("nan"))
        got = cp.estimate_static(prob, Qd, Kd, S_prev=prev if fuse else None, S_out=S_out)
        torch.cuda.synchronize()
        assert torch.equal(got, want)                      # same kernels on the same summaries: bit-identical
        S_ref = oracle_scores(cfg, Q, K, S_prev=prev_ref if fuse else None)
        compare_scores(got, S_ref)                         # and within 1e-9 of the oracle's ln S
        prev, prev_ref = (want, S_ref) if cfg is SMALL else (None, None)


def test_static_scratch_rejects_problems_beyond_its_size():
    big = cp.Problem(4, 32, 8, 131072, 128, 1024, 128, 32)      # summaries of 4 batch items: > 8 MiB
    assert cp.workspace_bytes(big) > cp.static_scratch_bytes()
    Q = torch.empty(16, dtype=torch.bfloat16, device="cuda")
    S = torch.empty(16, dtype=torch.float64, device="cuda")
    p = big.params()
    rc = cp.load_library().critiprefill_estimate_static(ctypes.byref(p), Q.data_ptr(), Q.data_ptr(), None,
                                                        S.data_ptr(), None)
    assert rc == 8 and "static" in cp.status_string(rc)
    # the paper's own operating point at 128K tokens (segment 512, block 32) needs about 20 MB: also refused
    paper = cp.Problem.from_config(CONFIGS["paper_128k"])
    assert cp.workspace_bytes(paper) > cp.static_scratch_bytes()
