"""critiprefill_estimate_static -- the entry point for callers that cannot allocate device memory
(its scratch is a fixed array inside the library) -- must give what critiprefill_estimate gives.

Collected last on purpose: the array is shared by every call in the process, so this runs after
all other tests and must also pass alone in a fresh process.
"""
import pytest
import torch

from paper_2409_12490_b200 import CONFIGS
from paper_2409_12490_b200 import binding as cp
from paper_2409_12490_b200.inputs import make_qkv

pytestmark = pytest.mark.gpu


def test_static_scratch_estimate_matches_workspace_estimate_twice():
    cfg = CONFIGS["C2"].with_(name="no_alloc", seq_len=2048, n_q_heads=4, n_kv_heads=2, segment_size=256,
                              block_size=64, budget_tokens=512, n_clusters=16)
    prob = cp.Problem.from_config(cfg)
    assert cp.workspace_bytes(prob) <= cp.static_scratch_bytes()
    ws = cp.alloc_workspace(prob)
    prev = None
    # two calls in a row on different inputs: the second sees the first one's leftovers in the array
    for layer in (0, 1):
        Q, K, _ = make_qkv(cfg, layer=layer)
        Q, K = Q.cuda(), K.cuda()
        want = cp.estimate(prob, Q, K, ws, S_prev=prev)
        S_out = torch.full_like(want, float("nan"))
        got = cp.estimate_static(prob, Q, K, S_prev=prev, S_out=S_out)
        torch.cuda.synchronize()
        fin = torch.isfinite(want)
        assert torch.equal(torch.isneginf(got), torch.isneginf(want))
        assert (got[fin] - want[fin]).abs().max().item() <= 1e-9
        prev = want


def test_static_scratch_rejects_problems_beyond_its_size():
    big = cp.Problem(4, 32, 8, 131072, 128, 1024, 128, 32)      # summaries of 4 batch items: > 8 MiB
    assert cp.workspace_bytes(big) > cp.static_scratch_bytes()
    Q = torch.empty(16, dtype=torch.bfloat16, device="cuda")
    S = torch.empty(16, dtype=torch.float64, device="cuda")
    p = big.params()
    import ctypes
    rc = cp.load_library().critiprefill_estimate_static(ctypes.byref(p), Q.data_ptr(), Q.data_ptr(), None,
                                                        S.data_ptr(), None)
    assert rc == 8 and "static" in cp.status_string(rc)
