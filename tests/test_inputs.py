"""The seeded generator: determinism, shapes, dtype, and the two structural properties it exists for."""
import numpy as np
import torch

from paper_2409_12490_b200 import CONFIGS
from paper_2409_12490_b200.inputs import make_qkv, make_uniform_qkv


def test_deterministic_and_shaped():
    cfg = CONFIGS["C1"]
    Q, K, V = make_qkv(cfg)
    Q2, K2, V2 = make_qkv(cfg, threads=2)
    assert torch.equal(Q, Q2) and torch.equal(K, K2) and torch.equal(V, V2)
    assert Q.shape == (1, 4, 1024, 64) and K.shape == (1, 2, 1024, 64) and Q.dtype == torch.float32
    Q3, _, _ = make_qkv(cfg, layer=1)
    assert not torch.equal(Q, Q3)
    assert 0.7 < Q.std() < 1.5 and 0.7 < K.std() < 1.5        # unit scale


def test_bf16_storage():
    cfg = CONFIGS["C2"].with_(seq_len=1024, n_q_heads=4, n_kv_heads=2)
    Q, K, V = make_qkv(cfg)
    assert Q.dtype == torch.bfloat16 and V.shape == (1, 2, 1024, 128)


def test_locality_of_token_wise_critical_sets():
    """Neighbouring queries share most of their top keys, distant ones do not (Section 2.2)."""
    cfg = CONFIGS["C1"]
    Q, K, _ = make_qkv(cfg)
    q, k = Q[0, 0].double().numpy(), K[0, 0].double().numpy()
    kk = 64

    def top(t):
        s = k[: t + 1] @ q[t]
        return set(np.argsort(-s)[:kk].tolist())

    near = len(top(900) & top(901)) / kk
    far = len(top(1000) & top(300)) / kk
    assert near > 0.8 and far < near


def test_uniform_generator():
    Q, K, V = make_uniform_qkv(2, 4, 2, 64, 16, dtype="f32", seed=3)
    assert Q.shape == (2, 4, 64, 16) and K.shape == (2, 2, 64, 16)
