"""Writes oracle_small_case.txt: results of the CPU oracle on one small seeded case.

The stored numbers come from `oracle/` alone (this script imports nothing else of the method) and guard the
oracle against unintended changes: a later edit of its arithmetic must change this file on purpose.  They are a
regression record, not a pin -- the pins are the closed forms, brute-force checks and library special cases in
tests/test_oracle_*.py.

Case: 2 query heads / 1 KV head, 256 tokens, head_dim 64, segment 64, block 16, budget 128 tokens (8 blocks: the 4 diagonal ones and 4 past ones),
two layers (the second fused onto the first with alpha = 0.25, Algorithm 1 line 14), inputs from the seeded generator.
Run:  python tests/golden/make_oracle_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2409_12490_b200.configs import CONFIGS  # noqa: E402
from paper_2409_12490_b200.inputs import make_qkv  # noqa: E402

CASE = dict(seq_len=256, n_q_heads=2, n_kv_heads=1, head_dim=64, segment_size=64, block_size=16, budget_tokens=128,
            n_clusters=4, dtype="f32")


def compute():
    cfg = CONFIGS["C1"].with_(name="golden", **CASE)
    out = {}
    S_prev = None
    for layer in (0, 1):
        Q, K, V = make_qkv(cfg, layer=layer)
        S = oracle.estimate(Q, K, cfg.segment_size, cfg.block_size, est_scale=1.0, alpha=0.25, S_prev=S_prev)
        idx, cnt = oracle.select(S, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
        O, lse = oracle.sparse_attention(Q, K, V, idx, cnt, cfg.segment_size, cfg.block_size, 1.0 / np.sqrt(cfg.head_dim))
        out[f"layer{layer}.lnS.row"] = S[0, 1, 3, :12]                      # head 1, segment 3, first 12 blocks
        out[f"layer{layer}.lnS.sum_finite"] = np.array([S[np.isfinite(S)].sum()])
        out[f"layer{layer}.idx.seg3"] = idx[0, :, 3].astype(np.float64).ravel()
        out[f"layer{layer}.cnt"] = cnt[0].astype(np.float64).ravel()
        out[f"layer{layer}.O.row200"] = O[0, 0, 200, :8]
        out[f"layer{layer}.lse"] = lse[0, 1, [0, 63, 64, 255]]
        S_prev = S
    return out


def main():
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_small_case.txt")
    with open(path, "w") as fh:
        fh.write("# Written by make_oracle_golden.py from oracle/ alone (regression record of the oracle, see that script).\n")
        for key, val in compute().items():
            fh.write(key + " " + " ".join(float(v).hex() for v in np.asarray(val, dtype=np.float64).ravel()) + "\n")
    print("wrote", path)


if __name__ == "__main__":
    main()
