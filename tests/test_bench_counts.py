"""The roofline numerator: bench.flop_counts must equal an explicit enumeration of the (query tile,
KV tile) pairs the sparse kernel issues, and the analytic totals (full listed tiles, causal-useful, dense)."""
import importlib.util
import os

from paper_2409_12490_b200 import CONFIGS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
spec = importlib.util.spec_from_file_location("bench", os.path.join(ROOT, "bench.py"))
bench = importlib.util.module_from_spec(spec)
spec.loader.exec_module(bench)


def enumerate_tiles(cfg):
    """Tile pairs per the kernel's unit rule: tile i of a segment streams the gathered past tiles,
    then the segment's own tiles 0..i."""
    r, k = cfg.r, cfg.budget_blocks
    pairs = 0
    for j in range(cfg.n1):
        cnt = min(k, (j + 1) * r)
        n_past_tiles = -(-(cnt - r) * cfg.block_size // 128)
        q_tiles = cfg.segment_size // 128
        for unit in range((q_tiles + 1) // 2):
            n_a = n_past_tiles + 2 * unit + 1
            pairs += n_a
            if 2 * unit + 1 < q_tiles:
                pairs += n_a + 1
    return pairs * cfg.n_q_heads * cfg.batch


def test_executed_flops_match_tile_enumeration():
    for name in ("C2", "C3", "C4", "C5", "paper_128k"):
        cfg = CONFIGS[name]
        fl = bench.flop_counts(cfg)
        assert fl["executed"] == enumerate_tiles(cfg) * 4 * 128 * 128 * cfg.head_dim
        assert fl["useful"] <= fl["executed"] <= fl["listed_full_tiles"]


def test_analytic_totals_at_c4():
    fl = bench.flop_counts(CONFIGS["C4"])
    assert abs(fl["listed_full_tiles"] / 1e12 - 8.693) < 1e-3      # every listed block against its whole segment
    assert abs(fl["useful"] / 1e12 - 7.595) < 1e-3
    assert abs(fl["dense"] / 1e12 - 140.74) < 1e-2
    assert abs(fl["executed"] / 1e12 - 7.731) < 1e-3
