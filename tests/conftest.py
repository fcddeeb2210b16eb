import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_terminal_summary(terminalreporter):
    """Every attention comparison of the run: plain max abs error, mean, and how many outputs were judged
    by the relative bound (|O| >= 2)."""
    try:
        from helpers import PARITY_RECORDS
    except Exception:  # pragma: no cover
        return
    if not PARITY_RECORDS:
        return
    tr = terminalreporter
    tr.write_sep("-", "attention parity records (GPU vs fp64 oracle)")
    for r in PARITY_RECORDS:
        tr.write_line(f"{r['case']}: elements {r['elements']}, max abs {r['max_abs_err']:.3e}, mean abs {r['mean_abs_err']:.3e}, "
                      f"n_big {r['n_big']}" + (f", max rel (|O|>=2) {r['max_rel_err_big']:.3e}" if r.get("max_rel_err_big") is not None else ""))
    worst = max(r["max_abs_err"] for r in PARITY_RECORDS)
    tr.write_line(f"worst plain max abs err over {len(PARITY_RECORDS)} comparisons: {worst:.3e}; "
                  f"comparisons with n_big > 0: {sum(1 for r in PARITY_RECORDS if r['n_big'])}")
