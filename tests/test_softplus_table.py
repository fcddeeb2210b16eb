"""The score kernel's table for ln(1 + exp(-x)) (host-side check of the generated coefficients).

The CUDA kernel evaluates ln(e^a + e^b) = max + f(|a - b|) with piecewise degree-11 polynomials whose
coefficients are compiled in from csrc/softplus_table.inc.  This test reads that file as text and checks the
polynomials against the definition in extended precision, so a stale or corrupted table fails here, on CPU."""
import os
import re

import numpy as np

import paper_2409_12490_b200

INC = os.path.join(os.path.dirname(paper_2409_12490_b200.__file__), "csrc", "softplus_table.inc")


def load_table():
    rows = []
    for line in open(INC):
        if line.lstrip().startswith("//"):
            continue
        vals = [float.fromhex(v) for v in re.findall(r"-?0x[0-9a-f.]+p[-+]?\d+", line)]
        if vals:
            rows.append(vals)
    return np.array(rows)


def evaluate(tab, x):
    i = np.minimum((x * 2.0).astype(int), len(tab) - 1)
    t = (x - (0.5 * i + 0.25)) * 4.0
    p = np.zeros_like(x)
    for k in range(tab.shape[1] - 1, -1, -1):
        p = p * t + tab[i, k]
    return p


def test_table_shape_and_accuracy():
    tab = load_table()
    assert tab.shape == (80, 12)
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.uniform(0.0, 40.0, 200000), np.arange(0, 80) * 0.5, np.nextafter(np.arange(1, 81) * 0.5, 0.0)])
    exact = np.log1p(np.exp(-x.astype(np.longdouble)))
    err = np.abs(evaluate(tab, x).astype(np.longdouble) - exact)
    assert float(err.max()) < 2e-15
    assert abs(evaluate(tab, np.array([0.0]))[0] - np.log(2.0)) < 1e-15


def test_pieces_join_and_the_cut_at_40_is_below_rounding():
    tab = load_table()
    edges = np.arange(1, 80) * 0.5
    left = evaluate(tab, np.nextafter(edges, 0.0))
    right = evaluate(tab, edges)
    assert np.abs(left - right).max() < 2e-15
    assert np.log1p(np.exp(-40.0)) < 5e-18          # what the kernel drops beyond the table
