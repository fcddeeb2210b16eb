"""The oracle's results on one small seeded case against the record in tests/golden/oracle_small_case.txt
(written by tests/golden/make_oracle_golden.py from oracle/ alone).  A regression guard: the oracle is what every
CUDA parity test trusts, so a change of its arithmetic has to show up here and be made on purpose."""
import importlib.util
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))


def _load_script():
    spec = importlib.util.spec_from_file_location("make_oracle_golden", os.path.join(HERE, "golden", "make_oracle_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def _read_record():
    rec = {}
    for line in open(os.path.join(HERE, "golden", "oracle_small_case.txt")):
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        rec[key] = np.array([float.fromhex(v) for v in vals])
    return rec


def test_oracle_reproduces_its_record():
    now = _load_script().compute()
    rec = _read_record()
    assert set(now) == set(rec)
    for key, val in now.items():
        val = np.asarray(val, dtype=np.float64).ravel()
        if ".idx." in key or key.endswith(".cnt"):
            assert np.array_equal(val, rec[key]), key
        else:
            assert np.allclose(val, rec[key], rtol=1e-12, atol=1e-13), key


def test_record_is_not_trivial():
    rec = _read_record()
    idx = rec["layer1.idx.seg3"].reshape(2, 8)
    assert (idx[:, 4:] == np.array([12, 13, 14, 15])).all()          # diagonal blocks of segment 3 (r = 4)
    assert (idx[:, :4] < 12).all() and (np.diff(idx[:, :4], axis=1) > 0).all()
    assert not np.array_equal(rec["layer0.lnS.row"], rec["layer1.lnS.row"])
