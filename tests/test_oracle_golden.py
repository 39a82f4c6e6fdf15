"""The oracle against its own stored results (tests/golden/tiny_path_oracle.txt, written by
tests/golden/make_golden.py from oracle/ alone): a change to the oracle's arithmetic shows up here and has to
be justified by the paper before the file is rewritten."""
import importlib.util
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))


def _load_maker():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    m = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(m)
    return m


def test_oracle_reproduces_its_stored_results():
    stored = {}
    with open(os.path.join(HERE, "golden", "tiny_path_oracle.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, v = line.rstrip("\n").split("\t")
            stored[name] = float(v)
    got = dict(_load_maker().entries())
    assert set(got) == set(stored)
    for name, v in got.items():
        assert np.isclose(v, stored[name], rtol=1e-11, atol=1e-13), (name, v, stored[name])
