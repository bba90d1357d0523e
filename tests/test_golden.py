"""The stored generator fixtures (written by tests/golden/make_golden.py from the oracle) still hold."""
import os

import numpy as np

from oracle import flora_oracle as orc

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _lines(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


def test_projection_fixture():
    rows = [[int(x, 16) for x in ln.split()] for ln in _lines("projection_seed42_r8_m24.txt")]
    A = orc.materialize_A(42, 8, 24)
    assert np.array_equal(A.view(np.uint32), np.array(rows, dtype=np.uint32))


def test_philox_fixture():
    for ln in _lines("philox_blocks.txt"):
        lhs, rhs = ln.split("->")
        v = [int(x, 16) for x in lhs.split()]
        assert [int(x) for x in orc.philox4x32_10(v[:4], v[4:])] == [int(x, 16) for x in rhs.split()]
