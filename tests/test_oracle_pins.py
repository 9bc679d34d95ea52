"""The committed oracle against every pin (CPU only)."""
import os

import pytest

import oracle
from oracle_pins import PINS, pin_paper_constants

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def read_golden(path=GOLDEN):
    vals = {}
    for line in open(path):
        line = line.split("#", 1)[0].strip()
        if line:
            name, val = line.split("=")
            vals[name.strip()] = float(val)
    return vals


@pytest.mark.parametrize("pin", PINS, ids=[p.__name__ for p in PINS])
def test_pin(pin):
    pin(oracle.load())


def test_paper_constants():
    g = read_golden()
    assert g["eps"] == 1e-4
    pin_paper_constants(oracle.load(), g)


def test_invalid_arguments_are_rejected():
    import numpy as np
    z = np.zeros((1, 1, 2, 4))
    with pytest.raises(ValueError):
        oracle.forward(z, z, z, 0.0, in_dtype=oracle.F64)          # lambda must be > 0 without A0
    with pytest.raises(ValueError):
        oracle.forward(z, z, z, 1.0, in_dtype=oracle.F64, eps=0.0)
