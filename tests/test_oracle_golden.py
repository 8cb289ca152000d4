"""The oracle against the closed-form fixture in tests/golden/closed_forms.txt."""
import math
import os

import numpy as np
import pytest

import oracle

_F = os.path.join(os.path.dirname(__file__), "golden", "closed_forms.txt")


def _cases():
    out = []
    with open(_F) as f:
        for line in f:
            line = line.split("#")[0].split()
            if line:
                out.append((line[0], int(line[1]), int(line[2]), int(line[3]), float(line[4]), float(line[5])))
    return out


@pytest.mark.parametrize("kind,V,arg,bits,H,c", _cases())
def test_closed_form_case(kind, V, arg, bits, H, c):
    x = np.full(V, -np.inf, np.float32)
    if kind == "uniform":
        x[:] = 0.5
    elif kind == "onehot":
        x[V // 3] = 4.0
    elif kind == "twopoint_ln3":
        # ln 3 is not a float32; the tolerance below covers its rounding (relative 3e-8)
        x[5], x[60] = np.float32(math.log(3.0)), 0.0
    elif kind == "subset":
        x[np.arange(arg) * 7] = -1.0
    r = oracle.signals(oracle.Batch(draft=x[None, None, :], entropy_in_bits=bool(bits)))
    # sequential double sums over V terms carry about V * 1e-16 of rounding
    tol = 1e-7 if kind == "twopoint_ln3" else max(1e-13, V * 2e-15)
    assert r["H"][0, 0] == pytest.approx(H, rel=tol, abs=1e-15)
    assert r["C"][0, 0] == pytest.approx(c, rel=tol)
