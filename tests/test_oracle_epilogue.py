"""Pins for the oracle's element-wise MLP step (SiLU(gate) * up, one rounding to FP16, thresholded list).

None of the expectations below comes from the functions under test: closed forms of the logistic function,
values of FP16 rounding worked out by hand from the format (10 fraction bits, ties to even), and a
brute-force list.
"""
import math

import numpy as np
import pytest

from oracle import celty_oracle as orc


def test_silu_closed_forms():
    assert orc.silu(0.0) == 0.0
    # SiLU(v) - SiLU(-v) = v (sigmoid(v) + sigmoid(-v) = 1)
    v = np.array([1e-9, 0.3, 1.0, 2.5, 7.0, 30.0, 700.0])
    assert np.allclose(orc.silu(v) - orc.silu(-v), v, rtol=1e-15, atol=0)
    # far out: the identity on the right, zero on the left (and no overflow warnings turned into NaN)
    assert orc.silu(800.0) == 800.0 and orc.silu(-800.0) == 0.0 and not np.isnan(orc.silu(-1e5))
    # slope one half at the origin
    assert abs(orc.silu(1e-8) / 1e-8 - 0.5) < 1e-7
    # the minimum: where 1 + v (1 - sigmoid(v)) = 0 the value is v + 1 (about -0.27846 at -1.27846)
    lo, hi = -2.0, -1.0
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        g = 1.0 + mid * (1.0 - 1.0 / (1.0 + math.exp(-mid)))
        lo, hi = (mid, hi) if g < 0 else (lo, mid)
    vmin = 0.5 * (lo + hi)
    assert abs(vmin + 1.2784645427610738) < 1e-12
    assert abs(float(orc.silu(vmin)) - (vmin + 1.0)) < 1e-15
    assert float(orc.silu(vmin)) < float(orc.silu(vmin - 1e-3)) and float(orc.silu(vmin)) < float(orc.silu(vmin + 1e-3))
    # against a literal evaluation with the math module
    for t in (-5.0, -0.7, 0.2, 3.3):
        assert float(orc.silu(t)) == t / (1.0 + math.exp(-t))


def test_swiglu_is_the_product():
    g = np.array([0.0, 1.0, -1.0, 2.0])
    u = np.array([5.0, 2.0, 4.0, -0.5])
    want = [0.0, 2.0 / (1.0 + math.exp(-1.0)), -4.0 / (1.0 + math.exp(1.0)), -1.0 / (1.0 + math.exp(-2.0))]
    assert np.allclose(orc.swiglu(g, u), want, rtol=1e-15, atol=0)


@pytest.mark.parametrize("value,bits", [
    (1.0, 0x3C00),
    (1.0 + 2.0 ** -11, 0x3C00),            # half way between 1 and 1 + 2^-10: the even neighbour is 1
    (1.0 + 3 * 2.0 ** -11, 0x3C02),        # half way between 0x3C01 and 0x3C02: even is 0x3C02
    (1.0 + 2.0 ** -11 + 2.0 ** -30, 0x3C01),   # just above the tie
    (1.0 + 2.0 ** -11 - 2.0 ** -30, 0x3C00),   # just below
    (-(1.0 + 3 * 2.0 ** -11), 0xBC02),
    (65504.0, 0x7BFF),                     # largest finite
    (65519.99, 0x7BFF),
    (65520.0, 0x7C00),                     # the tie between 65504 and 2^16 goes to the even side: infinity
    (2.0 ** -24, 0x0001),                  # smallest subnormal
    (2.0 ** -25, 0x0000),                  # tie between 0 and the smallest subnormal: even is 0
    (3 * 2.0 ** -25, 0x0002),              # tie between 1 and 2 subnormal steps: even is 2
    (2.0 ** -25 * 1.0000001, 0x0001),
    (2.0 ** -14, 0x0400),                  # smallest normal
    (2.0 ** -14 - 2.0 ** -25, 0x0400),     # tie between the largest subnormal 0x03FF and 0x0400: even is 0x0400
    (0.0, 0x0000), (-0.0, 0x8000),
    (0.1, 0x2E66),                         # 0.1 = 1.6 * 2^-4; fraction .6 * 1024 = 614.4 -> 614 = 0x266
])
def test_rounding_to_half_by_hand(value, bits):
    assert int(orc.to_half(np.array([value]))[0]) == bits


def test_rounding_to_half_is_monotone_and_exact_on_halves():
    allh = np.arange(0x0000, 0x7C00, dtype=np.uint16)          # every finite non-negative FP16 value
    vals = np.array([orc.half_to_double(int(b)) for b in allh[::37]])
    assert np.array_equal(orc.to_half(vals), allh[::37])        # exact values come back unchanged
    rng = np.random.default_rng(3)
    v = np.sort(rng.uniform(-65000, 65000, 5000))
    r = orc.to_half(v).view(np.float16).astype(np.float64)
    assert np.all(np.diff(r) >= 0)
    assert np.all(np.abs(r - v) <= np.maximum(np.abs(v) * 2.0 ** -11, 2.0 ** -25))   # within half a unit in the last place


def test_epilogue_list_by_brute_force():
    y = np.array([0.5, -3.0, 2.0, 0.0, 10.0, 1.0,        # gate
                  2.0, 100.0, -0.25, 7.0, 0.001, 1.0])   # up
    h, idx, val, n = orc.swiglu_epilogue(y, 0.2)
    want = []
    for i in range(6):
        g, u = y[i], y[6 + i]
        hv = float(np.float16(g / (1.0 + math.exp(-g)) * u))
        want.append(hv)
    assert [float(x) for x in h.view(np.float16)] == want
    keep = [i for i, hv in enumerate(want) if abs(hv) > np.float32(0.2)]
    assert idx.tolist() == keep and n == len(keep)
    assert [float(x) for x in val.view(np.float16)] == [want[i] for i in keep]
    # tau = 0 drops exactly the zeros (gate 0 gives h = 0)
    _, idx0, _, _ = orc.swiglu_epilogue(y, 0.0)
    assert 3 not in idx0.tolist() and set(idx0.tolist()) == {0, 1, 2, 4, 5}
