"""Pins for the GEGLU oracle (no GPU needed).

The paper gives the formula (Eq. 2) and no worked number, so the oracle is pinned to what the formula and mathematics
fix: the error function's Maclaurin series summed in 60-digit decimals (another formulation, another arithmetic),
scipy's normal distribution function as an independent library routine, closed forms and identities of GELU, and
the layout of the split (which half is gated, which index runs fastest).  A dropped factor 1/2, a missing 1/sqrt 2, a
swapped half or a transposed index fails at least one of them.
"""
import math
from decimal import Decimal, getcontext

import numpy as np
import pytest
import scipy.special

import oracle


def erf_series(x: float) -> Decimal:
    """erf(x) = 2/sqrt(pi) * sum_n (-1)^n x^(2n+1) / (n! (2n+1)), in 60-digit decimals."""
    getcontext().prec = 60
    xd = Decimal(x)
    term, total, n = xd, Decimal(0), 0   # term = x^(2n+1) / n!
    while True:
        add = term / (2 * n + 1)
        total += add if n % 2 == 0 else -add
        if abs(add) < Decimal(10) ** -55:
            break
        n += 1
        term = term * xd * xd / n
    pi = Decimal("3.14159265358979323846264338327950288419716939937510582097494")
    return 2 * total / pi.sqrt()


@pytest.mark.parametrize("g", [-6.0, -3.5, -2.0, -1.0, -0.3, -1e-3, 0.0, 1e-3, 0.25, 1.0, 1.7, 3.0, 5.5])
def test_gelu_against_the_error_function_series_in_decimals(g):
    getcontext().prec = 60
    gd = Decimal(g)
    want = gd / 2 * (1 + erf_series(g / math.sqrt(2.0)))
    # (the argument g / sqrt 2 is rounded to double before the series: the same rounding the oracle's libm call sees,
    # worth at most an ulp of the argument: compare to a relative 4e-15 plus the cancellation floor of the series)
    got = oracle.gelu(g)
    assert abs(Decimal(got) - want) <= abs(want) * Decimal("4e-13") + Decimal("1e-18")


def test_gelu_is_x_times_the_normal_distribution_function():
    g = np.linspace(-9.0, 9.0, 3601)
    want = g * scipy.special.ndtr(g)
    got = np.array([oracle.gelu(v) for v in g])
    np.testing.assert_allclose(got, want, rtol=1e-13, atol=1e-300)


def test_gelu_closed_forms_and_identities():
    assert oracle.gelu(0.0) == 0.0
    # GELU(g) - GELU(-g) = g: the odd part of g * Phi(g) is g / 2 + g / 2
    for g in (0.1, 0.5, 1.0, 2.5, 7.0):
        assert oracle.gelu(g) - oracle.gelu(-g) == pytest.approx(g, rel=1e-15)
    # far tails: the identity for large g, -g * phi(g)/g... -> 0 from below for very negative g
    assert oracle.gelu(12.0) == pytest.approx(12.0, rel=1e-15)
    assert -1e-30 < oracle.gelu(-12.0) < 0.0
    # the minimum of GELU: about -0.16997 at g about -0.75179
    gs = np.linspace(-1.0, -0.5, 5001)
    vals = np.array([oracle.gelu(v) for v in gs])
    assert gs[vals.argmin()] == pytest.approx(-0.75179, abs=2e-4)
    assert vals.min() == pytest.approx(-0.169971, abs=1e-6)
    # value at 1: Phi(1) = 0.8413447460685429...
    assert oracle.gelu(1.0) == pytest.approx(0.8413447460685429, rel=1e-15)


def test_which_half_is_gated_and_how_the_rows_are_laid_out():
    # row 0: a = (2, 3), g = (0, 50)  ->  2 * GELU(0) = 0,  3 * GELU(50) = 150
    # row 1: a = (1, 1), g = (1, -1)  ->  GELU(1), GELU(-1)
    x = np.array([[2.0, 3.0, 0.0, 50.0], [1.0, 1.0, 1.0, -1.0]], dtype=np.float32)
    out = oracle.geglu_forward(x)
    assert out.shape == (2, 2)
    assert out[0, 0] == 0.0 and out[0, 1] == pytest.approx(150.0, rel=1e-15)
    assert out[1, 0] == pytest.approx(0.8413447460685429, rel=1e-15)
    assert out[1, 1] == pytest.approx(-0.15865525393145707, rel=1e-14)
    # swapping the halves changes the result: the gate is the SECOND half
    swapped = oracle.geglu_forward(np.concatenate([x[:, 2:], x[:, :2]], axis=1))
    assert not np.allclose(out, swapped)


@pytest.mark.parametrize("dtype", [np.float16, np.float32])
def test_forward_is_the_formula_on_the_stored_values(dtype):
    g = np.random.default_rng(5)
    x = (g.standard_normal((7, 3, 2 * 24)) * 2.5).astype(dtype)
    out = oracle.geglu_forward(x)
    xd = x.astype(np.float64)
    want = xd[..., :24] * xd[..., 24:] * scipy.special.ndtr(xd[..., 24:])
    np.testing.assert_allclose(out, want, rtol=2e-13, atol=1e-300)
    # linear in the first half, and rows are independent
    x2 = x.copy()
    x2[..., :24] *= dtype(2.0)
    np.testing.assert_array_equal(oracle.geglu_forward(x2), 2.0 * out)
    np.testing.assert_array_equal(oracle.geglu_forward(x[3:4]), out[3:4])


def test_forward_edge_shapes_and_arguments():
    assert oracle.geglu_forward(np.zeros((0, 16), dtype=np.float16)).shape == (0, 8)
    assert oracle.geglu_forward(np.ones((5, 2), dtype=np.float16)).shape == (5, 1)
    with pytest.raises(ValueError):
        oracle.geglu_forward(np.zeros((4, 7), dtype=np.float16))
    with pytest.raises(TypeError):
        oracle.geglu_forward(np.zeros((4, 8), dtype=np.float64))
