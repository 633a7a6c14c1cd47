"""Pins of the oracle's AdamW sensitivity term (paper Sec. 4.3): exact rational examples, a closed form
for a constant gradient, and the defining property: it is the derivative of the AdamW direction with
respect to the gradient."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import snip_oracle as orc


def test_hand_worked_rational_examples():
    # v = 4, eps = 1: sqrt(v) = 2, d = 3; beta1 = 1/2, beta2 = 3/4, m = 3, g = 2:
    # T = (1/2)/3 - (1/4)*3*2/(2*9) = 1/6 - 1/12 = 1/12
    assert orc.adamw_sensitivity_sumsq([3.0], [4.0], [2.0], 0.5, 0.75, 1.0) == pytest.approx(float(Fraction(1, 144)), rel=1e-15)
    # two elements; second: v = 9, m = -1, g = 4, eps = 1: d = 4, T = (1/2)/4 + (1/4)*4/(3*16) = 1/8 + 1/48 = 7/48
    want = Fraction(1, 144) + Fraction(49, 2304)
    assert orc.adamw_sensitivity_sumsq([3.0, -1.0], [4.0, 9.0], [2.0, 4.0], 0.5, 0.75, 1.0) == pytest.approx(float(want), rel=1e-15)


def test_zero_first_moment_and_zero_second_moment():
    v = np.array([1.0, 4.0, 0.25])
    got = orc.adamw_sensitivity_sumsq(np.zeros(3), v, np.ones(3), 0.9, 0.999, 1e-3)
    assert got == pytest.approx(float(((0.1 / (np.sqrt(v) + 1e-3)) ** 2).sum()), rel=1e-14)
    # v == 0: only the first term, (1-beta1)/eps
    assert orc.adamw_sensitivity_sumsq([0.0], [0.0], [0.0], 0.9, 0.999, 1e-8) == pytest.approx((0.1 / 1e-8) ** 2, rel=1e-14)


def test_constant_gradient_closed_form():
    """m = g and v = g^2 (a gradient that never changed), eps = 0: T = (beta2 - beta1) / |g|."""
    g = np.array([0.5, -2.0, 3.0, -0.125])
    got = orc.adamw_sensitivity_sumsq(g, g * g, g, 0.9, 0.95, 0.0)
    assert got == pytest.approx(float((((0.95 - 0.9) / np.abs(g)) ** 2).sum()), rel=1e-12)


def test_is_the_derivative_of_the_adamw_direction():
    rng = np.random.default_rng(0)
    n = 64
    b1, b2, eps = 0.9, 0.95, 1e-3
    m_prev, v_prev, g = rng.normal(size=n), rng.uniform(0.1, 2.0, size=n), rng.normal(size=n)

    def direction(gg):
        m = b1 * m_prev + (1 - b1) * gg
        v = b2 * v_prev + (1 - b2) * gg * gg
        return m / (np.sqrt(v) + eps)

    h = 1e-6
    deriv = (direction(g + h) - direction(g - h)) / (2 * h)       # elementwise: the update is separable
    m = b1 * m_prev + (1 - b1) * g
    v = b2 * v_prev + (1 - b2) * g * g
    assert orc.adamw_sensitivity_sumsq(m, v, g, b1, b2, eps) == pytest.approx(float((deriv ** 2).sum()), rel=1e-7)
    # a dropped factor or a wrong power of (sqrt(v) + eps) would not survive this
    assert orc.adamw_sensitivity_sumsq(m, v, g, b1, b2, eps) != pytest.approx(float(((0.1 / (np.sqrt(v) + eps)) ** 2).sum()), rel=1e-3)
