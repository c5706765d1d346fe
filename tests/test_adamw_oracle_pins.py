"""Pins for the AdamW oracle that do not call back into it for expectations."""

import math

import numpy as np

from oracle import adamw_oracle as aw


def test_first_step_is_sign_of_gradient():
    """t = 1 from zero state: m_hat = g, v_hat = g^2, so the step is
    -lr * (g / (|g| + eps) + wd * p)."""
    rng = np.random.default_rng(0)
    p = rng.standard_normal(50)
    g = rng.standard_normal(50)
    z = np.zeros(50)
    p1, m1, v1 = aw.adamw_step(p, g, z, z, 1, lr=0.01, wd=0.1, beta1=0.9, beta2=0.95, eps=1e-8)
    assert np.allclose(m1, 0.1 * g, rtol=1e-14)
    assert np.allclose(v1, 0.05 * g * g, rtol=1e-14)
    assert np.allclose(p1, p - 0.01 * (g / (np.abs(g) + 1e-8) + 0.1 * p), rtol=1e-12, atol=1e-15)


def test_constant_gradient_keeps_bias_corrected_moments():
    """With the same gradient every step, m_hat = g and v_hat = g^2 at every t
    (geometric sums cancel the bias correction), so with wd = 0 the parameter
    moves by -lr * g / (|g| + eps) per step."""
    g = np.array([0.5, -2.0, 3.0])
    p = np.array([1.0, 1.0, 1.0])
    m = np.zeros(3)
    v = np.zeros(3)
    for t in range(1, 8):
        p, m, v = aw.adamw_step(p, g, m, v, t, lr=0.1, wd=0.0, eps=0.0)
        assert np.allclose(m, (1 - 0.9 ** t) * g, rtol=1e-13)
        assert np.allclose(v, (1 - 0.95 ** t) * g * g, rtol=1e-13)
        assert np.allclose(p, 1.0 - 0.1 * t * np.sign(g), rtol=1e-12)


def test_zero_gradient_only_decays():
    p = np.array([2.0, -4.0])
    z = np.zeros(2)
    p1, m1, v1 = aw.adamw_step(p, z, z, z, 1, lr=0.5, wd=0.1)
    assert np.array_equal(m1, z) and np.array_equal(v1, z)
    assert np.allclose(p1, p * (1 - 0.05), rtol=1e-15)


def test_hand_computed_second_step():
    """Scalars by hand: g1 = 1, g2 = -1, beta1 = 0.5, beta2 = 0.5, eps = 0, wd = 0, lr = 1.
    m1 = 0.5, v1 = 0.5; p1 = p0 - (0.5/0.5)/sqrt(0.5/0.5) = p0 - 1.
    m2 = 0.25 - 0.5 = -0.25, v2 = 0.25 + 0.5 = 0.75; m_hat = -0.25/0.75 = -1/3,
    v_hat = 0.75/0.75 = 1; p2 = p1 + 1/3."""
    p, m, v = np.array([3.0]), np.zeros(1), np.zeros(1)
    p, m, v = aw.adamw_step(p, np.array([1.0]), m, v, 1, lr=1.0, wd=0.0, beta1=0.5, beta2=0.5, eps=0.0)
    assert math.isclose(p[0], 2.0, rel_tol=1e-15)
    p, m, v = aw.adamw_step(p, np.array([-1.0]), m, v, 2, lr=1.0, wd=0.0, beta1=0.5, beta2=0.5, eps=0.0)
    assert math.isclose(m[0], -0.25) and math.isclose(v[0], 0.75)
    assert math.isclose(p[0], 2.0 + 1.0 / 3.0, rel_tol=1e-15)
