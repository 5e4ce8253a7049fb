"""Pins of the oracle's projection gate (Eq. 5-6) against closed forms and a brute-force loop."""
import math

import numpy as np
import pytest

import oracle


def _rng(seed):
    return np.random.default_rng(seed)


def test_zero_weights_give_half_of_each_path():
    r = _rng(0)
    ya, yb = r.standard_normal((7, 5)), r.standard_normal((7, 5))
    z = np.zeros((5, 5))
    np.testing.assert_allclose(oracle.gate_projection(ya, z), 0.5 * ya, rtol=0, atol=1e-15)
    np.testing.assert_allclose(oracle.gate_projection(ya, z, yb, z), 0.5 * (ya + yb), rtol=0, atol=1e-15)


def test_scaled_identity_is_an_elementwise_logistic():
    r = _rng(1)
    y = r.standard_normal((4, 6))
    c = 1.7
    want = y / (1.0 + np.exp(-c * y))
    np.testing.assert_allclose(oracle.gate_projection(y, c * np.eye(6)), want, rtol=1e-14)


def test_single_weight_entry_picks_input_column_not_output_column():
    # w[o, i] = 1 only: gate of output dimension o reads input dimension i (a transposed
    # weight would read dimension o of the input for output i instead)
    r = _rng(2)
    y = r.standard_normal((3, 4))
    o, i = 1, 3
    w = np.zeros((4, 4))
    w[o, i] = 1.0
    got = oracle.gate_projection(y, w)
    want = 0.5 * y
    want[:, o] = y[:, o] / (1.0 + np.exp(-y[:, i]))
    np.testing.assert_allclose(got, want, rtol=1e-14)


def test_brute_force_loops_on_a_tiny_case():
    r = _rng(3)
    ya, yb = r.standard_normal((3, 4)), r.standard_normal((3, 4))
    wa, wb = r.standard_normal((4, 4)), r.standard_normal((4, 4))
    want = np.zeros((3, 4))
    for t in range(3):
        for o in range(4):
            za = sum(wa[o][i] * ya[t][i] for i in range(4))
            zb = sum(wb[o][i] * yb[t][i] for i in range(4))
            want[t][o] = ya[t][o] / (1 + math.exp(-za)) + yb[t][o] / (1 + math.exp(-zb))
    np.testing.assert_allclose(oracle.gate_projection(ya, wa, yb, wb), want, rtol=1e-13)


def test_paths_are_independent_and_saturate():
    # the two sigmoids are independent (no normalisation across paths): with very large
    # positive pre-activations both gates are 1 and the paths simply add
    y = np.full((2, 3), 2.0)
    w = 50.0 * np.ones((3, 3))
    np.testing.assert_allclose(oracle.gate_projection(y, w, y, w), 2 * y, rtol=1e-12)
    # and with very negative ones both close
    np.testing.assert_allclose(oracle.gate_projection(y, -w, y, -w), 0 * y, atol=1e-100)


def test_shape_errors():
    with pytest.raises(ValueError):
        oracle.gate_projection(np.zeros((2, 3)), np.zeros((3, 4)))


def _loss(ya, wa, yb, wb, c):
    return float((oracle.gate_projection(ya, wa, yb, wb) * c).sum())


def test_backward_matches_central_differences_of_the_forward():
    # the forward oracle is pinned above; its numerical derivative pins the backward
    r = _rng(4)
    ya, yb = r.standard_normal((3, 4)), r.standard_normal((3, 4))
    wa, wb = r.standard_normal((4, 4)), r.standard_normal((4, 4))
    c = r.standard_normal((3, 4))              # upstream gradient: loss = sum(out * c)
    dya, dwa, dyb, dwb = oracle.gate_projection_backward(c, ya, wa, yb, wb)
    eps = 1e-6
    for arr, grad, which in ((ya, dya, 0), (wa, dwa, 1), (yb, dyb, 2), (wb, dwb, 3)):
        num = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            args = [ya.copy(), wa.copy(), yb.copy(), wb.copy()]
            args[which][idx] += eps
            up = _loss(*args, c)
            args[which][idx] -= 2 * eps
            num[idx] = (up - _loss(*args, c)) / (2 * eps)
        np.testing.assert_allclose(grad, num, rtol=1e-6, atol=1e-8)


def test_backward_zero_weights_closed_form():
    # w = 0: g = 1/2 everywhere, dz = dout * y / 4, so dy = dout / 2 and dw = (dout * y)^T y / 4
    r = _rng(5)
    y, c = r.standard_normal((5, 3)), r.standard_normal((5, 3))
    dy, dw = oracle.gate_projection_backward(c, y, np.zeros((3, 3)))
    np.testing.assert_allclose(dy, 0.5 * c, rtol=0, atol=1e-15)
    np.testing.assert_allclose(dw, (c * y).T @ y / 4.0, rtol=1e-14)


def test_backward_single_path_is_the_dual_path_with_a_dead_branch():
    r = _rng(6)
    y, c, w = r.standard_normal((4, 3)), r.standard_normal((4, 3)), r.standard_normal((3, 3))
    dy1, dw1 = oracle.gate_projection_backward(c, y, w)
    dy2, dw2, dyb, dwb = oracle.gate_projection_backward(c, y, w, np.zeros((4, 3)), w)
    np.testing.assert_allclose(dy1, dy2, rtol=0, atol=0)
    np.testing.assert_allclose(dw1, dw2, rtol=0, atol=0)
    np.testing.assert_allclose(dwb, 0 * dwb, atol=0)
