"""Pins of the oracle's rotary position embedding (the paper applies RoPE to Q and K with the
ORIGINAL token positions, before the shuffle: Sec. 4.2, App. B) against what the mathematics
fixes; CPU only."""
import math

import numpy as np
import pytest

import oracle
from oracle import CAUSAL


def test_position_zero_is_the_identity_and_norms_are_kept():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((2, 3, 5, 8))
    pos = np.array([0, 3, 0, 11, 7])
    y = oracle.rope(x, pos, base=50.0)
    assert np.array_equal(y[:, :, 0], x[:, :, 0]) and np.array_equal(y[:, :, 2], x[:, :, 2])
    # every pair (c, c + d/2) is rotated: its norm, and so the row norm, is unchanged
    half = 4
    pair = lambda a: a[..., :half] ** 2 + a[..., half:] ** 2
    assert np.abs(pair(y) - pair(x)).max() < 1e-12
    assert not np.allclose(y[:, :, 1], x[:, :, 1])


def test_hand_computed_two_pair_case():
    # d = 4, base = 10000: pair (0, 2) turns by 1 rad per position, pair (1, 3) by 0.01 rad
    x = np.array([[1.0, 2.0, 3.0, 4.0]])
    y = oracle.rope(x, np.array([2]), base=10000.0)
    a, b = 2.0 * 1.0, 2.0 * 10000.0 ** (-2.0 / 4.0)
    want = [1 * math.cos(a) - 3 * math.sin(a), 2 * math.cos(b) - 4 * math.sin(b),
            3 * math.cos(a) + 1 * math.sin(a), 4 * math.cos(b) + 2 * math.sin(b)]
    assert np.abs(y[0] - np.array(want)).max() < 1e-14
    assert abs(b - 0.02) < 1e-15


def test_scores_depend_on_the_position_difference_only():
    rng = np.random.default_rng(1)
    d = 16
    q, k = rng.standard_normal((1, d)), rng.standard_normal((1, d))
    base = 500.0
    ref = None
    for i, j in [(5, 2), (103, 100), (3, 0), (1000, 997)]:
        s = float(oracle.rope(q, np.array([i]), base)[0] @ oracle.rope(k, np.array([j]), base)[0])
        ref = s if ref is None else ref
        assert abs(s - ref) < 1e-9
    other = float(oracle.rope(q, np.array([5]), base)[0] @ oracle.rope(k, np.array([1]), base)[0])
    assert abs(other - ref) > 1e-3


def test_complex_multiplication_form_and_inverse():
    rng = np.random.default_rng(2)
    n, d, base = 9, 12, 77.0
    x = rng.standard_normal((n, d))
    pos = rng.integers(0, 50, size=n)
    y = oracle.rope(x, pos, base)
    z = (x[:, :d // 2] + 1j * x[:, d // 2:]) * np.exp(
        1j * pos[:, None] * base ** (-2.0 * np.arange(d // 2) / d))
    assert np.abs(y[:, :d // 2] - z.real).max() < 1e-12
    assert np.abs(y[:, d // 2:] - z.imag).max() < 1e-12
    assert np.abs(oracle.rope(y, pos, base, inverse=True) - x).max() < 1e-12
    # the inverse is the transpose: <rope(x), g> == <x, rope_inverse(g)>
    g = rng.standard_normal((n, d))
    assert abs((y * g).sum() - (x * oracle.rope(g, pos, base, inverse=True)).sum()) < 1e-10


def test_rope_uses_original_positions_under_the_shuffle():
    """RoPE before shuffling: rotating with the ORIGINAL positions and then running SA equals
    Alg. 1 carried out on the rotated tensors; rotating with slot indices instead (the mistake
    the paper warns about) gives something else."""
    rng = np.random.default_rng(3)
    B, H, n, d, w = 1, 2, 40, 8, 9
    q, k, v = (rng.standard_normal((B, H, n, d)) for _ in range(3))
    perm, inv = oracle.make_perm(5, 0, B, n)
    pos = np.arange(n)
    y = oracle.sa_forward(oracle.rope(q, pos), oracle.rope(k, pos), v, perm, inv, w, CAUSAL)[0]
    # Alg. 1 literally: gather rotated rows by perm, window in slot order, scatter back
    qp, kp, vp = (a[:, :, perm[0]] for a in (oracle.rope(q, pos), oracle.rope(k, pos), v))
    ident = np.arange(n, dtype=np.int32)[None]
    # causality still refers to original positions, so compare in the non-causal form
    y_nc = oracle.sa_forward(oracle.rope(q, pos), oracle.rope(k, pos), v, perm, inv, w, 0)[0]
    y_alg = oracle.sa_forward(qp, kp, vp, ident, ident, w, 0)[0][:, :, inv[0]]
    assert np.abs(y_nc - y_alg).max() < 1e-12
    wrong = oracle.sa_forward(oracle.rope(q, inv[0]), oracle.rope(k, inv[0]), v, perm, inv, w,
                              CAUSAL)[0]
    assert np.abs(wrong - y).max() > 1e-3


def test_rope_rejects_bad_shapes():
    with pytest.raises(ValueError):
        oracle.rope(np.zeros((3, 5)), np.arange(3))
    with pytest.raises(ValueError):
        oracle.rope(np.zeros((3, 4)), np.arange(2))


def test_gradient_through_the_rotation_by_finite_differences():
    """d/dq and d/dk of sum(dy * SA(rope(q), rope(k), v)) is the inverse rotation (the
    transpose) of the gradient with respect to the rotated tensors."""
    rng = np.random.default_rng(4)
    B, H, n, d, w = 1, 2, 10, 4, 5
    q, k, v = (rng.standard_normal((B, H, n, d)) for _ in range(3))
    dy = rng.standard_normal((B, H, n, d))
    perm, inv = oracle.make_perm(6, 0, B, n)
    pos = np.arange(n)
    f = lambda q_, k_: float((dy * oracle.sa_forward(oracle.rope(q_, pos), oracle.rope(k_, pos), v,
                                                     perm, inv, w, CAUSAL)[0]).sum())
    gq, gk, _, _ = oracle.backward(oracle.rope(q, pos), oracle.rope(k, pos), v, perm, inv, None, dy,
                                   w, CAUSAL)
    dq, dk = oracle.rope(gq, pos, inverse=True), oracle.rope(gk, pos, inverse=True)
    eps = 1e-6
    for arr, grad, which in ((q, dq, 0), (k, dk, 1)):
        flat = arr.reshape(-1)
        for e in rng.choice(flat.size, size=20, replace=False):
            old = flat[e]
            flat[e] = old + eps
            lp = f(q, k)
            flat[e] = old - eps
            lm = f(q, k)
            flat[e] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - grad.reshape(-1)[e]) <= 1e-7 * max(1.0, abs(fd)), (which, e)
