"""Pins of the oracle's load-balance loss L = alpha E sum_e f_e P_e (Section 5.1) and its gradient.

They use what the definition fixes without re-typing it: numbers worked by hand, the closed
forms at uniform and at saturated scores, a library softmax and bincount for the two factors,
shift invariance, central finite differences of the forward function for the gradient, and the
closed-form gradient at uniform scores."""
import numpy as np
import pytest
from scipy.special import softmax

from oracle import rr_oracle as orc

LN = np.log


def _first(c):
    return np.asarray(c, np.int32).reshape(-1, 1)


def test_hand_examples():
    # two tokens with g = (1/4, 3/4), both choosing expert 1: f = (0, 1), P = (1/4, 3/4), L = 2 * 3/4 alpha
    a = np.array([[0.0, LN(3)], [0.0, LN(3)]], np.float32)
    L, f, P = orc.aux_loss(a, _first([1, 1]), 0.5)
    assert f.tolist() == [0.0, 1.0]
    np.testing.assert_allclose(P, [0.25, 0.75], rtol=1e-7)
    assert abs(L - 0.75) < 1e-7
    # three experts: g_0 = (1, 2, 5)/8 choosing 2, g_1 = (5, 2, 1)/8 choosing 0:
    # f = (1/2, 0, 1/2), P = (3, 2, 3)/8, L = 3 alpha (3/16 + 3/16) = 9/8 alpha
    a = np.array([[0.0, LN(2), LN(5)], [LN(5), LN(2), 0.0]], np.float32)
    L, f, P = orc.aux_loss(a, _first([2, 0]), 1e-2)
    assert f.tolist() == [0.5, 0.0, 0.5]
    np.testing.assert_allclose(P, [0.375, 0.25, 0.375], rtol=1e-7)
    assert abs(L - 1.125e-2) < 1e-9
    # only column 0 of the choices counts
    te = np.array([[2, 1], [0, 1]], np.int32)
    assert orc.aux_loss(a, te, 1e-2)[0] == L


def test_uniform_scores_give_alpha_whatever_the_counts():
    rng = np.random.default_rng(0)
    for T, E in [(1, 1), (7, 3), (100, 8), (33, 64)]:
        a = np.full((T, E), 1.25, np.float32)
        L, f, P = orc.aux_loss(a, _first(rng.integers(0, E, T)), 0.3)
        assert abs(L - 0.3) < 1e-12 and abs(f.sum() - 1) < 1e-12
        np.testing.assert_allclose(P, 1.0 / E, rtol=1e-12)


def test_saturated_scores():
    # softmax -> one-hot: balanced first choices give alpha, all tokens on one expert give alpha E
    T, E = 64, 8
    c = np.arange(T) % E
    a = np.zeros((T, E), np.float32)
    a[np.arange(T), c] = 60.0
    assert abs(orc.aux_loss(a, _first(c), 1.0)[0] - 1.0) < 1e-9
    a[:] = 0
    a[:, 5] = 60.0
    assert abs(orc.aux_loss(a, _first(np.full(T, 5)), 1.0)[0] - E) < 1e-9


def test_factors_against_library_routines():
    rng = np.random.default_rng(1)
    for T, E, k in [(257, 8, 2), (1000, 64, 2), (50, 5, 1)]:
        a = (np.round(2.0 * rng.standard_normal((T, E)) * 1024) / 1024).astype(np.float32)   # multiples of 2^-10
        tab = orc.route(a, k, T, 1, 0)
        L, f, P = orc.aux_loss(a, tab.topk_expert, 1e-2)
        np.testing.assert_array_equal(f * T, np.bincount(a.argmax(1), minlength=E))
        np.testing.assert_allclose(P, softmax(a.astype(np.float64), axis=1).mean(0), rtol=1e-12)
        # shift invariance of the softmax: a per-token constant changes nothing
        a2 = (a.astype(np.float64) + np.round(rng.standard_normal((T, 1)) * 4) / 4).astype(np.float32)
        assert np.array_equal(a2.astype(np.float64) - a, np.broadcast_to((a2 - a)[:, :1], a.shape))   # exact shifts
        assert abs(orc.aux_loss(a2, tab.topk_expert, 1e-2)[0] - L) < 1e-12


def test_gradient_against_finite_differences():
    rng = np.random.default_rng(2)
    T, E, alpha = 9, 6, 0.7
    a = (np.round(rng.standard_normal((T, E)) * 2 * 256) / 256).astype(np.float32)   # multiples of 2^-8
    c = _first(rng.integers(0, E, T))
    L, f, _ = orc.aux_loss(a, c, alpha)
    g = orc.aux_loss_bwd(a, f, alpha, 1.0)
    h = 2.0 ** -9                                                                      # a +- h stays exact in fp32
    for i in range(T):
        for j in range(E):
            ap, am = a.copy(), a.copy()
            ap[i, j] += h
            am[i, j] -= h
            fd = (orc.aux_loss(ap, c, alpha)[0] - orc.aux_loss(am, c, alpha)[0]) / (2 * h)
            assert abs(fd - g[i, j]) < 2e-6 * alpha, (i, j, fd, g[i, j])
    # rows sum to zero (the softmax Jacobian annihilates constants); the scale is linear
    np.testing.assert_allclose(g.sum(1), 0, atol=1e-15)
    np.testing.assert_allclose(orc.aux_loss_bwd(a, f, alpha, -2.5), -2.5 * g, rtol=1e-14)


def test_gradient_closed_form_at_uniform_scores():
    # g = 1/E everywhere: dL/da_ij = alpha / T (f_j - 1/E)
    T, E, alpha = 12, 4, 2.0
    a = np.zeros((T, E), np.float32)
    f = np.array([0.5, 0.25, 0.25, 0.0])
    g = orc.aux_loss_bwd(a, f, alpha)
    np.testing.assert_allclose(g, np.broadcast_to(alpha / T * (f - 0.25), (T, E)), rtol=1e-14, atol=1e-18)


def test_bad_arguments():
    a = np.zeros((4, 3), np.float32)
    with pytest.raises(Exception):
        orc.aux_loss(a, _first([0, 1, 2, 3]), 1.0)      # a choice outside 0..E-1
