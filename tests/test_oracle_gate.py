"""Pins of the oracle's gate projection (Eq. 1: a_ij = w_j^T x_i) and its gradients.

None of them re-types the inner product or calls a matrix product for it: they use what the
definition fixes (selection by unit vectors, worked 2 x 2 numbers, linearity, central finite
differences of the forward function, the adjoint identity)."""
import numpy as np
import pytest

from oracle import rr_oracle as orc
from paper_2402_12399_b200 import synth


def _rand(T, E, d, seed, bf16=False):
    rng = np.random.default_rng(seed)
    h = rng.standard_normal((T, d)).astype(np.float32)
    w = rng.standard_normal((E, d)).astype(np.float32)
    if bf16:
        return synth.to_bf16_bits(h), synth.to_bf16_bits(w)
    return h, w


def test_hand_example():
    # x_0 = (1, 2), x_1 = (-3, 0.5); w_0 = (2, 0), w_1 = (1, 1), w_2 = (0.5, -4)
    h = np.array([[1.0, 2.0], [-3.0, 0.5]], np.float32)
    w = np.array([[2.0, 0.0], [1.0, 1.0], [0.5, -4.0]], np.float32)
    a = orc.gate_fwd(h, w)
    assert a.tolist() == [[2.0, 3.0, -7.5], [-6.0, -2.5, -3.5]]
    # L = a_02 + 2 a_10: dW_2 = x_0, dW_0 = 2 x_1, dW_1 = 0; dx_0 = w_2, dx_1 = 2 w_0
    dl = np.array([[0, 0, 1.0], [2.0, 0, 0]])
    dW, dh = orc.gate_bwd(dl, h, w)
    assert dW.tolist() == [[-6.0, 1.0], [0.0, 0.0], [1.0, 2.0]]
    assert dh.tolist() == [[0.5, -4.0], [4.0, 0.0]]


def test_unit_vectors_select_columns():
    h, _ = _rand(37, 5, 16, 1)
    w = np.zeros((5, 16), np.float32)
    cols = [3, 0, 15, 7, 7]
    for j, c in enumerate(cols):
        w[j, c] = 1.0
    a = orc.gate_fwd(h, w)
    for j, c in enumerate(cols):
        assert np.array_equal(a[:, j], h[:, c].astype(np.float64))


def test_bf16_bits_are_read_as_their_exact_values():
    hb, wb = _rand(9, 4, 32, 2, bf16=True)
    hf = (hb.astype(np.uint32) << 16).view(np.float32)
    wf = (wb.astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(orc.gate_fwd(hb, wb), orc.gate_fwd(hf, wf))


def test_linear_in_both_arguments():
    h1, w = _rand(11, 6, 24, 3)
    h2, w2 = _rand(11, 6, 24, 4)
    # sums of float32 values that stay exact in float32: use small integers
    h1, h2, w, w2 = (np.round(x * 4).astype(np.float32) for x in (h1, h2, w, w2))
    assert np.array_equal(orc.gate_fwd(h1 + h2, w), orc.gate_fwd(h1, w) + orc.gate_fwd(h2, w))
    assert np.array_equal(orc.gate_fwd(h1, w + w2), orc.gate_fwd(h1, w) + orc.gate_fwd(h1, w2))
    assert np.array_equal(orc.gate_fwd(h1, 3 * w), 3 * orc.gate_fwd(h1, w))


def test_gradients_against_finite_differences():
    h, w = _rand(7, 3, 10, 5)
    rng = np.random.default_rng(6)
    dl = rng.standard_normal((7, 3))
    dW, dh = orc.gate_bwd(dl, h, w)

    def loss(hh, ww):
        return float((orc.gate_fwd(hh, ww) * dl).sum())

    eps = 2.0 ** -6     # the forward is bilinear: central differences are exact up to rounding
    for (j, c) in [(0, 0), (2, 9), (1, 4)]:
        wp, wm = w.copy(), w.copy()
        wp[j, c] += eps
        wm[j, c] -= eps
        assert (loss(h, wp) - loss(h, wm)) / (2 * eps) == pytest.approx(dW[j, c], rel=1e-9, abs=1e-9)
    for (i, c) in [(0, 0), (6, 9), (3, 5)]:
        hp, hm = h.copy(), h.copy()
        hp[i, c] += eps
        hm[i, c] -= eps
        assert (loss(hp, w) - loss(hm, w)) / (2 * eps) == pytest.approx(dh[i, c], rel=1e-9, abs=1e-9)


def test_adjoint_identity():
    # <dl, a(h, w)> = <dW, w> = <dh, h> for the bilinear map
    h, w = _rand(13, 4, 8, 7)
    dl = np.random.default_rng(8).standard_normal((13, 4))
    dW, dh = orc.gate_bwd(dl, h, w)
    lhs = float((dl * orc.gate_fwd(h, w)).sum())
    assert float((dW * w).sum()) == pytest.approx(lhs, rel=1e-12)
    assert float((dh * h).sum()) == pytest.approx(lhs, rel=1e-12)


def test_bad_shapes_are_refused():
    h, w = _rand(4, 2, 8, 9)
    with pytest.raises(TypeError):
        orc.gate_fwd(h, synth.to_bf16_bits(w))
