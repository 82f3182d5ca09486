"""Pins for the oracle's output gate z = Swish(r) * LN(o) (Eq. attn_gla, the line forming Y_t) and
its derivative: library routines on the same rows, invariants of the normalisation, special values of
Swish, finite differences."""
import numpy as np
import pytest
import torch

import oracle


def _rows(seed, rows=7, d=24):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((rows, d)) * 3 + 1.5, rng.standard_normal((rows, d)) * 2,
            rng.standard_normal(d) + 1, rng.standard_normal(d))


def test_matches_library_layer_norm_and_silu():
    o, r, w, b = _rows(0)
    F = torch.nn.functional
    to = torch.from_numpy
    for ww, bb in [(w, b), (None, None), (w, None)]:
        ref = F.silu(to(r)) * F.layer_norm(to(o), (o.shape[1],), None if ww is None else to(ww),
                                           None if bb is None else to(bb), 1e-5)
        np.testing.assert_allclose(oracle.outgate(o, r, ww, bb, 1e-5), ref.numpy(), rtol=1e-12, atol=1e-13)


def test_normalisation_invariants():
    o, r, _, _ = _rows(1)
    big = np.full_like(r, 50.0)                 # Swish(50) = 50 up to 1e-20
    n = oracle.outgate(o, big, None, None, 0.0) / 50.0
    np.testing.assert_allclose(n.mean(axis=1), 0, atol=1e-13)
    np.testing.assert_allclose((n * n).mean(axis=1), 1, rtol=1e-12)
    # LN(a * o + c) = LN(o) for a > 0 when eps = 0; sign flips for a < 0
    np.testing.assert_allclose(oracle.outgate(3.5 * o - 2, big, None, None, 0.0) / 50.0, n, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(oracle.outgate(-o, big, None, None, 0.0) / 50.0, -n, rtol=1e-10, atol=1e-12)
    # eps enters under the root: a row of variance v is scaled by sqrt(v / (v + eps))
    v = o.var(axis=1, keepdims=True)
    np.testing.assert_allclose(oracle.outgate(o, big, None, None, 0.3) / 50.0, n * np.sqrt(v / (v + 0.3)), rtol=1e-12)


def test_swish_special_values_and_affine():
    o, _, w, b = _rows(2)
    z0 = oracle.outgate(o, np.zeros_like(o), w, b)
    assert np.all(z0 == 0)                                      # Swish(0) = 0
    zneg = oracle.outgate(o, np.full_like(o, -60.0), w, b)
    assert np.abs(zneg).max() < 1e-22                           # Swish(-60) = -60 e^-60
    # r = log 3: sigmoid = 3/4, Swish = 0.75 log 3; constant row -> LN gives the bias alone
    const = np.full((2, 24), 4.25)
    z = oracle.outgate(const, np.full_like(const, np.log(3.0)), w, b)
    np.testing.assert_allclose(z, np.broadcast_to(0.75 * np.log(3.0) * b, z.shape), rtol=1e-13)
    # two-element row (1, 3): mean 2, variance 1 -> LN = (-1, 1) at eps = 0
    z2 = oracle.outgate(np.array([[1.0, 3.0]]), np.full((1, 2), 50.0), np.array([2.0, 5.0]), np.array([0.5, -1.0]), 0.0)
    np.testing.assert_allclose(z2, [[50 * (-2 + 0.5), 50 * (5 - 1.0)]], rtol=1e-13)


@pytest.mark.parametrize("affine", [True, False])
def test_backward_finite_differences(affine):
    o, r, w, b = _rows(3, rows=4, d=8)
    if not affine:
        w = b = None
    rng = np.random.default_rng(4)
    dz = rng.standard_normal(o.shape)
    do, dr, dw, db = oracle.outgate_bwd(o, r, dz, w, b, 1e-5)
    f = lambda o_, r_, w_, b_: float((dz * oracle.outgate(o_, r_, w_, b_, 1e-5)).sum())
    h = 1e-6
    w1 = np.ones(8) if w is None else w
    b1 = np.zeros(8) if b is None else b
    for (arr, grad, which) in [(o, do, 0), (r, dr, 1), (w1, dw, 2), (b1, db, 3)]:
        for idx in np.ndindex(arr.shape):
            ap, am = arr.copy(), arr.copy()
            ap[idx] += h
            am[idx] -= h
            args_p = [o, r, w1, b1]
            args_m = [o, r, w1, b1]
            args_p[which], args_m[which] = ap, am
            fd = (f(*args_p) - f(*args_m)) / (2 * h)
            assert abs(fd - grad[idx]) <= 1e-7 * max(1.0, abs(fd)), (which, idx, fd, grad[idx])


def test_backward_against_library_autograd_and_row_sums():
    o, r, w, b = _rows(5)
    rng = np.random.default_rng(6)
    dz = rng.standard_normal(o.shape)
    F = torch.nn.functional
    to, tr, tw, tb = (torch.from_numpy(a.copy()).requires_grad_(True) for a in (o, r, w, b))
    (F.silu(tr) * F.layer_norm(to, (o.shape[1],), tw, tb, 1e-5) * torch.from_numpy(dz)).sum().backward()
    do, dr, dw, db = oracle.outgate_bwd(o, r, dz, w, b, 1e-5)
    for got, ref in [(do, to.grad), (dr, tr.grad), (dw, tw.grad), (db, tb.grad)]:
        np.testing.assert_allclose(got, ref.numpy(), rtol=1e-10, atol=1e-12)
    # the normalisation removes the row mean, so do sums to zero over every row
    np.testing.assert_allclose(do.sum(axis=1), 0, atol=1e-12)
    # and (eps = 0) it removes the component along o - mean as well
    do0 = oracle.outgate_bwd(o, r, dz, w, b, 0.0)[0]
    np.testing.assert_allclose((do0 * (o - o.mean(axis=1, keepdims=True))).sum(axis=1), 0, atol=1e-11)
