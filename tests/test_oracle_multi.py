"""Pins for the oracle's sums over several scan orders (Algorithm 2, bidirectional scanning, and
Algorithm 3, 4-directional scanning): what the sums must be when nothing decays, linearity, the
single-order special case against the C oracle's own direction handling, finite differences."""
import numpy as np
import pytest

import oracle


def _inputs(seed, B=1, H=2, gh=3, gw=4, dk=3, dv=4, decay=0.5):
    rng = np.random.default_rng(seed)
    L = gh * gw
    q, k = rng.standard_normal((B, L, H, dk)), rng.standard_normal((B, L, H, dk))
    v, dO = rng.standard_normal((B, L, H, dv)), rng.standard_normal((B, L, H, dv))
    a = -rng.random((B, L, H, dk)) * decay
    return q, k, v, a, dO


def test_without_decay_two_orders_are_full_attention_with_the_diagonal_twice():
    # alpha == 1: the forward order sums over s <= t, the flipped one over s >= t, so together every
    # pair once and the pair (t, t) twice: (Q K^T + diag(q_t . k_t)) V.  Column orders cover the same
    # pairs again, so all four orders give twice that.
    q, k, v, a, _ = _inputs(0, gh=4, gw=5)
    a = np.zeros_like(a)
    two = oracle.gla_fwd_multi(q, k, v, a, 4, 5, (0, 1))
    four = oracle.gla_fwd_multi(q, k, v, a, 4, 5, (0, 1, 2, 3))
    for h in range(2):
        A = q[0, :, h] @ k[0, :, h].T
        A = A + np.diag(np.diag(A))
        np.testing.assert_allclose(two[0, :, h], A @ v[0, :, h], rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(four[0, :, h], 2 * (A @ v[0, :, h]), rtol=1e-12, atol=1e-12)
    col = oracle.gla_fwd_multi(q, k, v, a, 4, 5, (2, 3))
    np.testing.assert_allclose(col, two, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("direction", [0, 1, 2, 3])
def test_one_order_is_the_plain_operator_in_that_order(direction):
    """The sum builds its orders with numpy flips and transposes and runs the plain row scan; the plain
    operator builds them inside the C code.  One order alone must agree."""
    q, k, v, a, dO = _inputs(1 + direction, B=2, gh=5, gw=3)
    np.testing.assert_allclose(oracle.gla_fwd_multi(q, k, v, a, 5, 3, (direction,)),
                               oracle.gla_fwd(q, k, v, a, 5, 3, direction), rtol=1e-13, atol=1e-13)
    for x, y in zip(oracle.gla_bwd_multi(q, k, v, a, dO, 5, 3, (direction,)),
                    oracle.gla_bwd(q, k, v, a, dO, 5, 3, direction)):
        np.testing.assert_allclose(x, y, rtol=1e-12, atol=1e-12)


def test_sum_is_linear_in_v_and_adds_over_orders():
    q, k, v, a, _ = _inputs(7)
    v2 = np.random.default_rng(8).standard_normal(v.shape)
    f = lambda vv, dirs=(0, 1, 2, 3): oracle.gla_fwd_multi(q, k, vv, a, 3, 4, dirs)
    np.testing.assert_allclose(f(2.0 * v - 3.0 * v2), 2.0 * f(v) - 3.0 * f(v2), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(f(v), f(v, (0, 3)) + f(v, (1, 2)), rtol=1e-12, atol=1e-12)
    # with decay the two row orders differ from the two column orders on a non-degenerate grid
    assert np.abs(f(v, (0, 1)) - f(v, (2, 3))).max() > 1e-3


@pytest.mark.parametrize("dirs", [(0, 1), (0, 1, 2, 3)])
def test_gradients_by_finite_differences(dirs):
    q, k, v, a, dO = _inputs(11, gh=2, gw=3, dk=2, dv=3)
    grads = oracle.gla_bwd_multi(q, k, v, a, dO, 2, 3, dirs)
    loss = lambda *x: float((oracle.gla_fwd_multi(*x, 2, 3, dirs) * dO).sum())
    args = [q, k, v, a]
    h = 1e-6
    for which, grad in enumerate(grads):
        arr = args[which]
        for idx in np.ndindex(arr.shape):
            ap, am = arr.copy(), arr.copy()
            ap[idx] += h
            am[idx] -= h
            pa, ma = list(args), list(args)
            pa[which], ma[which] = ap, am
            fd = (loss(*pa) - loss(*ma)) / (2 * h)
            assert abs(fd - grad[idx]) <= 2e-7 * max(1.0, abs(fd)), (which, idx, fd, grad[idx])
