"""Pins for the oracle's recurrence with the full gate G_t = alpha_t^T beta_t of Eq. gate_gla
(value-channel decay beta as well as key-channel decay alpha)."""
import numpy as np
import pytest

import oracle


def _inputs(seed, B=1, H=2, L=9, dk=3, dv=4):
    rng = np.random.default_rng(seed)
    q, k = rng.standard_normal((B, L, H, dk)), rng.standard_normal((B, L, H, dk))
    v, dO = rng.standard_normal((B, L, H, dv)), rng.standard_normal((B, L, H, dv))
    a = -rng.random((B, L, H, dk)) * 0.7
    bg = -rng.random((B, L, H, dv)) * 0.5
    return q, k, v, a, bg, dO


def test_beta_one_is_the_alpha_only_recurrence():
    q, k, v, a, bg, dO = _inputs(0)
    zero = np.zeros_like(bg)
    assert np.array_equal(oracle.gla_fwd_beta(q, k, v, a, zero, 3, 3, 2), oracle.gla_fwd(q, k, v, a, 3, 3, 2))
    g1 = oracle.gla_bwd_beta(q, k, v, a, zero, dO, 3, 3, 2)
    g0 = oracle.gla_bwd(q, k, v, a, dO, 3, 3, 2)
    for x, y in zip(g1[:4], g0):
        np.testing.assert_allclose(x, y, rtol=1e-14, atol=1e-14)


def test_parallel_form_written_out():
    # o_t[e] = sum_{s <= t} (sum_c q_tc k_sc e^{Lam_tc - Lam_sc}) v_se e^{M_te - M_se}, Lam / M inclusive prefix sums
    q, k, v, a, bg, _ = _inputs(1, L=12)
    o = oracle.gla_fwd_beta(q, k, v, a, bg, 1, 12, 0)
    Lam, M = np.cumsum(a, axis=1), np.cumsum(bg, axis=1)
    ref = np.zeros_like(v)
    for h in range(2):
        for t in range(12):
            for s in range(t + 1):
                w = np.sum(q[0, t, h] * k[0, s, h] * np.exp(Lam[0, t, h] - Lam[0, s, h]))
                ref[0, t, h] += w * v[0, s, h] * np.exp(M[0, t, h] - M[0, s, h])
    np.testing.assert_allclose(o, ref, rtol=1e-12, atol=1e-13)


def test_role_swap_of_the_two_gates():
    # with d_k = d_v the state of (k, v, alpha, beta) is the transpose of the state of (v, k, beta, alpha)
    rng = np.random.default_rng(2)
    L, d = 7, 3
    k, v = rng.standard_normal((1, L, 1, d)), rng.standard_normal((1, L, 1, d))
    a, bg = -rng.random((1, L, 1, d)), -rng.random((1, L, 1, d))
    eye = np.zeros((1, L, 1, d))
    # read out row c of the final state with a one-hot query at the last position only
    S1, S2 = np.zeros((d, d)), np.zeros((d, d))
    for c in range(d):
        qq = eye.copy()
        qq[0, L - 1, 0, c] = 1.0
        S1[c] = oracle.gla_fwd_beta(qq, k, v, a, bg, 1, L, 0)[0, L - 1, 0]
        S2[c] = oracle.gla_fwd_beta(qq, v, k, bg, a, 1, L, 0)[0, L - 1, 0]
    np.testing.assert_allclose(S1, S2.T, rtol=1e-13, atol=1e-14)


@pytest.mark.parametrize("direction", [0, 3])
def test_gradients_by_finite_differences(direction):
    q, k, v, a, bg, dO = _inputs(3, L=6)
    grads = oracle.gla_bwd_beta(q, k, v, a, bg, dO, 2, 3, direction)
    f = lambda *x: float((oracle.gla_fwd_beta(*x, 2, 3, direction) * dO).sum())
    args = [q, k, v, a, bg]
    h = 1e-6
    for which, grad in enumerate(grads):
        arr = args[which]
        for idx in np.ndindex(arr.shape):
            ap, am = arr.copy(), arr.copy()
            ap[idx] += h
            am[idx] -= h
            pa, ma = list(args), list(args)
            pa[which], ma[which] = ap, am
            fd = (f(*pa) - f(*ma)) / (2 * h)
            assert abs(fd - grad[idx]) <= 2e-7 * max(1.0, abs(fd)), (which, idx, fd, grad[idx])


def test_suffix_sum_identities_of_both_gate_gradients():
    q, k, v, a, bg, dO = _inputs(4, B=2, L=12)
    o = oracle.gla_fwd_beta(q, k, v, a, bg, 3, 4, 1)
    dq, dk, dv, da, db = oracle.gla_bwd_beta(q, k, v, a, bg, dO, 3, 4, 1)
    p = oracle.perm(1, 3, 4)                      # scan position -> token
    xa = (q * dq - k * dk)[:, p]
    xb = (o * dO - v * dv)[:, p]
    np.testing.assert_allclose(da[:, p], np.cumsum(xa[:, ::-1], axis=1)[:, ::-1], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(db[:, p], np.cumsum(xb[:, ::-1], axis=1)[:, ::-1], rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("direction", [0, 1, 2, 3])
def test_suffix_sum_identities_across_checkpoint_segments(direction):
    """Both identities on 200 scan positions, more than one stored-state segment of the backward sweep."""
    q, k, v, a, bg, dO = _inputs(5 + direction, B=1, L=200)
    a, bg = a * 0.4, bg * 0.4
    gh, gw = 10, 20
    o = oracle.gla_fwd_beta(q, k, v, a, bg, gh, gw, direction)
    dq, dk, dv, da, db = oracle.gla_bwd_beta(q, k, v, a, bg, dO, gh, gw, direction)
    p = oracle.perm(direction, gh, gw)
    xa = (q * dq - k * dk)[:, p]
    xb = (o * dO - v * dv)[:, p]
    np.testing.assert_allclose(da[:, p], np.cumsum(xa[:, ::-1], axis=1)[:, ::-1], rtol=1e-9, atol=1e-10)
    np.testing.assert_allclose(db[:, p], np.cumsum(xb[:, ::-1], axis=1)[:, ::-1], rtol=1e-9, atol=1e-10)
