"""Pins for the oracle's recurrence with a start state and a returned final state (Eq. attn_gla run
from S_in instead of zero): cutting a sequence in two and chaining the pieces through the state must
reproduce the uncut result, values and gradients; closed form of the final state under constant
decay; finite differences of the new arguments."""
import numpy as np
import pytest

import oracle


def _inputs(seed, B=2, H=2, L=12, dk=3, dv=4):
    rng = np.random.default_rng(seed)
    q, k = rng.standard_normal((B, L, H, dk)), rng.standard_normal((B, L, H, dk))
    v, dO = rng.standard_normal((B, L, H, dv)), rng.standard_normal((B, L, H, dv))
    a = -rng.random((B, L, H, dk)) * 0.7
    return q, k, v, a, dO


def test_zero_state_reduces_to_plain_recurrence():
    q, k, v, a, dO = _inputs(0)
    o0 = oracle.gla_fwd(q, k, v, a, 3, 4, 2)
    o1, s1 = oracle.gla_fwd_state(q, k, v, a, None, 3, 4, 2)
    o2, s2 = oracle.gla_fwd_state(q, k, v, a, np.zeros((2, 2, 3, 4)), 3, 4, 2)
    assert np.array_equal(o0, o1) and np.array_equal(o0, o2) and np.array_equal(s1, s2)
    g0 = oracle.gla_bwd(q, k, v, a, dO, 3, 4, 2)
    g1 = oracle.gla_bwd_state(q, k, v, a, dO, None, None, 3, 4, 2)
    for x, y in zip(g0, g1[:4]):
        assert np.array_equal(x, y)


def test_two_pieces_chained_equal_the_whole():
    q, k, v, a, dO = _inputs(1, L=12)
    rng = np.random.default_rng(11)
    s_in, ds_out = rng.standard_normal((2, 2, 3, 4)), rng.standard_normal((2, 2, 3, 4))
    # the whole: a 1 x 12 row; the pieces: 1 x 5 and 1 x 7
    o, s_out = oracle.gla_fwd_state(q, k, v, a, s_in, 1, 12, 0)
    cut = 5
    A = tuple(x[:, :cut] for x in (q, k, v, a, dO))
    Bp = tuple(x[:, cut:] for x in (q, k, v, a, dO))
    oA, sA = oracle.gla_fwd_state(*A[:4], s_in, 1, cut, 0)
    oB, sB = oracle.gla_fwd_state(*Bp[:4], sA, 1, 12 - cut, 0)
    np.testing.assert_allclose(np.concatenate([oA, oB], axis=1), o, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(sB, s_out, rtol=1e-13, atol=1e-13)
    # gradients: run the second piece first, hand its ds_in to the first as ds_out
    dq, dk, dv, da, ds_in = oracle.gla_bwd_state(q, k, v, a, dO, s_in, ds_out, 1, 12, 0)
    gB = oracle.gla_bwd_state(*Bp, sA, ds_out, 1, 12 - cut, 0)
    gA = oracle.gla_bwd_state(*A, s_in, gB[4], 1, cut, 0)
    for whole, pa, pb in zip((dq, dk, dv, da), gA[:4], gB[:4]):
        np.testing.assert_allclose(np.concatenate([pa, pb], axis=1), whole, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(gA[4], ds_in, rtol=1e-12, atol=1e-12)


def test_final_state_closed_form_constant_decay():
    # a == log(g) for every token and channel: S_out = g^L S_in + sum_t g^(L-1-t) k_t^T v_t
    rng = np.random.default_rng(2)
    L, dk, dv, g = 9, 2, 3, 0.8
    k, v = rng.standard_normal((1, L, 1, dk)), rng.standard_normal((1, L, 1, dv))
    s_in = rng.standard_normal((1, 1, dk, dv))
    a = np.full((1, L, 1, dk), np.log(g))
    _, s_out = oracle.gla_fwd_state(np.zeros_like(k), k, v, a, s_in, 3, 3, 0)
    ref = g ** L * s_in[0, 0]
    for t in range(L):
        ref = ref + g ** (L - 1 - t) * np.outer(k[0, t, 0], v[0, t, 0])
    np.testing.assert_allclose(s_out[0, 0], ref, rtol=1e-13)
    # reverse row order (direction 1) consumes the tokens back to front
    _, s_rev = oracle.gla_fwd_state(np.zeros_like(k), k, v, a, s_in, 3, 3, 1)
    ref = g ** L * s_in[0, 0]
    for t in range(L):
        ref = ref + g ** t * np.outer(k[0, t, 0], v[0, t, 0])
    np.testing.assert_allclose(s_rev[0, 0], ref, rtol=1e-13)


@pytest.mark.parametrize("direction", [0, 3])
def test_state_gradients_by_finite_differences(direction):
    q, k, v, a, dO = _inputs(3, B=1, H=2, L=6, dk=2, dv=3)
    rng = np.random.default_rng(33)
    s_in, ds_out = rng.standard_normal((1, 2, 2, 3)), rng.standard_normal((1, 2, 2, 3))

    def loss(q_, k_, v_, a_, s_):
        o, s_out = oracle.gla_fwd_state(q_, k_, v_, a_, s_, 2, 3, direction)
        return float((o * dO).sum() + (s_out * ds_out).sum())

    grads = oracle.gla_bwd_state(q, k, v, a, dO, s_in, ds_out, 2, 3, direction)
    args = [q, k, v, a, s_in]
    h = 1e-6
    for which, grad in zip(range(5), grads):
        arr = args[which]
        for idx in np.ndindex(arr.shape):
            ap, am = arr.copy(), arr.copy()
            ap[idx] += h
            am[idx] -= h
            pa, ma = list(args), list(args)
            pa[which], ma[which] = ap, am
            fd = (loss(*pa) - loss(*ma)) / (2 * h)
            assert abs(fd - grad[idx]) <= 2e-7 * max(1.0, abs(fd)), (which, idx, fd, grad[idx])


@pytest.mark.parametrize("direction", [0, 1, 2, 3])
def test_two_pieces_chained_equal_the_whole_across_checkpoint_segments(direction):
    """A 300-position sequence cut at 170: both pieces are longer than one stored-state segment of
    the backward sweep, so ds_in, da and the other gradients are pinned where states are recomputed.
    The cut is made in scan order (pieces are 1 x n rows holding the tokens in the order visited)."""
    B, H, dk, dv, gh, gw, cut = 1, 2, 3, 4, 15, 20, 170
    L = gh * gw
    q, k, v, a, dO = _inputs(40 + direction, B=B, H=H, L=L, dk=dk, dv=dv)
    a = a * 0.3
    rng = np.random.default_rng(41)
    s_in, ds_out = rng.standard_normal((B, H, dk, dv)), rng.standard_normal((B, H, dk, dv))
    o, s_out = oracle.gla_fwd_state(q, k, v, a, s_in, gh, gw, direction)
    dq, dk_, dv_, da, ds_in = oracle.gla_bwd_state(q, k, v, a, dO, s_in, ds_out, gh, gw, direction)
    idx = np.arange(L)
    col = idx.reshape(gh, gw).T.ravel()
    p = {0: idx, 1: idx[::-1], 2: col, 3: col[::-1]}[direction]          # scan position -> token
    sq, sk, sv, sa, sdO = (x[:, p] for x in (q, k, v, a, dO))
    A = tuple(x[:, :cut] for x in (sq, sk, sv, sa, sdO))
    Bp = tuple(x[:, cut:] for x in (sq, sk, sv, sa, sdO))
    oA, sA = oracle.gla_fwd_state(*A[:4], s_in, 1, cut, 0)
    oB, sB = oracle.gla_fwd_state(*Bp[:4], sA, 1, L - cut, 0)
    np.testing.assert_allclose(np.concatenate([oA, oB], axis=1), o[:, p], rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(sB, s_out, rtol=1e-11, atol=1e-11)
    gB = oracle.gla_bwd_state(*Bp, sA, ds_out, 1, L - cut, 0)
    gA = oracle.gla_bwd_state(*A, s_in, gB[4], 1, cut, 0)
    for whole, pa, pb in zip((dq, dk_, dv_, da), gA[:4], gB[:4]):
        np.testing.assert_allclose(np.concatenate([pa, pb], axis=1), whole[:, p], rtol=1e-9, atol=1e-10)
    np.testing.assert_allclose(gA[4], ds_in, rtol=1e-9, atol=1e-10)
