"""Pins for the fp64 GLA oracle: each test checks it against something the definition or the
mathematics fixes independently of the oracle's own loops."""
import numpy as np
import pytest

import oracle


def _rand(rng, B, L, H, dk, dv, decay_scale=0.3):
    q = rng.standard_normal((B, L, H, dk))
    k = rng.standard_normal((B, L, H, dk))
    v = rng.standard_normal((B, L, H, dv))
    a = -np.abs(rng.standard_normal((B, L, H, dk))) * decay_scale
    return q, k, v, a


def _scan_orders(gh, gw):
    """The four orders built with numpy reshapes only (independent of the oracle's C code)."""
    idx = np.arange(gh * gw)
    col = idx.reshape(gh, gw).T.ravel()
    return {0: idx, 1: idx[::-1].copy(), 2: col, 3: col[::-1].copy()}


def _parallel_literal(q, k, v, a):
    """O = ((Q*Bc)(K/Bc)^T * M) V with Bc_t = prod_{r<=t} alpha_r, M lower-triangular incl. diagonal."""
    L = q.shape[0]
    Bc = np.exp(np.cumsum(a, axis=0))
    M = np.tril(np.ones((L, L)))
    return (((q * Bc) @ (k / Bc).T) * M) @ v


def _parallel_stable(q, k, v, a):
    """A_ts = sum_c q_tc k_sc exp(Lam_tc - Lam_sc) for s <= t, built entry by entry."""
    L = q.shape[0]
    Lam = np.cumsum(a, axis=0)
    A = np.zeros((L, L))
    for t in range(L):
        for s in range(t + 1):
            A[t, s] = np.sum(q[t] * k[s] * np.exp(Lam[t] - Lam[s]))
    return A @ v, A


def test_matches_literal_parallel_form_tiny():
    rng = np.random.default_rng(1)
    q, k, v, a = _rand(rng, 2, 12, 3, 5, 4)
    o = oracle.gla_fwd(q, k, v, a, 3, 4)
    for b in range(2):
        for h in range(3):
            ref = _parallel_literal(q[b, :, h], k[b, :, h], v[b, :, h], a[b, :, h])
            np.testing.assert_allclose(o[b, :, h], ref, rtol=1e-11, atol=1e-11)


def test_matches_stable_parallel_form_longer():
    rng = np.random.default_rng(2)
    q, k, v, a = _rand(rng, 1, 160, 2, 6, 7, decay_scale=1.5)   # literal form would lose digits here
    o = oracle.gla_fwd(q, k, v, a, 10, 16)
    for h in range(2):
        ref, _ = _parallel_stable(q[0, :, h], k[0, :, h], v[0, :, h], a[0, :, h])
        np.testing.assert_allclose(o[0, :, h], ref, rtol=1e-11, atol=1e-11)


def test_alpha_one_is_causal_linear_attention():
    """Eq. attn_simple: with no decay S_t is a running sum, so O = tril(Q K^T) V."""
    rng = np.random.default_rng(3)
    q, k, v, a = _rand(rng, 1, 48, 2, 8, 8)
    o = oracle.gla_fwd(q, k, v, np.zeros_like(a), 6, 8)
    for h in range(2):
        ref = np.tril(q[0, :, h] @ k[0, :, h].T) @ v[0, :, h]
        np.testing.assert_allclose(o[0, :, h], ref, rtol=1e-12, atol=1e-12)


def test_constant_decay_closed_form():
    """alpha == gamma for every token and channel gives weights gamma^(t-s): the token that
    enters at step s is decayed once per later step, never at its own step."""
    rng = np.random.default_rng(4)
    L, gamma = 40, 0.9
    q, k, v, a = _rand(rng, 1, L, 1, 4, 3)
    a[:] = np.log(gamma)
    o = oracle.gla_fwd(q, k, v, a, 5, 8)
    t = np.arange(L)
    Dm = np.where(t[:, None] >= t[None, :], gamma ** (t[:, None] - t[None, :]).clip(0), 0.0)
    ref = ((q[0, :, 0] @ k[0, :, 0].T) * Dm) @ v[0, :, 0]
    np.testing.assert_allclose(o[0, :, 0], ref, rtol=1e-12, atol=1e-12)


def test_fast_decay_and_single_token_limits():
    rng = np.random.default_rng(5)
    q, k, v, a = _rand(rng, 1, 20, 2, 6, 5)
    o = oracle.gla_fwd(q, k, v, np.full_like(a, -60.0), 4, 5)
    ref = np.sum(q * k, axis=-1, keepdims=True) * v          # o_t = (q_t . k_t) v_t
    np.testing.assert_allclose(o, ref, rtol=1e-12, atol=1e-12)
    q1, k1, v1, a1 = _rand(rng, 2, 1, 2, 6, 5)
    o1 = oracle.gla_fwd(q1, k1, v1, a1, 1, 1)                # L = 1: gate is irrelevant
    np.testing.assert_allclose(o1, np.sum(q1 * k1, -1, keepdims=True) * v1, rtol=1e-13, atol=1e-13)


def test_bilinear_in_qk_and_linear_in_v():
    rng = np.random.default_rng(6)
    q, k, v, a = _rand(rng, 1, 30, 2, 4, 4)
    q2, k2, v2, _ = _rand(rng, 1, 30, 2, 4, 4)
    f = lambda qq, kk, vv: oracle.gla_fwd(qq, kk, vv, a, 5, 6)
    np.testing.assert_allclose(f(q + 2 * q2, k, v), f(q, k, v) + 2 * f(q2, k, v), rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(f(q, k - 3 * k2, v), f(q, k, v) - 3 * f(q, k2, v), rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(f(q, k, v + v2), f(q, k, v) + f(q, k, v2), rtol=1e-11, atol=1e-11)


@pytest.mark.parametrize("direction", [0, 1, 2, 3])
def test_direction_equals_permute_scan_unpermute(direction):
    rng = np.random.default_rng(7)
    gh, gw = 3, 5
    q, k, v, a = _rand(rng, 2, gh * gw, 2, 4, 3)
    p = _scan_orders(gh, gw)[direction]
    o_dir = oracle.gla_fwd(q, k, v, a, gh, gw, direction)
    # permute tokens into scan order, run the plain row-major scan on a 1 x L grid, un-permute
    o_seq = oracle.gla_fwd(q[:, p], k[:, p], v[:, p], a[:, p], 1, gh * gw, 0)
    ref = np.empty_like(o_seq)
    ref[:, p] = o_seq
    np.testing.assert_array_equal(o_dir, ref)
    if direction != 0:
        assert not np.allclose(o_dir, oracle.gla_fwd(q, k, v, a, gh, gw, 0))


def _loss(q, k, v, a, dO, gh, gw, direction):
    return float(np.sum(dO * oracle.gla_fwd(q, k, v, a, gh, gw, direction)))


@pytest.mark.parametrize("direction", [0, 3])
def test_backward_matches_central_finite_differences(direction):
    rng = np.random.default_rng(8)
    gh, gw = 3, 4
    q, k, v, a = _rand(rng, 1, gh * gw, 2, 3, 4)
    dO = rng.standard_normal(v.shape)
    grads = oracle.gla_bwd(q, k, v, a, dO, gh, gw, direction)
    args = [q, k, v, a]
    h = 1e-6
    for which in range(4):
        g = grads[which]
        flat_idx = rng.choice(g.size, size=25, replace=False)
        for fi in flat_idx:
            idx = np.unravel_index(fi, g.shape)
            plus = [x.copy() for x in args]
            minus = [x.copy() for x in args]
            plus[which][idx] += h
            minus[which][idx] -= h
            fd = (_loss(*plus, dO, gh, gw, direction) - _loss(*minus, dO, gh, gw, direction)) / (2 * h)
            assert abs(fd - g[idx]) <= 1e-7 * max(1.0, abs(fd)), (which, idx, fd, g[idx])


def test_backward_long_sequence_crosses_checkpoints():
    """dV = A^T dO and dQ, dK from the explicit attention matrix A of the stable parallel form;
    L = 200 spans several checkpoint segments of the oracle's backward sweep."""
    rng = np.random.default_rng(9)
    L = 200
    q, k, v, a = _rand(rng, 1, L, 1, 3, 4, decay_scale=0.2)
    dO = rng.standard_normal(v.shape)
    dq, dk, dv, da = oracle.gla_bwd(q, k, v, a, dO, 10, 20)
    _, A = _parallel_stable(q[0, :, 0], k[0, :, 0], v[0, :, 0], a[0, :, 0])
    np.testing.assert_allclose(dv[0, :, 0], A.T @ dO[0, :, 0], rtol=1e-10, atol=1e-10)
    # dA = dO V^T on the causal support; dq_t = sum_s dA_ts k_s exp(Lam_t - Lam_s)
    Lam = np.cumsum(a[0, :, 0], axis=0)
    dA = np.tril(dO[0, :, 0] @ v[0, :, 0].T)
    dq_ref = np.zeros_like(dq[0, :, 0])
    dk_ref = np.zeros_like(dq_ref)
    for t in range(L):
        for s in range(t + 1):
            w = np.exp(Lam[t] - Lam[s])
            dq_ref[t] += dA[t, s] * k[0, s, 0] * w
            dk_ref[s] += dA[t, s] * q[0, t, 0] * w
    np.testing.assert_allclose(dq[0, :, 0], dq_ref, rtol=1e-10, atol=1e-10)
    np.testing.assert_allclose(dk[0, :, 0], dk_ref, rtol=1e-10, atol=1e-10)


@pytest.mark.parametrize("direction", [0, 1, 2])
def test_gate_gradient_suffix_sum_identity(direction):
    """da_t = sum over scan positions at or after t of (q*dq - k*dk); hence da at the first
    scan position is 0, and sum_t q_t.dq_t = <dO, O>."""
    rng = np.random.default_rng(10)
    gh, gw = 4, 6
    q, k, v, a = _rand(rng, 2, gh * gw, 2, 5, 3)
    dO = rng.standard_normal(v.shape)
    dq, dk, dv, da = oracle.gla_bwd(q, k, v, a, dO, gh, gw, direction)
    p = _scan_orders(gh, gw)[direction]
    x = (q * dq - k * dk)[:, p]                                # scan order
    suffix = np.cumsum(x[:, ::-1], axis=1)[:, ::-1]
    np.testing.assert_allclose(da[:, p], suffix, rtol=1e-10, atol=1e-10)
    np.testing.assert_allclose(da[:, p[0]], 0.0, atol=1e-10)
    o = oracle.gla_fwd(q, k, v, a, gh, gw, direction)
    np.testing.assert_allclose(np.sum(q * dq), np.sum(dO * o), rtol=1e-11)
    np.testing.assert_allclose(np.sum(v * dv), np.sum(dO * o), rtol=1e-11)


@pytest.mark.parametrize("direction", [0, 1, 2, 3])
def test_gate_gradient_suffix_sum_identity_across_checkpoint_segments(direction):
    """The same identity on 200 scan positions (10 x 20 grid): the oracle's backward sweep restarts
    from a stored state several times on the way, so a slip in how the gate gradient uses the
    recomputed states would break the running sum here while leaving short sequences intact."""
    rng = np.random.default_rng(20 + direction)
    gh, gw = 10, 20
    q, k, v, a = _rand(rng, 1, gh * gw, 2, 4, 3, decay_scale=0.25)
    dO = rng.standard_normal(v.shape)
    dq, dk, dv, da = oracle.gla_bwd(q, k, v, a, dO, gh, gw, direction)
    p = _scan_orders(gh, gw)[direction]
    x = (q * dq - k * dk)[:, p]
    suffix = np.cumsum(x[:, ::-1], axis=1)[:, ::-1]
    np.testing.assert_allclose(da[:, p], suffix, rtol=1e-9, atol=1e-10)
    np.testing.assert_allclose(da[:, p[0]], 0.0, atol=1e-10)


def test_threads_do_not_change_results():
    rng = np.random.default_rng(11)
    q, k, v, a = _rand(rng, 2, 64, 3, 8, 8)
    dO = rng.standard_normal(v.shape)
    np.testing.assert_array_equal(oracle.gla_fwd(q, k, v, a, 8, 8, 2, threads=1),
                                  oracle.gla_fwd(q, k, v, a, 8, 8, 2, threads=4))
    g1 = oracle.gla_bwd(q, k, v, a, dO, 8, 8, 1, threads=1)
    g4 = oracle.gla_bwd(q, k, v, a, dO, 8, 8, 1, threads=4)
    for x, y in zip(g1, g4):
        np.testing.assert_array_equal(x, y)
