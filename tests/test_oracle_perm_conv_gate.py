"""Pins for the oracle's scan orders, SREM depthwise convolution and gate transform."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
NAMES = {"row_fwd": 0, "row_rev": 1, "col_fwd": 2, "col_rev": 3}


def _golden_orders():
    orders, cycles = {}, {}
    with open(os.path.join(GOLDEN, "scan_orders_2x3.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, *rest = line.split()
            if name in NAMES:
                orders[name] = np.array([int(x) for x in rest])
            else:
                cycles[name] = rest
    return orders, cycles


def test_perm_matches_hand_worked_orders():
    orders, _ = _golden_orders()
    for name, d in NAMES.items():
        np.testing.assert_array_equal(oracle.perm(d, 2, 3), orders[name])


@pytest.mark.parametrize("gh,gw", [(2, 3), (3, 5), (4, 4), (1, 7), (6, 1)])
def test_perm_is_bijection_and_relations(gh, gw):
    L = gh * gw
    p = {d: oracle.perm(d, gh, gw) for d in range(4)}
    for d in range(4):
        assert sorted(p[d].tolist()) == list(range(L))
        inv = np.empty(L, dtype=np.int64)
        inv[p[d]] = np.arange(L)
        np.testing.assert_array_equal(p[d][inv], np.arange(L))
    np.testing.assert_array_equal(p[0], np.arange(L))
    np.testing.assert_array_equal(p[1], p[0][::-1])
    np.testing.assert_array_equal(p[2], np.arange(L).reshape(gh, gw).T.ravel())
    np.testing.assert_array_equal(p[3], p[2][::-1])


def _run_schedule(gh, gw, op_for_block, nblocks):
    """Apply flip / transpose block after block to the token-id sequence, tracking the matrix shape."""
    seq, shape, seen = np.arange(gh * gw), (gh, gw), []
    for l in range(1, nblocks + 1):
        seen.append(seq.copy())
        if op_for_block(l) == "flip":
            seq = seq[::-1].copy()
        else:
            seq = seq.reshape(shape).T.ravel().copy()
            shape = (shape[1], shape[0])
    return seen


@pytest.mark.parametrize("gh,gw", [(2, 3), (3, 5), (4, 4)])
def test_block_by_block_schedules_cycle_through_the_four_orders(gh, gw):
    _, cycles = _golden_orders()
    alg1 = _run_schedule(gh, gw, lambda l: "transpose" if l % 2 == 0 else "flip", 5)
    alg4 = _run_schedule(gh, gw, lambda l: "flip" if l % 2 == 0 else "transpose", 5)
    for seen, key in ((alg1, "alg1_cycle"), (alg4, "alg4_cycle")):
        for seq, name in zip(seen, cycles[key]):
            np.testing.assert_array_equal(seq, oracle.perm(NAMES[name], gh, gw))


# ---------------------------------------------------------------- depthwise conv

def test_conv_identity_init_returns_input_bit_exact():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((2, 20, 6))
    w = np.zeros((3, 3, 6))
    w[1, 1] = 1.0
    for d in range(4):
        np.testing.assert_array_equal(oracle.dwconv(x, w, None, 4, 5, d), x)


def test_conv_all_ones_counts_taps():
    want = np.loadtxt(os.path.join(GOLDEN, "dwconv_ones_3x4.txt"))
    y = oracle.dwconv(np.ones((1, 12, 2)), np.ones((3, 3, 2)), None, 3, 4, 0)
    np.testing.assert_array_equal(y[0, :, 0].reshape(3, 4), want)
    np.testing.assert_array_equal(y[0, :, 1].reshape(3, 4), want)


def test_conv_is_cross_correlation_with_zero_padding():
    """A single bright pixel at (i0,j0) and tap (u,v): y[i0-(u-1), j0-(v-1)] = w[u,v]."""
    gh, gw = 5, 6
    w = np.arange(1, 10, dtype=np.float64).reshape(3, 3, 1)
    x = np.zeros((1, gh * gw, 1))
    i0, j0 = 2, 3
    x[0, i0 * gw + j0, 0] = 1.0
    y = oracle.dwconv(x, w, None, gh, gw, 0)[0, :, 0].reshape(gh, gw)
    for u in range(3):
        for v in range(3):
            assert y[i0 - (u - 1), j0 - (v - 1)] == w[u, v, 0]
    assert np.count_nonzero(y) == 9
    # bias is added once per output
    yb = oracle.dwconv(x, w, np.array([0.5]), gh, gw, 0)[0, :, 0].reshape(gh, gw)
    np.testing.assert_allclose(yb, y + 0.5)


def _conv_direct(x2d, w):
    """Plain 3x3 zero-padded cross-correlation written with shifted slices (numpy only)."""
    R, C, D = x2d.shape
    pad = np.zeros((R + 2, C + 2, D))
    pad[1:-1, 1:-1] = x2d
    out = np.zeros_like(x2d)
    for u in range(3):
        for v in range(3):
            out += w[u, v] * pad[u:u + R, v:v + C]
    return out


@pytest.mark.parametrize("gh,gw", [(3, 3), (4, 7), (8, 8)])
def test_conv_in_reoriented_layout_equals_canonical_conv_with_transformed_kernel(gh, gw):
    rng = np.random.default_rng(1)
    D = 5
    x = rng.standard_normal((2, gh * gw, D))
    w = rng.standard_normal((3, 3, D))
    kernels = {0: w, 1: w[::-1, ::-1], 2: w.transpose(1, 0, 2), 3: w.transpose(1, 0, 2)[::-1, ::-1]}
    for d in range(4):
        y = oracle.dwconv(x, w, None, gh, gw, d)
        for b in range(2):
            ref = _conv_direct(x[b].reshape(gh, gw, D), kernels[d]).reshape(gh * gw, D)
            np.testing.assert_allclose(y[b], ref, rtol=1e-13, atol=1e-13)


# ---------------------------------------------------------------- gate transform

def test_gate_is_log_of_sigmoid_power():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((2, 7, 3, 4)) * 3
    tau = np.array([16.0, 4.0, 1.0])
    a = oracle.gate(x, tau)
    alpha = (1.0 / (1.0 + np.exp(-x))) ** (1.0 / tau[None, None, :, None])     # Eq. gate_gla
    np.testing.assert_allclose(np.exp(a), alpha, rtol=1e-13)
    from scipy.special import log_expit
    np.testing.assert_allclose(a, log_expit(x) / tau[None, None, :, None], rtol=1e-14, atol=0)
    assert (a < 0).all()


def test_gate_extreme_logits_stay_finite():
    x = np.array([-800.0, -40.0, 0.0, 40.0, 800.0]).reshape(1, 5, 1, 1)
    a = oracle.gate(x, np.array([2.0]))[0, :, 0, 0]
    np.testing.assert_allclose(a[0], -400.0)                 # logsigmoid(x) -> x for x << 0
    np.testing.assert_allclose(a[2], np.log(0.5) / 2)
    assert a[4] == 0.0 or abs(a[4]) < 1e-300
    assert np.isfinite(a).all()


# ---- reverse mode of the SREM convolution --------------------------------------------------------
@pytest.mark.parametrize("direction", [0, 1, 2, 3])
def test_conv_backward_matches_central_finite_differences(direction):
    rng = np.random.default_rng(20 + direction)
    gh, gw, D, B = 4, 5, 3, 2
    x = rng.standard_normal((B, gh * gw, D))
    w = rng.standard_normal((3, 3, D))
    bias = rng.standard_normal(D)
    dy = rng.standard_normal((B, gh * gw, D))
    dx, dw, db = oracle.dwconv_bwd(x, w, dy, gh, gw, direction)
    loss = lambda xx, ww, bb: float((dy * oracle.dwconv(xx, ww, bb, gh, gw, direction)).sum())
    h = 1e-6
    for arr, grad, which in ((x, dx, 0), (w, dw, 1), (bias, db, 2)):
        for _ in range(6):
            idx = tuple(rng.integers(0, n) for n in arr.shape)
            plus, minus = arr.copy(), arr.copy()
            plus[idx] += h
            minus[idx] -= h
            args_p = [x, w, bias]
            args_m = [x, w, bias]
            args_p[which], args_m[which] = plus, minus
            fd = (loss(*args_p) - loss(*args_m)) / (2 * h)
            assert abs(fd - grad[idx]) <= 1e-7 * max(1.0, abs(fd)), (which, idx, fd, grad[idx])


@pytest.mark.parametrize("direction", [0, 1, 2, 3])
def test_conv_backward_is_the_adjoint_of_the_forward_map(direction):
    """<dy, conv(x)> = <dx, x> (the map is linear in x without bias), and likewise in w."""
    rng = np.random.default_rng(30 + direction)
    gh, gw, D = 5, 3, 4
    x = rng.standard_normal((1, gh * gw, D))
    w = rng.standard_normal((3, 3, D))
    dy = rng.standard_normal((1, gh * gw, D))
    dx, dw, db = oracle.dwconv_bwd(x, w, dy, gh, gw, direction)
    y = oracle.dwconv(x, w, None, gh, gw, direction)
    assert abs((dy * y).sum() - (dx * x).sum()) <= 1e-12 * np.abs(dy * y).sum()
    assert abs((dy * y).sum() - (dw * w).sum()) <= 1e-12 * np.abs(dy * y).sum()
    np.testing.assert_allclose(db, dy.sum(axis=(0, 1)), rtol=1e-13)


def test_conv_backward_of_identity_filter_and_single_pixel():
    """Identity-initialised filter (centre tap 1): dx == dy.  A 1 x 1 image only ever touches the
    centre tap: dw is x*dy there and 0 elsewhere."""
    rng = np.random.default_rng(40)
    gh, gw, D = 4, 4, 2
    w = np.zeros((3, 3, D))
    w[1, 1] = 1.0
    x = rng.standard_normal((2, gh * gw, D))
    dy = rng.standard_normal((2, gh * gw, D))
    dx, _, _ = oracle.dwconv_bwd(x, w, dy, gh, gw, 3)
    np.testing.assert_array_equal(dx, dy)
    x1, dy1 = rng.standard_normal((1, 1, D)), rng.standard_normal((1, 1, D))
    _, dw1, _ = oracle.dwconv_bwd(x1, rng.standard_normal((3, 3, D)), dy1, 1, 1, 0)
    want = np.zeros((3, 3, D))
    want[1, 1] = (x1 * dy1)[0, 0]
    np.testing.assert_allclose(dw1, want, rtol=1e-15)
