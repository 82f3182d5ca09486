"""fp64 CPU oracle for the DiG token-mixer hot path.  TEST INFRASTRUCTURE ONLY.

Thin ctypes loader around ``dig_oracle.c`` (plain C, fp64, token-by-token).  Only the test
suite, the smoke check and the benchmark's CPU-baseline leg may import this package; the
product path never does.  Nothing here shares code with the CUDA library.

All tensors are numpy float64, C-contiguous, layout ``[B, L, H, d]`` with ``L = grid_h*grid_w``
in canonical row-major token order.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dig_oracle.c")
_LIB = os.path.join(_HERE, "libdig_oracle.so")
_lock = threading.Lock()
_lib = None

ROW_FWD, ROW_REV, COL_FWD, COL_REV = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over (batch, head) pairs only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            build()
            lib = ctypes.CDLL(_LIB)
            dp = ctypes.POINTER(ctypes.c_double)
            lib.dig_oracle_perm.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                            ctypes.POINTER(ctypes.c_longlong)]
            lib.dig_oracle_gate.argtypes = [dp, dp, dp, ctypes.c_longlong, ctypes.c_longlong,
                                            ctypes.c_int, ctypes.c_int]
            lib.dig_oracle_gla_fwd.argtypes = [dp] * 5 + [ctypes.c_int] * 8
            lib.dig_oracle_gla_bwd.argtypes = [dp] * 9 + [ctypes.c_int] * 8
            lib.dig_oracle_gla_fwd_state.argtypes = [dp] * 7 + [ctypes.c_int] * 8
            lib.dig_oracle_gla_bwd_state.argtypes = [dp] * 12 + [ctypes.c_int] * 8
            lib.dig_oracle_gla_fwd_beta.argtypes = [dp] * 6 + [ctypes.c_int] * 8
            lib.dig_oracle_gla_bwd_beta.argtypes = [dp] * 11 + [ctypes.c_int] * 8
            lib.dig_oracle_dwconv.argtypes = [dp] * 4 + [ctypes.c_int] * 5
            lib.dig_oracle_dwconv_bwd.argtypes = [dp] * 6 + [ctypes.c_int] * 5
            lib.dig_oracle_outgate_fwd.argtypes = [dp] * 5 + [ctypes.c_longlong, ctypes.c_int, ctypes.c_double]
            lib.dig_oracle_outgate_bwd.argtypes = [dp] * 9 + [ctypes.c_longlong, ctypes.c_int, ctypes.c_double]
            _lib = lib
    return _lib


def _f64(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def perm(direction: int, grid_h: int, grid_w: int) -> np.ndarray:
    """perm[p] = canonical token (y*grid_w + x) visited at scan position p."""
    out = np.empty(grid_h * grid_w, dtype=np.int64)
    rc = _load().dig_oracle_perm(direction, grid_h, grid_w,
                                 out.ctypes.data_as(ctypes.POINTER(ctypes.c_longlong)))
    _check(rc, "perm")
    return out


def gate(x, tau_per_head) -> np.ndarray:
    """a = logsigmoid(x) / tau[h]  (log of Eq. gate_gla's alpha).  x: [B, L, H, d_k]."""
    x = _f64(x)
    B, L, H, dk = x.shape
    tau = _f64(tau_per_head)
    assert tau.shape == (H,)
    out = np.empty_like(x)
    _check(_load().dig_oracle_gate(_p(x), _p(tau), _p(out), B, L, H, dk), "gate")
    return out


def gla_fwd(q, k, v, a, grid_h, grid_w, direction=ROW_FWD, threads=1) -> np.ndarray:
    """o_t = q_t S_t with S_t = diag(exp(a_t)) S_{t-1} + k_t^T v_t, scanned in `direction`."""
    q, k, v, a = map(_f64, (q, k, v, a))
    B, L, H, dk = q.shape
    dv = v.shape[-1]
    assert L == grid_h * grid_w and k.shape == q.shape == a.shape and v.shape == (B, L, H, dv)
    out = np.empty_like(v)
    _check(_load().dig_oracle_gla_fwd(_p(q), _p(k), _p(v), _p(a), _p(out), B, H, grid_h, grid_w,
                                      dk, dv, direction, threads), "gla_fwd")
    return out


def gla_bwd(q, k, v, a, dout, grid_h, grid_w, direction=ROW_FWD, threads=1):
    """Gradients (dq, dk, dv, da) of <dout, gla_fwd(q,k,v,a)>."""
    q, k, v, a, dout = map(_f64, (q, k, v, a, dout))
    B, L, H, dk = q.shape
    dv_ = v.shape[-1]
    assert L == grid_h * grid_w and dout.shape == v.shape
    dq, dk_, da = np.empty_like(q), np.empty_like(q), np.empty_like(q)
    dv = np.empty_like(v)
    _check(_load().dig_oracle_gla_bwd(_p(q), _p(k), _p(v), _p(a), _p(dout), _p(dq), _p(dk_),
                                      _p(dv), _p(da), B, H, grid_h, grid_w, dk, dv_, direction,
                                      threads), "gla_bwd")
    return dq, dk_, dv, da


def dwconv(x, w, bias, grid_h, grid_w, direction=ROW_FWD) -> np.ndarray:
    """3x3 depthwise conv of the SREM module on the re-oriented token matrix.
    x: [B, L, D] canonical order, w: [3, 3, D], bias: [D] or None."""
    x, w = _f64(x), _f64(w)
    B, L, D = x.shape
    assert L == grid_h * grid_w and w.shape == (3, 3, D)
    bp = None
    if bias is not None:
        bias = _f64(bias)
        assert bias.shape == (D,)
        bp = _p(bias)
    y = np.empty_like(x)
    _check(_load().dig_oracle_dwconv(_p(x), _p(w), bp, _p(y), B, grid_h, grid_w, D, direction),
           "dwconv")
    return y


def dwconv_bwd(x, w, dy, grid_h, grid_w, direction=ROW_FWD, with_bias=True):
    """Gradients (dx, dw, dbias) of <dy, dwconv(x, w, bias)>; dbias is None if with_bias is False."""
    x, w, dy = _f64(x), _f64(w), _f64(dy)
    B, L, D = x.shape
    assert L == grid_h * grid_w and w.shape == (3, 3, D) and dy.shape == x.shape
    dx, dw = np.empty_like(x), np.empty_like(w)
    db = np.empty(D, dtype=np.float64) if with_bias else None
    _check(_load().dig_oracle_dwconv_bwd(_p(x), _p(w), _p(dy), _p(dx), _p(dw), None if db is None else _p(db),
                                         B, grid_h, grid_w, D, direction), "dwconv_bwd")
    return dx, dw, db


def _opt(a, d):
    if a is None:
        return None, None
    a = _f64(a)
    assert a.shape == (d,)
    return a, _p(a)


def outgate(o, r, ln_w=None, ln_b=None, eps=1e-5) -> np.ndarray:
    """z = Swish(r) * LN(o) per row of the last axis (Eq. attn_gla, the line forming Y_t)."""
    o, r = _f64(o), _f64(r)
    assert o.shape == r.shape
    d = o.shape[-1]
    (_w, wp), (_b, bp) = _opt(ln_w, d), _opt(ln_b, d)
    z = np.empty_like(o)
    _check(_load().dig_oracle_outgate_fwd(_p(o), _p(r), wp, bp, _p(z), o.size // d, d, float(eps)), "outgate")
    return z


def outgate_bwd(o, r, dz, ln_w=None, ln_b=None, eps=1e-5):
    """Gradients (do, dr, dln_w, dln_b) of <dz, outgate(o, r, ln_w, ln_b)>; the affine gradients are
    those with respect to a weight of ones / a bias of zeros where the argument is None."""
    o, r, dz = _f64(o), _f64(r), _f64(dz)
    assert o.shape == r.shape == dz.shape
    d = o.shape[-1]
    (_w, wp), (_b, bp) = _opt(ln_w, d), _opt(ln_b, d)
    do, dr = np.empty_like(o), np.empty_like(o)
    dw, db = np.empty(d), np.empty(d)
    _check(_load().dig_oracle_outgate_bwd(_p(o), _p(r), wp, bp, _p(dz), _p(do), _p(dr), _p(dw), _p(db),
                                          o.size // d, d, float(eps)), "outgate_bwd")
    return do, dr, dw, db


def gla_fwd_state(q, k, v, a, s_in, grid_h, grid_w, direction=ROW_FWD, threads=1):
    """gla_fwd started from state s_in ([B, H, d_k, d_v] or None = zero); returns (out, s_out)."""
    q, k, v, a = map(_f64, (q, k, v, a))
    B, L, H, dk = q.shape
    dv = v.shape[-1]
    assert L == grid_h * grid_w and k.shape == q.shape == a.shape and v.shape == (B, L, H, dv)
    sp = None
    if s_in is not None:
        s_in = _f64(s_in)
        assert s_in.shape == (B, H, dk, dv)
        sp = _p(s_in)
    out, s_out = np.empty_like(v), np.empty((B, H, dk, dv))
    _check(_load().dig_oracle_gla_fwd_state(_p(q), _p(k), _p(v), _p(a), sp, _p(out), _p(s_out), B, H, grid_h,
                                            grid_w, dk, dv, direction, threads), "gla_fwd_state")
    return out, s_out


def gla_bwd_state(q, k, v, a, dout, s_in, ds_out, grid_h, grid_w, direction=ROW_FWD, threads=1):
    """Gradients (dq, dk, dv, da, ds_in) of <dout, out> + <ds_out, s_out> for gla_fwd_state."""
    q, k, v, a, dout = map(_f64, (q, k, v, a, dout))
    B, L, H, dk = q.shape
    dv_ = v.shape[-1]
    assert L == grid_h * grid_w and dout.shape == v.shape
    sp = dp_ = None
    if s_in is not None:
        s_in = _f64(s_in)
        assert s_in.shape == (B, H, dk, dv_)
        sp = _p(s_in)
    if ds_out is not None:
        ds_out = _f64(ds_out)
        assert ds_out.shape == (B, H, dk, dv_)
        dp_ = _p(ds_out)
    dq, dk_, da = np.empty_like(q), np.empty_like(q), np.empty_like(q)
    dv = np.empty_like(v)
    ds_in = np.empty((B, H, dk, dv_))
    _check(_load().dig_oracle_gla_bwd_state(_p(q), _p(k), _p(v), _p(a), _p(dout), sp, dp_, _p(dq), _p(dk_),
                                            _p(dv), _p(da), _p(ds_in), B, H, grid_h, grid_w, dk, dv_, direction,
                                            threads), "gla_bwd_state")
    return dq, dk_, dv, da, ds_in


def gla_fwd_beta(q, k, v, a, bg, grid_h, grid_w, direction=ROW_FWD, threads=1) -> np.ndarray:
    """gla_fwd with the full gate of Eq. gate_gla: S_t = diag(e^a_t) S_{t-1} diag(e^bg_t) + k_t^T v_t.
    bg = log(beta), [B, L, H, d_v]."""
    q, k, v, a, bg = map(_f64, (q, k, v, a, bg))
    B, L, H, dk = q.shape
    dv = v.shape[-1]
    assert L == grid_h * grid_w and k.shape == q.shape == a.shape and v.shape == (B, L, H, dv) == bg.shape
    out = np.empty_like(v)
    _check(_load().dig_oracle_gla_fwd_beta(_p(q), _p(k), _p(v), _p(a), _p(bg), _p(out), B, H, grid_h, grid_w,
                                           dk, dv, direction, threads), "gla_fwd_beta")
    return out


def gla_bwd_beta(q, k, v, a, bg, dout, grid_h, grid_w, direction=ROW_FWD, threads=1):
    """Gradients (dq, dk, dv, da, dbg) of <dout, gla_fwd_beta(q, k, v, a, bg)>."""
    q, k, v, a, bg, dout = map(_f64, (q, k, v, a, bg, dout))
    B, L, H, dk = q.shape
    dv_ = v.shape[-1]
    assert L == grid_h * grid_w and dout.shape == v.shape == bg.shape
    dq, dk_, da = np.empty_like(q), np.empty_like(q), np.empty_like(q)
    dv, db = np.empty_like(v), np.empty_like(v)
    _check(_load().dig_oracle_gla_bwd_beta(_p(q), _p(k), _p(v), _p(a), _p(bg), _p(dout), _p(dq), _p(dk_), _p(dv),
                                           _p(da), _p(db), B, H, grid_h, grid_w, dk, dv_, direction, threads),
           "gla_bwd_beta")
    return dq, dk_, dv, da, db


# ---- several scan orders summed (Algorithm 2: bidirectional, Algorithm 3: 4-directional scanning) ----
def _scan_order(direction: int, grid_h: int, grid_w: int) -> np.ndarray:
    """Token visited at each position after the re-orderings the algorithms apply to the sequence:
    nothing, flip, flatten(transpose(reshape2d)), and flip of the transposed sequence."""
    idx = np.arange(grid_h * grid_w)
    if direction in (COL_FWD, COL_REV):
        idx = idx.reshape(grid_h, grid_w).T.reshape(-1)
    if direction in (ROW_REV, COL_REV):
        idx = idx[::-1]
    return np.ascontiguousarray(idx)


def gla_fwd_multi(q, k, v, a, grid_h, grid_w, directions, threads=1) -> np.ndarray:
    """z_out = sum over the listed scan orders of GLA(re-ordered sequence) brought back to the input
    order, written out as the algorithms do: permute, run the recurrence on the plain sequence, undo
    the permutation, add."""
    q, k, v, a = _f64(q), _f64(k), _f64(v), _f64(a)
    L = grid_h * grid_w
    out = np.zeros_like(v)
    for d in directions:
        p = _scan_order(d, grid_h, grid_w)
        o = gla_fwd(q[:, p], k[:, p], v[:, p], a[:, p], 1, L, ROW_FWD, threads=threads)
        back = np.empty_like(o)
        back[:, p] = o
        out += back
    return out


def gla_bwd_multi(q, k, v, a, dout, grid_h, grid_w, directions, threads=1):
    """Gradients of <dout, gla_fwd_multi(...)> with respect to q, k, v and a: the sum over the scan
    orders of the single-order gradients, each computed on the re-ordered sequence and brought back."""
    q, k, v, a, dout = _f64(q), _f64(k), _f64(v), _f64(a), _f64(dout)
    L = grid_h * grid_w
    tot = [np.zeros_like(q), np.zeros_like(k), np.zeros_like(v), np.zeros_like(a)]
    for d in directions:
        p = _scan_order(d, grid_h, grid_w)
        gs = gla_bwd(q[:, p], k[:, p], v[:, p], a[:, p], dout[:, p], 1, L, ROW_FWD, threads=threads)
        for t, g_ in zip(tot, gs):
            back = np.empty_like(g_)
            back[:, p] = g_
            t += back
    return tuple(tot)
