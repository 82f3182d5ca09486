"""ctypes binding of the C-ABI CUDA library (include/dig_gla.h).

Argument marshalling only: every function forwards torch CUDA tensors as raw device pointers
to the entry point of the same name, on torch's current stream.  There is no CPU path: if the
shared library is missing, loading fails with an error that says how to build it.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdig_gla.so")

DIG_OK = 0
DIG_ERR_INVALID_ARG, DIG_ERR_UNSUPPORTED, DIG_ERR_WORKSPACE, DIG_ERR_CUDA, DIG_ERR_TIMEOUT = 1, 2, 3, 4, 5
DIG_ERR_SCRATCH_LIMIT = 6
DIG_ERR_RANGE = 7
DIG_GLA_STATIC_SCRATCH_BYTES = 16 << 20
DIG_F32, DIG_BF16, DIG_BF16_F32OUT = 0, 1, 2
DIG_ROW_FWD, DIG_ROW_REV, DIG_COL_FWD, DIG_COL_REV = 0, 1, 2, 3
DIG_IMPL_AUTO, DIG_IMPL_FMA, DIG_IMPL_TENSOR, DIG_IMPL_MMA = 0, 1, 2, 3

EXPORTS = ("dig_set_impl", "dig_gla_query_impl", "dig_gla_workspace_bytes", "dig_gate_logsigmoid",
           "dig_gla_fwd", "dig_gla_fwd_static", "dig_gla_bwd", "dig_gla_fwd_state", "dig_gla_bwd_state",
           "dig_gla_fwd_multi", "dig_gla_bwd_multi", "dig_gla_multi_workspace_bytes",
           "dig_gla_fwd_beta", "dig_gla_bwd_beta", "dig_gla_beta_workspace_bytes", "dig_gla_fwd_outgate", "dig_srem_dwconv", "dig_srem_dwconv_bwd",
           "dig_srem_dwconv_bwd_workspace_bytes", "dig_gla_outgate_fwd", "dig_gla_outgate_bwd",
           "dig_gla_outgate_bwd_workspace_bytes", "dig_last_device_status", "dig_selftest_wait_timeout",
           "dig_status_string", "dig_profile_enable", "dig_profile_kernels", "dig_profile_read")

_lib = None


class DigError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (dig_status {status})")


def lib() -> ctypes.CDLL:
    """The loaded shared library with argtypes set.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2405_18428_b200.build` "
                "(needs nvcc); this package has no CPU fallback")
        L = ctypes.CDLL(LIB_PATH)
        vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.dig_set_impl.argtypes = [i]
        L.dig_set_impl.restype = i
        L.dig_gla_query_impl.argtypes = [i] * 5
        L.dig_gla_query_impl.restype = i
        L.dig_gla_workspace_bytes.argtypes = [i] * 9
        L.dig_gla_workspace_bytes.restype = sz
        L.dig_gate_logsigmoid.argtypes = [vp, ctypes.POINTER(ctypes.c_float), vp, i, i, i, i, i, vp]
        L.dig_gate_logsigmoid.restype = i
        L.dig_gla_fwd.argtypes = [vp] * 5 + [i] * 9 + [vp, sz, vp]
        L.dig_gla_fwd.restype = i
        L.dig_gla_fwd_static.argtypes = [vp] * 5 + [i] * 9 + [vp]
        L.dig_gla_fwd_static.restype = i
        L.dig_gla_bwd.argtypes = [vp] * 9 + [i] * 9 + [vp, sz, vp]
        L.dig_gla_bwd.restype = i
        L.dig_gla_multi_workspace_bytes.argtypes = [i] * 9
        L.dig_gla_multi_workspace_bytes.restype = sz
        L.dig_gla_fwd_multi.argtypes = [vp] * 5 + [i] * 7 + [ctypes.c_uint, i] + [vp, sz, vp]
        L.dig_gla_fwd_multi.restype = i
        L.dig_gla_bwd_multi.argtypes = [vp] * 9 + [i] * 7 + [ctypes.c_uint, i] + [vp, sz, vp]
        L.dig_gla_bwd_multi.restype = i
        L.dig_gla_fwd_outgate.argtypes = [vp] * 7 + [ctypes.c_float, vp, vp] + [i] * 9 + [vp, sz, vp]
        L.dig_gla_fwd_outgate.restype = i
        L.dig_gla_beta_workspace_bytes.argtypes = [i] * 9
        L.dig_gla_beta_workspace_bytes.restype = sz
        L.dig_gla_fwd_beta.argtypes = [vp] * 6 + [i] * 9 + [vp, sz, vp]
        L.dig_gla_fwd_beta.restype = i
        L.dig_gla_bwd_beta.argtypes = [vp] * 11 + [i] * 9 + [vp, sz, vp]
        L.dig_gla_bwd_beta.restype = i
        L.dig_gla_fwd_state.argtypes = [vp] * 7 + [i] * 9 + [vp, sz, vp]
        L.dig_gla_fwd_state.restype = i
        L.dig_gla_bwd_state.argtypes = [vp] * 12 + [i] * 9 + [vp, sz, vp]
        L.dig_gla_bwd_state.restype = i
        L.dig_srem_dwconv.argtypes = [vp] * 4 + [i] * 6 + [vp]
        L.dig_srem_dwconv.restype = i
        L.dig_srem_dwconv_bwd_workspace_bytes.argtypes = [i] * 4
        L.dig_srem_dwconv_bwd_workspace_bytes.restype = ctypes.c_size_t
        L.dig_srem_dwconv_bwd.argtypes = [vp] * 6 + [i] * 6 + [vp, ctypes.c_size_t, vp]
        L.dig_srem_dwconv_bwd.restype = i
        ll, fl = ctypes.c_longlong, ctypes.c_float
        L.dig_gla_outgate_fwd.argtypes = [vp] * 5 + [ll, i, fl, i, vp]
        L.dig_gla_outgate_fwd.restype = i
        L.dig_gla_outgate_bwd_workspace_bytes.argtypes = [ll, i]
        L.dig_gla_outgate_bwd_workspace_bytes.restype = ctypes.c_size_t
        L.dig_gla_outgate_bwd.argtypes = [vp] * 9 + [ll, i, fl, i, vp, ctypes.c_size_t, vp]
        L.dig_gla_outgate_bwd.restype = i
        L.dig_last_device_status.argtypes = [vp]
        L.dig_last_device_status.restype = i
        L.dig_selftest_wait_timeout.argtypes = [ctypes.c_uint, vp]
        L.dig_selftest_wait_timeout.restype = i
        L.dig_status_string.argtypes = [i]
        L.dig_status_string.restype = ctypes.c_char_p
        L.dig_profile_enable.argtypes = [i]
        L.dig_profile_enable.restype = i
        L.dig_profile_kernels.argtypes = []
        L.dig_profile_kernels.restype = i
        L.dig_profile_read.argtypes = [i, ctypes.c_char_p, i, ctypes.POINTER(i), ctypes.POINTER(ctypes.c_float)]
        L.dig_profile_read.restype = i
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().dig_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != DIG_OK:
        raise DigError(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _storage(dtype: int) -> torch.dtype:
    return torch.float32 if dtype == DIG_F32 else torch.bfloat16


def _out_storage(dtype: int) -> torch.dtype:
    return torch.bfloat16 if dtype == DIG_BF16 else torch.float32


def _dtype_of(t: torch.Tensor, f32_out: bool = False) -> int:
    if t.dtype == torch.float32:
        return DIG_F32
    if t.dtype == torch.bfloat16:
        return DIG_BF16_F32OUT if f32_out else DIG_BF16
    raise TypeError(f"unsupported storage type {t.dtype}")


def _dev(t: torch.Tensor, dtype: torch.dtype, shape=None, name="tensor"):
    if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise ValueError(f"{name}: need a contiguous CUDA tensor of {dtype}, got {t.dtype} on {t.device}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: shape {tuple(t.shape)} != {tuple(shape)}")
    return t.data_ptr()


def dig_set_impl(impl: int) -> None:
    _check(lib().dig_set_impl(impl), "dig_set_impl")


def dig_gla_query_impl(d_k, d_v, chunk, dtype, backward) -> int:
    return lib().dig_gla_query_impl(d_k, d_v, chunk, dtype, int(backward))


def dig_gla_workspace_bytes(B, H, grid_h, grid_w, d_k, d_v, chunk, dtype, backward) -> int:
    return lib().dig_gla_workspace_bytes(B, H, grid_h, grid_w, d_k, d_v, chunk, dtype, int(backward))


def dig_gate_logsigmoid(g: torch.Tensor, tau_per_head, gate: torch.Tensor | None = None) -> torch.Tensor:
    """gate = logsigmoid(g) / tau[h]; g: [B, L, H, d_k] (fp32 or bf16), returns fp32."""
    B, L, H, dk = g.shape
    dtype = _dtype_of(g)
    if gate is None:
        gate = torch.empty(g.shape, dtype=torch.float32, device=g.device)
    tau = (ctypes.c_float * H)(*[float(x) for x in tau_per_head])
    _check(lib().dig_gate_logsigmoid(_dev(g, _storage(dtype), name="g"), tau,
                                     _dev(gate, torch.float32, g.shape, "gate"), B, L, H, dk, dtype,
                                     _stream()), "dig_gate_logsigmoid")
    return gate


def _workspace(ws, need, device):
    if ws is None:
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device=device)
    return ws


def dig_gla_fwd(q, k, v, gate, grid_h, grid_w, chunk=64, direction=DIG_ROW_FWD, *, f32_out=False,
                out=None, workspace=None) -> torch.Tensor:
    B, L, H, dk = q.shape
    dv = v.shape[-1]
    dtype = _dtype_of(q, f32_out)
    st = _storage(dtype)
    if out is None:
        out = torch.empty((B, L, H, dv), dtype=_out_storage(dtype), device=q.device)
    need = dig_gla_workspace_bytes(B, H, grid_h, grid_w, dk, dv, chunk, dtype, 0)
    workspace = _workspace(workspace, need, q.device)
    _check(lib().dig_gla_fwd(_dev(q, st, name="q"), _dev(k, st, q.shape, "k"),
                             _dev(v, st, (B, L, H, dv), "v"), _dev(gate, torch.float32, q.shape, "gate"),
                             _dev(out, _out_storage(dtype), (B, L, H, dv), "out"),
                             B, H, grid_h, grid_w, dk, dv, chunk, direction, dtype,
                             workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                             _stream()), "dig_gla_fwd")
    return out


def dig_gla_fwd_static(q, k, v, gate, out, grid_h, grid_w, chunk=64, direction=DIG_ROW_FWD) -> torch.Tensor:
    """dig_gla_fwd for callers that cannot allocate: the scratch is a fixed array inside the
    library, so `out` must be given and nothing is allocated here either.  `out` is bf16 for bf16
    inputs unless it is an fp32 tensor, which selects the fp32-output variant."""
    B, L, H, dk = q.shape
    dv = v.shape[-1]
    dtype = _dtype_of(q, f32_out=(q.dtype == torch.bfloat16 and out.dtype == torch.float32))
    st = _storage(dtype)
    _check(lib().dig_gla_fwd_static(_dev(q, st, name="q"), _dev(k, st, q.shape, "k"),
                                    _dev(v, st, (B, L, H, dv), "v"), _dev(gate, torch.float32, q.shape, "gate"),
                                    _dev(out, _out_storage(dtype), (B, L, H, dv), "out"),
                                    B, H, grid_h, grid_w, dk, dv, chunk, direction, dtype, _stream()),
           "dig_gla_fwd_static")
    return out


def dig_gla_bwd(q, k, v, gate, d_out, grid_h, grid_w, chunk=64, direction=DIG_ROW_FWD, *,
                f32_out=False, grads=None, workspace=None):
    """Returns (dq, dk, dv, dgate)."""
    B, L, H, dk = q.shape
    dv = v.shape[-1]
    dtype = _dtype_of(q, f32_out)
    st, ost = _storage(dtype), _out_storage(dtype)
    if grads is None:
        grads = (torch.empty(q.shape, dtype=ost, device=q.device),
                 torch.empty(q.shape, dtype=ost, device=q.device),
                 torch.empty(v.shape, dtype=ost, device=q.device),
                 torch.empty(q.shape, dtype=torch.float32, device=q.device))
    dq, dk_, dv_, dgate = grads
    need = dig_gla_workspace_bytes(B, H, grid_h, grid_w, dk, dv, chunk, dtype, 1)
    workspace = _workspace(workspace, need, q.device)
    _check(lib().dig_gla_bwd(_dev(q, st, name="q"), _dev(k, st, q.shape, "k"),
                             _dev(v, st, (B, L, H, dv), "v"), _dev(gate, torch.float32, q.shape, "gate"),
                             _dev(d_out, st, v.shape, "d_out"),
                             _dev(dq, ost, q.shape, "dq"), _dev(dk_, ost, q.shape, "dk"),
                             _dev(dv_, ost, v.shape, "dv"), _dev(dgate, torch.float32, q.shape, "dgate"),
                             B, H, grid_h, grid_w, dk, dv, chunk, direction, dtype,
                             workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                             _stream()), "dig_gla_bwd")
    return dq, dk_, dv_, dgate


def _mask(directions) -> int:
    m = 0
    for d in directions:
        m |= 1 << int(d)
    return m


def dig_gla_multi_workspace_bytes(B, H, grid_h, grid_w, d_k, d_v, chunk, dtype, backward) -> int:
    return lib().dig_gla_multi_workspace_bytes(B, H, grid_h, grid_w, d_k, d_v, chunk, dtype, int(backward))


def dig_gla_fwd_multi(q, k, v, gate, grid_h, grid_w, directions, chunk=64, *, f32_out=False, out=None,
                      workspace=None) -> torch.Tensor:
    """Sum of dig_gla_fwd over the scan orders in `directions` (an iterable of dig_dir values)."""
    B, L, H, dk = q.shape
    dv = v.shape[-1]
    dtype = _dtype_of(q, f32_out)
    st = _storage(dtype)
    if out is None:
        out = torch.empty((B, L, H, dv), dtype=_out_storage(dtype), device=q.device)
    need = dig_gla_multi_workspace_bytes(B, H, grid_h, grid_w, dk, dv, chunk, dtype, 0)
    workspace = _workspace(workspace, need, q.device)
    _check(lib().dig_gla_fwd_multi(_dev(q, st, name="q"), _dev(k, st, q.shape, "k"), _dev(v, st, (B, L, H, dv), "v"),
                                   _dev(gate, torch.float32, q.shape, "gate"),
                                   _dev(out, _out_storage(dtype), (B, L, H, dv), "out"),
                                   B, H, grid_h, grid_w, dk, dv, chunk, _mask(directions), dtype,
                                   workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream()),
           "dig_gla_fwd_multi")
    return out


def dig_gla_bwd_multi(q, k, v, gate, d_out, grid_h, grid_w, directions, chunk=64, *, f32_out=False, grads=None,
                      workspace=None):
    """Gradients of <d_out, dig_gla_fwd_multi(...)>: returns (dq, dk, dv, dgate)."""
    B, L, H, dk = q.shape
    dv = v.shape[-1]
    dtype = _dtype_of(q, f32_out)
    st, ost = _storage(dtype), _out_storage(dtype)
    if grads is None:
        grads = (torch.empty(q.shape, dtype=ost, device=q.device), torch.empty(q.shape, dtype=ost, device=q.device),
                 torch.empty(v.shape, dtype=ost, device=q.device), torch.empty(q.shape, dtype=torch.float32, device=q.device))
    dq, dk_, dv_, dgate = grads
    need = dig_gla_multi_workspace_bytes(B, H, grid_h, grid_w, dk, dv, chunk, dtype, 1)
    workspace = _workspace(workspace, need, q.device)
    _check(lib().dig_gla_bwd_multi(_dev(q, st, name="q"), _dev(k, st, q.shape, "k"), _dev(v, st, (B, L, H, dv), "v"),
                                   _dev(gate, torch.float32, q.shape, "gate"), _dev(d_out, st, v.shape, "d_out"),
                                   _dev(dq, ost, q.shape, "dq"), _dev(dk_, ost, q.shape, "dk"),
                                   _dev(dv_, ost, v.shape, "dv"), _dev(dgate, torch.float32, q.shape, "dgate"),
                                   B, H, grid_h, grid_w, dk, dv, chunk, _mask(directions), dtype,
                                   workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream()),
           "dig_gla_bwd_multi")
    return dq, dk_, dv_, dgate


def dig_srem_dwconv(x, w, bias, grid_h, grid_w, direction=DIG_ROW_FWD, *, f32_out=False, y=None):
    """x: [B, L, D] canonical token order; w: [3, 3, D]; bias: [D] or None."""
    B, L, D = x.shape
    if L != grid_h * grid_w:
        raise ValueError("x: L != grid_h*grid_w")
    dtype = _dtype_of(x, f32_out)
    st = _storage(dtype)
    if y is None:
        y = torch.empty(x.shape, dtype=_out_storage(dtype), device=x.device)
    _check(lib().dig_srem_dwconv(_dev(x, st, name="x"), _dev(w, st, (3, 3, D), "w"),
                                 None if bias is None else _dev(bias, st, (D,), "bias"),
                                 _dev(y, _out_storage(dtype), x.shape, "y"),
                                 B, grid_h, grid_w, D, direction, dtype, _stream()), "dig_srem_dwconv")
    return y


def dig_srem_dwconv_bwd(x, w, dy, grid_h, grid_w, direction=DIG_ROW_FWD, *, with_bias=True, f32_out=False,
                        workspace=None):
    """Reverse mode of dig_srem_dwconv: returns (dx, dw, dbias); dw and dbias are fp32, dbias None
    unless `with_bias`."""
    B, L, D = x.shape
    if L != grid_h * grid_w:
        raise ValueError("x.shape[1] must equal grid_h * grid_w")
    st = x.dtype
    dtype = _dtype_of(x, f32_out)
    need = lib().dig_srem_dwconv_bwd_workspace_bytes(B, grid_h, grid_w, D)
    if need == 0:
        raise ValueError("dig_srem_dwconv_bwd: unsupported sizes")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
    dx = torch.empty(x.shape, dtype=_out_storage(dtype), device=x.device)
    dw = torch.empty((3, 3, D), dtype=torch.float32, device=x.device)
    db = torch.empty((D,), dtype=torch.float32, device=x.device) if with_bias else None
    _check(lib().dig_srem_dwconv_bwd(_dev(x, st, name="x"), _dev(w, st, (3, 3, D), "w"), _dev(dy, st, x.shape, "dy"),
                                     _dev(dx, _out_storage(dtype), x.shape, "dx"),
                                     _dev(dw, torch.float32, (3, 3, D), "dw"),
                                     None if db is None else _dev(db, torch.float32, (D,), "dbias"),
                                     B, grid_h, grid_w, D, direction, dtype,
                                     _dev(workspace, torch.uint8, name="workspace"), workspace.numel(), _stream()),
           "dig_srem_dwconv_bwd")
    return dx, dw, db


def dig_last_device_status() -> int:
    return lib().dig_last_device_status(_stream())


def dig_selftest_wait_timeout(limit_us: int = 1000) -> None:
    """Launches the kernel whose only wait expires after limit_us; dig_last_device_status then reports it."""
    _check(lib().dig_selftest_wait_timeout(int(limit_us), _stream()), "dig_selftest_wait_timeout")


def dig_profile_enable(on: bool) -> None:
    _check(lib().dig_profile_enable(int(on)), "dig_profile_enable")


def dig_profile_read() -> dict:
    """{kernel name: (launches, total milliseconds)} for the launches recorded since enabling."""
    out = {}
    for idx in range(lib().dig_profile_kernels()):
        name = ctypes.create_string_buffer(64)
        n, ms = ctypes.c_int(0), ctypes.c_float(0)
        _check(lib().dig_profile_read(idx, name, 64, ctypes.byref(n), ctypes.byref(ms)), "dig_profile_read")
        if n.value:
            out[name.value.decode()] = (n.value, ms.value)
    return out


def _affine(t, d, name):
    return None if t is None else _dev(t, torch.float32, (d,), name)


def dig_gla_outgate_fwd(o, r, ln_w=None, ln_b=None, eps=1e-5, *, f32_out=False):
    """z = Swish(r) * LN(o) over the last axis; o, r: [..., d_v]; ln_w, ln_b: fp32 [d_v] or None."""
    d = o.shape[-1]
    dtype = _dtype_of(o, f32_out)
    z = torch.empty(o.shape, dtype=_out_storage(dtype), device=o.device)
    _check(lib().dig_gla_outgate_fwd(_dev(o, o.dtype, name="o"), _dev(r, o.dtype, o.shape, "r"),
                                     _affine(ln_w, d, "ln_w"), _affine(ln_b, d, "ln_b"),
                                     _dev(z, z.dtype, name="z"), o.numel() // d, d, float(eps), dtype, _stream()),
           "dig_gla_outgate_fwd")
    return z


def dig_gla_outgate_bwd(o, r, dz, ln_w=None, ln_b=None, eps=1e-5, *, affine_grads=True, f32_out=False,
                        workspace=None):
    """Returns (d_o, d_r, dln_w, dln_b); the last two are fp32 [d_v], or None without `affine_grads`."""
    d = o.shape[-1]
    rows = o.numel() // d
    dtype = _dtype_of(o, f32_out)
    d_o = torch.empty(o.shape, dtype=_out_storage(dtype), device=o.device)
    d_r = torch.empty_like(d_o)
    dw = db = None
    wsp, wsn = None, 0
    if affine_grads:
        dw = torch.empty(d, dtype=torch.float32, device=o.device)
        db = torch.empty(d, dtype=torch.float32, device=o.device)
        if workspace is None:
            workspace = torch.empty(lib().dig_gla_outgate_bwd_workspace_bytes(rows, d), dtype=torch.uint8,
                                    device=o.device)
        wsp, wsn = _dev(workspace, torch.uint8, name="workspace"), workspace.numel()
    _check(lib().dig_gla_outgate_bwd(_dev(o, o.dtype, name="o"), _dev(r, o.dtype, o.shape, "r"),
                                     _affine(ln_w, d, "ln_w"), _affine(ln_b, d, "ln_b"),
                                     _dev(dz, o.dtype, o.shape, "dz"), _dev(d_o, d_o.dtype, name="d_o"),
                                     _dev(d_r, d_r.dtype, name="d_r"),
                                     None if dw is None else dw.data_ptr(), None if db is None else db.data_ptr(),
                                     rows, d, float(eps), dtype, wsp, wsn, _stream()), "dig_gla_outgate_bwd")
    return d_o, d_r, dw, db


def _state(t, shape, name):
    return None if t is None else _dev(t, torch.float32, shape, name)


def dig_gla_fwd_state(q, k, v, gate, s_in, grid_h, grid_w, chunk=64, direction=DIG_ROW_FWD, *, f32_out=False,
                      want_s_out=True, workspace=None):
    """dig_gla_fwd started from state s_in ([B, H, d_k, d_v] fp32 or None); returns (out, s_out)."""
    B, L, H, dk = q.shape
    dv = v.shape[-1]
    dtype = _dtype_of(q, f32_out)
    st = _storage(dtype)
    out = torch.empty((B, L, H, dv), dtype=_out_storage(dtype), device=q.device)
    s_out = torch.empty((B, H, dk, dv), dtype=torch.float32, device=q.device) if want_s_out else None
    need = dig_gla_workspace_bytes(B, H, grid_h, grid_w, dk, dv, chunk, dtype, 0)
    workspace = _workspace(workspace, need, q.device)
    _check(lib().dig_gla_fwd_state(_dev(q, st, name="q"), _dev(k, st, q.shape, "k"), _dev(v, st, (B, L, H, dv), "v"),
                                   _dev(gate, torch.float32, q.shape, "gate"), _state(s_in, (B, H, dk, dv), "s_in"),
                                   _dev(out, _out_storage(dtype), (B, L, H, dv), "out"),
                                   _state(s_out, (B, H, dk, dv), "s_out"),
                                   B, H, grid_h, grid_w, dk, dv, chunk, direction, dtype,
                                   workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream()),
           "dig_gla_fwd_state")
    return out, s_out


def dig_gla_bwd_state(q, k, v, gate, d_out, s_in, ds_out, grid_h, grid_w, chunk=64, direction=DIG_ROW_FWD, *,
                      f32_out=False, workspace=None):
    """Returns (dq, dk, dv, dgate, ds_in) for the loss <d_out, out> + <ds_out, s_out>."""
    B, L, H, dk = q.shape
    dv = v.shape[-1]
    dtype = _dtype_of(q, f32_out)
    st, ost = _storage(dtype), _out_storage(dtype)
    dq = torch.empty(q.shape, dtype=ost, device=q.device)
    dk_ = torch.empty(q.shape, dtype=ost, device=q.device)
    dv_ = torch.empty(v.shape, dtype=ost, device=q.device)
    dgate = torch.empty(q.shape, dtype=torch.float32, device=q.device)
    ds_in = torch.empty((B, H, dk, dv), dtype=torch.float32, device=q.device)
    need = dig_gla_workspace_bytes(B, H, grid_h, grid_w, dk, dv, chunk, dtype, 1)
    workspace = _workspace(workspace, need, q.device)
    _check(lib().dig_gla_bwd_state(_dev(q, st, name="q"), _dev(k, st, q.shape, "k"), _dev(v, st, (B, L, H, dv), "v"),
                                   _dev(gate, torch.float32, q.shape, "gate"), _dev(d_out, st, v.shape, "d_out"),
                                   _state(s_in, (B, H, dk, dv), "s_in"), _state(ds_out, (B, H, dk, dv), "ds_out"),
                                   _dev(dq, ost, q.shape, "dq"), _dev(dk_, ost, q.shape, "dk"),
                                   _dev(dv_, ost, v.shape, "dv"), _dev(dgate, torch.float32, q.shape, "dgate"),
                                   _dev(ds_in, torch.float32, (B, H, dk, dv), "ds_in"),
                                   B, H, grid_h, grid_w, dk, dv, chunk, direction, dtype,
                                   workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream()),
           "dig_gla_bwd_state")
    return dq, dk_, dv_, dgate, ds_in


def dig_gla_fwd_beta(q, k, v, gate, bgate, grid_h, grid_w, chunk=64, direction=DIG_ROW_FWD, *, f32_out=False,
                     workspace=None) -> torch.Tensor:
    """dig_gla_fwd with the value-channel gate: bgate = log(beta), fp32 [B, L, H, d_v]."""
    B, L, H, dk = q.shape
    dv = v.shape[-1]
    dtype = _dtype_of(q, f32_out)
    st = _storage(dtype)
    need = lib().dig_gla_beta_workspace_bytes(B, H, grid_h, grid_w, dk, dv, chunk, dtype, 0)
    if need == 0:
        raise DigError(DIG_ERR_UNSUPPORTED, "dig_gla_beta_workspace_bytes")
    workspace = _workspace(workspace, need, q.device)
    out = torch.empty((B, L, H, dv), dtype=_out_storage(dtype), device=q.device)
    _check(lib().dig_gla_fwd_beta(_dev(q, st, name="q"), _dev(k, st, q.shape, "k"), _dev(v, st, (B, L, H, dv), "v"),
                                  _dev(gate, torch.float32, q.shape, "gate"), _dev(bgate, torch.float32, v.shape, "bgate"),
                                  _dev(out, _out_storage(dtype), name="out"),
                                  B, H, grid_h, grid_w, dk, dv, chunk, direction, dtype,
                                  workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream()),
           "dig_gla_fwd_beta")
    return out


def dig_gla_bwd_beta(q, k, v, gate, bgate, d_out, grid_h, grid_w, chunk=64, direction=DIG_ROW_FWD, *,
                     f32_out=False, workspace=None):
    """Returns (dq, dk, dv, dgate, dbgate)."""
    B, L, H, dk = q.shape
    dv = v.shape[-1]
    dtype = _dtype_of(q, f32_out)
    st, ost = _storage(dtype), _out_storage(dtype)
    need = lib().dig_gla_beta_workspace_bytes(B, H, grid_h, grid_w, dk, dv, chunk, dtype, 1)
    if need == 0:
        raise DigError(DIG_ERR_UNSUPPORTED, "dig_gla_beta_workspace_bytes")
    workspace = _workspace(workspace, need, q.device)
    dq = torch.empty(q.shape, dtype=ost, device=q.device)
    dk_ = torch.empty(q.shape, dtype=ost, device=q.device)
    dv_ = torch.empty(v.shape, dtype=ost, device=q.device)
    dgate = torch.empty(q.shape, dtype=torch.float32, device=q.device)
    dbgate = torch.empty(v.shape, dtype=torch.float32, device=q.device)
    _check(lib().dig_gla_bwd_beta(_dev(q, st, name="q"), _dev(k, st, q.shape, "k"), _dev(v, st, (B, L, H, dv), "v"),
                                  _dev(gate, torch.float32, q.shape, "gate"), _dev(bgate, torch.float32, v.shape, "bgate"),
                                  _dev(d_out, st, v.shape, "d_out"),
                                  _dev(dq, ost, name="dq"), _dev(dk_, ost, name="dk"), _dev(dv_, ost, name="dv"),
                                  _dev(dgate, torch.float32, name="dgate"), _dev(dbgate, torch.float32, name="dbgate"),
                                  B, H, grid_h, grid_w, dk, dv, chunk, direction, dtype,
                                  workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream()),
           "dig_gla_bwd_beta")
    return dq, dk_, dv_, dgate, dbgate


def dig_gla_fwd_outgate(q, k, v, gate, r, grid_h, grid_w, chunk=64, direction=DIG_ROW_FWD, *, ln_w=None, ln_b=None,
                        eps=1e-5, f32_out=False, want_out=True, workspace=None):
    """dig_gla_fwd and the output gate z = Swish(r) * LN(out) in one call; returns (out or None, z)."""
    B, L, H, dk = q.shape
    dv = v.shape[-1]
    dtype = _dtype_of(q, f32_out)
    st, ost = _storage(dtype), _out_storage(dtype)
    out = torch.empty((B, L, H, dv), dtype=ost, device=q.device) if want_out else None
    z = torch.empty((B, L, H, dv), dtype=ost, device=q.device)
    need = dig_gla_workspace_bytes(B, H, grid_h, grid_w, dk, dv, chunk, dtype, 0)
    workspace = _workspace(workspace, need, q.device)
    _check(lib().dig_gla_fwd_outgate(_dev(q, st, name="q"), _dev(k, st, q.shape, "k"), _dev(v, st, (B, L, H, dv), "v"),
                                     _dev(gate, torch.float32, q.shape, "gate"), _dev(r, st, v.shape, "r"),
                                     _affine(ln_w, dv, "ln_w"), _affine(ln_b, dv, "ln_b"), float(eps),
                                     None if out is None else out.data_ptr(), z.data_ptr(),
                                     B, H, grid_h, grid_w, dk, dv, chunk, direction, dtype,
                                     workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream()),
           "dig_gla_fwd_outgate")
    return out, z
