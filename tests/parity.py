"""Shared helpers of the GPU parity tests: run the CUDA path through the C-ABI binding and the
fp64 oracle on the same seeded inputs, and measure max|err| / RMS(ref) per output tensor."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2405_18428_b200 import dig
from paper_2405_18428_b200.inputs import Workload, make_inputs

TOL_F32 = 1e-4       # fp32 storage, fp32 FMA arithmetic
TOL_BF16 = 2e-2      # bf16 inputs, fp32 accumulation
TOL_GATE = 1e-6      # elementwise fp32 transform


def rel_err(got, ref) -> float:
    got = np.asarray(got, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref ** 2)))
    if rms == 0.0:          # an identically-zero reference (e.g. the gate gradient of a 1-token
        rms = 1.0           # sequence): fall back to the absolute error
    return float(np.abs(got - ref).max() / rms)


def to_dev(x: np.ndarray, wl: Workload) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    return t.to(torch.bfloat16) if wl.dtype == "bf16" else t      # values are bf16-exact already


def oracle_threads() -> int:
    import os
    return max(1, min(16, len(os.sched_getaffinity(0))))


def oracle_all(wl: Workload, x: dict, direction: int, backward: bool):
    a = oracle.gate(x["g"], x["tau"])
    thr = oracle_threads()
    o = oracle.gla_fwd(x["q"], x["k"], x["v"], a, wl.grid_h, wl.grid_w, direction, threads=thr)
    ref = {"gate": a, "out": o}
    if backward:
        dq, dk, dv, da = oracle.gla_bwd(x["q"], x["k"], x["v"], a, x["dO"], wl.grid_h, wl.grid_w,
                                        direction, threads=thr)
        ref.update(dq=dq, dk=dk, dv=dv, dgate=da)
    return ref


def gpu_all(wl: Workload, x: dict, direction: int, backward: bool, chunk=None, f32_out=True):
    chunk = wl.chunk if chunk is None else chunk
    q, k, v, g = (to_dev(x[n], wl) for n in ("q", "k", "v", "g"))
    gate = dig.dig_gate_logsigmoid(g, x["tau"])
    out = dig.dig_gla_fwd(q, k, v, gate, wl.grid_h, wl.grid_w, chunk, direction, f32_out=f32_out)
    got = {"gate": gate, "out": out}
    if backward:
        dO = to_dev(x["dO"], wl)
        dq, dk, dv, dgate = dig.dig_gla_bwd(q, k, v, gate, dO, wl.grid_h, wl.grid_w, chunk, direction,
                                            f32_out=f32_out)
        got.update(dq=dq, dk=dk, dv=dv, dgate=dgate)
    torch.cuda.synchronize()
    assert dig.dig_last_device_status() == dig.DIG_OK
    return {n: t.float().cpu().numpy() for n, t in got.items()}


def check_workload(wl: Workload, direction: int, *, chunk=None, backward=None, x=None, ref=None):
    """Full element-by-element comparison; returns the per-tensor errors."""
    backward = wl.backward if backward is None else backward
    x = make_inputs(wl, conv=False) if x is None else x
    ref = oracle_all(wl, x, direction, backward) if ref is None else ref
    got = gpu_all(wl, x, direction, backward, chunk=chunk, f32_out=True)
    tol = TOL_F32 if wl.dtype == "f32" else TOL_BF16
    errs = {}
    for name, r in ref.items():
        errs[name] = rel_err(got[name], r)
        limit = TOL_GATE if name == "gate" else tol
        assert np.isfinite(got[name]).all(), f"{wl.name} dir {direction}: {name} has non-finite values"
        assert errs[name] <= limit, f"{wl.name} dir {direction} chunk {chunk}: {name} err {errs[name]:.3e} > {limit}"
    if wl.dtype == "bf16":
        # bf16-stored results are exactly the fp32 results rounded to nearest-even bf16
        got16 = gpu_all(wl, x, direction, backward, chunk=chunk, f32_out=False)
        for name in ref:
            if name in ("gate", "dgate"):
                np.testing.assert_array_equal(got16[name], got[name])
            else:
                want = torch.from_numpy(got[name]).to(torch.bfloat16).float().numpy()
                np.testing.assert_array_equal(got16[name], want, err_msg=f"{name}: bf16 store != RNE(fp32 result)")
    return errs
