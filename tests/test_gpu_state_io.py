"""GPU parity of the recurrence with a start state / final state (dig_gla_fwd_state, dig_gla_bwd_state)
against the fp64 oracle, through the C ABI, on every kernel family."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_18428_b200.inputs import Workload, make_inputs
from parity import TOL_BF16, TOL_F32, oracle_threads, rel_err, to_dev

pytestmark = pytest.mark.gpu


def _run(wl, direction, seed, with_ds_out=True):
    from paper_2405_18428_b200 import dig
    x = make_inputs(wl, conv=False)
    rng = np.random.default_rng(seed)
    shape = (wl.B, wl.H, wl.d_k, wl.d_v)
    s_in = rng.standard_normal(shape).astype(np.float32)
    ds_out = rng.standard_normal(shape).astype(np.float32) if with_ds_out else None
    a = oracle.gate(x["g"], x["tau"])
    thr = oracle_threads()
    ro, rs = oracle.gla_fwd_state(x["q"], x["k"], x["v"], a, s_in, wl.grid_h, wl.grid_w, direction, threads=thr)
    rg = oracle.gla_bwd_state(x["q"], x["k"], x["v"], a, x["dO"], s_in, ds_out, wl.grid_h, wl.grid_w, direction,
                              threads=thr)
    q, k, v, g, dO = (to_dev(x[n], wl) for n in ("q", "k", "v", "g", "dO"))
    gate = dig.dig_gate_logsigmoid(g, x["tau"])
    ts = torch.from_numpy(s_in).cuda()
    tds = None if ds_out is None else torch.from_numpy(ds_out).cuda()
    out, s_out = dig.dig_gla_fwd_state(q, k, v, gate, ts, wl.grid_h, wl.grid_w, wl.chunk, direction, f32_out=wl.dtype == "bf16")
    grads = dig.dig_gla_bwd_state(q, k, v, gate, dO, ts, tds, wl.grid_h, wl.grid_w, wl.chunk, direction,
                                  f32_out=wl.dtype == "bf16")
    torch.cuda.synchronize()
    assert dig.dig_last_device_status() == dig.DIG_OK
    tol = TOL_BF16 if wl.dtype == "bf16" else TOL_F32
    errs = {"out": rel_err(out.float().cpu().numpy(), ro), "s_out": rel_err(s_out.cpu().numpy(), rs)}
    for name, got, ref in zip(("dq", "dk", "dv", "dgate", "ds_in"), grads, rg):
        errs[name] = rel_err(got.float().cpu().numpy(), ref)
    assert all(e <= tol for e in errs.values()), errs
    return errs


@pytest.mark.parametrize("direction", [0, 3])
def test_tensor_family(direction):
    wl = Workload("st", B=2, H=3, grid_h=12, grid_w=14, d_k=64, d_v=64, chunk=64, dtype="bf16", backward=True,
                  tau=(16.0, 4.0, 2.0), seed=21)          # 168 tokens: two full chunks and a ragged one
    print(_run(wl, direction, 1))


@pytest.mark.parametrize("d,B,H,direction", [(64, 20, 16, 2), (72, 10, 16, 1), (64, 1, 2, 0)])
def test_tensor_family_uncut_sequences(d, B, H, direction):
    """More sequences than CTAs stay resident (or a single tile per sequence): the forward pass then runs
    the forward sweep alone, which takes the start state as its entry state and writes the final state."""
    g = (8, 24) if B > 1 else (4, 9)
    wl = Workload("st1", B=B, H=H, grid_h=g[0], grid_w=g[1], d_k=d, d_v=d, chunk=64, dtype="bf16", backward=True,
                  tau=(16.0, 4.0), seed=25)
    print(_run(wl, direction, 6))


@pytest.mark.parametrize("d,B,H,direction", [(64, 20, 16, 3), (72, 10, 16, 0)])
def test_plain_entry_points_on_uncut_sequences(d, B, H, direction):
    """The same regime through dig_gla_fwd / dig_gla_bwd: the backward pass then runs the local sweep that
    only stores the per-chunk states (nothing asks for the gradient of a start state)."""
    from parity import check_workload
    wl = Workload("st2", B=B, H=H, grid_h=8, grid_w=24, d_k=d, d_v=d, chunk=64, dtype="bf16", backward=True,
                  tau=(16.0, 4.0), seed=26)
    print(check_workload(wl, direction))


@pytest.mark.parametrize("direction", [1, 2])
def test_mma_family(direction):
    wl = Workload("st", B=1, H=2, grid_h=9, grid_w=10, d_k=72, d_v=72, chunk=64, dtype="bf16", backward=True,
                  tau=(16.0, 4.0), seed=22)
    print(_run(wl, direction, 2))
    print(_run(wl.scaled(d_k=24, d_v=40, chunk=16), direction, 3))


def test_fma_family_fp32():
    wl = Workload("st", B=1, H=2, grid_h=7, grid_w=9, d_k=24, d_v=40, chunk=16, dtype="f32", backward=True,
                  tau=(16.0, 2.0), seed=23)
    print(_run(wl, 3, 4))
    print(_run(wl, 0, 5, with_ds_out=False))


def test_two_pieces_chained_on_the_gpu_equal_the_whole():
    """A 1 x 256 row cut into 1 x 128 pieces: outputs and final state of the chained pieces against the
    uncut call (both on the GPU; the pieces see the same tf32 rounding per chunk, so they agree closely)."""
    from paper_2405_18428_b200 import dig
    wl = Workload("cut", B=2, H=2, grid_h=1, grid_w=256, d_k=64, d_v=64, chunk=64, dtype="bf16", backward=False, seed=24)
    x = make_inputs(wl, conv=False)
    q, k, v, g = (to_dev(x[n], wl) for n in ("q", "k", "v", "g"))
    gate = dig.dig_gate_logsigmoid(g, x["tau"])
    whole, s_whole = dig.dig_gla_fwd_state(q, k, v, gate, None, 1, 256, 64, 0, f32_out=True)
    cut = lambda t, lo, hi: t[:, lo:hi].contiguous()
    oA, sA = dig.dig_gla_fwd_state(cut(q, 0, 128), cut(k, 0, 128), cut(v, 0, 128), cut(gate, 0, 128), None, 1, 128, 64, 0,
                                   f32_out=True)
    oB, sB = dig.dig_gla_fwd_state(cut(q, 128, 256), cut(k, 128, 256), cut(v, 128, 256), cut(gate, 128, 256), sA, 1, 128,
                                   64, 0, f32_out=True)
    torch.cuda.synchronize()
    ref = whole.cpu().numpy().astype(np.float64)
    assert rel_err(torch.cat([oA, oB], dim=1).cpu().numpy(), ref) <= 1e-5
    assert rel_err(sB.cpu().numpy(), s_whole.cpu().numpy().astype(np.float64)) <= 1e-5
