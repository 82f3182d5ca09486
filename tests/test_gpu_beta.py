"""GPU parity of gated linear attention with the full gate alpha^T beta of Eq. gate_gla
(dig_gla_fwd_beta, dig_gla_bwd_beta) against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_18428_b200.inputs import CONFIGS, Workload, make_inputs, round_to_bf16
from parity import TOL_BF16, TOL_F32, oracle_threads, rel_err, to_dev

pytestmark = pytest.mark.gpu


def _run(wl, direction, seed, tau_v=8.0):
    from paper_2405_18428_b200 import dig
    x = make_inputs(wl, conv=False)
    rng = np.random.default_rng(seed)
    gb = rng.standard_normal((wl.B, wl.grid_h * wl.grid_w, wl.H, wl.d_v)).astype(np.float32)
    if wl.dtype == "bf16":
        gb = round_to_bf16(gb)
    a = oracle.gate(x["g"], x["tau"])
    bg = oracle.gate(gb, np.full(wl.H, tau_v, dtype=np.float32))          # log(beta) = logsigmoid / tau
    thr = oracle_threads()
    ro = oracle.gla_fwd_beta(x["q"], x["k"], x["v"], a, bg, wl.grid_h, wl.grid_w, direction, threads=thr)
    rg = oracle.gla_bwd_beta(x["q"], x["k"], x["v"], a, bg, x["dO"], wl.grid_h, wl.grid_w, direction, threads=thr)
    q, k, v, g, dO = (to_dev(x[n], wl) for n in ("q", "k", "v", "g", "dO"))
    gate = dig.dig_gate_logsigmoid(g, x["tau"])
    bgate = dig.dig_gate_logsigmoid(to_dev(gb, wl), np.full(wl.H, tau_v, dtype=np.float32))
    if wl.dtype == "f32":
        # fp32 storage: one pass, held to the fp32 bound (the kernels split every operand into two tf32 parts)
        out = dig.dig_gla_fwd_beta(q, k, v, gate, bgate, wl.grid_h, wl.grid_w, wl.chunk, direction)
        grads = dig.dig_gla_bwd_beta(q, k, v, gate, bgate, dO, wl.grid_h, wl.grid_w, wl.chunk, direction)
        torch.cuda.synchronize()
        assert dig.dig_last_device_status() == dig.DIG_OK
        assert all(t.dtype == torch.float32 for t in (out, *grads))
        errs = {n: rel_err(t.cpu().numpy(), r) for n, t, r in zip(("out", "dq", "dk", "dv", "dgate", "dbgate"), (out, *grads), (ro, *rg))}
        assert all(np.isfinite(e) and e <= TOL_F32 for e in errs.values()), errs
        return errs
    res = {}
    for f32_out in (True, False):
        out = dig.dig_gla_fwd_beta(q, k, v, gate, bgate, wl.grid_h, wl.grid_w, wl.chunk, direction, f32_out=f32_out)
        grads = dig.dig_gla_bwd_beta(q, k, v, gate, bgate, dO, wl.grid_h, wl.grid_w, wl.chunk, direction, f32_out=f32_out)
        torch.cuda.synchronize()
        assert dig.dig_last_device_status() == dig.DIG_OK
        res[f32_out] = dict(zip(("out", "dq", "dk", "dv", "dgate", "dbgate"), (out, *grads)))
    errs = {n: rel_err(t.cpu().numpy(), r) for (n, t), r in zip(res[True].items(), (ro, *rg))}
    assert all(np.isfinite(e) and e <= TOL_BF16 for e in errs.values()), errs
    # bf16-stored results are exactly the fp32 results rounded to nearest-even bf16; the gate gradients are fp32 in both
    for n in ("out", "dq", "dk", "dv"):
        assert torch.equal(res[False][n], res[True][n].to(torch.bfloat16)), n
    for n in ("dgate", "dbgate"):
        assert torch.equal(res[False][n], res[True][n]), n
    return errs


@pytest.mark.parametrize("direction", [0, 1, 2, 3])
def test_small_ragged_all_directions(direction):
    wl = Workload("beta", B=2, H=3, grid_h=7, grid_w=9, d_k=24, d_v=40, chunk=16, dtype="bf16", backward=True,
                  tau=(16.0, 2.0, 1.0), seed=31)
    print(_run(wl, direction, direction))


@pytest.mark.parametrize("d,chunk", [(64, 64), (72, 64), (64, 32), (8, 16)])
def test_head_and_chunk_sizes(d, chunk):
    wl = Workload("beta", B=1, H=2, grid_h=12, grid_w=11, d_k=d, d_v=d, chunk=chunk, dtype="bf16", backward=True,
                  tau=(16.0, 4.0), seed=32)
    print(_run(wl, 2, 5))


def test_long_sequence_many_chunks():
    wl = CONFIGS["C5"].scaled(B=1, H=2, grid_h=40, grid_w=40, backward=True)       # 1600 tokens, 25 chunks, d = 72
    print(_run(wl, 3, 6))


def test_beta_one_equals_the_alpha_only_entry_point():
    """With beta == 1 the full-gate kernels compute what the alpha-only kernels of their own family
    (the warp-level one) compute, bit for bit; against the family that serves the alpha-only entry
    point by default the two agree within the parity bound."""
    from paper_2405_18428_b200 import dig
    from parity import TOL_BF16, rel_err
    wl = Workload("beta1", B=1, H=2, grid_h=8, grid_w=16, d_k=72, d_v=72, chunk=64, dtype="bf16", backward=True, seed=33)
    x = make_inputs(wl, conv=False)
    q, k, v, g, dO = (to_dev(x[n], wl) for n in ("q", "k", "v", "g", "dO"))
    gate = dig.dig_gate_logsigmoid(g, x["tau"])
    zero = torch.zeros(v.shape, dtype=torch.float32, device="cuda")
    b = dig.dig_gla_fwd_beta(q, k, v, gate, zero, 8, 16, 64, 1, f32_out=True)
    gb = dig.dig_gla_bwd_beta(q, k, v, gate, zero, dO, 8, 16, 64, 1, f32_out=True)
    dig.dig_set_impl(dig.DIG_IMPL_MMA)
    try:
        a = dig.dig_gla_fwd(q, k, v, gate, 8, 16, 64, 1, f32_out=True)
        ga = dig.dig_gla_bwd(q, k, v, gate, dO, 8, 16, 64, 1, f32_out=True)
    finally:
        dig.dig_set_impl(dig.DIG_IMPL_AUTO)
    assert torch.equal(a, b)
    for x1, x2 in zip(ga, gb[:4]):
        assert torch.equal(x1, x2)
    a = dig.dig_gla_fwd(q, k, v, gate, 8, 16, 64, 1, f32_out=True)
    ga = dig.dig_gla_bwd(q, k, v, gate, dO, 8, 16, 64, 1, f32_out=True)
    for x1, x2 in zip((a,) + tuple(ga), (b,) + tuple(gb[:4])):
        assert rel_err(x1.cpu().numpy(), x2.cpu().numpy().astype("float64")) <= TOL_BF16


@pytest.mark.parametrize("direction", [0, 1, 2, 3])
def test_fp32_storage_small_ragged_all_directions(direction):
    wl = Workload("beta32", B=2, H=3, grid_h=7, grid_w=9, d_k=24, d_v=40, chunk=16, dtype="f32", backward=True,
                  tau=(16.0, 2.0, 1.0), seed=35)
    print(_run(wl, direction, 10 + direction))


@pytest.mark.parametrize("d,chunk", [(64, 64), (72, 64), (64, 32)])
def test_fp32_storage_head_and_chunk_sizes(d, chunk):
    wl = Workload("beta32", B=1, H=2, grid_h=20, grid_w=13, d_k=d, d_v=d, chunk=chunk, dtype="f32", backward=True,
                  tau=(16.0, 4.0), seed=36)
    print(_run(wl, 1, 7))


def test_fp32_storage_alpha_only_stays_with_the_fma_family():
    """Without the value-channel gate, fp32 storage is served by the fp32 FMA kernels."""
    from paper_2405_18428_b200 import dig
    assert dig.dig_gla_query_impl(64, 64, 64, dig.DIG_F32, 1) == dig.DIG_IMPL_FMA
