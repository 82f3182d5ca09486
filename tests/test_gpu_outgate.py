"""GPU parity of the output gate z = Swish(r) * LN(o) (Eq. attn_gla) and its reverse mode against the
fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_18428_b200.inputs import CONFIGS, round_to_bf16
from parity import rel_err

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-5     # a few dozen fp32 operations per value, row sums of <= 128 terms
RTOL_BF16_OUT = 2.0 ** -8   # one bf16 rounding of each result (half an ulp = 2^-9 of the value), elementwise


def _case(shape, dtype, affine, seed, eps=1e-5):
    from paper_2405_18428_b200 import dig
    rng = np.random.default_rng(seed)
    d = shape[-1]
    mk = lambda a: round_to_bf16(a.astype(np.float32)) if dtype == "bf16" else a.astype(np.float32)
    o = mk(rng.standard_normal(shape) * 3 + 0.5)
    r = mk(rng.standard_normal(shape) * 2)
    dz = mk(rng.standard_normal(shape))
    w = (rng.standard_normal(d) * 0.3 + 1).astype(np.float32) if affine else None
    b = (rng.standard_normal(d) * 0.3).astype(np.float32) if affine else None
    tt = torch.bfloat16 if dtype == "bf16" else torch.float32
    dev = lambda a: torch.from_numpy(a).cuda().to(tt)
    dw_ = None if w is None else torch.from_numpy(w).cuda()
    db_ = None if b is None else torch.from_numpy(b).cuda()
    ref = oracle.outgate(o, r, w, b, eps)
    z = dig.dig_gla_outgate_fwd(dev(o), dev(r), dw_, db_, eps, f32_out=True)
    assert z.dtype == torch.float32
    assert rel_err(z.cpu().numpy(), ref) <= TOL_F32
    rdo, rdr, rdw, rdb = oracle.outgate_bwd(o, r, dz, w, b, eps)
    d_o, d_r, dlw, dlb = dig.dig_gla_outgate_bwd(dev(o), dev(r), dev(dz), dw_, db_, eps, f32_out=True)
    assert rel_err(d_o.cpu().numpy(), rdo) <= TOL_F32
    assert rel_err(d_r.cpu().numpy(), rdr) <= TOL_F32
    assert rel_err(dlw.cpu().numpy(), rdw) <= TOL_F32
    assert rel_err(dlb.cpu().numpy(), rdb) <= TOL_F32
    if dtype == "bf16":
        z16 = dig.dig_gla_outgate_fwd(dev(o), dev(r), dw_, db_, eps)
        assert z16.dtype == torch.bfloat16 and torch.equal(z16, z.to(torch.bfloat16))
        np.testing.assert_allclose(z16.float().cpu().numpy(), ref, rtol=RTOL_BF16_OUT, atol=1e-5)
        o16, r16, w2, b2 = dig.dig_gla_outgate_bwd(dev(o), dev(r), dev(dz), dw_, db_, eps)
        assert torch.equal(o16, d_o.to(torch.bfloat16)) and torch.equal(r16, d_r.to(torch.bfloat16))
        assert torch.equal(w2, dlw) and torch.equal(b2, dlb)          # fixed summation order
        o3, r3, w3, b3 = dig.dig_gla_outgate_bwd(dev(o), dev(r), dev(dz), dw_, db_, eps, affine_grads=False)
        assert w3 is None and b3 is None and torch.equal(o3, o16) and torch.equal(r3, r16)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d", [8, 24, 64, 72, 128])
def test_outgate_small_ragged(dtype, d):
    # 3 * 37 * 5 = 555 rows: not a multiple of the rows a CTA takes per pass, for either lane grouping
    _case((3, 37, 5, d), dtype, affine=(d != 24), seed=d)


def test_outgate_single_row_and_extremes():
    from paper_2405_18428_b200 import dig
    _case((1, 1, 1, 64), "f32", True, 1)
    o = torch.full((4, 64), 2.5, device="cuda")                 # constant rows: LN = bias (0)
    r = torch.tensor([-100.0, -20.0, 0.0, 30.0], device="cuda")[:, None].expand(4, 64).contiguous()
    z = dig.dig_gla_outgate_fwd(o, r)
    assert torch.isfinite(z).all() and float(z.abs().max()) == 0.0
    o = torch.randn(4, 64, device="cuda")
    z = dig.dig_gla_outgate_fwd(o, r)
    assert torch.isfinite(z).all() and float(z[:3].abs().max()) < 1e-6      # Swish(-100), Swish(-20), Swish(0)


@pytest.mark.parametrize("cfg", ["C2", "C5"])
def test_outgate_benchmark_shapes(cfg):
    wl = CONFIGS[cfg]
    _case((wl.B, wl.grid_h * wl.grid_w, wl.H, wl.d_v), "bf16", True, 3)


def test_outgate_argument_checks():
    from paper_2405_18428_b200 import dig
    o = torch.zeros(4, 20, device="cuda")                       # d_v not a multiple of 8
    with pytest.raises(dig.DigError):
        dig.dig_gla_outgate_fwd(o, o)
    o = torch.zeros(40, 64, device="cuda")
    with pytest.raises(dig.DigError):
        dig.dig_gla_outgate_bwd(o, o, o, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))


# ---- forward pass and output gate in one call -------------------------------------------------------
@pytest.mark.parametrize("d,chunk,direction", [(64, 64, 0), (64, 64, 3), (72, 64, 2), (64, 32, 1)])
@pytest.mark.parametrize("f32_out", [True, False])
def test_fwd_outgate_one_call(d, chunk, direction, f32_out):
    """Against the oracle (recurrence, then gate, on the stored form of the outputs) and against the two
    public calls made one after the other, on every kernel family."""
    from paper_2405_18428_b200 import dig
    from paper_2405_18428_b200.inputs import Workload, make_inputs
    from parity import TOL_BF16, to_dev
    wl = Workload("fo", B=2, H=3, grid_h=12, grid_w=14, d_k=d, d_v=d, chunk=chunk, dtype="bf16", backward=False,
                  tau=(16.0, 4.0, 2.0), seed=51)
    x = make_inputs(wl, conv=False)
    rng = np.random.default_rng(52)
    r = round_to_bf16(rng.standard_normal(x["v"].shape).astype(np.float32) * 2)
    w = (rng.standard_normal(d) * 0.3 + 1).astype(np.float32)
    b = (rng.standard_normal(d) * 0.3).astype(np.float32)
    q, k, v, g = (to_dev(x[n], wl) for n in ("q", "k", "v", "g"))
    gate = dig.dig_gate_logsigmoid(g, x["tau"])
    tr, tw, tb = to_dev(r, wl), torch.from_numpy(w).cuda(), torch.from_numpy(b).cuda()
    out, z = dig.dig_gla_fwd_outgate(q, k, v, gate, tr, wl.grid_h, wl.grid_w, chunk, direction, ln_w=tw, ln_b=tb,
                                     f32_out=f32_out)
    _, z_only = dig.dig_gla_fwd_outgate(q, k, v, gate, tr, wl.grid_h, wl.grid_w, chunk, direction, ln_w=tw, ln_b=tb,
                                        f32_out=f32_out, want_out=False)
    # the two public calls one after the other
    out2 = dig.dig_gla_fwd(q, k, v, gate, wl.grid_h, wl.grid_w, chunk, direction, f32_out=f32_out)
    assert torch.equal(out, out2) and torch.equal(z, z_only)
    # oracle on the values the gate actually sees (the stored outputs), so only the gate's own arithmetic differs
    ref = oracle.outgate(out.float().cpu().numpy(), r, w, b, 1e-5)
    got = z.float().cpu().numpy()
    if f32_out:
        assert rel_err(got, ref) <= 1e-5
    else:
        np.testing.assert_allclose(got, ref, rtol=RTOL_BF16_OUT, atol=1e-5)
    # and end to end against the oracle's own recurrence (fp32 results; with bf16 results the two roundings
    # of the heavy-tailed z dominate a max-over-RMS measure, and the stored-form check above covers them)
    if f32_out:
        a = oracle.gate(x["g"], x["tau"])
        ref_full = oracle.outgate(oracle.gla_fwd(x["q"], x["k"], x["v"], a, wl.grid_h, wl.grid_w, direction), r, w, b, 1e-5)
        assert rel_err(got, ref_full) <= TOL_BF16
