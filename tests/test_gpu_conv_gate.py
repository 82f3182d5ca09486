"""GPU parity of the SREM depthwise conv and the gate transform against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_18428_b200.inputs import CONFIGS, Workload, make_inputs, round_to_bf16

pytestmark = pytest.mark.gpu


def _conv_case(B, gh, gw, D, dtype, direction, bias, seed=0):
    from paper_2405_18428_b200 import dig
    from parity import rel_err
    rng = np.random.default_rng(seed)
    mk = (lambda a: round_to_bf16(a.astype(np.float32))) if dtype == "bf16" else (lambda a: a.astype(np.float32))
    x = mk(rng.standard_normal((B, gh * gw, D)))
    w = mk(rng.standard_normal((3, 3, D)) / 3)
    bvec = mk(rng.standard_normal(D)) if bias else None
    ref = oracle.dwconv(x, w, bvec, gh, gw, direction)
    tt = torch.bfloat16 if dtype == "bf16" else torch.float32
    dev = lambda a: None if a is None else torch.from_numpy(a).cuda().to(tt)
    y32 = dig.dig_srem_dwconv(dev(x), dev(w), dev(bvec), gh, gw, direction, f32_out=True)
    err = rel_err(y32.float().cpu().numpy(), ref)
    assert err <= 1e-5, err           # 9 fp32 FMAs per output
    if dtype == "bf16":
        y16 = dig.dig_srem_dwconv(dev(x), dev(w), dev(bvec), gh, gw, direction)
        assert torch.equal(y16, y32.to(torch.bfloat16))
    return err


@pytest.mark.parametrize("direction", [0, 1, 2, 3])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_conv_small_ragged(direction, dtype):
    # grid not a multiple of the tile, channels not a multiple of the channel block
    _conv_case(2, 11, 19, 72, dtype, direction, bias=(direction % 2 == 0), seed=direction)


def test_conv_tiny_grids():
    for gh, gw in [(1, 1), (1, 5), (3, 1), (2, 2)]:
        _conv_case(1, gh, gw, 8, "f32", 3, bias=True)


def test_conv_identity_init_is_exact():
    from paper_2405_18428_b200 import dig
    x = torch.randn(2, 16 * 24, 136, device="cuda").to(torch.bfloat16)
    w = torch.zeros(3, 3, 136, device="cuda", dtype=torch.bfloat16)
    w[1, 1] = 1
    for d in range(4):
        assert torch.equal(dig.dig_srem_dwconv(x, w, None, 16, 24, d), x)


@pytest.mark.parametrize("cfg", ["C2", "C5"])
def test_conv_benchmark_shapes(cfg):
    from paper_2405_18428_b200 import dig
    from parity import rel_err
    wl = CONFIGS[cfg]
    x = make_inputs(wl, gla=False, conv=True)
    D = wl.H * wl.d_v
    xs, ws = torch.from_numpy(x["conv_x"]).cuda().to(torch.bfloat16), torch.from_numpy(x["conv_w"]).cuda().to(torch.bfloat16)
    for d in wl.directions:
        ref = oracle.dwconv(x["conv_x"], x["conv_w"], None, wl.grid_h, wl.grid_w, d)
        y = dig.dig_srem_dwconv(xs, ws, None, wl.grid_h, wl.grid_w, d, f32_out=True)
        assert rel_err(y.cpu().numpy(), ref) <= 1e-5


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_gate_transform(dtype):
    from paper_2405_18428_b200 import dig
    from parity import rel_err, TOL_GATE
    rng = np.random.default_rng(1)
    g = rng.standard_normal((2, 50, 5, 24)).astype(np.float32) * 4
    g[0, 0, 0, :6] = [-100, -30, 0, 30, 100, 88.5]
    if dtype == "bf16":
        g = round_to_bf16(g)
    tau = np.array([16, 4, 1, 2, 0.5], dtype=np.float32)
    ref = oracle.gate(g, tau)
    t = torch.from_numpy(g).cuda()
    got = dig.dig_gate_logsigmoid(t.to(torch.bfloat16) if dtype == "bf16" else t, tau).cpu().numpy()
    assert np.isfinite(got).all() and (got <= 0).all()
    assert rel_err(got, ref) <= TOL_GATE
    np.testing.assert_allclose(got, ref, rtol=3e-6, atol=1e-30)


# ---- reverse mode of the SREM convolution ----------------------------------------------------------
def _conv_bwd_case(B, gh, gw, D, dtype, direction, with_bias, seed=0):
    from paper_2405_18428_b200 import dig
    from parity import rel_err
    rng = np.random.default_rng(100 + seed)
    mk = lambda a: round_to_bf16(a.astype(np.float32)) if dtype == "bf16" else a.astype(np.float32)
    x = mk(rng.standard_normal((B, gh * gw, D)))
    dy = mk(rng.standard_normal((B, gh * gw, D)))
    w = mk(rng.standard_normal((3, 3, D)) / 3)
    rdx, rdw, rdb = oracle.dwconv_bwd(x, w, dy, gh, gw, direction, with_bias)
    tt = torch.bfloat16 if dtype == "bf16" else torch.float32
    dev = lambda a: torch.from_numpy(a).cuda().to(tt)
    dx, dw, db = dig.dig_srem_dwconv_bwd(dev(x), dev(w), dev(dy), gh, gw, direction, with_bias=with_bias, f32_out=True)
    assert dx.dtype == torch.float32 and dw.dtype == torch.float32
    assert rel_err(dx.cpu().numpy(), rdx) <= 1e-5            # 9 fp32 FMAs per output
    assert rel_err(dw.cpu().numpy(), rdw) <= 1e-5            # fp32 sums of B*gh*gw products, blocked
    if with_bias:
        assert rel_err(db.cpu().numpy(), rdb) <= 1e-5
    else:
        assert db is None and rdb is None
    if dtype == "bf16":
        dx16, dw2, _ = dig.dig_srem_dwconv_bwd(dev(x), dev(w), dev(dy), gh, gw, direction, with_bias=False)
        assert torch.equal(dx16, dx.to(torch.bfloat16))
        assert torch.equal(dw2, dw)                          # fixed summation order


@pytest.mark.parametrize("direction", [0, 1, 2, 3])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_conv_bwd_small_ragged(direction, dtype):
    # 2*11*19 = 418 pixels: three full slabs and a ragged one; 72 channels: a partial channel block
    _conv_bwd_case(2, 11, 19, 72, dtype, direction, with_bias=(direction % 2 == 0), seed=direction)


def test_conv_bwd_tiny_grids():
    for gh, gw in [(1, 1), (1, 5), (3, 1), (2, 2)]:
        _conv_bwd_case(1, gh, gw, 8, "f32", 2, with_bias=True)


@pytest.mark.parametrize("cfg", ["C2", "C5"])
def test_conv_bwd_benchmark_shapes(cfg):
    from paper_2405_18428_b200 import dig
    from parity import rel_err
    wl = CONFIGS[cfg]
    x = make_inputs(wl, gla=False, conv=True)
    D = wl.H * wl.d_v
    rng = np.random.default_rng(7)
    dy = round_to_bf16(rng.standard_normal(x["conv_x"].shape).astype(np.float32))
    xs, ws, dys = (torch.from_numpy(a).cuda().to(torch.bfloat16) for a in (x["conv_x"], x["conv_w"], dy))
    d = wl.directions[-1]
    rdx, rdw, rdb = oracle.dwconv_bwd(x["conv_x"], x["conv_w"], dy, wl.grid_h, wl.grid_w, d, True)
    dx, dw, db = dig.dig_srem_dwconv_bwd(xs, ws, dys, wl.grid_h, wl.grid_w, d, f32_out=True)
    assert rel_err(dx.cpu().numpy(), rdx) <= 1e-5
    assert rel_err(dw.cpu().numpy(), rdw) <= 1e-5
    assert rel_err(db.cpu().numpy(), rdb) <= 1e-5


def test_conv_bwd_rejects_short_workspace():
    from paper_2405_18428_b200 import dig
    x = torch.zeros(1, 16, 8, device="cuda")
    w = torch.zeros(3, 3, 8, device="cuda")
    ws = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(RuntimeError):
        dig.dig_srem_dwconv_bwd(x, w, x, 4, 4, 0, workspace=ws)


@pytest.mark.parametrize("dtype,direction,bias", [("f32", 1, True), ("bf16", 2, True), ("bf16", 3, False)])
def test_conv_many_tiles_per_cta(dtype, direction, bias):
    """3 x 96 x 96 pixels x 136 channels: 1728 tiles, which selects the strip-walking kernel (8 row segments
    per strip, ragged last channel block, every scan order's tap permutation, bf16 and fp32 storage and output)."""
    _conv_case(3, 96, 96, 136, dtype, direction, bias=bias, seed=9)
    _conv_bwd_case(3, 96, 96, 136, dtype, direction, with_bias=bias, seed=9)      # dx runs through the same kernel


@pytest.mark.parametrize("dtype,direction", [("bf16", 0), ("f32", 3)])
def test_conv_strips_ragged_and_persistent(dtype, direction):
    """16 x 45 x 100 pixels x 264 channels: 13 strips per image row of which the last is 4 columns wide, a last
    channel block of 8 channels, and more strips (624) than CTAs stay resident, so some CTAs walk two strips."""
    _conv_case(16, 45, 100, 264, dtype, direction, bias=True, seed=11)
    _conv_bwd_case(16, 45, 100, 264, dtype, direction, with_bias=True, seed=11)      # dx by the same kernel, dw by the strip walk of x and dy


@pytest.mark.parametrize("gh,gw", [(2, 2048), (1, 4100), (300, 9)])
def test_conv_strips_flat_and_narrow_grids(gh, gw):
    """Grids of one or two rows (a strip is then only halo rows plus them) and grids narrower than two strips,
    large enough in the other extent to select the strip-walking kernels."""
    _conv_case(8, gh, gw, 136, "bf16", 2, bias=True, seed=12)
    _conv_bwd_case(8, gh, gw, 136, "bf16", 1, with_bias=True, seed=12)
