"""GPU parity of the sums over several scan orders (Algorithm 2, bidirectional, and Algorithm 3,
4-directional scanning) against the fp64 oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

from paper_2405_18428_b200.inputs import CONFIGS, Workload, make_inputs

pytestmark = pytest.mark.gpu


def _check(wl, dirs):
    import oracle
    from paper_2405_18428_b200 import dig
    from parity import TOL_BF16, oracle_threads, rel_err, to_dev
    x = make_inputs(wl, conv=False)
    q, k, v, g, dO = (to_dev(x[n], wl) for n in ("q", "k", "v", "g", "dO"))
    gate = dig.dig_gate_logsigmoid(g, x["tau"])
    a = oracle.gate(x["g"], x["tau"])
    thr = oracle_threads()
    ref = (oracle.gla_fwd_multi(x["q"], x["k"], x["v"], a, wl.grid_h, wl.grid_w, dirs, threads=thr),
           *oracle.gla_bwd_multi(x["q"], x["k"], x["v"], a, x["dO"], wl.grid_h, wl.grid_w, dirs, threads=thr))
    names = ("out", "dq", "dk", "dv", "dgate")
    got32 = (dig.dig_gla_fwd_multi(q, k, v, gate, wl.grid_h, wl.grid_w, dirs, wl.chunk, f32_out=True),
             *dig.dig_gla_bwd_multi(q, k, v, gate, dO, wl.grid_h, wl.grid_w, dirs, wl.chunk, f32_out=True))
    got16 = (dig.dig_gla_fwd_multi(q, k, v, gate, wl.grid_h, wl.grid_w, dirs, wl.chunk),
             *dig.dig_gla_bwd_multi(q, k, v, gate, dO, wl.grid_h, wl.grid_w, dirs, wl.chunk))
    torch.cuda.synchronize()
    assert dig.dig_last_device_status() == dig.DIG_OK
    errs = {}
    for n, g32, g16, r in zip(names, got32, got16, ref):
        g32 = g32.float().cpu().numpy()
        assert np.isfinite(g32).all(), n
        errs[n] = rel_err(g32, r)
        assert errs[n] <= TOL_BF16, (n, dirs, errs[n])
        # the bf16 results are the fp32 sums rounded once
        want = g32 if n == "dgate" else torch.from_numpy(g32).to(torch.bfloat16).float().numpy()
        np.testing.assert_array_equal(g16.float().cpu().numpy(), want, err_msg=n)
    return errs


@pytest.mark.parametrize("dirs", [(0, 1), (2, 3), (0, 1, 2, 3)])
def test_c2_full_size(dirs):
    print(dirs, {k: f"{v:.2e}" for k, v in _check(CONFIGS["C2"], dirs).items()})


@pytest.mark.parametrize("dirs", [(0, 1), (2, 3), (0, 1, 2, 3)])
def test_long_sequences_d72_ragged(dirs):
    """4 heads of the XL width on a 90 x 91 grid: 8190 tokens, a ragged last tile, columns that straddle tiles."""
    wl = CONFIGS["C5"].scaled(H=4, grid_h=90, grid_w=91)
    print(dirs, {k: f"{v:.2e}" for k, v in _check(wl, dirs).items()})


def test_one_direction_equals_the_plain_entry_points():
    from paper_2405_18428_b200 import dig
    from parity import to_dev
    wl = Workload("m1", B=2, H=2, grid_h=12, grid_w=17, d_k=64, d_v=64, chunk=64, dtype="bf16", seed=5)
    x = make_inputs(wl, conv=False)
    q, k, v, g, dO = (to_dev(x[n], wl) for n in ("q", "k", "v", "g", "dO"))
    gate = dig.dig_gate_logsigmoid(g, x["tau"])
    for d in range(4):
        assert torch.equal(dig.dig_gla_fwd_multi(q, k, v, gate, 12, 17, (d,)), dig.dig_gla_fwd(q, k, v, gate, 12, 17, 64, d))
        for a, b in zip(dig.dig_gla_bwd_multi(q, k, v, gate, dO, 12, 17, (d,)), dig.dig_gla_bwd(q, k, v, gate, dO, 12, 17, 64, d)):
            assert torch.equal(a, b)


def test_bad_masks_and_unsupported_shapes_are_refused():
    from paper_2405_18428_b200 import dig
    t = torch.zeros(1, 16, 1, 64, dtype=torch.bfloat16, device="cuda")
    gate = torch.zeros(1, 16, 1, 64, dtype=torch.float32, device="cuda")
    with pytest.raises(dig.DigError) as e:
        dig.dig_gla_fwd_multi(t, t, t, gate, 4, 4, ())
    assert e.value.status == dig.DIG_ERR_INVALID_ARG
    t32 = torch.zeros(1, 16, 1, 64, device="cuda")
    assert dig.dig_gla_multi_workspace_bytes(1, 1, 4, 4, 64, 64, 64, dig.DIG_F32, 0) == 0
    with pytest.raises(dig.DigError):
        dig.dig_gla_fwd_multi(t32, t32, t32, gate, 4, 4, (0, 1))
