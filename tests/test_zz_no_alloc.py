"""dig_gla_fwd_static: the forward call for callers that cannot allocate device memory.

Some users of the library run where no allocator may be called: the host application owns all of
the GPU's memory and hands over only inputs and outputs, or a cudaMalloc in the middle of a
latency-critical loop would synchronise the device.  The entry point tested here takes no
workspace: its scratch is a fixed 16 MiB array inside the library.  It must give what dig_gla_fwd
gives with a caller-allocated workspace, also on a second call that finds the first call's
leftovers in the shared array.

This file sorts last on purpose, so a run that stops at the first failure has already run every
other test.  It passes alone in a fresh process as well as after the rest of the suite.
"""
import numpy as np
import pytest

from paper_2405_18428_b200.inputs import Workload, make_inputs

pytestmark = pytest.mark.gpu


def _inputs(wl):
    import torch
    from parity import to_dev
    from paper_2405_18428_b200 import dig
    x = make_inputs(wl, conv=False)
    q, k, v, g = (to_dev(x[n], wl) for n in ("q", "k", "v", "g"))
    gate = dig.dig_gate_logsigmoid(g, x["tau"])
    torch.cuda.synchronize()
    return q, k, v, gate


def test_static_scratch_forward_matches_workspace_forward_twice():
    import torch
    import oracle
    from parity import TOL_BF16, rel_err
    from paper_2405_18428_b200 import dig

    # two different problems back to back: the second finds the first one's states in the array,
    # and has more chunks per sequence and another scan order, so stale entries would show
    first = Workload("static-a", B=2, H=3, grid_h=16, grid_w=12, d_k=64, d_v=64, chunk=64, dtype="bf16",
                     tau=(16.0, 4.0), seed=11)
    second = Workload("static-b", B=1, H=2, grid_h=9, grid_w=31, d_k=64, d_v=64, chunk=64, dtype="bf16",
                      tau=(4.0,), seed=12)
    for wl, direction in ((first, 0), (second, 3)):
        x = make_inputs(wl, conv=False)
        q, k, v, gate = _inputs(wl)
        want = dig.dig_gla_fwd(q, k, v, gate, wl.grid_h, wl.grid_w, wl.chunk, direction, f32_out=True)
        out = torch.full(want.shape, float("nan"), dtype=torch.float32, device="cuda")   # caller-owned output
        dig.dig_gla_fwd_static(q, k, v, gate, out, wl.grid_h, wl.grid_w, wl.chunk, direction)   # first call on the device: set-up
        torch.cuda.synchronize()
        # a second call must leave both torch's allocator and the device's free memory untouched
        out.fill_(float("nan"))
        torch.cuda.synchronize()
        held, (free0, _) = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()
        dig.dig_gla_fwd_static(q, k, v, gate, out, wl.grid_h, wl.grid_w, wl.chunk, direction)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == held
        assert torch.cuda.mem_get_info()[0] == free0
        assert dig.dig_last_device_status() == dig.DIG_OK
        got = out.cpu().numpy()
        assert np.isfinite(got).all()
        # the header promises the same kernels on other scratch memory: the same bits
        np.testing.assert_array_equal(got, want.cpu().numpy())
        # and, like every other entry point, it is held against the fp64 oracle
        a = oracle.gate(x["g"], x["tau"])
        ref = oracle.gla_fwd(x["q"], x["k"], x["v"], a, wl.grid_h, wl.grid_w, direction)
        err = rel_err(got, ref)
        assert err <= TOL_BF16, f"{wl.name}: static-scratch forward differs from the oracle by {err:.3e}"


def test_static_scratch_rejects_problems_beyond_its_limit():
    import torch
    from paper_2405_18428_b200 import dig

    # 64 x 64 grid, 48 sequences: the chunk states alone need about 50 MB, more than the 16 MiB array
    B, H, gh, gw, d = 4, 12, 64, 64, 64
    need = dig.dig_gla_workspace_bytes(B, H, gh, gw, d, d, 64, dig.DIG_BF16, 0)
    assert need > dig.DIG_GLA_STATIC_SCRATCH_BYTES
    t = torch.zeros((B, gh * gw, H, d), dtype=torch.bfloat16, device="cuda")
    gate = torch.zeros((B, gh * gw, H, d), dtype=torch.float32, device="cuda")
    out = torch.zeros_like(t)
    with pytest.raises(dig.DigError) as e:
        dig.dig_gla_fwd_static(t, t, t, gate, out, gh, gw, 64, 0)
    assert e.value.status == dig.DIG_ERR_SCRATCH_LIMIT
    assert "built-in scratch" in str(e.value)
