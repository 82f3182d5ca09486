"""GPU parity at the edges of the operator's domain, on both tensor-core families: gates close to the
documented limit of the in-chunk decay, no decay at all (plain causal linear attention, Eq.
attn_simple), one-row and one-column grids in every scan order, all-zero inputs, and chunk pairs that
straddle two sequences."""
import numpy as np
import pytest
import torch

from paper_2405_18428_b200.inputs import Workload, make_inputs, round_to_bf16
from parity import check_workload

pytestmark = pytest.mark.gpu

FAMILIES = [("tensor", 64, 64), ("tensor", 72, 64), ("tensor", 64, 32), ("mma", 72, 64), ("mma", 64, 32)]


@pytest.fixture(autouse=True)
def _force_family(request):
    """Tests parametrised over a family run with that family forced."""
    from paper_2405_18428_b200 import dig
    family = getattr(request.node, "callspec", None) and request.node.callspec.params.get("family")
    if family:
        dig.dig_set_impl({"tensor": dig.DIG_IMPL_TENSOR, "mma": dig.DIG_IMPL_MMA}[family])
    yield
    dig.dig_set_impl(dig.DIG_IMPL_AUTO)


def _wl(d, chunk, **kw):
    base = dict(B=1, H=2, grid_h=12, grid_w=16, d_k=d, d_v=d, chunk=chunk, dtype="bf16", backward=True, tau=(1.0, 1.0), seed=41)
    base.update(kw)
    return Workload("edge", **base)


def _with_gate_logit(wl, logit):
    """Inputs whose gate is the same for every token and channel: logsigmoid(logit) / tau, tau = 1."""
    x = make_inputs(wl, conv=False)
    x["g"] = np.full_like(x["g"], round_to_bf16(np.float32(logit)))
    return x


@pytest.mark.parametrize("family,d,chunk", FAMILIES)
def test_strong_constant_decay(family, d, chunk):
    # log alpha = -1 per token: the gate summed over a 64-token chunk reaches -64, exp(+-64) is used inside
    wl = _wl(d, chunk)
    x = _with_gate_logit(wl, np.log(np.exp(-1.0) / (1.0 - np.exp(-1.0))))
    print(family, check_workload(wl, 0, x=x))
    print(family, check_workload(wl, 3, x=x))


@pytest.mark.parametrize("family,d,chunk", FAMILIES)
def test_no_decay_is_causal_linear_attention(family, d, chunk):
    # temperature 1e6: log alpha is about -1e-6 per token, alpha = 1 to six digits; the state only accumulates
    wl = _wl(d, chunk, tau=(1e6, 1e6))
    print(family, check_workload(wl, 1))


@pytest.mark.parametrize("family,d,chunk", FAMILIES)
@pytest.mark.parametrize("direction", [0, 1, 2, 3])
def test_one_row_and_one_column_grids(family, d, chunk, direction):
    check_workload(_wl(d, chunk, grid_h=1, grid_w=150, tau=(16.0, 2.0)), direction)
    check_workload(_wl(d, chunk, grid_h=150, grid_w=1, tau=(16.0, 2.0)), direction)


@pytest.mark.parametrize("family,d,chunk", FAMILIES)
def test_all_zero_inputs_give_zeros(family, d, chunk):
    from paper_2405_18428_b200 import dig
    wl = _wl(d, chunk)
    z = lambda dd: torch.zeros(wl.B, wl.L, wl.H, dd, device="cuda", dtype=torch.bfloat16)
    gate = torch.zeros(wl.B, wl.L, wl.H, d, device="cuda")
    out = dig.dig_gla_fwd(z(d), z(d), z(d), gate, wl.grid_h, wl.grid_w, chunk, 2)
    grads = dig.dig_gla_bwd(z(d), z(d), z(d), gate, z(d), wl.grid_h, wl.grid_w, chunk, 2)
    torch.cuda.synchronize()
    assert dig.dig_last_device_status() == dig.DIG_OK
    for t in (out, *grads):
        assert torch.count_nonzero(t) == 0


@pytest.mark.parametrize("family,d,chunk", FAMILIES)
def test_odd_chunk_count_with_several_sequences(family, d, chunk):
    # 11 x 15 = 165 tokens: an odd number of chunks per sequence (3 of 64, or 6 of 32 with a ragged last one),
    # 3 x 3 = 9 sequences, so consecutive chunk ids pair up across sequence boundaries
    wl = _wl(d, chunk, B=3, H=3, grid_h=11, grid_w=15, tau=(16.0, 4.0, 1.0))
    print(family, check_workload(wl, 2))


def test_families_are_the_intended_ones():
    """Left to itself the library serves every bf16 shape of this file with the tcgen05 kernels; the
    warp-level family takes them when it is forced."""
    from paper_2405_18428_b200 import dig
    for _, d, chunk in FAMILIES:
        assert dig.dig_gla_query_impl(d, d, chunk, dig.DIG_BF16, 1) == dig.DIG_IMPL_TENSOR
    dig.dig_set_impl(dig.DIG_IMPL_MMA)
    try:
        for family, d, chunk in FAMILIES:
            if family == "mma":
                assert dig.dig_gla_query_impl(d, d, chunk, dig.DIG_BF16, 1) == dig.DIG_IMPL_MMA
    finally:
        dig.dig_set_impl(dig.DIG_IMPL_AUTO)


def _constant_gate_case(per_token, d=64):
    from paper_2405_18428_b200 import dig
    from parity import to_dev
    wl = _wl(d, 64, grid_h=10, grid_w=20)
    x = make_inputs(wl, conv=False)
    gate = np.full(x["q"].shape, per_token, dtype=np.float32)
    q, k, v, dO = (to_dev(x[n], wl) for n in ("q", "k", "v", "dO"))
    return wl, x, gate, (q, k, v, torch.from_numpy(gate).cuda(), dO)


@pytest.mark.parametrize("d", [64, 72])
def test_fast_decay_inside_the_range_is_worked_in_sub_chunks(d):
    """log alpha = -1.9 per token: 64 tokens sum to -122, far beyond what one fp16 tile can centre; the tcgen05
    kernels fall back to 8-token sub-chunks (8 x 1.9 = 15.2 < 15.9) and still match the oracle."""
    import oracle
    from paper_2405_18428_b200 import dig
    from parity import TOL_BF16, rel_err
    wl, x, gate, (q, k, v, g, dO) = _constant_gate_case(-1.9, d)
    out = dig.dig_gla_fwd(q, k, v, g, wl.grid_h, wl.grid_w, 64, 2, f32_out=True)
    grads = dig.dig_gla_bwd(q, k, v, g, dO, wl.grid_h, wl.grid_w, 64, 2, f32_out=True)
    torch.cuda.synchronize()
    assert dig.dig_last_device_status() == dig.DIG_OK
    a = gate.astype(np.float64)
    ref = (oracle.gla_fwd(x["q"], x["k"], x["v"], a, wl.grid_h, wl.grid_w, 2),
           *oracle.gla_bwd(x["q"], x["k"], x["v"], a, x["dO"], wl.grid_h, wl.grid_w, 2))
    for name, got, want in zip(("out", "dq", "dk", "dv", "dgate"), (out, *grads), ref):
        got = got.float().cpu().numpy()
        assert np.isfinite(got).all(), name
        assert rel_err(got, want) <= TOL_BF16, (name, rel_err(got, want))


def test_decay_beyond_the_range_is_reported_not_silent():
    """log alpha = -3 per token: even 8 tokens sum to -24.  The call must say so through the device status
    (DIG_ERR_RANGE), return finite numbers, and the status must be cleared by the query."""
    from paper_2405_18428_b200 import dig
    wl, x, gate, (q, k, v, g, dO) = _constant_gate_case(-3.0)
    out = dig.dig_gla_fwd(q, k, v, g, wl.grid_h, wl.grid_w, 64, 0, f32_out=True)
    torch.cuda.synchronize()
    assert dig.dig_last_device_status() == dig.DIG_ERR_RANGE
    assert dig.dig_last_device_status() == dig.DIG_OK
    assert torch.isfinite(out).all()
    grads = dig.dig_gla_bwd(q, k, v, g, dO, wl.grid_h, wl.grid_w, 64, 0, f32_out=True)
    torch.cuda.synchronize()
    assert dig.dig_last_device_status() == dig.DIG_ERR_RANGE
    for t in grads:
        assert torch.isfinite(t).all()
    assert "range" in dig.status_string(dig.DIG_ERR_RANGE)


def test_a_wait_that_nothing_satisfies_expires_and_is_reported_once():
    """Every wait inside the kernels is bounded.  A dedicated kernel waits 2 ms on a barrier nobody arrives
    on: the device status must say so exactly once, and the library must keep working afterwards."""
    from paper_2405_18428_b200 import dig
    assert dig.dig_last_device_status() == dig.DIG_OK
    dig.dig_selftest_wait_timeout(2000)
    assert dig.dig_last_device_status() == dig.DIG_ERR_TIMEOUT
    assert dig.dig_last_device_status() == dig.DIG_OK
    check_workload(_wl(64, 64), 0)
