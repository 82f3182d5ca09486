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
