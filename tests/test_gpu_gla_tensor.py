"""GPU parity of the tensor-core (tcgen05) kernel family against the fp64 oracle, through the C-ABI."""
import numpy as np
import pytest

from paper_2405_18428_b200.inputs import CONFIGS, Workload, make_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _force_tensor():
    from paper_2405_18428_b200 import dig
    dig.dig_set_impl(dig.DIG_IMPL_TENSOR)
    yield
    dig.dig_set_impl(dig.DIG_IMPL_AUTO)


def _supported(wl, backward):
    from paper_2405_18428_b200 import dig
    return dig.dig_gla_query_impl(wl.d_k, wl.d_v, wl.chunk, dig.DIG_BF16, backward) == dig.DIG_IMPL_TENSOR


@pytest.mark.parametrize("direction", [0, 1, 2, 3])
def test_small_ragged_all_directions(direction):
    """9x15 grid: 135 tokens = 2 full chunks and a tail of 7; mixed gate temperatures."""
    from parity import check_workload
    wl = Workload("ragged", B=2, H=3, grid_h=9, grid_w=15, d_k=64, d_v=64, chunk=64, dtype="bf16",
                  backward=True, tau=(16.0, 4.0, 1.0), seed=3)
    bwd = _supported(wl, True)
    if not _supported(wl, False):
        pytest.skip("tensor family does not cover this shape")
    errs = check_workload(wl, direction, backward=bwd)
    print("ragged", direction, errs)


def test_single_chunk_and_single_token():
    from parity import check_workload
    for gh, gw in [(1, 1), (8, 8), (5, 13)]:
        wl = Workload("tiny", B=1, H=1, grid_h=gh, grid_w=gw, d_k=64, d_v=64, chunk=64, dtype="bf16",
                      backward=True, seed=gh)
        check_workload(wl, 3, backward=_supported(wl, True))


@pytest.mark.parametrize("cfg,direction", [("C2", 0), ("C2", 1), ("C2", 2), ("C2", 3), ("C3", 0), ("C4", 0), ("C4", 2)])
def test_benchmark_configs_full_size(cfg, direction):
    from parity import check_workload
    wl = CONFIGS[cfg]
    if not _supported(wl, False):
        pytest.skip("tensor family does not cover this shape")
    errs = check_workload(wl, direction, backward=_supported(wl, True))
    print(cfg, direction, {k: f"{v:.2e}" for k, v in errs.items()})


def test_repeat_runs_are_bit_identical():
    from parity import gpu_all
    wl = CONFIGS["C2"].scaled(B=2)
    bwd = _supported(wl, True)
    x = make_inputs(wl, conv=False)
    a = gpu_all(wl, x, 2, bwd)
    b = gpu_all(wl, x, 2, bwd)
    for n in a:
        np.testing.assert_array_equal(a[n], b[n])
