"""GPU parity of the warp-MMA kernel family (mma.sync tf32; bf16 storage, any head size that is a
multiple of 8, chunks of 16 to 128 tokens) against the fp64 oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

from paper_2405_18428_b200.inputs import CONFIGS, Workload, make_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _force_mma():
    from paper_2405_18428_b200 import dig
    dig.dig_set_impl(dig.DIG_IMPL_MMA)
    yield
    dig.dig_set_impl(dig.DIG_IMPL_AUTO)


def test_auto_picks_this_family_where_tcgen05_does_not_apply():
    from paper_2405_18428_b200 import dig
    dig.dig_set_impl(dig.DIG_IMPL_AUTO)
    assert dig.dig_gla_query_impl(72, 72, 64, dig.DIG_BF16, 1) == dig.DIG_IMPL_TENSOR     # the paper's XL head size
    assert dig.dig_gla_query_impl(64, 64, 32, dig.DIG_BF16, 1) == dig.DIG_IMPL_TENSOR
    assert dig.dig_gla_query_impl(64, 64, 64, dig.DIG_BF16, 1) == dig.DIG_IMPL_TENSOR
    assert dig.dig_gla_query_impl(24, 40, 16, dig.DIG_BF16, 1) == dig.DIG_IMPL_MMA        # d_k != d_v, other head sizes
    assert dig.dig_gla_query_impl(72, 72, 64, dig.DIG_F32, 1) == dig.DIG_IMPL_FMA
    dig.dig_set_impl(dig.DIG_IMPL_MMA)
    assert dig.dig_gla_query_impl(72, 72, 64, dig.DIG_F32, 1) < 0          # fp32 storage is not served


@pytest.mark.parametrize("direction", [0, 1, 2, 3])
def test_small_ragged_all_directions_fwd_bwd(direction):
    """7x9 grid (63 tokens, chunk 16 -> ragged tail of 15), non-square, d_k != d_v, neither a multiple of 16."""
    from parity import check_workload
    wl = Workload("ragged", B=2, H=3, grid_h=7, grid_w=9, d_k=24, d_v=40, chunk=16, dtype="bf16",
                  backward=True, tau=(16.0, 2.0, 1.0), seed=3)
    check_workload(wl, direction)


@pytest.mark.parametrize("chunk", [16, 32, 64])
@pytest.mark.parametrize("d", [8, 64, 72, 128])
def test_head_and_chunk_sizes_fwd_bwd(chunk, d):
    from paper_2405_18428_b200 import dig
    from parity import check_workload
    if dig.dig_gla_query_impl(d, d, chunk, dig.DIG_BF16, 1) < 0:
        pytest.skip("does not fit shared memory")
    wl = Workload("sizes", B=1, H=2, grid_h=12, grid_w=11, d_k=d, d_v=d, chunk=chunk, dtype="bf16",
                  backward=True, tau=(16.0, 4.0), seed=4)
    check_workload(wl, 2)


def test_chunk128_forward():
    from parity import check_workload
    wl = Workload("c128", B=1, H=2, grid_h=20, grid_w=13, d_k=64, d_v=64, chunk=128, dtype="bf16",
                  backward=False, seed=5)
    check_workload(wl, 3)


def test_c2_on_this_family():
    from parity import check_workload
    errs = check_workload(CONFIGS["C2"], 1)
    print("C2 mma dir1", errs)


def test_single_token_and_single_chunk():
    from parity import check_workload
    check_workload(Workload("one", B=1, H=1, grid_h=1, grid_w=1, d_k=8, d_v=8, chunk=16, dtype="bf16",
                            backward=True, seed=6), 0)
    check_workload(Workload("onechunk", B=1, H=1, grid_h=4, grid_w=4, d_k=8, d_v=16, chunk=16, dtype="bf16",
                            backward=True, seed=7), 3)


def test_repeat_runs_are_bit_identical():
    from parity import gpu_all
    wl = Workload("rep", B=1, H=2, grid_h=16, grid_w=16, d_k=72, d_v=72, chunk=64, dtype="bf16", backward=True, seed=8)
    x = make_inputs(wl, conv=False)
    a = gpu_all(wl, x, 1, True)
    b = gpu_all(wl, x, 1, True)
    for n in a:
        np.testing.assert_array_equal(a[n], b[n])
