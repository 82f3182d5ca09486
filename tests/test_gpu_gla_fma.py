"""GPU parity of the fp32-FMA kernel family against the fp64 oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

from paper_2405_18428_b200.inputs import CONFIGS, Workload, make_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _force_fma():
    from paper_2405_18428_b200 import dig
    dig.dig_set_impl(dig.DIG_IMPL_FMA)
    yield
    dig.dig_set_impl(dig.DIG_IMPL_AUTO)


def test_c1_fp32_forward():
    from parity import check_workload
    errs = check_workload(CONFIGS["C1"], 0)
    print("C1 fma", errs)


@pytest.mark.parametrize("direction", [0, 1, 2, 3])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_small_ragged_all_directions_fwd_bwd(direction, dtype):
    """7x9 grid (63 tokens, chunk 16 -> ragged tail of 15), non-square, d_k != d_v."""
    from parity import check_workload
    wl = Workload("ragged", B=2, H=3, grid_h=7, grid_w=9, d_k=24, d_v=40, chunk=16, dtype=dtype,
                  backward=True, tau=(16.0, 2.0, 1.0), seed=3)
    check_workload(wl, direction)


@pytest.mark.parametrize("chunk", [16, 32, 64])
def test_chunk_sizes_fwd_bwd_fp32(chunk):
    from parity import check_workload
    wl = Workload("chunks", B=1, H=2, grid_h=12, grid_w=11, d_k=64, d_v=64, chunk=chunk, dtype="f32",
                  backward=True, tau=(16.0, 4.0), seed=4)
    check_workload(wl, 2)


def test_chunk128_forward_and_d72():
    from parity import check_workload
    wl = Workload("c128", B=1, H=2, grid_h=20, grid_w=13, d_k=64, d_v=64, chunk=128, dtype="f32",
                  backward=False, seed=5)
    check_workload(wl, 3)
    check_workload(wl.scaled(d_k=72, d_v=72, chunk=64, backward=True), 1)


def test_c2_bf16_storage_on_fma_family():
    from parity import check_workload
    errs = check_workload(CONFIGS["C2"], 2)
    print("C2 fma dir2", errs)


def test_single_token_and_single_chunk():
    from parity import check_workload
    check_workload(Workload("one", B=1, H=1, grid_h=1, grid_w=1, d_k=8, d_v=8, chunk=16, dtype="f32",
                            backward=True, seed=6), 0)
    check_workload(Workload("onechunk", B=1, H=1, grid_h=4, grid_w=4, d_k=8, d_v=16, chunk=16, dtype="f32",
                            backward=True, seed=7), 3)


def test_repeat_runs_are_bit_identical():
    from parity import gpu_all
    wl = CONFIGS["C1"].scaled(backward=True)
    x = make_inputs(wl, conv=False)
    a = gpu_all(wl, x, 1, True)
    b = gpu_all(wl, x, 1, True)
    for n in a:
        np.testing.assert_array_equal(a[n], b[n])
