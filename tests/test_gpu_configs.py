"""GPU parity at the benchmark configurations that the other files do not cover: the d = 72 workload
(C5) and the chunk sweep of C4, with whichever kernel family the library picks for them."""
import numpy as np
import pytest

from paper_2405_18428_b200.inputs import CONFIGS

pytestmark = pytest.mark.gpu


def _family(wl, chunk, backward):
    from paper_2405_18428_b200 import dig
    return dig.dig_gla_query_impl(wl.d_k, wl.d_v, chunk, dig.DIG_BF16, backward)


def test_c5_full_size_column_reverse():
    """128 x 128 grid, 16 heads of 72 channels, forward and backward, column-major reverse scan."""
    from parity import check_workload
    errs = check_workload(CONFIGS["C5"], 3)
    print("C5 dir 3", {k: f"{v:.2e}" for k, v in errs.items()})


@pytest.mark.parametrize("direction", [0, 1, 2])
def test_c5_other_directions_four_heads(direction):
    from parity import check_workload
    check_workload(CONFIGS["C5"].scaled(H=4), direction)


@pytest.mark.parametrize("chunk", [32, 64, 128])
def test_c4_chunk_sweep(chunk):
    """112 x 112 grid: 64 does not divide the column length, so column orders straddle columns.
    Every chunk size must be served by some kernel family, forward and backward."""
    from paper_2405_18428_b200 import dig
    from parity import check_workload
    wl = CONFIGS["C4"]
    assert _family(wl, chunk, False) > 0
    assert _family(wl, chunk, True) > 0
    errs = check_workload(wl, 2, chunk=chunk, backward=True)
    print("C4 chunk", chunk, {k: f"{v:.2e}" for k, v in errs.items()})


def test_chunk_size_does_not_change_the_result_beyond_rounding():
    from parity import gpu_all
    from paper_2405_18428_b200.inputs import make_inputs
    wl = CONFIGS["C4"].scaled(H=2)
    x = make_inputs(wl, conv=False)
    a = gpu_all(wl, x, 0, True, chunk=32)
    b = gpu_all(wl, x, 0, True, chunk=64)
    for n in a:
        rms = np.sqrt(np.mean(a[n].astype(np.float64) ** 2))
        assert np.abs(a[n].astype(np.float64) - b[n]).max() <= 2e-2 * rms, n


def test_chunk128_forward_on_the_fma_family_matches_too():
    """Forcing the fp32-FMA family keeps a real 128-token chunk (forward only there)."""
    from paper_2405_18428_b200 import dig
    from parity import check_workload
    dig.dig_set_impl(dig.DIG_IMPL_FMA)
    try:
        check_workload(CONFIGS["C4"].scaled(H=2), 1, chunk=128, backward=False)
    finally:
        dig.dig_set_impl(dig.DIG_IMPL_AUTO)
