"""Host-side checks of the C-ABI library: it loads, exports what the header declares, and rejects
bad arguments before touching the GPU (no kernel is launched here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2405_18428_b200 import build, dig
    build.build()
    return dig.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "dig_gla.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dig_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    from paper_2405_18428_b200 import dig
    names = _declared()
    assert set(names) == set(dig.EXPORTS)
    for n in names:
        assert getattr(L, n) is not None


def test_status_strings(L):
    seen = {L.dig_status_string(i).decode() for i in range(8)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert L.dig_status_string(99).decode() == "unknown status"


def test_workspace_bytes(L):
    # forward: states [B*H][N][dk][dv] + gamma [B*H][N][dk], fp32, each block 256-byte aligned
    n = L.dig_gla_workspace_bytes(1, 6, 16, 16, 64, 64, 64, 0, 0)
    assert n == 6 * 4 * 64 * 64 * 4 + 6 * 4 * 64 * 4
    # backward: + dstates, carry and the state after the last chunk [B*H][dk][dv]
    assert L.dig_gla_workspace_bytes(1, 6, 16, 16, 64, 64, 64, 0, 1) == 2 * n + 6 * 64 * 64 * 4
    # bf16 storage: sized for whichever family may serve the call, so at least what the per-chunk families need
    assert L.dig_gla_workspace_bytes(1, 6, 16, 16, 64, 64, 64, 1, 0) >= n
    assert L.dig_gla_workspace_bytes(1, 6, 16, 16, 64, 64, 64, 1, 1) >= 2 * n + 6 * 64 * 64 * 4
    # ragged tail: 10x10 = 100 tokens in chunks of 64 -> 2 chunks
    assert L.dig_gla_workspace_bytes(1, 1, 10, 10, 8, 8, 64, 1, 0) == 2 * 8 * 8 * 4 + 256
    for bad in [(0, 6, 16, 16, 64, 64, 64, 0, 0), (1, 6, 16, 16, 60, 64, 64, 0, 0),
                (1, 6, 16, 16, 64, 136, 64, 0, 0), (1, 6, 16, 16, 64, 64, 48, 0, 0),
                (1, 6, 16, 16, 64, 64, 64, 7, 0)]:
        assert L.dig_gla_workspace_bytes(*bad) == 0


def test_query_impl(L):
    from paper_2405_18428_b200 import dig
    assert L.dig_gla_query_impl(64, 64, 64, dig.DIG_F32, 0) == dig.DIG_IMPL_FMA
    assert L.dig_gla_query_impl(64, 64, 64, dig.DIG_F32, 1) == dig.DIG_IMPL_FMA
    assert L.dig_gla_query_impl(60, 64, 64, dig.DIG_F32, 0) == -dig.DIG_ERR_INVALID_ARG
    # fp32-FMA backward at chunk 128 does not fit in shared memory
    assert L.dig_gla_query_impl(64, 64, 128, dig.DIG_F32, 1) == -dig.DIG_ERR_UNSUPPORTED
    assert L.dig_set_impl(5) == dig.DIG_ERR_INVALID_ARG
    assert L.dig_set_impl(dig.DIG_IMPL_AUTO) == dig.DIG_OK


def test_bad_arguments_are_rejected_on_the_host(L):
    from paper_2405_18428_b200 import dig
    p = ctypes.c_void_p
    ok = 0x1000          # never dereferenced: validation fails first
    geom = (1, 6, 16, 16, 64, 64, 64, 0, 0)
    assert L.dig_gla_fwd(None, ok, ok, ok, ok, *geom, ok, 1 << 30, None) == dig.DIG_ERR_INVALID_ARG
    assert L.dig_gla_fwd(ok + 4, ok, ok, ok, ok, *geom, ok, 1 << 30, None) == dig.DIG_ERR_INVALID_ARG
    assert L.dig_gla_fwd(ok, ok, ok, ok, ok, 1, 6, 16, 16, 64, 64, 64, 4, 0, ok, 1 << 30, None) == dig.DIG_ERR_INVALID_ARG
    assert L.dig_gla_fwd(ok, ok, ok, ok, ok, 1, 6, 16, 16, 64, 64, 24, 0, 0, ok, 1 << 30, None) == dig.DIG_ERR_INVALID_ARG
    assert L.dig_gla_fwd(ok, ok, ok, ok, ok, *geom, None, 0, None) == dig.DIG_ERR_WORKSPACE
    assert L.dig_gla_fwd(ok, ok, ok, ok, ok, *geom, ok, 16, None) == dig.DIG_ERR_WORKSPACE
    assert L.dig_gla_bwd(ok, ok, ok, ok, None, ok, ok, ok, ok, *geom, ok, 1 << 30, None) == dig.DIG_ERR_INVALID_ARG
    assert L.dig_gla_bwd(ok, ok, ok, ok, ok, ok, ok, ok, ok, 1, 6, 16, 16, 64, 64, 128, 0, 0, ok, 1 << 30, None) == dig.DIG_ERR_UNSUPPORTED
    assert L.dig_srem_dwconv(ok, ok, None, None, 1, 8, 8, 64, 0, 0, None) == dig.DIG_ERR_INVALID_ARG
    assert L.dig_srem_dwconv(ok, ok, None, ok, 1, 8, 8, 60, 0, 0, None) == dig.DIG_ERR_INVALID_ARG
    assert L.dig_srem_dwconv(ok, ok, None, ok, 1, 8, 8, 64, 9, 0, None) == dig.DIG_ERR_INVALID_ARG
    tau = (ctypes.c_float * 2)(1.0, 1.0)
    assert L.dig_gate_logsigmoid(ok, tau, None, 1, 4, 2, 8, 0, None) == dig.DIG_ERR_INVALID_ARG
    assert L.dig_gate_logsigmoid(ok, None, ok, 1, 4, 2, 8, 0, None) == dig.DIG_ERR_INVALID_ARG


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    from paper_2405_18428_b200 import dig
    monkeypatch.setattr(dig, "_lib", None)
    monkeypatch.setattr(dig, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError, match="no CPU fallback"):
        dig.lib()
