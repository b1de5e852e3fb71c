"""CPU-only checks of the boundary: the shared library loads, exports every symbol that
include/bcs.h declares, and its host-side entry points (no kernel launch) behave."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2205_10072_b200 import build_ext
    build_ext.build()
    import paper_2205_10072_b200 as bcs
    return bcs


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(bcs_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert {"bcs_build", "bcs_build_batch", "bcs_expand", "bcs_checksum", "bcs_skips", "bcs_q",
            "bcs_batch_plan", "bcs_status_str", "bcs_build_to_host", "bcs_build_workspace_bytes",
            "bcs_build_batch_workspace_bytes", "bcs_validate", "bcs_build_static", "bcs_simulate", "bcs_prepare",
            "bcs_build_prepared", "bcs_prepare_workspace_bytes", "bcs_prepare_codes", "bcs_prepare_rows", "bcs_allgather_tables", "bcs_circulant_rounds"} <= set(names)
    dll = ctypes.CDLL(lib.lib_path())
    for n in names:
        assert hasattr(dll, n), n
        assert callable(getattr(lib, n)), "binding lacks %s" % n


def test_q_and_skips_host_side(lib):
    assert lib.bcs_q(0) == -1 and lib.bcs_q(1) == 0 and lib.bcs_q(2) == 1
    assert lib.bcs_q(1024) == 10 and lib.bcs_q(1025) == 11 and lib.bcs_q(2**31 - 1) == 31
    assert lib.bcs_skips(1) == [1]
    assert lib.bcs_skips(20) == [1, 2, 3, 5, 10, 20]            # caption of Table 1
    assert lib.bcs_skips(33) == [1, 2, 3, 5, 9, 17, 33]         # caption of Table 2
    assert lib.bcs_skips(31) == [1, 2, 4, 8, 16, 31]            # caption of Table 4
    assert lib.bcs_skips(2**30 - 1) == [2**k for k in range(30)] + [2**30 - 1]
    with pytest.raises(lib.BcsError) as e:
        lib.bcs_skips(0)
    assert e.value.status == 2
    with pytest.raises(lib.BcsError) as e:
        lib.bcs_skips(2**31)
    assert e.value.status == 4


def test_status_strings(lib):
    assert [lib.bcs_status_str(i) for i in range(6)] == [
        "BCS_OK", "BCS_ERR_ARG", "BCS_ERR_RANGE", "BCS_ERR_ALIGN", "BCS_ERR_UNSUPPORTED",
        "BCS_ERR_CUDA"]
    assert lib.bcs_status_str(99) == "BCS_ERR_UNKNOWN"


def test_batch_plan_host_side(lib):
    plan = lib.bcs_batch_plan([2, 3, 20, 1, 1025])
    assert plan.rank_off.tolist() == [0, 2, 5, 25, 26, 1051]
    assert plan.entry_off.tolist() == [0, 2, 8, 108, 108, 108 + 1025 * 11]
    # tiles of 512 ranks and q rounds of align16(p) bytes of scratch for a p above 1024 only: a
    # smaller p is built by one CTA that keeps everything in shared memory
    assert plan.tile_off.tolist() == [0, 0, 0, 0, 0, 3]
    assert plan.copy_off.tolist() == [0, 0, 0, 0, 0, 11 * 1040]
    assert plan.total_tiles == 3 and plan.workspace_bytes() == 4352 + 11 * 1040
    small = lib.bcs_batch_plan([1024, 7, 1])
    assert small.total_tiles == 0 and small.total_copy == 0 and small.workspace_bytes() == 256
    assert plan.skips_tab[2].tolist()[:6] == [1, 2, 3, 5, 10, 20]
    assert plan.skips_tab[3].tolist()[:2] == [1, 0]
    # full_tab[d] = skip code of rank skips[d]-1: p = 20, skips 1 2 3 5 10 20:
    # 0 -> {}, 1 -> {0}, 2 -> {1}, 4 = 3+1 -> {2,0}, 9 = 5+3+1 -> {3,2,0}, 19 = 10+5+3+1
    assert plan.full_tab[2].tolist()[:6] == [0, 1, 2, 5, 13, 29]
    assert plan.total_ranks == 1051
    with pytest.raises(lib.BcsError):
        lib.bcs_batch_plan([5, 0])


def test_argument_errors_need_no_gpu(lib):
    """Validation happens before any CUDA call: these return an error code on a CPU-only box."""
    L = lib.lib()
    assert L.bcs_build(0, 0, 0, None, None, None, 0, None) == 2
    assert L.bcs_build(2**31, 0, 1, None, None, None, 0, None) == 4
    assert L.bcs_build(10, 5, 4, None, None, None, 0, None) == 2
    assert L.bcs_build(10, 0, 11, None, None, None, 0, None) == 2
    assert L.bcs_build(10, 0, 10, None, None, None, 0, None) == 1
    assert L.bcs_build(10, 0, 10, 8, None, None, 0, None) == 3   # misaligned pointer
    assert L.bcs_build(1, 0, 1, None, None, None, 0, None) == 0  # q == 0: nothing to do
    assert L.bcs_build(10, 3, 3, None, None, None, 0, None) == 0 # empty range
    assert L.bcs_build_workspace_bytes(2**20 + 1, 0, 2**20 + 1) == 4194560 + 21 * 1048592
    assert L.bcs_build_workspace_bytes(0, 0, 0) == 0
    assert L.bcs_build_batch_workspace_bytes(1000, 9008) == 4096 + 9008
    assert L.bcs_expand(10, 0, 0, 10, 16, 16, 16, None) == 1     # n == 0
    assert L.bcs_expand(10, 4, 0, 10, None, 16, 16, None) == 1
    assert L.bcs_expand(10, 4, 0, 10, 16, 16, 8, None) == 3
    assert L.bcs_checksum(16, 8, 2, 16, None) == 3               # first index not a multiple of 4
    assert L.bcs_checksum(16, 8, 0, None, None) == 1
    assert L.bcs_build_batch(None, None, None, None, None, None, None, 3, 10, 40, 1, 48, 16, None, None, 0,
                             None) == 1
    assert L.bcs_prepare_codes(0, 16, 1 << 20, None) == 2
    assert L.bcs_prepare_codes(1000, None, 0, None) == 1
    assert L.bcs_prepare_codes(1000, 16, 64, None) == 1                       # workspace too small
    assert L.bcs_prepare_codes(1000, 8, 1 << 20, None) == 3                    # misaligned workspace
    assert L.bcs_prepare_rows(1000, 8, 100, 16, 16, 1 << 20, None) == 3        # r_begin not a multiple of 16
    assert L.bcs_prepare_rows(1000, 16, 1001, 16, 16, 1 << 20, None) == 2
    assert L.bcs_prepare_rows(1000, 16, 100, 24, 16, 1 << 20, None) == 3       # misaligned rows
    assert L.bcs_prepare_rows(1000, 16, 16, None, 16, 1 << 20, None) == 0      # empty range
    assert L.bcs_prepare_workspace_bytes(1000) == 4096 + 10 * 1008
    assert L.bcs_expand(10, 4, 0, 10, None, None, None, None) == 1             # no table to write to
    assert L.bcs_build_to_host(10, 0, 10, None, None, 16, 1024, None) == 1
    assert L.bcs_build_to_host(10, 0, 10, 16, None, 16, 16, None) == 1   # staging too small
