"""The C-ABI library builds for sm_100a, loads without a GPU and exports every symbol the
header declares; host-side argument validation rejects bad calls before any launch."""
import ctypes as C
import os
import re

import pytest

from paper_2605_09503_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "pq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pq_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_named_entry_points():
    names = declared_symbols()
    for required in ["pq_calib_stats", "pq_select_perm", "pq_accept", "pq_quant_act_nvfp4", "pq_quant_weight",
                     "pq_gemm_w4a4", "pq_group_error"]:
        assert required in names


def test_library_exports_every_declared_symbol(L):
    raw = C.CDLL(binding.LIB_PATH)
    for name in declared_symbols():
        assert hasattr(raw, name), f"{name} declared in include/pq.h but not exported"
        assert name in binding._SIGNATURES, f"{name} has no Python binding"


def test_status_strings_and_sizes(L):
    assert binding.status_string(0) == "ok"
    for code in range(1, 8):
        assert binding.status_string(code) not in ("ok", "unknown status")
    assert L.pq_version() >= 1
    assert binding.sf_bytes(256, 512, binding.PQ_SF_LINEAR) == 256 * 32
    assert binding.sf_bytes(130, 512, binding.PQ_SF_TCGEN05) == 2 * 8 * 512
    assert binding.sf_bytes(130, 500, binding.PQ_SF_LINEAR) == 0
    assert binding.workspace_bytes(binding.OP_CALIB_STATS, 4608, 3072) == 36 * 3072 * (8 + 4)
    # group error: fp32 per (chunk, order, group) for candidate orders, fp64 per (slab, group) otherwise
    assert binding.workspace_bytes(binding.OP_GROUP_ERROR, 5, 4096, 0, 1) >= 1 * 256 * 8
    assert binding.workspace_bytes(binding.OP_GROUP_ERROR, 4608, 3072, 0, 6) >= 288 * 6 * 192 * 4
    assert binding.workspace_bytes(binding.OP_GROUP_ERROR, 130, 512, 0, 7) >= 3 * 7 * 32 * 4
    assert binding.workspace_bytes(binding.OP_GEMM, 128, 64, 128) >= 4
    assert binding.workspace_bytes(99, 1, 1) == 0


def test_argument_errors_are_caught_on_the_host(L):
    """No launch happens for these calls, so they run without a GPU.  The fake pointers are
    never dereferenced."""
    p = C.c_void_p(0x1000)       # 16- and 256-byte aligned, never touched
    odd = C.c_void_p(0x1008)
    fmt4 = binding.pq_format(1, 4, 32)
    assert L.pq_calib_stats(None, 8, 64, 64, p, p, p, 1 << 20, None) == 1            # NULL
    assert L.pq_calib_stats(p, 0, 64, 64, p, p, p, 1 << 20, None) == 2               # rows
    assert L.pq_calib_stats(p, 8, 60, 64, p, p, p, 1 << 20, None) == 2               # K % 8
    assert L.pq_calib_stats(odd, 8, 64, 64, p, p, p, 1 << 20, None) == 3             # alignment
    assert L.pq_calib_stats(p, 8, 64, 68, p, p, p, 1 << 20, None) == 3               # ld % 8
    assert L.pq_calib_stats(p, 8, 64, 64, p, p, p, 16, None) == 5                    # workspace
    assert L.pq_select_perm(p, 8, p, 8, 20000, 5, p, p, 1 << 30, None) == 2          # K too large
    assert L.pq_select_perm(p, 8, p, 8, 64, 0, p, p, 1 << 20, None) == 2             # J
    assert L.pq_select_perm(p, 8, p, 8, 64, 5, p, None, 0, None) == 5                # the sort keys need a workspace
    assert L.pq_select_perm(p, 8, p, 8, 64, 5, p, odd, 1 << 20, None) == 3           # ... 256-byte aligned
    assert L.pq_order_by_absmax(p, 64, p, None, 0, None) == 5
    assert L.pq_hadamard_quant_nvfp4(None, 8, 64, 64, None, p, p, p, 0, None, None) == 1          # NULL input
    assert L.pq_hadamard_quant_nvfp4(p, 8, 64, 64, None, p, p, None, 0, None, None) == 1           # codes without scales
    assert L.pq_hadamard_quant_nvfp4(p, 8, 64, 64, None, None, None, None, 0, None, None) == 1     # nothing to write
    assert L.pq_hadamard_quant_nvfp4(p, 8, 80, 80, None, p, p, p, 0, None, None) == 2              # 5 * 16: no transform
    assert L.pq_hadamard_quant_nvfp4(p, 8, 48, 48, None, p, p, p, 0, None, None) == 2              # segments of 4
    assert L.pq_hadamard_quant_nvfp4(p, 8, 96, 96, None, p, p, p, 1, None, None) == 2              # K % 64 for the TC layout
    assert L.pq_hadamard_quant_nvfp4(p, 8, 64, 64, odd, p, p, p, 0, None, None) == 3               # misaligned order
    assert L.pq_calib_sum(p, 8, 64, 64, p, None, 0, None) == 5
    assert L.pq_order_by_variance(p, p, 0, 64, p, p, 1 << 20, None) == 2                           # rows
    assert L.pq_order_round_robin(p, 64, 24, p, p, 1 << 20, None) == 2                             # K % group
    assert L.pq_selftest_wait_expiry(None, 4, 1000, p, None) == 1
    assert L.pq_selftest_wait_expiry(p, 4, 0, p, None) == 2                           # limit out of range
    assert L.pq_selftest_wait_expiry(p, 4, 10 ** 12, p, None) == 2
    assert L.pq_group_error(p, 8, 64, 64, binding.pq_format(1, 4, 48), None, None, 1, p, p, 1 << 20, None) == 4
    assert L.pq_group_error(p, 8, 64, 64, binding.pq_format(0, 4, 16), None, None, 1, p, p, 1 << 20, None) == 1
    assert L.pq_group_error(p, 8, 64, 64, fmt4, None, None, 3, p, p, 1 << 20, None) == 2   # P>1 w/o perms
    assert L.pq_accept(p, p, None, 0, 4, 0.0, p, p, None, None) == 2
    assert L.pq_quant_act_nvfp4(p, 8, 72, 72, p, p, p, 0, None) == 2                 # K % 16
    assert L.pq_quant_act_nvfp4(p, 8, 80, 80, p, p, p, 1, None) == 2                 # K % 64 for TC layout
    assert L.pq_quant_act_nvfp4(p, 8, 64, 64, p, p, p, 7, None) == 4                 # layout
    assert L.pq_quant_weight(p, 8, 64, 64, None, p, p, p, 0, p, p, 256, None) == 1   # select without table
    assert L.pq_fakequant_int(p, 8, 64, 64, binding.pq_format(0, 4, 16), None, p, 64, None) == 4
    assert L.pq_fakequant_int(p, 8, 96, 96, binding.pq_format(1, 3, 64), None, p, 96, None) == 2
    assert L.pq_gemm_w4a4(p, p, p, p, p, p, 128, 128, 96, p, 128, p, 256, None) == 2  # K % 64
    assert L.pq_gemm_w4a4(p, p, p, p, p, p, 128, 100, 64, p, 104, p, 256, None) == 2  # N % 8
    assert L.pq_gemm_w4a4(p, p, p, p, p, p, 128, 128, 64, p, 128, None, 0, None) == 5
