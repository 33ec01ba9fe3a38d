"""Host-side checks of the C ABI: the library loads, exports what the header declares,
sizes and argument errors are answered without touching a GPU."""

import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "tl_e0m4.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tl_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound(lib):
    declared = _declared_symbols()
    assert "tl_e0m4_matmul" in declared and "tl_e0m4_quantize" in declared
    handle = ctypes.CDLL(lib.LIB_PATH)
    for name in declared:
        assert hasattr(handle, name), name
    assert sorted(lib.SYMBOLS) == declared


def test_packed_sizes(lib):
    assert lib.tl_e0m4_packed_sizes(4096, 4096) == (4096 * 4096 // 2, 32 * 4096 * 4)
    assert lib.tl_e0m4_packed_sizes(13696, 5120) == (13696 * 5120 // 2, 107 * 5120 * 4)
    assert lib.tl_e0m4_packed_sizes(4096, 4096, 64) == (4096 * 4096 // 2, 64 * 4096 * 4)
    assert lib.tl_e0m4_packed_sizes(13696, 5120, 32) == (13696 * 5120 // 2, 428 * 5120 * 4)
    for K, N, group in [(100, 16, 128), (128, 24, 128), (128, 16, 48), (128, 16, 16), (128, 16, 256), (64, 16, 64),
                        (0, 16, 128), (128, -16, 128)]:
        with pytest.raises(lib.TlError) as err:
            lib.tl_e0m4_packed_sizes(K, N, group)
        assert err.value.status == 2  # TL_ERR_SHAPE


def test_stage_switches_at_sixteen_tokens_and_kernel_at_eight(lib):
    for M in (1, 2, 8, 9, 16):
        assert lib.tl_e0m4_matmul_stage(M) == lib.TL_STAGE_DECODE
    for M in (17, 64, 128, 4096):
        assert lib.tl_e0m4_matmul_stage(M) == lib.TL_STAGE_PREFILL
    # what really runs: the register kernel up to 8 tokens, the tensor-core kernel from 9
    for M in (1, 2, 8):
        assert lib.tl_e0m4_matmul_kernel(M, 4096, 4096) == lib.TL_KERNEL_REGISTER
    for M in (9, 16, 17, 4096):
        assert lib.tl_e0m4_matmul_kernel(M, 4096, 4096) == lib.TL_KERNEL_TENSOR


def test_tuning_overrides_are_read_by_sizing_and_dispatch_and_can_be_restored(lib):
    L = lib.lib()
    assert L.tl_e0m4_tuning_set(b"no_such_key", 1) == 10  # TL_ERR_KEY
    try:
        lib.tl_e0m4_tuning_set("register_max_m", 16)
        assert lib.tl_e0m4_matmul_kernel(12, 4096, 4096) == lib.TL_KERNEL_REGISTER
        lib.tl_e0m4_tuning_set("register_max_m", -1)
        assert lib.tl_e0m4_matmul_kernel(12, 4096, 4096) == lib.TL_KERNEL_TENSOR
        base = lib.tl_e0m4_matmul_workspace(200, 2048, 512)
        lib.tl_e0m4_tuning_set("ksplit", 4)
        forced = lib.tl_e0m4_matmul_workspace(200, 2048, 512)
        assert forced > 0 and forced >= base
    finally:
        lib.tl_e0m4_tuning_set(None)
    assert lib.tl_e0m4_matmul_workspace(200, 2048, 512) == base


def test_argument_errors_come_back_before_any_launch(lib):
    L = lib.lib()
    before = lib.tl_e0m4_launch_count()
    a = 0x10000  # fake, aligned, never dereferenced: the checks below fail first
    assert L.tl_e0m4_quantize(None, 0, 128, 16, 128, a, a, None) == 1
    assert L.tl_e0m4_quantize(a, 7, 128, 16, 128, a, a, None) == 4
    assert L.tl_e0m4_quantize(a, 0, 130, 16, 128, a, a, None) == 2
    assert L.tl_e0m4_quantize(a + 4, 0, 128, 16, 128, a, a, None) == 3
    assert L.tl_e0m4_dequant(a, None, 128, 16, 128, a, None) == 1
    assert L.tl_e0m4_dequant(a, a, 128, 8, 128, a, None) == 2
    assert L.tl_e0m4_dequant(a, a, 128, 16, 128, a + 8, None) == 3
    assert L.tl_e0m4_matmul(a, a, a, None, 1, 128, 16, 128, None, 0, None) == 1
    assert L.tl_e0m4_matmul(a, a, a, a, 0, 128, 16, 128, None, 0, None) == 2
    assert L.tl_e0m4_matmul(a, a, a, a, 1, 128, 16, 48, None, 0, None) == 2
    assert L.tl_e0m4_matmul(a, a + 2, a, a, 1, 128, 16, 128, None, 0, None) == 3
    assert L.tl_e0m4_matmul_host(a, a, a, a, 1, 128, 16, 128, a, 16, None) == 5
    import ctypes
    prob = lib.Problem(a, a, a, a, 128, 16)
    pp = ctypes.cast(ctypes.pointer(prob), ctypes.c_void_p)
    assert L.tl_e0m4_matmul_batch(None, 1, 1, 128, a, 1 << 30, None) == 1
    assert L.tl_e0m4_matmul_batch(pp, 0, 1, 128, a, 1 << 30, None) == 2
    assert L.tl_e0m4_matmul_batch(pp, 1, 129, 128, a, 1 << 30, None) == 2
    assert L.tl_e0m4_matmul_batch(pp, 1, 1, 128, a, 16, None) == 5
    bad = lib.Problem(a, a + 4, a, a, 128, 16)
    assert L.tl_e0m4_matmul_batch(ctypes.cast(ctypes.pointer(bad), ctypes.c_void_p), 1, 1, 128, a, 1 << 30, None) == 3
    # the list scratch covers both kernels: the GEMV kernel's slots and 148 slots of 128 x 128 fp32 sums
    assert lib.tl_e0m4_matmul_batch_workspace() >= max(lib.tl_e0m4_matmul_workspace(1, 128, 16), 148 * 128 * 128 * 4)
    assert lib.tl_e0m4_launch_count() == before


def test_status_strings(lib):
    assert lib.tl_status_string(0) == "ok"
    assert "align" in lib.tl_status_string(3)
    assert lib.tl_status_string(99) == "unknown status"


def test_host_staging_size(lib):
    need = lib.tl_e0m4_matmul_host_staging(3, 256, 48)
    assert need >= 3 * 256 * 2 + 3 * 48 * 2 and need % 256 == 0


def test_e0m8_sizes_and_argument_errors(lib):
    assert lib.tl_e0m8_packed_sizes(4096, 4096) == (4096 * 4096, 32 * 4096 * 4)
    assert lib.tl_e0m8_packed_sizes(13696, 5120) == (13696 * 5120, 107 * 5120 * 4)
    for K, N, group in [(100, 16, 128), (128, 24, 128), (128, 16, 64), (128, 16, 32), (0, 16, 128)]:
        with pytest.raises(lib.TlError) as err:
            lib.tl_e0m8_packed_sizes(K, N, group)
        assert err.value.status == 2  # TL_ERR_SHAPE: groups of 128 only
    L = lib.lib()
    before = lib.tl_e0m4_launch_count()
    a = 0x10000  # fake, aligned, never dereferenced: the checks below fail first
    assert L.tl_e0m8_quantize(None, 0, 128, 16, 128, a, a, None) == 1
    assert L.tl_e0m8_quantize(a, 7, 128, 16, 128, a, a, None) == 4
    assert L.tl_e0m8_quantize(a, 0, 128, 16, 64, a, a, None) == 2
    assert L.tl_e0m8_quantize(a, 0, 128, 16, 128, a + 4, a, None) == 3
    assert L.tl_e0m8_dequant(a, a, 128, 16, 128, None, None) == 1
    assert L.tl_e0m8_dequant(a, a, 130, 16, 128, a, None) == 2
    assert L.tl_e0m8_matmul(a, a, a, None, 1, 128, 16, 128, None, 0, None) == 1
    assert L.tl_e0m8_matmul(a, a, a, a, 0, 128, 16, 128, None, 0, None) == 2
    assert L.tl_e0m8_matmul(a, a, a, a, 1, 128, 16, 32, None, 0, None) == 2
    assert L.tl_e0m8_matmul(a, a, a + 8, a, 1, 128, 16, 128, None, 0, None) == 3
    assert L.tl_e0m8_matmul_add(a, a, a, None, a, 1, 128, 16, 128, None, 0, None) == 1
    assert L.tl_e0m8_matmul_bias(a, a, a, a + 2, a, 1, 128, 16, 128, None, 0, None) == 3
    assert L.tl_e0m8_matmul_swiglu(a, a, a, a, 1 << 21, 128, 16, 128, None, 0, None) == 2
    prob = lib.Problem(a, a, a, a, 128, 16)
    arr = (lib.Problem * 1)(prob)
    ptr = ctypes.cast(arr, ctypes.c_void_p)
    assert L.tl_e0m8_matmul_batch(None, 1, 1, 128, a, 1 << 30, None) == 1
    assert L.tl_e0m8_matmul_batch(ptr, 0, 1, 128, a, 1 << 30, None) == 2
    assert L.tl_e0m8_matmul_batch(ptr, 1, 129, 128, a, 1 << 30, None) == 2
    assert L.tl_e0m8_matmul_batch(ptr, 1, 1, 64, a, 1 << 30, None) == 2
    assert L.tl_e0m8_matmul_batch(ptr, 1, 1, 128, None, 1 << 30, None) == 1
    assert L.tl_e0m8_matmul_batch(ptr, 1, 1, 128, a, 16, None) == 5  # TL_ERR_WORKSPACE
    assert lib.tl_e0m4_launch_count() == before
    assert lib.tl_e0m8_matmul_workspace(1, 100, 16) == 0


def test_chain_argument_errors_come_back_before_any_launch(lib):
    L = lib.lib()
    a = 0x10000
    st = lib.Step(a, a, a, a, None, 128, 16, 0, 0, 0, 0.0)
    ptr = lambda s: ctypes.cast(ctypes.pointer(s), ctypes.c_void_p)
    big = 1 << 30
    before = lib.tl_e0m4_launch_count()
    assert L.tl_e0m4_matmul_chain(None, 1, 1, 128, a, big, None) == 1
    assert L.tl_e0m4_matmul_chain(ptr(st), 0, 1, 128, a, big, None) == 2
    assert L.tl_e0m4_matmul_chain(ptr(st), 1, 9, 128, a, big, None) == 2       # more than 8 tokens
    assert L.tl_e0m4_matmul_chain(ptr(st), 1, 1, 128, a, 16, None) == 5        # workspace too small
    assert L.tl_e0m4_matmul_chain(ptr(lib.Step(a, a, a, a, None, 128, 16, 1, 0, 0, 0.0)), 1, 1, 128, a, big, None) == 1
    assert L.tl_e0m4_matmul_chain(ptr(lib.Step(a, a, a, a, a + 2, 128, 16, 2, 0, 0, 0.0)), 1, 1, 128, a, big, None) == 3
    assert L.tl_e0m4_matmul_chain(ptr(lib.Step(a, a, a, a, None, 128, 16, 7, 0, 0, 0.0)), 1, 1, 128, a, big, None) == 2
    assert L.tl_e0m4_matmul_chain(ptr(lib.Step(a, a, a, a, None, 100, 16, 0, 0, 0, 0.0)), 1, 1, 128, a, big, None) == 2
    assert L.tl_e0m4_matmul_chain(ptr(lib.Step(a, a, a, a, None, 128, 16, 0, 0, 1, -1.0)), 1, 1, 128, a, big, None) == 2
    assert lib.tl_e0m4_launch_count() == before
