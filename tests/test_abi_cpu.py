"""CPU-side checks of the C-ABI: the library loads, exports every declared
symbol, and host validation returns the documented status codes before any
device work."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2603_16590_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared_symbols():
    names = set()
    for header in sorted(os.listdir(os.path.join(ROOT, "include"))):
        assert header.endswith(".h")
        src = open(os.path.join(ROOT, "include", header)).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        names |= set(re.findall(r"\b(batq_[a-z0-9_]+)\s*\(", src))
    return sorted(names)


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = _declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
        assert n in binding.SIGNATURES, n
    assert sorted(binding.SIGNATURES) == names


def test_status_strings_and_version(lib):
    assert lib.batq_version() >= 100
    seen = {lib.batq_status_string(i) for i in range(9)}
    assert len(seen) == 9 and b"ok" in seen


def test_sf_and_weight_sizes(lib):
    assert lib.batq_sf_bytes(128, 1024, binding.SF_ROWMAJOR) == 128 * 32
    assert lib.batq_sf_bytes(128, 1024, binding.SF_MMA) == 1 * 8 * 512          # k=32 -> 8 atoms
    assert lib.batq_sf_bytes(129, 1024, binding.SF_MMA) == 2 * 8 * 512
    assert lib.batq_sf_bytes(1, 96, binding.SF_MMA) == 1 * 2 * 512              # k=3 -> padded to 8 blocks
    assert lib.batq_sf_bytes(5, 100, binding.SF_MMA) == 0                        # n % 32 != 0
    assert lib.batq_sf_bytes(5, 64, 7) == 0
    assert lib.batq_weight_bytes(1024, 1024) == 1024 * 512 + 8 * 8 * 512
    assert lib.batq_weight_bytes(0, 1024) == 0


def test_host_validation_without_a_device(lib):
    h = C.c_void_p()
    f = np.zeros(64 * 4, np.float32)
    p = f.ctypes.data
    assert lib.batq_transform_create(None, 128, 4, 8, p, 0, p, 0, None, None) == 1
    assert lib.batq_transform_create(C.byref(h), 128, 4, 8, None, 0, p, 0, None, None) == 1
    assert lib.batq_transform_create(C.byref(h), 128, 4, 8, p, 0, p, 0, p, None) == 1
    assert lib.batq_transform_create(C.byref(h), 100, 4, 8, p, 0, p, 0, None, None) == 2
    assert lib.batq_transform_create(C.byref(h), 128, 4, 4, p, 0, p, 0, None, None) == 2
    assert lib.batq_transform_create(C.byref(h), 128, 3, 11, p, 0, p, 0, None, None) == 2
    assert lib.batq_transform_create(C.byref(h), 128, 4, 8, p, 5, p, 0, None, None) == 2
    # quantize: shape / alignment / null, checked before any launch
    assert lib.batq_quantize_act(None, 16, 4, 100, 100, 16, 16, 0, None) == 2
    assert lib.batq_quantize_act(None, 16, 4, 128, 64, 16, 16, 0, None) == 2     # ld < n
    assert lib.batq_quantize_act(None, None, 4, 128, 128, 16, 16, 0, None) == 1
    assert lib.batq_quantize_act(None, 8, 4, 128, 128, 16, 16, 0, None) == 3      # x not 16-byte aligned
    assert lib.batq_quantize_act(None, 16, 4, 128, 132, 16, 16, 0, None) == 3     # ld % 8
    assert lib.batq_quantize_act(None, 16, 4, 128, 128, 16, 16, 9, None) == 4     # layout
    assert lib.batq_quantize_act(None, 16, 0, 128, 128, None, None, 0, None) == 0  # s == 0 no-op
    assert lib.batq_quantize_act(None, 16, 4, 128, 128, None, 16, 0, None) == 1
    assert lib.batq_gemm_mxfp4(16, 16, None, 4, 16, 0, 128, None) == 1
    assert lib.batq_linear_w4a4(None, None, 16, 4, 128, 16, 0, 128, 1024, 0, None) == 1
    assert lib.batq_prepare_weight(None, 16, 4, 100, 100, None, None, 1024, C.byref(h), None) == 2
    assert lib.batq_prepare_weight(None, 16, 4, 128, 128, None, None, None, C.byref(h), None) == 1
    assert lib.batq_prepare_weight(None, 16, 4, 128, 128, None, None, 512, C.byref(h), None) == 3
    assert lib.batq_linear_workspace_bytes(None, 4) == 0
    assert lib.batq_linear_kernel_launches(None, None, 4) == 0
    assert lib.batq_weight_destroy(None) == 0 and lib.batq_transform_destroy(None) == 0
    assert lib.batq_gemm_mxfp8_mxfp4(16, 16, None, 4, 16, 0, 128, None) == 1
    assert lib.batq_linear_w4a8(None, None, 16, 4, 128, 16, 0, 128, 1024, 0, None) == 1
    h2 = C.c_void_p()
    assert lib.batq_weight_import(16, 16, 0, 64, 1024, C.byref(h2), None) == 2      # shape before anything else
    assert lib.batq_weight_import(None, 16, 8, 64, 1024, C.byref(h2), None) == 1
    assert lib.batq_weight_import(16, 16, 8, 64, 1000, C.byref(h2), None) == 3      # weight_buf not 1024-byte aligned
    # host entry points: a NULL weight is refused before anything touches a device
    assert lib.batq_linear_w4a4_host(None, None, 16, 4, 16, 0, 16, 16, 1024, 0, None) == 1
    assert lib.batq_linear_w4a4_host_async(None, None, 16, 4, 16, 0, 16, 16, 1024, 0, None) == 1
    assert lib.batq_linear_w4a8_host_async(None, None, 16, 4, 16, 0, 16, 16, 1024, 0, None) == 1
    assert lib.batq_linear_w4a8_workspace_bytes(None, 4) == 0
    assert lib.batq_transform_set_bf16_intermediates(None, 1) == 1
    assert lib.batq_debug_mma_peak(0, 100, 10, 0, None, None) == 2
    assert lib.batq_debug_mma_peak(0, 256, 0, 0, None, None) == 2
    # the loop with a load stream: a weight is needed as soon as something is loaded
    assert lib.batq_debug_mma_peak_with_loads(None, 1, 256, 10, 10, 0, None, None, None) == 2
    assert lib.batq_debug_mma_peak_with_loads(None, 1, 256, 0, 0, 0, None, None, None) == 2
    assert lib.batq_debug_mma_peak_with_loads(None, 1, 100, 10, 0, 0, None, None, None) == 2


def test_debug_hooks_are_not_in_the_public_header():
    src = open(os.path.join(ROOT, "include", "batq.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    assert "batq_debug_" not in src
