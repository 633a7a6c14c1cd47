"""The C-ABI library builds, loads without a GPU, exports every symbol the header declares and
rejects bad arguments on the host (no compute call is made here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "snip.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2602_01410_b200 import build
    return ctypes.CDLL(build.build())


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(snip_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 13
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_entry_points():
    src = open(os.path.join(ROOT, "paper_2602_01410_b200", "api.py")).read()
    for n in declared_symbols():
        assert f'"{n}"' in src, n


def test_version_and_status_strings(lib):
    assert lib.snip_version() >= 100
    lib.snip_status_string.restype = ctypes.c_char_p
    assert lib.snip_status_string(0) == b"SNIP_OK"
    assert lib.snip_status_string(7) == b"SNIP_ERR_TIMEOUT"
    assert lib.snip_status_string(99) == b"SNIP_ERR_UNKNOWN"


def test_quantize_sizes_and_shape_errors(lib):
    sz = ctypes.c_size_t
    i64 = ctypes.c_int64
    lib.snip_quantize_sizes.argtypes = [i64, i64, ctypes.c_int, ctypes.c_int, ctypes.c_uint32] + [ctypes.POINTER(sz)] * 3
    cb, sb, wb = sz(), sz(), sz()
    assert lib.snip_quantize_sizes(256, 320, 1, 0, 0, cb, sb, wb) == 0
    assert cb.value == 256 * 320 and sb.value == 4 * 3 * 256
    assert lib.snip_quantize_sizes(256, 320, 2, 1, 0, cb, sb, wb) == 0
    assert cb.value == 256 * 320 // 2 + 64 and sb.value == 4 * 2 * 320
    assert lib.snip_quantize_sizes(256, 320, 2, 2, 0, cb, sb, wb) == 0
    assert sb.value == 4 * 2 * 3
    assert lib.snip_quantize_sizes(256, 320, 0, 2, 0, cb, sb, wb) == 0 and cb.value == 0 and sb.value == 0
    assert wb.value > 0
    assert lib.snip_quantize_sizes(100, 320, 1, 0, 0, cb, sb, wb) == 2   # SNIP_ERR_SHAPE
    assert lib.snip_quantize_sizes(256, 320, 7, 0, 0, cb, sb, wb) == 1   # SNIP_ERR_ARG


def test_host_side_argument_checks(lib):
    vp, i64, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t
    lib.snip_quantize.argtypes = [vp, i64, i64, i64, ctypes.c_int, ctypes.c_int, ctypes.c_uint32, vp, vp, vp, vp, vp, sz, vp]
    assert lib.snip_quantize(None, 128, 128, 128, 1, 0, 0, None, None, None, None, None, 0, None) == 1
    assert lib.snip_quantize(0x1000, 100, 128, 128, 1, 0, 0, 0x2000, 0x3000, None, None, None, 0, None) == 2
    assert lib.snip_quantize(0x1004, 128, 128, 128, 1, 0, 0, 0x2000, 0x3000, None, None, None, 0, None) == 3
    # statistics need a workspace
    assert lib.snip_quantize(0x1000, 128, 128, 128, 1, 0, 2, 0x2000, 0x3000, 0x4000, None, None, 0, None) == 5
    lib.snip_workspace_size.argtypes = [ctypes.c_int, i64, i64, i64, ctypes.c_int, ctypes.c_int, ctypes.POINTER(sz), ctypes.POINTER(sz)]
    g, l = sz(), sz()
    assert lib.snip_workspace_size(0, 512, 512, 512, 1, 1, g, l) == 0
    assert g.value >= 4 and l.value >= 2 * 512 * 512
    assert lib.snip_workspace_size(3, 512, 512, 512, 1, 1, g, l) == 1
    lin = [vp, vp, vp, i64, i64, i64, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, vp, vp, sz, vp]
    lib.snip_linear_fwd.argtypes = lin
    # mixing BF16 with a quantized operand is rejected; too small a workspace is rejected
    assert lib.snip_linear_fwd(0x1000, 0x2000, 0x3000, 128, 128, 128, 0, 1, 0, None, None, 0x4000, 1 << 30, None) == 4
    assert lib.snip_linear_fwd(0x1000, 0x2000, 0x3000, 128, 128, 128, 1, 1, 0, None, None, 0x4000, 16, None) == 5


def test_host_side_checks_of_the_added_options(lib):
    vp, i64, sz, i32, u32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint32
    psz = ctypes.POINTER(sz)
    # sizes of the 32-long tile kinds (a scale per 1x32 / 32x1 tile) and of the two-level form (two 512-byte atoms per 128x128 tile)
    lib.snip_quantize_sizes.argtypes = [i64, i64, i32, i32, u32, psz, psz, psz]
    cb, sb, wb = sz(), sz(), sz()
    assert lib.snip_quantize_sizes(256, 320, 1, 3, 0, cb, sb, wb) == 0 and sb.value == 4 * 10 * 256
    assert lib.snip_quantize_sizes(256, 320, 2, 4, 1, cb, sb, wb) == 0 and sb.value == 4 * 8 * 320
    assert lib.snip_quantize_sizes(256, 320, 1, 5, 0, cb, sb, wb) == 1      # the 16-long kinds have their own entry points
    lib.snip_quantize_nvfp4_sizes.argtypes = [i64, i64, psz, psz]
    assert lib.snip_quantize_nvfp4_sizes(256, 320, cb, sb) == 0
    assert cb.value == 256 * 320 // 2 + 64 and sb.value == 2 * 3 * 1024
    assert lib.snip_quantize_nvfp4_sizes(256, 100, cb, sb) == 2
    # 32-long tiles exist for the power-of-two rule only: the paper-rule entry point refuses them before touching a device
    lib.snip_quantize.argtypes = [vp, i64, i64, i64, i32, i32, u32, vp, vp, vp, vp, vp, sz, vp]
    assert lib.snip_quantize(0x1000, 128, 128, 128, 1, 3, 0, 0x2000, 0x3000, None, None, None, 0, None) == 4
    lib.snip_quantize_mx.argtypes = [vp, i64, i64, i64, i32, i32, u32, vp, vp, vp, vp, vp, sz, vp]
    assert lib.snip_quantize_mx(0x1000, 128, 128, 128, 1, 3, 1, 0x2000, 0x3000, None, None, None, 0, None) == 4   # 1x32 tiles are stored as they are
    assert lib.snip_quantize_mx(0x1000, 128, 128, 128, 1, 4, 0, 0x2000, 0x3000, None, None, None, 0, None) == 4   # 32x1 tiles transposed
    # two-level quantizer: missing bound, misaligned pointers, statistics without a workspace
    lib.snip_quantize_nvfp4_dual.argtypes = [vp, i64, i64, i64, vp, vp, vp, vp, vp, vp, vp, i32, ctypes.c_uint64, vp, sz, vp]
    q = lib.snip_quantize_nvfp4_dual
    assert q(0x1000, 128, 128, 128, None, 0x2000, 0x3000, None, 0x4000, 0x5000, None, 0, 0, None, 0, None) == 1
    assert q(0x1000, 128, 100, 128, 0x100, 0x2000, 0x3000, None, 0x4000, 0x5000, None, 0, 0, None, 0, None) == 2
    assert q(0x1000, 128, 128, 128, 0x102, 0x2000, 0x3000, None, 0x4000, 0x5000, None, 0, 0, None, 0, None) == 3
    assert q(0x1000, 128, 128, 128, 0x100, 0x2000, 0x3000, 0x6000, 0x4000, 0x5000, 0x6020, 0, 0, None, 0, None) == 5
    assert q(0x1000, 128, 128, 128, 0x100, 0x2000, 0x3000, None, 0x4000, 0x5000, None, 7, 0, None, 0, None) == 1    # unknown rounding mode
    # the composition refuses a workspace that is too small
    lib.snip_linear_fwd_bwd_nvfp4_workspace.argtypes = [i64, i64, i64, psz]
    assert lib.snip_linear_fwd_bwd_nvfp4_workspace(512, 512, 512, wb) == 0 and wb.value > 6 * 512 * 512 // 2
    lib.snip_linear_fwd_bwd_nvfp4.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, vp, i32, ctypes.c_uint64, vp, vp, sz, vp]
    assert lib.snip_linear_fwd_bwd_nvfp4(0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000, 512, 512, 512, 0, 0x100, 0, 0, None, 0x7000, 64, None) == 5
