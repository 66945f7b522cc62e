"""CPU-side checks of the C ABI: the library builds, exports every declared symbol, and rejects bad arguments
on the host before any launch."""
import ctypes as C
import os
import re

import pytest

from paper_2407_09453_b200 import bsp, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return bsp.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "bsp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bsp_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert set(bsp.EXPORTS) <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings(lib):
    assert bsp.status_string(bsp.OK) == "ok"
    assert "8x8" in bsp.status_string(bsp.ERR_BLOCK)


def test_host_validation_without_gpu(lib):
    good = bsp.wdesc(64, 64, 3, 3, 8, 8, bsp.BF16)
    assert bsp.bsp_mask_workspace_bytes(good) >= 256 + 64 * 8
    assert bsp.bsp_packed_bytes(good, 32) > 32 * 8 * 8 * 9 * 2
    one = C.c_void_p(256)      # a non-null dummy address: every call below must fail before touching it
    def mask(wd, n_zero=1, norm=0, scope=0, W=one, g=one, ws=one):
        return lib.bsp_mask(C.byref(wd), W, norm, scope, C.c_int64(n_zero), g, None, ws, None)
    assert mask(bsp.wdesc(64, 64, 3, 3, 8, 4, bsp.BF16)) == bsp.ERR_BLOCK
    assert mask(bsp.wdesc(64, 60, 3, 3, 8, 8, bsp.BF16)) == bsp.ERR_SHAPE
    assert mask(bsp.wdesc(64, 3, 7, 7, 8, 8, bsp.BF16)) == bsp.ERR_SHAPE     # a 3-channel first layer
    assert mask(bsp.wdesc(64, 64, 3, 3, 8, 8, bsp.I32)) == bsp.ERR_DTYPE
    assert mask(good, n_zero=65) == bsp.ERR_CAPACITY
    assert mask(good, n_zero=9, scope=1) == bsp.ERR_CAPACITY
    assert mask(good, W=None) == bsp.ERR_NULL
    assert lib.bsp_mask(None, one, 0, 0, C.c_int64(0), one, None, one, None) == bsp.ERR_NULL
    h = bsp.Bcsr(256, 256, 256, 256, 32)
    xd = bsp.XDesc(1, 8, 8, 1, 1, 1, 1)
    def conv(wd, h=h, xd=xd, ytype=bsp.F32, X=one, Y=one):
        return lib.bsp_conv2d(C.byref(wd), C.byref(h), C.byref(xd), X, None, Y, ytype, one, None)
    assert conv(good, ytype=bsp.I32) == bsp.ERR_DTYPE
    assert conv(bsp.wdesc(64, 64, 3, 3, 8, 8, bsp.I8), ytype=bsp.F32) == bsp.ERR_DTYPE
    assert conv(good, xd=bsp.XDesc(1, 1, 1, 1, 1, 0, 0)) == bsp.ERR_SHAPE    # kernel larger than padded input
    assert conv(good, xd=bsp.XDesc(1, 8, 8, 0, 1, 1, 1)) == bsp.ERR_SHAPE
    assert conv(good, h=bsp.Bcsr(256, 256, 256, 0, 32)) == bsp.ERR_NULL
    assert conv(good, h=bsp.Bcsr(256, 256, 256, 256, 65)) == bsp.ERR_INDEX
    assert conv(good, X=C.c_void_p(260)) == bsp.ERR_SHAPE                    # misaligned activations
    assert lib.bsp_gemm(C.byref(good), C.byref(h), one, C.c_int64(4), None, one, bsp.F32, one, None) == bsp.ERR_SHAPE
    assert lib.bsp_compact(C.byref(good), one, one, one, one, None, None, C.c_int64(-1), one, None) == bsp.ERR_CAPACITY
    assert lib.bsp_check(None, None) == bsp.ERR_NULL


def test_product_kernel_name():
    """Every layer the API accepts takes the one product kernel, whatever its type, taps and strides (a host-side
    answer: no GPU needed)."""
    import torch
    for dt in (torch.bfloat16, torch.int8, torch.float32):
        wd = bsp.wdesc(64, 64, 3, 3, 8, 8, dt)
        assert bsp.conv_kernel_name(wd, bsp.XDesc(2, 14, 14, 1, 1, 1, 1)) == "gemm_tc_kernel"
        assert bsp.conv_kernel_name(wd, bsp.XDesc(2, 14, 14, 2, 2, 1, 1)) == "gemm_tc_kernel"
        assert bsp.conv_kernel_name(bsp.wdesc(64, 48, 1, 1, 8, 8, dt), bsp.XDesc(2, 7, 7, 1, 1, 0, 0)) == "gemm_tc_kernel"
    assert bsp.conv_kernel_name(bsp.wdesc(64, 64, 5, 5, 8, 8, torch.bfloat16), bsp.XDesc(2, 20, 20, 3, 3, 2, 2)) == "gemm_tc_kernel"
