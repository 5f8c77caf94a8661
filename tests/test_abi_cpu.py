"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares, its host
helpers agree with the documented layouts, and argument errors are returned without touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2602_17681_b200 import build
    build.build_library()
    from paper_2602_17681_b200 import binding
    return binding


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "latmix.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(latmix_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(B):
    names = declared_symbols()
    assert {"latmix_fold_weights", "latmix_quantize_mx", "latmix_linear", "latmix_mx_gemm"} <= set(names)
    lib = ctypes.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert set(B.EXPORTS) == set(names)          # the binding covers the header, name for name


def test_sizes_and_scale_offsets(B):
    assert B.mx_sizes(4096, 4096, B.MXFP4, B.SF_LINEAR) == (4096 * 2048, 4096 * 128)
    assert B.mx_sizes(4096, 4096, B.MXFP8, B.SF_TCGEN05) == (4096 * 4096, 32 * 32 * 512)
    # padding: 130 rows -> 2 row tiles; 96 elements = 3 blocks -> 8 blocks = 2 k-tiles
    assert B.mx_sizes(130, 96, B.MXINT8, B.SF_TCGEN05) == (130 * 96, 2 * 2 * 512)
    assert B.mx_sizes(130, 96, B.MXINT4, B.SF_TCGEN05) == (130 * 96, 2 * 2 * 512)     # one E4M3 byte per element
    # NVFP4: blocks of 16 (tiles of 128 rows x 4 blocks, blocks padded to 16), plus the 16-byte tensor-scale trailer
    assert B.mx_sizes(4096, 4096, B.NVFP4, B.SF_TCGEN05) == (4096 * 2048, 32 * 64 * 512 + 16)
    assert B.mx_sizes(130, 192, B.NVFP4, B.SF_TCGEN05) == (130 * 96, 2 * 4 * 512 + 16)
    assert B.mx_sizes(3, 64, B.NVFP4, B.SF_LINEAR) == (3 * 32, 16 + 16)
    assert B.tensor_scale_offset(130, 192, B.NVFP4, B.SF_TCGEN05) == 2 * 4 * 512
    assert B.tensor_scale_offset(130, 192, B.MXFP4, B.SF_TCGEN05) == ctypes.c_size_t(-1).value
    assert B.scale_offset_fmt(129, 5, 130, 192, B.NVFP4, B.SF_TCGEN05) == (1 * 4 + 1) * 512 + 1 * 16 + 0 * 4 + 1
    assert B.scale_offset_fmt(129, 5, 130, 192, B.NVFP4, B.SF_LINEAR) == 129 * 12 + 5
    assert B.scale_offset_fmt(0, 12, 130, 192, B.NVFP4, B.SF_LINEAR) == ctypes.c_size_t(-1).value
    assert B.scale_offset_fmt(7, 3, 130, 192, B.MXFP8, B.SF_TCGEN05) == B.scale_offset(7, 3, 130, 192, B.SF_TCGEN05)
    with pytest.raises(B.LatmixError):
        B.mx_sizes(4, 96, B.NVFP4)
    rows, K = 300, 1088
    seen = set()
    cb, sb = B.mx_sizes(rows, K, B.MXFP8, B.SF_TCGEN05)
    for r in range(rows):
        for kb in range(K // 32):
            off = B.scale_offset(r, kb, rows, K, B.SF_TCGEN05)
            tile = (r // 128) * (((K // 32 + 7) // 8) * 2) + kb // 4
            assert off == tile * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + kb % 4
            assert off < sb and off not in seen
            seen.add(off)
            assert B.scale_offset(r, kb, rows, K, B.SF_LINEAR) == r * (K // 32) + kb
    assert B.scale_offset(rows, 0, rows, K, B.SF_TCGEN05) == ctypes.c_size_t(-1).value
    assert B.scale_offset(0, K // 32, rows, K, B.SF_LINEAR) == ctypes.c_size_t(-1).value


def test_shape_and_argument_errors_need_no_device(B):
    with pytest.raises(B.LatmixError) as e:
        B.mx_sizes(4, 100, B.MXFP8)
    assert e.value.code == B.ERR_SHAPE
    with pytest.raises(B.LatmixError) as e:
        B.mx_sizes(4, 96, B.MXFP4)                 # FP4 packs two codes per byte and needs K % 64 == 0
    assert e.value.code == B.ERR_SHAPE
    with pytest.raises(B.LatmixError) as e:
        B.mx_sizes(4, 128, 7)
    assert e.value.code == B.ERR_INVALID_ARG
    lib = B._lib
    # null pointers / misaligned pointers / too small workspace are refused before any CUDA call
    assert lib.latmix_quantize_mx(None, B.BF16, None, None, 4, 128, B.MXFP4, B.SF_LINEAR, 16, 16, None, 16, 256, 0, None) == B.ERR_INVALID_ARG
    assert lib.latmix_quantize_mx(None, B.BF16, None, None, 0, 128, B.MXFP4, B.SF_LINEAR, None, None, None, None, 0, 0, None) == B.OK   # empty input
    assert lib.latmix_quantize_mx(24, B.BF16, None, None, 4, 128, B.MXFP4, B.SF_LINEAR, 16, 32, None, 64, 256, 0, None) == B.ERR_INVALID_ARG
    assert lib.latmix_quantize_mx(32, B.BF16, None, None, 4, 100, B.MXFP4, B.SF_LINEAR, 16, 32, None, 64, 256, 0, None) == B.ERR_SHAPE
    assert lib.latmix_quantize_mx(32, B.BF16, None, None, 4, 128, B.MXFP4, B.SF_LINEAR, 16, 32, None, 64, 8, 0, None) == B.ERR_WORKSPACE
    assert lib.latmix_linear(32, B.BF16, 32, None, 32, 32, None, 128, 256, 256, B.MXFP4, 32, 256, 64, 256, 0, None) == B.ERR_WORKSPACE
    assert lib.latmix_mx_gemm(32, 32, 32, 32, None, 128, 256, 256, B.MXFP4, 32, 100, 64, 256, 0, None) == B.ERR_SHAPE
    assert lib.latmix_fold_weights(32, None, 32, B.BF16, None, 256, 64, B.MXFP4, B.SF_TCGEN05, 32, 32, 32, None, 64, 256, 0, None) == B.ERR_WORKSPACE
    # two-sided fold: nothing to fold; a shift without its matrix; workspace without the N x K intermediate
    two = lib.latmix_fold_weights_two_sided
    assert two(None, None, 32, B.BF16, None, None, None, 256, 64, B.MXFP4, B.SF_TCGEN05, 32, 32, 32, None, 64, 1 << 30, 0, None) == B.ERR_INVALID_ARG
    assert two(None, 32, 32, B.BF16, None, 32, None, 256, 64, B.MXFP4, B.SF_TCGEN05, 32, 32, 32, None, 64, 1 << 30, 0, None) == B.ERR_INVALID_ARG
    assert two(32, None, 32, B.BF16, None, None, 32, 256, 64, B.MXFP4, B.SF_TCGEN05, 32, 32, 32, None, 64, 1 << 30, 0, None) == B.ERR_INVALID_ARG
    assert two(32, None, 32, B.F32, None, 32, None, 256, 64, B.MXFP4, B.SF_TCGEN05, 32, 32, 32, None, 64, 256 + 2048 + 256, 0, None) == B.ERR_WORKSPACE
    assert two(32, None, 32, B.BF16, None, 32, None, 250, 64, B.MXFP4, B.SF_TCGEN05, 32, 32, 32, None, 64, 1 << 30, 0, None) == B.ERR_SHAPE
    # transformation MSE: a transform comes with its inverse; results must be given; workspace
    mse = lib.latmix_transformation_mse
    assert mse(32, B.BF16, 32, None, None, 64, 256, B.MXFP4, 32, 32, 64, 1 << 30, 0, None) == B.ERR_INVALID_ARG
    assert mse(32, B.BF16, None, None, None, 64, 256, B.MXFP4, None, 32, 64, 1 << 30, 0, None) == B.ERR_INVALID_ARG
    assert mse(32, B.BF16, None, None, None, 64, 256, B.MXFP4, 32, 32, 64, 4096, 0, None) == B.ERR_WORKSPACE
    assert mse(32, B.BF16, None, None, None, 0, 256, B.MXFP4, 32, 32, 64, 4096, 0, None) in (B.OK, B.ERR_CUDA, B.ERR_UNSUPPORTED)   # empty: device check only
    for code in range(8):
        assert B.status_string(code) != "unknown status"
    assert B.workspace_bytes(B.OP_LINEAR, 4096, 4096, 14336, B.MXFP4) == 256 + 4096 * 2048 + 32 * 32 * 512
    assert B.workspace_bytes(B.OP_FOLD_WEIGHTS, 0, 4096, 14336, B.MXFP4) == 256 + 4096 * 8 + 3 * 4096 * 4096 * 2
    K, N = 4096, 4096
    assert B.workspace_bytes(B.OP_FOLD_TWO_SIDED, 0, K, N, B.MXFP4) == 256 + K * 8 + N * 4 + 12 * K * N + 6 * N * N + 6 * K * K
    M = 2048
    assert B.workspace_bytes(B.OP_TRANSFORMATION_MSE, M, K, 0, B.MXFP4) == 256 + M * K // 2 + M * K // 32 + 2 * 4 * M * K + 6 * M * K + 6 * K * K


def test_no_device_means_loud_failure(B):
    """Without a CUDA device the compute calls must fail, never fall back to a CPU path."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    buf = (ctypes.c_uint8 * 4096)()
    p = ctypes.addressof(buf)
    p = (p + 255) // 256 * 256
    rc = B._lib.latmix_quantize_mx(p, B.BF16, None, None, 1, 64, B.MXFP4, B.SF_LINEAR, p + 512, p + 1024, None, p + 2048, 256, 0, None)
    assert rc in (B.ERR_CUDA, B.ERR_UNSUPPORTED)


def test_product_package_does_not_import_the_oracle():
    """No file of the product package imports, includes or executes anything under oracle/."""
    pkg = os.path.join(ROOT, "paper_2602_17681_b200")
    pat = re.compile(r"^\s*(from\s+\S*oracle|import\s+\S*oracle|#include\s+.*oracle)|oracle/|latmix_oracle", re.M)
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not pat.search(text), f
