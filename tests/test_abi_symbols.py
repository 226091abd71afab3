"""The C-ABI library builds, loads and exports every entry point that include/edgelora.h declares.

No compute call is made here; on a machine without a GPU the calls that need one must fail with an
error code rather than fall back to anything.
"""
import ctypes
import os
import re
import shutil

import pytest

from paper_2507_01438_b200 import binding as B
from paper_2507_01438_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "edgelora.h")


@pytest.fixture(scope="module")
def lib():
    if shutil.which("nvcc") or os.path.exists(libbuild.NVCC):
        libbuild.build()
    assert os.path.exists(B.LIB_PATH), "libedgelora.so missing and nvcc not available"
    return B.lib()


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(edgelora_[a-z0-9_]+)\s*\(", text)))


def test_header_and_binding_agree(lib):
    names = declared_symbols()
    assert "edgelora_pool_create" in names and "edgelora_lora_linear" in names
    assert "edgelora_pool_load_slot" in names and "edgelora_pool_destroy" in names
    assert sorted(B.EXPORTS) == names
    for n in names:
        assert hasattr(B, n) or n == "edgelora_strerror"       # same names above the boundary


def test_every_declared_symbol_is_exported(lib):
    for n in declared_symbols():
        getattr(lib, n)                                          # raises AttributeError if missing


def test_checked_build_exports_the_same_symbols():
    # the checked variant (-DEDGELORA_CHECKED) is the same sources and must offer the same boundary
    if not (shutil.which("nvcc") or os.path.exists(libbuild.NVCC)):
        pytest.skip("no nvcc to build the checked variant with")
    path = libbuild.build(checked=True)
    checked = ctypes.CDLL(path)
    for n in declared_symbols():
        getattr(checked, n)
    assert checked.edgelora_build_is_checked() == 1


def test_host_only_calls(lib):
    assert B.strerror(0) == "ok" and "rank" in B.strerror(B.ERR_RANK_TOO_LARGE)
    # 2 * R_pad * (h_in + h_out) bytes per slot, ranks padded to 16 / 32 / 64
    assert B.edgelora_pool_bytes_required(4096, 4096, 32, 16) == 32 * 2 * 16 * 8192
    assert B.edgelora_pool_bytes_required(14336, 4096, 1000, 64) == 1000 * 2 * 64 * 18432
    assert B.edgelora_pool_bytes_required(256, 256, 4, 8) == 4 * 2 * 16 * 512
    for bad in [(4097, 4096, 1, 8), (4096, 4, 1, 8), (64, 64, 0, 8), (64, 64, 1, 0), (64, 64, 70000, 8)]:
        with pytest.raises(B.EdgeLoraError) as e:
            B.edgelora_pool_bytes_required(*bad)
        assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.EdgeLoraError) as e:
        B.edgelora_pool_bytes_required(64, 64, 1, 65)
    assert e.value.code == B.ERR_RANK_TOO_LARGE
    assert lib.edgelora_pool_destroy(None) == B.ERR_INVALID_ARG
    assert lib.edgelora_pool_load_slot(None, 0, 1, ctypes.c_float(1.0), None, None) == B.ERR_INVALID_ARG


def test_no_cpu_fallback_without_a_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(B.EdgeLoraError) as e:
        B.edgelora_pool_create(256, 256, 4, 8)
    assert e.value.code == B.ERR_CUDA
