"""CPU-side checks of the C-ABI library: it builds, loads, exports what include/sg.h
declares, and rejects bad arguments before touching the GPU."""
import ctypes
import os
import re

import pytest

from paper_2202_03293_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "sg.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sg_[a-z0-9_]+)\s*\(", text)))


def test_header_and_binding_agree(lib):
    syms = declared_symbols()
    assert "sg_matmul" in syms and "sg_conv1d_nwc_wcf" in syms and "sg_conv2d_nhwc_hwcf" in syms
    for s in syms:
        assert hasattr(lib, s), f"libsg.so does not export {s}"
    assert sorted(binding.EXPORTS) == syms


def test_version_and_status_strings(lib):
    assert binding.sg_version() >= 100
    seen = {binding.status_string(c) for c in range(7)}
    assert len(seen) == 7 and "ok" in seen
    assert "unknown" in binding.status_string(99)


def test_argument_validation_needs_no_gpu(lib):
    null = ctypes.c_void_p(0)
    fake = ctypes.c_void_p(4096)      # never dereferenced: every call below returns before any launch
    i3 = (ctypes.c_int64 * 3)(1, 1, 1)
    i4 = (ctypes.c_int64 * 4)(1, 1, 1, 1)
    mm = lib.sg_matmul
    assert mm(-1, 4, 4, fake, 4, 1, fake, 4, 1, fake, 4, 1, 0, 0, null) == 1           # negative size
    assert mm(4, 4, 4, fake, 4, 1, fake, 4, 1, fake, 4, 1, 7, 0, null) == 2            # unknown dtype
    assert mm(4, 4, 4, fake, 4, 1, fake, 4, 1, fake, 4, 1, 0, 5, null) == 2            # unknown mode
    assert mm(4, 4, 4, null, 4, 1, fake, 4, 1, fake, 4, 1, 0, 0, null) == 1            # null input
    assert mm(4, 4, 4, fake, 4, 1, fake, 4, 1, null, 4, 1, 0, 0, null) == 1            # null output
    assert mm(4, 4, 4, ctypes.c_void_p(4098), 4, 1, fake, 4, 1, fake, 4, 1, 0, 0, null) == 3   # misaligned f32
    assert mm(4, 4, 4, fake, -4, 1, fake, 4, 1, fake, 4, 1, 0, 0, null) == 1           # negative stride
    assert mm(0, 4, 4, null, 4, 1, null, 4, 1, null, 4, 1, 0, 0, null) == 0            # empty output: no-op
    assert mm(4, 0, 4, fake, 4, 1, fake, 4, 1, fake, 4, 1, 1, 1, null) == 0
    assert mm(2 ** 31, 4, 4, fake, 4, 1, fake, 4, 1, fake, 4, 1, 0, 0, null) == 2      # beyond int32 extents
    assert mm(4, 4, 0, null, 4, 1, null, 4, 1, fake, 4, 1, 0, 1, null) == 0            # K = 0, accumulate: no-op

    c1 = lib.sg_conv1d_nwc_wcf
    assert c1(1, 8, 4, 3, 4, 9, 1, 1, fake, i3, fake, i3, fake, i3, 0, 0, null) == 1   # W_in too small (needs 10)
    assert c1(1, 8, 4, 3, 4, 10, 0, 1, fake, i3, fake, i3, fake, i3, 0, 0, null) == 1  # stride 0
    assert c1(1, 8, 4, 3, 4, 10, 1, 1, fake, None, fake, i3, fake, i3, 0, 0, null) == 1  # null stride array
    assert c1(0, 8, 4, 3, 4, 10, 1, 1, null, i3, null, i3, null, i3, 0, 0, null) == 0
    c2 = lib.sg_conv2d_nhwc_hwcf
    assert c2(1, 4, 4, 2, 3, 3, 2, 5, 6, 1, 1, 1, 1, fake, i4, fake, i4, fake, i4, 1, 0, null) == 1  # H_in too small
    assert c2(1, 4, 4, 2, 3, 3, 2, 6, 6, 1, 1, 1, 0, fake, i4, fake, i4, fake, i4, 1, 0, null) == 1  # dilation 0
    assert c2(1, 4, 0, 2, 3, 3, 2, 6, 6, 1, 1, 1, 1, null, i4, null, i4, null, i4, 1, 0, null) == 0
    assert lib.sg_set_kernel_override(9) == 1
    assert lib.sg_set_kernel_override(0) == 0
    # an output stride of 0 along a dimension with more than one element: the elements would coincide
    assert mm(4, 4, 4, fake, 4, 1, fake, 4, 1, fake, 0, 1, 0, 0, null) == 1
    assert mm(4, 4, 4, fake, 4, 1, fake, 4, 1, fake, 4, 0, 0, 0, null) == 1
    o3 = (ctypes.c_int64 * 3)(1, 0, 1)
    assert c1(1, 8, 4, 3, 4, 10, 1, 1, fake, i3, fake, i3, fake, o3, 0, 0, null) == 1
    o4 = (ctypes.c_int64 * 4)(1, 1, 1, 0)
    assert c2(1, 4, 4, 2, 3, 3, 2, 6, 6, 1, 1, 1, 1, fake, i4, fake, i4, fake, o4, 1, 0, null) == 1
    assert lib.sg_copy2d(4, 4, fake, 4, 1, fake, 0, 1, 0, null) == 1
    assert lib.sg_transpose2d(4, 4, fake, 4, 1, fake, 4, 0, 0, null) == 1
    assert lib.sg_colred2d(4, 4, fake, 4, 1, fake, 0, 0, 0, null) == 1
    assert lib.sg_rowred2d(4, 1, fake, 4, 1, fake, 0, 0, 0, null) == 1
    # the time-out self-test takes a bounded budget only
    assert lib.sg_selftest_wait_timeout(0, null) == 1
    assert lib.sg_selftest_wait_timeout(10 ** 9, null) == 1
    # null result pointers are ignored
    lib.sg_last_stream_k(None)
    lib.sg_last_tile_choice(None)
    assert binding.sg_last_kernel_name() == ""


def test_oracle_header_and_library_agree():
    """oracle/sg_ref.h declares the reference counterparts of the entry points; libsgref.so exports each of them."""
    from oracle import ref
    text = open(os.path.join(ROOT, "oracle", "sg_ref.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    syms = sorted(set(re.findall(r"\b(sg_ref_[a-z0-9_]+)\s*\(", text)))
    assert {"sg_ref_matmul", "sg_ref_conv1d_nwc_wcf", "sg_ref_conv2d_nhwc_hwcf"} <= set(syms)
    L = ref.lib()
    for s in syms:
        assert hasattr(L, s), f"libsgref.so does not export {s}"
    # and the product's header does not mention the oracle
    assert "sg_ref" not in open(os.path.join(ROOT, "include", "sg.h")).read()


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "libsg.so"))
    with pytest.raises(RuntimeError, match="no non-CUDA fallback"):
        binding.lib()
