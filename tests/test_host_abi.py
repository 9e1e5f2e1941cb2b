"""Host logic of the C-ABI library, no GPU needed: it loads, exports what include/division.h declares,
and its size arithmetic agrees with the CPU checker's closed form (Sec. 4.1: cached tuple (H^L, V^H, Delta, delta))."""
import ctypes
import os
import re

import pytest

from oracle import division_oracle as orc
from paper_2208_04187_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built_library():
    build.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "division.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(div_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert set(names) == set(binding.EXPORTED_SYMBOLS)
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in names:
        assert getattr(lib, name) is not None


DESCS = [
    (64, 64, 112, 112, 8, 2, "f32", "f32"), (64, 512, 28, 28, 8, 2, "f32", "f32"), (64, 2048, 7, 7, 8, 2, "f32", "f32"),
    (128, 512, 4, 4, 8, 2, "f32", "f32"), (128, 160, 32, 32, 4, 4, "bf16", "bf16"), (1, 1, 3, 3, 2, 2, "f32", "f32"),
    (3, 5, 7, 9, 4, 1, "f32", "bf16"), (2, 3, 5, 6, 1, 8, "bf16", "f32"), (1, 1, 1, 1, 8, 2, "f32", "f32"),
    (7, 3, 100, 30, 64, 4, "f32", "f32"), (5, 2, 33, 17, 12, 2, "f32", "f32"),
]


@pytest.mark.parametrize("d", DESCS)
def test_compressed_bytes_matches_closed_form(d):
    n, c, h, w, b, q, xd, ld = d
    got = binding.div_compressed_bytes(binding.make_desc(*d))
    ref = orc.compressed_layout(n, c, h, w, b, q, xd, ld)
    for field in ("lfc_off", "lfc_bytes", "packed_off", "packed_bytes", "stats_off", "stats_bytes",
                  "total_bytes", "closed_form_bytes", "raw_bytes"):
        assert getattr(got, field) == getattr(ref, field), field
    assert got.workspace_bytes >= 64 + 32 * n and got.workspace_bytes % 256 == 0


@pytest.mark.parametrize("d", DESCS)
def test_planegroup_bytes_matches_closed_form(d):
    """Per-plane form: the same sections with 4 bytes of (delta, Delta) per plane and no scratch."""
    n, c, h, w, b, q, xd, ld = d
    got = binding.div_planegroup_bytes(binding.make_desc(*d))
    ref = orc.plane_layout(n, c, h, w, b, q, xd, ld)
    for field in ("lfc_off", "lfc_bytes", "packed_off", "packed_bytes", "stats_off", "stats_bytes",
                  "total_bytes", "closed_form_bytes", "raw_bytes"):
        assert getattr(got, field) == getattr(ref, field), field
    assert got.workspace_bytes == 0 and got.stats_bytes == 4 * n * c


def test_planegroup_refuses_too_many_planes_and_bad_flags():
    L = binding.lib()
    out = binding.DivLayout()
    assert L.div_planegroup_bytes(ctypes.byref(binding.make_desc(2 ** 30, 2, 1, 1, 8, 2)), ctypes.byref(out)) == binding.DIV_ERR_SHAPE
    assert L.div_planegroup_bytes(ctypes.byref(binding.make_desc(2 ** 30 - 1, 2, 1, 1, 8, 2)), ctypes.byref(out)) == binding.DIV_OK
    assert L.div_planegroup_bytes(None, ctypes.byref(out)) == binding.DIV_ERR_NULL
    d = binding.make_desc(2, 3, 8, 8, 8, 2)
    assert L.div_planegroup_compress(ctypes.byref(d), None, None, 0, 0, None, 0) == binding.DIV_ERR_NULL
    assert L.div_planegroup_compress(ctypes.byref(d), 16, 32, 0, 0, None, 4) == binding.DIV_ERR_PARAM
    assert L.div_planegroup_compress(ctypes.byref(d), 16, 36, 1 << 20, 0, None, 0) == binding.DIV_ERR_ALIGN
    assert L.div_planegroup_compress(ctypes.byref(d), 16, 32, 8, 0, None, 0) == binding.DIV_ERR_CAPACITY
    assert L.div_planegroup_decompress(ctypes.byref(d), 16, 8, 32, None) == binding.DIV_ERR_CAPACITY
    assert L.div_planegroup_decompress(ctypes.byref(d), 16, 1 << 20, 34, None) == binding.DIV_ERR_ALIGN


@pytest.mark.parametrize("d", [(2, 3, 8, 8, 8, 4, 2, "f32", "f32"), (3, 5, 8, 16, 24, 8, 2, "f32", "bf16"),
                               (1, 2, 5, 9, 7, 4, 4, "bf16", "bf16"), (2, 2, 3, 3, 3, 8, 8, "f32", "f32"),
                               (4, 7, 1, 14, 14, 8, 1, "f32", "f32")])
def test_3d_bytes_match_the_closed_form(d):
    m, c, dd, h, w, b, q, xd, ld = d
    got = binding.div_compressed_bytes_3d(binding.make_desc_3d(*d))
    ref = orc.layout_3d(m, c, dd, h, w, b, q, xd, ld)
    for field in ("lfc_off", "lfc_bytes", "packed_off", "packed_bytes", "stats_off", "stats_bytes",
                  "total_bytes", "closed_form_bytes", "raw_bytes"):
        assert getattr(got, field) == getattr(ref, field), field


def test_mask_bytes_and_host_checks():
    L = binding.lib()
    for total in (1, 31, 32, 33, 49, 12544, 64 * 64 * 112 * 112):
        assert binding.div_mask_bytes(total) == orc.mask_bytes(total)
    out = ctypes.c_uint64(0)
    assert L.div_mask_bytes(0, ctypes.byref(out)) == binding.DIV_ERR_SHAPE
    assert L.div_mask_bytes((1 << 40) + 1, ctypes.byref(out)) == binding.DIV_ERR_SHAPE
    assert L.div_mask_bytes(5, None) == binding.DIV_ERR_NULL
    assert L.div_relu_forward(None, 16, 32, 64, 8, 0, None) == binding.DIV_ERR_NULL
    assert L.div_relu_forward(16, 16, 32, 64, 8, 7, None) == binding.DIV_ERR_PARAM
    assert L.div_relu_forward(16, 18, 32, 64, 8, 0, None) == binding.DIV_ERR_ALIGN
    assert L.div_relu_forward(16, 16, 32, 3, 8, 0, None) == binding.DIV_ERR_CAPACITY
    assert L.div_dropout_forward(16, 16, 32, 64, 8, 0, 1, 65537, None) == binding.DIV_ERR_PARAM
    assert L.div_mask_backward(32, 3, 16, 16, 8, 0, None) == binding.DIV_ERR_CAPACITY
    assert L.div_mask_backward(32, 64, 16, 16, 0, 0, None) == binding.DIV_ERR_SHAPE


def test_bad_descriptors_are_refused_on_the_host():
    L = binding.lib()
    out = binding.DivLayout()

    def status(*d):
        return L.div_compressed_bytes(ctypes.byref(binding.make_desc(*d)), ctypes.byref(out))

    assert status(1, 1, 8, 8, 8, 2) == binding.DIV_OK
    assert status(0, 1, 8, 8, 8, 2) == binding.DIV_ERR_SHAPE
    assert status(1, 1, 0, 8, 8, 2) == binding.DIV_ERR_SHAPE
    assert status(1, 1, -3, 8, 8, 2) == binding.DIV_ERR_SHAPE
    assert status(1, 1 << 12, 1 << 10, 1 << 10, 8, 2) == binding.DIV_ERR_SHAPE      # c*h*w = 2^32
    assert status(1, (1 << 12) - 1, 1 << 10, 1 << 10, 8, 2) == binding.DIV_OK
    assert status(1 << 31, 1, 8, 8, 8, 2) == binding.DIV_ERR_SHAPE
    assert status(1, 1, 8, 8, 0, 2) == binding.DIV_ERR_PARAM
    for q in (0, 3, 5, 16, 32):
        assert status(1, 1, 8, 8, 8, q) == binding.DIV_ERR_PARAM
    bad = binding.make_desc(1, 1, 8, 8, 8, 2)
    bad.x_dtype = 7
    assert L.div_compressed_bytes(ctypes.byref(bad), ctypes.byref(out)) == binding.DIV_ERR_PARAM
    assert L.div_compressed_bytes(None, ctypes.byref(out)) == binding.DIV_ERR_NULL
    assert L.div_compressed_bytes(ctypes.byref(bad), None) == binding.DIV_ERR_NULL
    with pytest.raises(binding.DivisionError):
        binding.div_compressed_bytes(binding.make_desc(1, 1, 8, 8, 8, 3))


def test_null_and_misaligned_pointers_are_refused_before_any_launch():
    L = binding.lib()
    d = binding.make_desc(2, 3, 8, 8, 8, 2)
    lo = binding.div_compressed_bytes(d)
    ws = int(lo.workspace_bytes)
    cap = int(lo.total_bytes)
    assert L.div_compress(ctypes.byref(d), None, 256, cap, 512, ws, 0, None) == binding.DIV_ERR_NULL
    assert L.div_compress(ctypes.byref(d), 256, 512, cap, None, ws, 0, None) == binding.DIV_ERR_NULL
    assert L.div_compress(ctypes.byref(d), 260, 512, cap, 1024, ws, 0, None) == binding.DIV_ERR_ALIGN
    assert L.div_compress(ctypes.byref(d), 256, 512, cap - 1, 1024, ws, 0, None) == binding.DIV_ERR_CAPACITY
    assert L.div_compress(ctypes.byref(d), 256, 512, cap, 1024, ws - 1, 0, None) == binding.DIV_ERR_CAPACITY
    assert L.div_compress_ex(ctypes.byref(d), 256, 512, cap, 1024, ws, 0, None, 0x80) == binding.DIV_ERR_PARAM
    assert L.div_decompress(ctypes.byref(d), None, cap, 512, None) == binding.DIV_ERR_NULL
    assert L.div_decompress(ctypes.byref(d), 256, cap, 520, None) == binding.DIV_ERR_ALIGN
    assert L.div_decompress(ctypes.byref(d), 256, cap - 1, 512, None) == binding.DIV_ERR_CAPACITY


def test_status_strings():
    for code in range(8):
        assert binding.status_string(code)
    assert binding.status_string(0) == "ok"
