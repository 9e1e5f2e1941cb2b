"""Parity of 3-D activation maps (appendix "Compression of 1D and 3D Activation Maps") with the checker's 3-D
functions, through the C ABI: exact equality of the whole blob and of the reconstruction."""
import numpy as np
import pytest
import torch

from oracle import division_oracle as orc
from paper_2208_04187_b200 import binding, build

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built_library():
    build.build()
    binding.lib()


def volume(shape, seed, dtype):
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal(shape) * (1 + rng.random(shape[:2] + (1, 1, 1)))).astype(np.float32)
    return orc.f32_to_bf16_bits(x) if dtype == "bf16" else x


def run(x, block, q, seed, xd, ld):
    m, c, d, h, w = x.shape
    desc = binding.make_desc_3d(m, c, d, h, w, block, q, xd, ld)
    lo = binding.div_compressed_bytes_3d(desc)
    t = torch.from_numpy(x)
    xdev = (t.view(torch.bfloat16) if xd == "bf16" else t).cuda()
    blob = torch.full((int(lo.total_bytes) + 64,), 0x5A, dtype=torch.uint8, device="cuda")   # stale bytes everywhere ...
    blob[int(lo.lfc_bytes):int(lo.packed_off)] = 0                                          # ... but in the padding,
    blob[int(lo.packed_off + lo.packed_bytes):int(lo.stats_off)] = 0                        # which is never written
    ws = torch.empty(int(lo.workspace_bytes), dtype=torch.uint8, device="cuda")
    out = torch.empty_like(xdev)
    s = torch.cuda.current_stream().cuda_stream
    binding.div_compress_3d(desc, xdev.data_ptr(), blob.data_ptr(), int(lo.total_bytes), ws.data_ptr(), ws.numel(), seed, s)
    binding.div_decompress_3d(desc, blob.data_ptr(), int(lo.total_bytes), out.data_ptr(), s)
    torch.cuda.synchronize()
    got = out.view(torch.int16).cpu().numpy().view(np.uint16) if xd == "bf16" else out.cpu().numpy()
    return lo, blob.cpu().numpy(), (orc.bf16_bits_to_f32(got) if xd == "bf16" else got)


CASES = [
    ((2, 3, 8, 8, 8), 4, 2, "f32", "f32"), ((2, 2, 16, 8, 24), 8, 2, "f32", "f32"), ((1, 3, 5, 9, 7), 4, 4, "f32", "bf16"),
    ((2, 2, 3, 3, 3), 8, 8, "bf16", "bf16"), ((3, 2, 6, 10, 4), 3, 1, "f32", "f32"), ((2, 5, 1, 14, 14), 8, 2, "f32", "f32"),
    ((2, 4, 2, 12, 20), 8, 2, "bf16", "f32"), ((1, 1, 1, 1, 1), 8, 2, "f32", "f32"), ((3, 3, 7, 5, 3), 2, 2, "f32", "f32"),
    ((2, 8, 16, 28, 28), 8, 2, "f32", "f32"), ((2, 3, 4, 4, 33), 16, 4, "f32", "f32"),
    ((1, 3, 1, 3, 4), 4, 2, "f32", "f32"), ((2, 5, 6, 10, 24), 12, 4, "bf16", "bf16"), ((2, 4, 9, 8, 16), 16, 8, "f32", "f32"),
    ((3, 2, 5, 7, 12), 4, 1, "f32", "f32"), ((1, 2, 40, 12, 8), 8, 2, "f32", "bf16"),
    # W % 4 == 0 and B in {4, 8}: the strip statistics kernel; ragged depth and height, a last block of 4 columns,
    # warps that straddle volumes and samples
    ((3, 5, 6, 10, 12), 4, 2, "f32", "f32"), ((2, 3, 9, 7, 16), 4, 4, "bf16", "bf16"), ((5, 1, 4, 4, 8), 4, 2, "f32", "f32"),
    ((7, 3, 3, 5, 12), 8, 8, "f32", "bf16"), ((2, 2, 17, 9, 40), 8, 2, "bf16", "f32"),
]


@pytest.mark.parametrize("shape,block,q,xd,ld", CASES)
def test_3d_matches_the_checker(shape, block, q, xd, ld):
    x = volume(shape, 12, xd)
    ref = orc.compress_3d(x, block, q, 77, xd, ld)
    lo, blob, xhat = run(x, block, q, 77, xd, ld)
    for f in ("lfc_off", "lfc_bytes", "packed_off", "packed_bytes", "stats_off", "stats_bytes", "total_bytes",
              "closed_form_bytes", "raw_bytes"):
        assert getattr(lo, f) == getattr(ref.layout, f), f
    np.testing.assert_array_equal(blob[:lo.total_bytes], ref.blob(), err_msg="blob bytes")
    assert (blob[lo.total_bytes:] == 0x5A).all()
    np.testing.assert_array_equal(xhat, orc.decompress_3d(ref), err_msg="reconstruction")


def test_depth_one_equals_the_2d_entry_points():
    x = volume((2, 6, 1, 28, 28), 5, "f32")
    _, blob3, xhat3 = run(x, 8, 2, 9, "f32", "f32")
    codec = binding.Codec(2, 6, 28, 28, 8, 2)
    codec.blob.zero_()
    codec.compress(torch.from_numpy(x[:, :, 0]).cuda(), seed=9)
    xhat2 = codec.decompress()
    torch.cuda.synchronize()
    np.testing.assert_array_equal(blob3[:codec.blob.numel()], codec.blob.cpu().numpy())
    np.testing.assert_array_equal(xhat3[:, :, 0], xhat2.cpu().numpy())


def test_argument_checks():
    L = binding.lib()
    import ctypes
    out = binding.DivLayout()
    assert L.div_compressed_bytes_3d(ctypes.byref(binding.make_desc_3d(1, 1, 0, 2, 2, 8, 2)), ctypes.byref(out)) == binding.DIV_ERR_SHAPE
    assert L.div_compressed_bytes_3d(ctypes.byref(binding.make_desc_3d(1, 1 << 12, 1 << 10, 1 << 5, 1 << 5, 8, 2)), ctypes.byref(out)) == binding.DIV_ERR_SHAPE
    assert L.div_compressed_bytes_3d(ctypes.byref(binding.make_desc_3d(1, 1, 2, 2, 2, 8, 3)), ctypes.byref(out)) == binding.DIV_ERR_PARAM
    d = binding.make_desc_3d(2, 2, 4, 4, 4, 4, 2)
    assert L.div_compress_3d(ctypes.byref(d), 16, 32, 8, 64, 1 << 20, 0, None) == binding.DIV_ERR_CAPACITY
    assert L.div_compress_3d(ctypes.byref(d), 16, 36, 1 << 20, 64, 1 << 20, 0, None) == binding.DIV_ERR_ALIGN
    assert L.div_decompress_3d(ctypes.byref(d), None, 8, 32, None) == binding.DIV_ERR_NULL
