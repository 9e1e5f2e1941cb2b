"""Seeded random shapes through every entry point against the checker (exact equality).  The shapes are small, so
the checker finishes in milliseconds; they mix block sizes, bit widths, dtypes and ragged sides so that every
kernel-selection branch is reached with geometry nobody picked by hand."""
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


def dev(a, dtype):
    t = torch.from_numpy(a)
    return (t.view(torch.bfloat16) if dtype == "bf16" else t).cuda()


def host(t, dtype):
    if dtype == "bf16":
        return orc.bf16_bits_to_f32(t.view(torch.int16).cpu().numpy().view(np.uint16))
    return t.cpu().numpy()


def draw(rng, shape, dtype):
    x = (rng.standard_normal(shape) * 10.0 ** rng.integers(-2, 3)).astype(np.float32)
    if rng.random() < 0.3:
        x = np.maximum(x, 0)                      # ReLU-like maps with constant tiles
    return orc.f32_to_bf16_bits(x) if dtype == "bf16" else x


def pick(rng):
    block = int(rng.choice([1, 2, 3, 4, 4, 8, 8, 8, 12, 16, 32, 64]))
    q = int(rng.choice([1, 2, 2, 4, 8]))
    xd = str(rng.choice(["f32", "f32", "bf16"]))
    ld = str(rng.choice(["f32", "bf16"]))
    return block, q, xd, ld


@pytest.mark.parametrize("seed", range(60))
def test_random_2d_maps_per_sample_and_per_plane(seed):
    rng = np.random.default_rng(1000 + seed)
    n, c = int(rng.integers(1, 4)), int(rng.integers(1, 24))
    h, w = int(rng.integers(1, 40)), int(rng.choice([rng.integers(1, 40), 4 * rng.integers(1, 12)]))
    block, q, xd, ld = pick(rng)
    x = draw(rng, (n, c, h, w), xd)
    flags = int(rng.choice([0, 0, binding.DIV_FLAG_NO_STRIP_KERNEL, binding.DIV_FLAG_NO_LAGGED_KERNEL,
                            binding.DIV_FLAG_NO_STRIP_KERNEL | binding.DIV_FLAG_NO_LAGGED_KERNEL,
                            binding.DIV_FLAG_FORCE_TWO_PASS]))
    ref = orc.compress(x, block, q, seed, xd, ld)
    codec = binding.Codec(n, c, h, w, block, q, xd, ld)
    codec.blob.zero_()
    codec.compress(dev(x, xd), seed=seed, flags=flags)
    xhat = codec.decompress()
    torch.cuda.synchronize()
    assert codec.device_status() == binding.DIV_OK
    np.testing.assert_array_equal(codec.blob.cpu().numpy(), ref.blob(), err_msg=f"per-sample blob {x.shape} B={block} Q={q} flags={flags}")
    np.testing.assert_array_equal(host(xhat, xd), orc.decompress(ref))
    refp = orc.compress_planes(x, block, q, seed, xd, ld)
    pg = binding.PlaneGroupCodec(n, c, h, w, block, q, xd, ld)
    pg.blob.zero_()
    pg.compress(dev(x, xd), seed=seed, flags=int(rng.choice([0, 0, binding.DIV_FLAG_FORCE_TWO_PASS])))
    xhatp = pg.decompress()
    torch.cuda.synchronize()
    np.testing.assert_array_equal(pg.blob.cpu().numpy(), refp.blob(), err_msg=f"per-plane blob {x.shape} B={block} Q={q}")
    np.testing.assert_array_equal(host(xhatp, xd), orc.decompress_planes(refp))


@pytest.mark.parametrize("seed", range(30))
def test_random_1d_and_3d_maps(seed):
    rng = np.random.default_rng(2000 + seed)
    block, q, xd, ld = pick(rng)
    m, c = int(rng.integers(1, 4)), int(rng.integers(1, 30))
    n1 = int(rng.choice([rng.integers(1, 200), 4 * rng.integers(1, 64)]))
    x = draw(rng, (m, c, n1), xd)
    ref = orc.compress_1d(x, block, q, seed, xd, ld)
    codec = binding.Codec(m, c, 1, n1, block, q, xd, ld)
    codec.blob.zero_()
    codec.compress(dev(x.reshape(m, c, 1, n1), xd), seed=seed)
    xhat = codec.decompress()
    torch.cuda.synchronize()
    np.testing.assert_array_equal(codec.blob.cpu().numpy(), ref.blob(), err_msg=f"1-D blob {x.shape} B={block} Q={q}")
    np.testing.assert_array_equal(host(xhat, xd).reshape(m, c, n1), orc.decompress_1d(ref))

    d3, h3, w3 = int(rng.integers(1, 10)), int(rng.integers(1, 12)), int(rng.choice([rng.integers(1, 14), 4 * rng.integers(1, 5)]))
    c3 = int(rng.integers(1, 5))
    y = draw(rng, (m, c3, d3, h3, w3), xd)
    ref3 = orc.compress_3d(y, block, q, seed, xd, ld)
    desc = binding.make_desc_3d(m, c3, d3, h3, w3, block, q, xd, ld)
    lo = binding.div_compressed_bytes_3d(desc)
    blob = torch.zeros(int(lo.total_bytes), dtype=torch.uint8, device="cuda")
    ws = torch.empty(int(lo.workspace_bytes), dtype=torch.uint8, device="cuda")
    yd = dev(y, xd)
    out = torch.empty_like(yd)
    s = torch.cuda.current_stream().cuda_stream
    binding.div_compress_3d(desc, yd.data_ptr(), blob.data_ptr(), blob.numel(), ws.data_ptr(), ws.numel(), seed, s)
    binding.div_decompress_3d(desc, blob.data_ptr(), blob.numel(), out.data_ptr(), s)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(blob.cpu().numpy(), ref3.blob(), err_msg=f"3-D blob {y.shape} B={block} Q={q}")
    np.testing.assert_array_equal(host(out, xd), orc.decompress_3d(ref3))
