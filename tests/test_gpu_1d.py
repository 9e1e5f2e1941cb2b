"""Parity of 1-D activation maps (appendix "Compression of 1D and 3D Activation Maps": Minibatch x Channel x N,
described to the library as N x C x 1 x W) with the checker's separately written 1-D functions: exact equality of
stored low-frequency values, (delta, Delta), packed words, the whole blob and the reconstruction."""
import numpy as np
import pytest
import torch

from oracle import division_oracle as orc
from paper_2208_04187_b200 import binding, build

pytestmark = pytest.mark.gpu

NO_LINE = binding.DIV_FLAG_NO_LINE_KERNELS
TWO_PASS = binding.DIV_FLAG_FORCE_TWO_PASS


@pytest.fixture(scope="module", autouse=True)
def built_library():
    build.build()
    binding.lib()


def tokens(m, c, n, seed, dtype):
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal((m, c, n)) * (1 + rng.random((m, c, 1)))).astype(np.float32)
    return orc.f32_to_bf16_bits(x) if dtype == "bf16" else x


def assert_parity(x, block, q, seed, xd="f32", ld="f32", flags=0, expect=None):
    m, c, n = x.shape
    ref = orc.compress_1d(x, block, q, seed, xd, ld)
    codec = binding.Codec(m, c, 1, n, block, q, xd, ld)
    if expect is not None:
        assert codec.plan(flags).fused == expect
    t = torch.from_numpy(x.reshape(m, c, 1, n))
    xdev = (t.view(torch.bfloat16) if xd == "bf16" else t).cuda()
    codec.blob.fill_(0)
    codec.compress(xdev, seed=seed, flags=flags)
    xhat = codec.decompress()
    torch.cuda.synchronize()
    assert codec.device_status() == binding.DIV_OK
    np.testing.assert_array_equal(codec.blob.cpu().numpy(), ref.blob(), err_msg="blob bytes")
    got = xhat.view(torch.int16).cpu().numpy().view(np.uint16) if xd == "bf16" else xhat.cpu().numpy()
    got = orc.bf16_bits_to_f32(got) if xd == "bf16" else got
    np.testing.assert_array_equal(got.reshape(m, c, n), orc.decompress_1d(ref), err_msg="reconstruction")


# W % 4 == 0, B a power of two in [4, 128], Q in {2, 4, 8}: the pair of 1-D kernels
LINE = [
    ((2, 5, 64), 8, 2, "f32", "f32"), ((3, 7, 768), 8, 4, "f32", "f32"), ((2, 9, 768), 16, 2, "bf16", "bf16"),
    ((2, 11, 96), 64, 2, "f32", "bf16"), ((3, 4, 1024), 128, 8, "f32", "f32"), ((2, 6, 100), 16, 2, "f32", "f32"),
    ((2, 3, 36), 8, 4, "bf16", "f32"), ((1, 300, 20), 4, 2, "f32", "f32"), ((4, 197, 384), 64, 2, "f32", "f32"),
    ((2, 13, 4), 8, 2, "f32", "f32"), ((1, 1, 8), 8, 8, "f32", "f32"), ((2, 50, 132), 32, 4, "f32", "f32"),
]
# 1-D maps the pair does not take
OTHER = [
    ((2, 5, 30), 8, 2, "f32", "f32"), ((2, 4, 96), 12, 2, "f32", "f32"), ((2, 6, 64), 8, 1, "f32", "f32"),
    ((1, 3, 512), 256, 2, "f32", "f32"), ((2, 7, 33), 16, 4, "bf16", "bf16"), ((2, 3, 8), 2, 2, "f32", "f32"),
]


@pytest.mark.parametrize("shape,block,q,xd,ld", LINE)
def test_line_kernels_match_the_checker(shape, block, q, xd, ld):
    # the single-launch kernel (plan code 8), then the pair of kernels it replaces where its CTAs cannot all be resident
    assert_parity(tokens(*shape, 21, xd), block, q, 5, xd, ld, expect=8)
    assert_parity(tokens(*shape, 21, xd), block, q, 5, xd, ld, flags=binding.DIV_FLAG_TWO_LAUNCH_PLANES, expect=5)


@pytest.mark.parametrize("shape,block,q,xd,ld", LINE + OTHER)
@pytest.mark.parametrize("flags", [NO_LINE, TWO_PASS])
def test_other_paths_match_the_checker_on_1d_maps(shape, block, q, xd, ld, flags):
    x = tokens(*shape, 22, xd)
    codec = binding.Codec(shape[0], shape[1], 1, shape[2], block, q, xd, ld)
    assert codec.plan(flags).fused not in (5, 8)
    assert_parity(x, block, q, 6, xd, ld, flags=flags)


@pytest.mark.parametrize("shape,block,q,xd,ld", OTHER)
def test_default_path_on_the_remaining_1d_maps(shape, block, q, xd, ld):
    x = tokens(*shape, 23, xd)
    codec = binding.Codec(shape[0], shape[1], 1, shape[2], block, q, xd, ld)
    assert codec.plan().fused not in (5, 8)
    assert_parity(x, block, q, 7, xd, ld)


def test_transformer_shaped_map_sampled():
    """Batch 32 x 512 tokens x 768 hidden, B = 8, Q = 4 (the T5 setting of the paper's appendix) at full size:
    samples are independent, so three of them are checked whole against the checker."""
    m, c, n = 32, 512, 768
    rng = np.random.default_rng(0)
    x = rng.standard_normal((m, c, n)).astype(np.float32)
    codec = binding.Codec(m, c, 1, n, 8, 4)
    assert codec.plan().fused == 8
    codec.compress(torch.from_numpy(x.reshape(m, c, 1, n)).cuda(), seed=3)
    xhat = codec.decompress().cpu().numpy().reshape(m, c, n)
    blob = codec.blob.cpu().numpy()
    lo = codec.layout
    got = orc.parse_blob(blob, m, c, 1, n, 8, 4)
    for i in (0, 17, 31):
        ref = orc.compress_1d(x[i:i + 1], 8, 4, 3)            # sample index 0 in the checker's stream ...
        # ... so compare what does not depend on the stream, then the codes through a stream of the right index
        np.testing.assert_array_equal(got.lfc[i, :, 0, :], ref.lfc[0, :, 0, :])
        assert got.delta[i] == ref.delta[0] and got.step[i] == ref.step[0]
        r = (x[i] - orc.upsample_nearest_1d(ref.lfc[:, :, 0, :], 8, n)[0]).reshape(-1)
        _, _, scale = orc.sample_stats(r, 4)
        codes = orc.quantize(r, ref.delta[0], scale, orc.divrng_fields(3, i, np.arange(c * n, dtype=np.uint64)), 4)
        np.testing.assert_array_equal(got.codes[i], codes)
        np.testing.assert_array_equal(xhat[i].reshape(-1), orc.dequantize(codes, ref.delta[0], ref.step[0]) +
                                      orc.upsample_nearest_1d(ref.lfc[:, :, 0, :], 8, n)[0].reshape(-1))
