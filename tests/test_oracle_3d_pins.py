"""Pins of the checker's 3-D form (appendix "Compression of 1D and 3D Activation Maps": Minibatch x Channel x N x N x N,
pooling and up-sampling over B x B x B blocks).  No GPU needed."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import division_oracle as orc


def volume(m, c, d, h, w, seed):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((m, c, d, h, w)) * (1 + rng.random((m, c, 1, 1, 1)))).astype(np.float32)


@pytest.mark.parametrize("dims,block", [((8, 8, 8), 4), ((16, 8, 24), 8), ((5, 9, 7), 4), ((3, 3, 3), 8), ((6, 10, 4), 3),
                                        ((2, 12, 20), 8)])
def test_lfc_3d_is_library_average_pooling(dims, block):
    x = volume(2, 3, *dims, 1)
    b = min(block, max(dims))
    k = tuple(min(b, s) for s in dims)          # torch refuses a window longer than a side; a shorter side is one block
    ref = F.avg_pool3d(torch.from_numpy(x).double(), k, k, ceil_mode=True, count_include_pad=False).numpy()
    got = orc.lfc_mean_3d(x, block)
    assert got.shape == ref.shape
    np.testing.assert_allclose(got, ref, rtol=0, atol=3e-6 * np.abs(x).max())
    if all(s % b == 0 for s in dims):
        assert got.shape[2:] == tuple(s // b for s in dims)            # the paper's floor(N/B) shapes when B divides N


def test_upsampling_3d_is_library_nearest_interpolation():
    lfc = volume(2, 3, 2, 3, 4, 2)
    ref = F.interpolate(torch.from_numpy(lfc), scale_factor=4, mode="nearest").numpy()
    np.testing.assert_array_equal(orc.upsample_nearest_3d(lfc, 4, 8, 12, 16), ref)
    np.testing.assert_array_equal(orc.upsample_nearest_3d(lfc, 4, 7, 10, 13), ref[:, :, :7, :10, :13])


@pytest.mark.parametrize("hw,block,q", [((16, 24), 8, 2), ((14, 14), 8, 4), ((7, 9), 4, 8), ((5, 6), 16, 1)])
def test_depth_one_is_the_2d_form(hw, block, q):
    """A 3-D map of depth 1 is a 2-D map: the separately written 3-D functions give the same bytes."""
    h, w = hw
    x = volume(2, 3, 1, h, w, 4)
    a = orc.compress_3d(x, block, q, 9)
    b = orc.compress(x[:, :, 0], block, q, 9)
    np.testing.assert_array_equal(a.lfc[:, :, 0], b.lfc)
    np.testing.assert_array_equal(a.words, b.words)
    np.testing.assert_array_equal(a.blob(), b.blob())
    np.testing.assert_array_equal(orc.decompress_3d(a)[:, :, 0], orc.decompress(b))


def test_constant_volume_block_zero_sum_and_sizes():
    x = np.full((2, 2, 8, 8, 8), -1.25, np.float32)
    comp = orc.compress_3d(x, 4, 2, 1)
    assert np.all(comp.lfc == -1.25) and np.all(comp.step == 0) and not comp.codes.any()
    np.testing.assert_array_equal(orc.decompress_3d(comp), x)
    y = volume(1, 2, 8, 8, 8, 3)
    lfc = orc.lfc_mean_3d(y, 4)
    res = (y.astype(np.float64) - orc.upsample_nearest_3d(lfc, 4, 8, 8, 8)).reshape(1, 2, 2, 4, 2, 4, 2, 4).sum((3, 5, 7))
    assert np.abs(res).max() < 1e-4
    lo = orc.layout_3d(3, 5, 8, 16, 24, 8, 2)
    assert lo.closed_form_bytes == 3 * 5 * 1 * 2 * 3 * 4 + 3 * 5 * 8 * 16 * 24 * 2 // 8 + 8 * 3
    assert lo.raw_bytes / lo.closed_form_bytes == pytest.approx(4 / (4 / 512 + 2 / 8), rel=3e-3)     # B^3 = 512 elements per low-frequency value


@pytest.mark.parametrize("q", [1, 2, 4, 8])
def test_error_bound_end_codes_and_unbiasedness(q):
    x = volume(2, 3, 6, 10, 12, 5)
    comp = orc.compress_3d(x, 4, q, 3)
    xhat = orc.decompress_3d(comp)
    err = np.abs(xhat.astype(np.float64) - x)
    assert (err <= comp.step[:, None, None, None, None] * (1 + 1e-5) + 1e-6).all()
    r = (x - orc.upsample_nearest_3d(comp.lfc, 4, 6, 10, 12)).reshape(2, -1)
    for i in range(2):
        assert comp.codes[i][r[i].argmin()] == 0 and comp.codes[i][r[i].argmax()] == (1 << q) - 1
    if q == 2:
        small = volume(1, 1, 4, 4, 4, 6)
        acc = np.zeros(small.shape)
        for s in range(400):
            acc += orc.decompress_3d(orc.compress_3d(small, 4, 2, 50 + s))
        step = float(orc.compress_3d(small, 4, 2, 0).step[0])
        z = (acc / 400 - small) / (0.5 * step / 20.0)
        assert np.abs(z).max() < 5 and abs(z.mean()) < 0.5
