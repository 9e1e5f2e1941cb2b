"""Pins of the checker's 1-D form (appendix "Compression of 1D and 3D Activation Maps": Minibatch x Channel x N,
pooling and up-sampling along the last axis).  No GPU needed."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import division_oracle as orc


def tokens(m, c, n, seed):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((m, c, n)) * (1 + rng.random((m, c, 1)))).astype(np.float32)


@pytest.mark.parametrize("n,block", [(64, 8), (768, 16), (96, 64), (40, 4), (30, 8), (77, 16), (5, 8), (100, 12)])
def test_lfc_1d_is_library_average_pooling(n, block):
    x = tokens(2, 3, n, 1)
    b = min(block, n)
    ref = F.avg_pool1d(torch.from_numpy(x).double(), b, b, ceil_mode=True, count_include_pad=False).numpy()
    got = orc.lfc_mean_1d(x, block)
    assert got.shape == ref.shape == (2, 3, -(-n // b))
    np.testing.assert_allclose(got, ref, rtol=0, atol=2e-6 * np.abs(x).max())
    if n % b == 0:
        assert got.shape[2] == n // b                              # the paper's floor(N/B) when B divides N


def test_upsampling_1d_is_library_nearest_interpolation():
    lfc = tokens(2, 3, 6, 2)
    ref = F.interpolate(torch.from_numpy(lfc), scale_factor=8, mode="nearest").numpy()
    np.testing.assert_array_equal(orc.upsample_nearest_1d(lfc, 8, 48), ref)
    np.testing.assert_array_equal(orc.upsample_nearest_1d(lfc, 8, 43), ref[:, :, :43])


def test_constant_rows_and_zero_residual_sum():
    x = np.full((2, 3, 32), 2.5, np.float32)
    comp = orc.compress_1d(x, 8, 2, 1)
    assert np.all(comp.lfc == 2.5) and np.all(comp.step == 0) and not comp.codes.any()
    np.testing.assert_array_equal(orc.decompress_1d(comp), x)
    y = tokens(2, 3, 64, 3)
    lfc = orc.lfc_mean_1d(y, 8)
    res = (y.astype(np.float64) - orc.upsample_nearest_1d(lfc, 8, 64)).reshape(2, 3, 8, 8).sum(-1)
    assert np.abs(res).max() < 1e-5                                # each block's residual sums to zero


@pytest.mark.parametrize("n,block,q", [(64, 8, 2), (96, 16, 4), (30, 8, 8), (128, 64, 2), (5, 8, 1)])
def test_1d_form_equals_the_2d_form_on_a_map_of_height_one(n, block, q):
    """A 1-D map is a 2-D map with one row: the separately written 1-D functions give the same bytes."""
    x = tokens(3, 4, n, 4)
    a = orc.compress_1d(x, block, q, 9)
    b = orc.compress(x[:, :, None, :], block if block <= n else n, q, 9)
    np.testing.assert_array_equal(a.lfc, b.lfc)
    np.testing.assert_array_equal(a.delta, b.delta)
    np.testing.assert_array_equal(a.words, b.words)
    np.testing.assert_array_equal(a.blob(), b.blob())
    np.testing.assert_array_equal(orc.decompress_1d(a), orc.decompress(b)[:, :, 0, :])


@pytest.mark.parametrize("q", [1, 2, 4, 8])
def test_error_bound_and_end_codes(q):
    x = tokens(2, 5, 96, 5)
    comp = orc.compress_1d(x, 16, q, 3)
    xhat = orc.decompress_1d(comp)
    err = np.abs(xhat.astype(np.float64) - x)
    assert (err <= comp.step[:, None, None] * (1 + 1e-5) + 1e-6).all()
    r = (x - orc.upsample_nearest_1d(comp.lfc[:, :, 0, :], 16, 96)).reshape(2, -1)
    for i in range(2):
        assert comp.codes[i][r[i].argmin()] == 0 and comp.codes[i][r[i].argmax()] == (1 << q) - 1


def test_unbiased_over_seeds():
    x = tokens(1, 2, 32, 6)
    acc = np.zeros(x.shape)
    seeds = 500
    for s in range(seeds):
        acc += orc.decompress_1d(orc.compress_1d(x, 8, 2, 100 + s))
    step = float(orc.compress_1d(x, 8, 2, 0).step[0])
    z = (acc / seeds - x) / (0.5 * step / np.sqrt(seeds))
    assert np.abs(z).max() < 5 and abs(z.mean()) < 0.5
