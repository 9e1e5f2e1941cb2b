"""Pins of the CPU checker (oracle/) against what the paper and the mathematics fix.

None of these needs a GPU.  Each test names the statement it pins:
Sec. 4.1 / 4.2, Eq. 9 (Quant), Eq. 10 (reconstruction), Theorem 3A, and the footnotes of Sec. 4.1.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import division_oracle as orc
from paper_2208_04187_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")


def golden_values():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, value, tol, _ = [s.strip() for s in line.split("|", 3)]
            out[name] = (float(value), float(tol))
    return out


def relu_map(shape, seed):
    return synth.activation_map(*shape, "relu", seed)


def bn_map(shape, seed):
    return synth.activation_map(*shape, "bn", seed)


# ---------------------------------------------------------------------------------------
# low-frequency component: Sec. 4.1 (average pooling, window = stride = B) and its footnote
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("shape,block", [((2, 3, 16, 24), 8), ((2, 3, 12, 8), 4), ((1, 5, 32, 16), 16),
                                         ((2, 2, 6, 10), 2)])
def test_lfc_equals_library_avg_pool_on_divisible_shapes(shape, block):
    x = bn_map(shape, 11)
    ref = F.avg_pool2d(torch.from_numpy(x).double(), block, block).numpy()
    got = orc.lfc_mean_f32(x, block)
    assert got.shape == ref.shape
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-6 * np.abs(x).max())
    np.testing.assert_allclose(orc.lfc_mean_f64(x, block), ref, rtol=0, atol=1e-12)


@pytest.mark.parametrize("shape,block", [((2, 3, 28, 14), 8), ((1, 4, 7, 7), 8), ((2, 2, 9, 13), 4),
                                         ((1, 3, 14, 30), 12)])
def test_lfc_tail_tiles_average_in_bounds_elements(shape, block):
    """Ceil grid; a partial tile divides by its in-bounds count (library: ceil_mode pooling)."""
    x = bn_map(shape, 12)
    ref = F.avg_pool2d(torch.from_numpy(x).double(), block, block, ceil_mode=True,
                       count_include_pad=False).numpy()
    got = orc.lfc_mean_f32(x, block)
    assert got.shape == ref.shape == (shape[0], shape[1], -(-shape[2] // block), -(-shape[3] // block))
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-6 * np.abs(x).max())


def test_block_sum_order_is_columns_first_pairwise_trees():
    """The block sum is a balanced pairwise tree down the rows of every tile column, then the same tree across
    the column sums.  One 8 x 8 tile on which this order, the rows-first order and a running sum round
    differently in fp32 (2^24 + 1 is not representable and rounds to 2^24); the expected value is worked out
    by hand, not by the checker:
        column 0 = (1, 2^24, 1, -2^24, 0, ...):  (1 + 2^24) + (1 - 2^24) = 2^24 + (-16777215) = 1
        column 1 = (1, 0,    1, 0,     0, ...):  (1 + 0) + (1 + 0) = 2
        across the columns: (1 + 2) + 0 + ... = 3, mean = 3 / 64        (the exact sum is 4)."""
    big = np.float32(2.0 ** 24)
    tile = np.zeros((8, 8), dtype=np.float32)
    tile[:4, 0] = [1, big, 1, -big]
    tile[:4, 1] = [1, 0, 1, 0]
    got = orc.lfc_mean_f32(tile[None, None], 8)
    assert got.shape == (1, 1, 1, 1)
    assert got[0, 0, 0, 0] == np.float32(3.0 / 64.0)

    def tree(values):
        v = [np.float32(a) for a in values]
        while len(v) > 1:
            v = [np.float32(v[i] + v[i + 1]) for i in range(0, len(v), 2)]
        return v[0]

    # the other orders give other numbers on this tile, so the pin tells them apart
    rows_first = tree([tree(tile[r, :]) for r in range(8)])          # (2 + 2^24) + (2 - 2^24) = 4
    running = np.float32(0)
    for v in tile.T.reshape(-1):                                     # column by column, one element after the other
        running = np.float32(running + v)                            # ((1 + 2^24) + 1) - 2^24 = 0, then + 2
    assert rows_first == np.float32(4) and running == np.float32(2)
    assert float(tile.astype(np.float64).sum()) == 4.0
    # the same tile inside a larger map, next to ordinary tiles, and as a partial tile (5 in-bounds rows)
    x = bn_map((1, 2, 16, 16), 21)
    x[0, 1, 8:16, 0:8] = tile
    assert orc.lfc_mean_f32(x, 8)[0, 1, 1, 0] == np.float32(3.0 / 64.0)
    part = np.zeros((1, 1, 13, 8), dtype=np.float32)
    part[0, 0, 8:13, :] = tile[:5]
    assert orc.lfc_mean_f32(part, 8)[0, 0, 1, 0] == np.float32(np.float32(3.0) / np.float32(40.0))


def test_side_shorter_than_block_gives_1x1_plane_mean():
    """Sec. 4.1 footnote: N < B makes the low-frequency map Minibatch x Channel x 1 x 1."""
    x = bn_map((3, 5, 7, 7), 13)
    got = orc.lfc_mean_f32(x, 8)
    assert got.shape == (3, 5, 1, 1)
    np.testing.assert_allclose(got[..., 0, 0], x.astype(np.float64).mean(axis=(2, 3)), atol=1e-6)
    x = bn_map((2, 4, 4, 4), 14)
    np.testing.assert_allclose(orc.lfc_mean_f32(x, 8)[..., 0, 0], x.astype(np.float64).mean(axis=(2, 3)),
                               atol=1e-6)


def test_upsample_is_nearest_interpolation():
    lfc = bn_map((2, 3, 4, 5), 15)
    ref = F.interpolate(torch.from_numpy(lfc), scale_factor=8, mode="nearest").numpy()
    np.testing.assert_array_equal(orc.upsample_nearest(lfc, 8, 32, 40), ref)
    # cropped for tails: element (h, w) reads tile (h // B, w // B)
    up = orc.upsample_nearest(lfc, 8, 28, 35)
    for (h, w) in [(0, 0), (7, 8), (27, 34), (16, 15)]:
        np.testing.assert_array_equal(up[:, :, h, w], lfc[:, :, h // 8, w // 8])


def test_block_one_keeps_everything_in_the_lfc():
    """B = 1: LFC = x exactly, HFC = 0, Delta = 0, exact reconstruction."""
    x = relu_map((2, 3, 5, 6), 16)
    comp = orc.compress(x, 1, 2, seed=3)
    np.testing.assert_array_equal(comp.lfc, x)
    assert not comp.codes.any()
    np.testing.assert_array_equal(comp.step, 0)
    np.testing.assert_array_equal(comp.delta, 0)
    np.testing.assert_array_equal(orc.decompress(comp), x)


def test_constant_tensor_reconstructs_exactly():
    x = np.full((2, 3, 16, 12), 1.7, dtype=np.float32)
    for lfc_dtype in ("f32", "bf16"):
        comp = orc.compress(x, 8, 2, seed=5, lfc_dtype=lfc_dtype)
        assert not comp.codes.any() and not comp.words.any()
        np.testing.assert_array_equal(comp.step, 0)
        xhat = orc.decompress(comp)
        if lfc_dtype == "f32":
            np.testing.assert_array_equal(comp.delta, 0)
            np.testing.assert_array_equal(xhat, x)
        else:   # the bf16 rounding of the mean lands in the (constant) residual, so it comes back
            np.testing.assert_allclose(xhat, x, rtol=1e-7)


def test_tile_residuals_sum_to_zero():
    """Definition of a mean: per tile, sum of (x - mean) is zero up to rounding."""
    x = bn_map((2, 4, 28, 20), 17)
    lfc = orc.lfc_mean_f32(x, 8)
    r = x.astype(np.float64) - orc.upsample_nearest(lfc, 8, 28, 20)
    t, rows, cols = orc._tiles(r, 8)
    sums = t.sum(axis=(-1, -2))
    assert np.abs(sums).max() <= 64 * 2e-7 * np.abs(x).max()


def test_residual_uses_the_stored_bf16_lfc():
    x = bn_map((2, 3, 16, 16), 18)
    comp = orc.compress(x, 8, 4, seed=0, lfc_dtype="bf16")
    # stored values are representable in bf16 and within half a bf16 ulp of the exact mean
    np.testing.assert_array_equal(orc.round_to_dtype(comp.lfc, "bf16"), comp.lfc)
    exact = orc.lfc_mean_f64(x, 8)
    assert np.abs(comp.lfc - exact).max() <= 2.0 ** -8 * np.abs(exact).max()
    # decoding with the stored values meets the one-step error bound (it would not with the exact mean)
    xhat = orc.decompress(comp)
    assert np.all(np.abs(xhat - x).reshape(2, -1) <= comp.step[:, None] * (1 + 1e-5) + 1e-6)


def test_bf16_rounding_is_nearest_even():
    vals = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -2.5, 3.1415927, 1e-30],
                    dtype=np.float32)
    ref = torch.from_numpy(vals).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(orc.round_to_dtype(vals, "bf16"), ref)
    big = bn_map((1, 1, 64, 64), 19).reshape(-1)
    ref = torch.from_numpy(big).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(orc.round_to_dtype(big, "bf16"), ref)


# ---------------------------------------------------------------------------------------
# quantiser: Eq. 9 and the two footnotes on stochastic rounding
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("qbits", [1, 2, 4, 8])
def test_dequantisation_error_is_at_most_one_step(qbits):
    """|H^H_hat - H^H| <= Delta = (max - min)/(2^Q - 1), element by element."""
    x = relu_map((3, 4, 16, 16), 20 + qbits)
    comp = orc.compress(x, 8, qbits, seed=7)
    r = (x - orc.upsample_nearest(comp.lfc, 8, 16, 16)).reshape(3, -1)
    for i in range(3):
        hh = orc.dequantize(comp.codes[i], comp.delta[i], comp.step[i])
        span = r[i].max() - r[i].min()
        assert comp.step[i] == pytest.approx(span / (2 ** qbits - 1), rel=1e-6)
        assert comp.delta[i] == r[i].min()
        assert np.abs(hh - r[i]).max() <= comp.step[i] * (1 + 1e-5)
    xhat = orc.decompress(comp)
    assert np.all(np.abs(xhat - x).reshape(3, -1) <= comp.step[:, None] * (1 + 1e-5) + 1e-6)


def test_error_shrinks_with_more_bits():
    x = relu_map((2, 4, 16, 16), 30)
    errs = [np.abs(orc.decompress(orc.compress(x, 8, q, seed=1)) - x).mean() for q in (1, 2, 4, 8)]
    assert errs[0] > errs[1] > errs[2] > errs[3]
    span = 2.0 * np.abs(x).max()
    assert np.abs(orc.decompress(orc.compress(x, 8, 8, seed=1)) - x).max() <= span / 255


def test_extremes_get_end_codes_for_every_seed():
    """t = 0 has no fractional part, so the minimum always codes 0; the maximum always 2^Q - 1."""
    x = bn_map((3, 2, 8, 8), 31)
    for seed in range(50):
        comp = orc.compress(x, 4, 2, seed=seed)
        r = (x - orc.upsample_nearest(comp.lfc, 4, 8, 8)).reshape(3, -1)
        for i in range(3):
            assert comp.codes[i, r[i].argmin()] == 0
            assert comp.codes[i, r[i].argmax()] == 3


def test_stats_are_per_sample():
    x = bn_map((4, 3, 8, 8), 32)
    x[1] *= 10.0
    x[3] *= 0.01
    comp = orc.compress(x, 8, 2, seed=0)
    assert comp.delta.shape == (4,) and comp.step.shape == (4,)
    r = (x - orc.upsample_nearest(comp.lfc, 8, 8, 8)).reshape(4, -1)
    np.testing.assert_array_equal(comp.delta, r.min(axis=1))
    np.testing.assert_allclose(comp.step, (r.max(axis=1) - r.min(axis=1)) / 3, rtol=1e-6)
    for i in range(4):   # each sample uses its whole code range
        assert comp.codes[i].min() == 0 and comp.codes[i].max() == 3


def _bias_z_scores(x, block, qbits, n_seeds, rounding="paper-unbiased"):
    """z-score per element of mean_over_seeds(dequant(quant(r))) - r."""
    lfc = orc.lfc_mean_f32(x, block)
    n, c, h, w = x.shape
    r = (x - orc.upsample_nearest(lfc, block, h, w)).reshape(n, -1)
    e = np.arange(r.shape[1], dtype=np.uint64)
    zs = []
    for i in range(n):
        delta, step, scale = orc.sample_stats(r[i], qbits)
        acc = np.zeros(r.shape[1], dtype=np.float64)
        for seed in range(n_seeds):
            fields = orc.divrng_fields(seed, i, e)
            if rounding == "reversed":       # the literal (garbled) footnote: up with probability 1 - frac
                fields = (65535 - fields.astype(np.int64)).astype(np.uint16)
                codes = orc.quantize(r[i], delta, scale, fields, qbits)
                t = (r[i] - delta) * scale
                codes = np.where(t == np.floor(t), codes, 2 * np.floor(t).astype(np.int64) + 1 - codes)
            else:
                codes = orc.quantize(r[i], delta, scale, fields, qbits)
            acc += orc.dequantize(codes, delta, step).astype(np.float64)
        mean = acc / n_seeds
        t = (r[i].astype(np.float64) - float(delta)) * float(scale)
        p = t - np.floor(t)
        sigma = float(step) * np.sqrt(np.maximum(p * (1 - p), 0) / n_seeds) + 1e-6 * float(step)
        zs.append((mean - r[i]) / sigma)
    return np.concatenate(zs)


def test_stochastic_rounding_is_unbiased_over_1e4_seeds():
    """Sec. 4.1 footnote: E[dequant(quant(h))] = h.  Mean over 10^4 seeds within 3 sigma."""
    x = bn_map((1, 2, 8, 8), 33)
    z = _bias_z_scores(x, 4, 2, 10_000)
    assert np.mean(np.abs(z) <= 3.0) >= 0.99
    assert np.abs(z).max() <= 4.5


def test_unbiasedness_pin_catches_the_reversed_footnote():
    """Rounding up with probability 1 - frac(t) (the footnote read literally) fails the same statistic."""
    x = bn_map((1, 2, 8, 8), 33)
    z = _bias_z_scores(x, 4, 2, 300, rounding="reversed")
    assert np.mean(np.abs(z) <= 3.0) < 0.5


def test_brute_force_on_a_tiny_tensor():
    """1x2x3x3, B=2, Q=2 with dyadic values: every step redone in exact rationals, and the rounding
    probabilities by running all 65536 values of the random field through the quantiser."""
    x = np.array([[[[0.0, 1.0, 0.5], [2.0, 1.0, 0.25], [3.5, 0.5, 1.5]],
                   [[0.75, 0.25, 0.0], [0.5, 0.5, 1.0], [0.125, 0.375, 2.0]]]], dtype=np.float32)
    n, c, h, w, b, q = 1, 2, 3, 3, 2, 2
    xf = [[[Fraction(float(x[0, cc, hh, ww])) for ww in range(w)] for hh in range(h)] for cc in range(c)]
    lfc = {}
    for cc in range(c):
        for bh in range(2):
            for bw in range(2):
                cells = [xf[cc][hh][ww] for hh in range(bh * b, min(h, bh * b + b))
                         for ww in range(bw * b, min(w, bw * b + b))]
                lfc[cc, bh, bw] = sum(cells) / len(cells)
    r = [xf[cc][hh][ww] - lfc[cc, hh // b, ww // b] for cc in range(c) for hh in range(h) for ww in range(w)]
    lo, hi = min(r), max(r)
    step = (hi - lo) / 3
    comp = orc.compress(x, b, q, seed=0)
    for (cc, bh, bw), v in lfc.items():
        assert Fraction(float(comp.lfc[0, cc, bh, bw])) == v
    assert Fraction(float(comp.delta[0])) == lo
    assert abs(Fraction(float(comp.step[0])) - step) <= step * Fraction(1, 2 ** 22)
    delta, st, scale = orc.sample_stats(np.array([float(v) for v in r], dtype=np.float32), q)
    all_fields = np.arange(65536, dtype=np.uint16)
    for e, rv in enumerate(r):
        t = (rv - lo) * Fraction(float(scale))             # scale is an fp32 number; t stays exact here
        f = t.numerator // t.denominator
        p = t - f
        codes = orc.quantize(np.full(65536, float(rv), dtype=np.float32), delta, scale, all_fields, q)
        ups = int((codes.astype(np.int64) == min(f + 1, 3)).sum()) if p > 0 else 0
        expected_ups = -((-p.numerator * 65536) // p.denominator)        # ceil(p * 65536) fields lie below p
        if f >= 3:
            assert np.all(codes == 3)
        else:
            assert ups == expected_ups
            assert set(np.unique(codes).tolist()) <= {f, f + 1}
        # and the code actually emitted uses the field DIVRNG gives this element
        fld = int(orc.divrng_fields(0, 0, np.array([e]))[0])
        assert comp.codes[0, e] == min(f + (1 if Fraction(fld, 65536) < p else 0), 3)


# ---------------------------------------------------------------------------------------
# random numbers (DIVRNG-v1 is this build's definition; pinned by its statistics)
# ---------------------------------------------------------------------------------------
def _py_field(seed, n, e):
    m = (1 << 64) - 1
    z = (seed ^ (0x9E3779B97F4A7C15 * (n + 1))) & m
    z = (z + 0xD1B54A32D192ED03 * ((e >> 2) + 1)) & m
    for _ in range(2):
        z ^= z >> 32
        z = (z * 0xD6E8FEB86659FD93) & m
    z ^= z >> 32
    return (z >> (16 * (e & 3))) & 0xFFFF


def test_rng_matches_big_integer_arithmetic():
    for seed, n in [(0, 0), (1, 0), (0, 1), (2 ** 63 + 12345, 77), (2 ** 64 - 1, 2 ** 31 - 2)]:
        e = np.array([0, 1, 2, 3, 4, 5, 1023, 2 ** 20 + 3, 2 ** 32 - 1], dtype=np.uint64)
        got = orc.divrng_fields(seed, n, e)
        assert got.tolist() == [_py_field(seed, n, int(v)) for v in e]


def test_rng_fields_are_uniform_and_uncorrelated():
    m = 1 << 18
    e = np.arange(m, dtype=np.uint64)
    streams = {(s, n): orc.divrng_fields(s, n, e).astype(np.float64) for s, n in
               [(0, 0), (0, 1), (1, 0), (12345, 7)]}
    for f in streams.values():
        for byte in (f.astype(np.int64) >> 8, f.astype(np.int64) & 0xFF):
            counts = np.bincount(byte, minlength=256)
            chi2 = ((counts - m / 256) ** 2 / (m / 256)).sum()
            assert chi2 < 255 + 5 * np.sqrt(2 * 255)
        bits = ((f.astype(np.int64)[:, None] >> np.arange(16)) & 1).mean(axis=0)
        assert np.abs(bits - 0.5).max() < 5 * 0.5 / np.sqrt(m)
        assert abs(f.mean() / 65536 - 0.5) < 5 / np.sqrt(12 * m)
    lim = 5 / np.sqrt(m)

    def corr(a, b):
        return abs(np.corrcoef(a, b)[0, 1])

    f = streams[(0, 0)]
    for lag in (1, 2, 3, 4, 5, 8, 64):              # within a 64-bit word and across words
        assert corr(f[:-lag], f[lag:]) < lim
    assert corr(streams[(0, 0)], streams[(0, 1)]) < lim    # neighbouring samples
    assert corr(streams[(0, 0)], streams[(1, 0)]) < lim    # neighbouring seeds


def test_same_seed_same_blob_other_seed_other_codes():
    x = relu_map((2, 3, 16, 16), 40)
    a = orc.compress(x, 8, 2, seed=9)
    b = orc.compress(x, 8, 2, seed=9)
    c = orc.compress(x, 8, 2, seed=10)
    np.testing.assert_array_equal(a.blob(), b.blob())
    np.testing.assert_array_equal(a.lfc, c.lfc)
    np.testing.assert_array_equal(a.delta, c.delta)
    np.testing.assert_array_equal(a.step, c.step)
    assert (a.codes != c.codes).mean() > 0.05


# ---------------------------------------------------------------------------------------
# packing and sizes
# ---------------------------------------------------------------------------------------
def test_pack_layout_by_hand():
    # Q = 2, codes 0,1,2,3,0,1,2,3,... : every byte is 0b11100100 = 0xE4
    codes = np.tile(np.array([0, 1, 2, 3], dtype=np.uint8), 8)
    np.testing.assert_array_equal(orc.pack_codes(codes, 2), np.array([0xE4E4E4E4, 0xE4E4E4E4], dtype=np.uint32))
    # first element sits in the lowest bits; a short tail leaves the high bits zero
    np.testing.assert_array_equal(orc.pack_codes(np.array([3], dtype=np.uint8), 2), [3])
    np.testing.assert_array_equal(orc.pack_codes(np.array([0, 0, 1], dtype=np.uint8), 2), [1 << 4])
    np.testing.assert_array_equal(orc.pack_codes(np.array([0xA, 0x5, 0xF], dtype=np.uint8), 4), [0xF5A])
    np.testing.assert_array_equal(orc.pack_codes(np.array([1, 2, 3, 4, 5], dtype=np.uint8), 8),
                                  [0x04030201, 0x05])
    np.testing.assert_array_equal(orc.pack_codes(np.array([1, 0, 1, 1] + [0] * 29, dtype=np.uint8), 1),
                                  [0b1101, 0])


@pytest.mark.parametrize("qbits", [1, 2, 4, 8])
def test_unpack_inverts_pack(qbits):
    rng = np.random.default_rng(qbits)
    for total in (1, 31, 32, 33, 1000):
        codes = rng.integers(0, 1 << qbits, size=total).astype(np.uint8)
        words = orc.pack_codes(codes, qbits)
        assert words.size == -(-total * qbits // 32)
        np.testing.assert_array_equal(orc.unpack_codes(words, qbits, total), codes)


def test_blob_round_trip_and_sections():
    x = relu_map((2, 3, 14, 14), 41)
    for lfc_dtype in ("f32", "bf16"):
        comp = orc.compress(x, 8, 2, seed=4, lfc_dtype=lfc_dtype)
        blob = comp.blob()
        lo = comp.layout
        assert blob.size == lo.total_bytes and lo.packed_off % 128 == 0 and lo.stats_off % 128 == 0
        back = orc.parse_blob(blob, 2, 3, 14, 14, 8, 2, "f32", lfc_dtype)
        np.testing.assert_array_equal(back.lfc, comp.lfc)
        np.testing.assert_array_equal(back.codes, comp.codes)
        np.testing.assert_array_equal(back.delta, comp.delta)
        np.testing.assert_array_equal(orc.decompress(back), orc.decompress(comp))


def test_compressed_bytes_closed_form_and_ratios():
    """N*C*ceil(H/B)*ceil(W/B)*sizeof(lfc) + ceil(N*C*H*W*Q/32)*4 + 8N; > 10x at the paper's settings."""
    lo = orc.compressed_layout(64, 64, 112, 112, 8, 2)
    assert lo.lfc_bytes == 64 * 64 * 14 * 14 * 4
    assert lo.packed_bytes == 64 * 64 * 112 * 112 * 2 // 8
    assert lo.stats_bytes == 512
    assert lo.closed_form_bytes == 3211264 + 12845056 + 512
    assert lo.raw_bytes / lo.closed_form_bytes == pytest.approx(12.80, abs=0.005)
    for (c, s, ratio) in [(512, 28, 12.06), (1024, 14, 12.06), (2048, 7, 12.06)]:
        lo = orc.compressed_layout(64, c, s, s, 8, 2)
        assert lo.raw_bytes / lo.closed_form_bytes == pytest.approx(ratio, abs=0.005)
    lo = orc.compressed_layout(128, 512, 4, 4, 8, 2)
    assert lo.raw_bytes / lo.closed_form_bytes == pytest.approx(7.98, abs=0.01)
    for (b, q, ratio) in [(4, 2, 5.33), (4, 4, 3.20), (8, 2, 7.11), (8, 4, 3.76)]:
        lo = orc.compressed_layout(128, 160, 32, 32, b, q, "bf16", "bf16")
        assert lo.raw_bytes / lo.closed_form_bytes == pytest.approx(ratio, abs=0.006)
    # odd sizes: word count rounds up, tail grid is the ceil grid
    lo = orc.compressed_layout(1, 1, 3, 3, 2, 2)
    assert (lo.lfc_bytes, lo.packed_bytes, lo.stats_bytes) == (16, 4, 8)
    assert orc.compressed_layout(3, 5, 7, 9, 4, 1).packed_bytes == 4 * -(-945 // 32)
    # the blob the checker builds has exactly the predicted size
    x = relu_map((3, 5, 7, 9), 42)
    comp = orc.compress(x, 4, 1, seed=0)
    assert comp.blob().size == comp.layout.total_bytes
    assert comp.words.size * 4 == comp.layout.packed_bytes


def test_paper_printed_values():
    g = golden_values()
    v, tol = g["theorem3a_rate_side7_B8_Q2"]
    assert orc.paper_conv_block_rate(7, 8, 2) == pytest.approx(v, abs=tol)
    # and the theorem's closed formula, typed from the theorem statement
    closed = 9.0 / (4.0 / min(64, 49) + 2 / 4.0 + 8.0 / 49 + 1 / 8.0)
    assert orc.paper_conv_block_rate(7, 8, 2) == pytest.approx(closed, rel=1e-12)
    assert all(orc.paper_conv_block_rate(s, 8, 2) >= orc.paper_conv_block_rate(7, 8, 2) for s in range(7, 225))
    v, tol = g["lfc_share_percent_B8_bf16"]
    lo = orc.compressed_layout(4, 8, 64, 64, 8, 2, "f32", "bf16")
    assert 100.0 * lo.lfc_bytes / lo.raw_bytes == pytest.approx(v, abs=tol)
    v, tol = g["hfc_bytes_per_plane_side8_Q2"]
    lo = orc.compressed_layout(1, 1, 8, 8, 8, 2)
    assert lo.packed_bytes + 4 == v      # the paper counts 4 bytes of bf16 (Delta, delta) per plane
