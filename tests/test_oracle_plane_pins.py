"""Pins of the per-plane variant of the CPU checker: one bfloat16 (delta, Delta) pair per
(sample, channel) plane, the grouping behind the paper's N^2*Q/8 + 4 bytes per channel
(Sec. 4.1, proof of Theorem 3A).  No GPU needed.
"""
import os

import numpy as np
import pytest

from oracle import division_oracle as orc
from paper_2208_04187_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")


def golden(name):
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith(name):
                return float(line.split("|")[1])
    raise KeyError(name)


def all_finite_bf16():
    """Every finite bfloat16 number, ascending (brute-force table, no bit tricks)."""
    bits = np.arange(1 << 16, dtype=np.uint32)
    vals = (bits << np.uint32(16)).view(np.float32)
    vals = vals[np.isfinite(vals)]
    return np.unique(vals)            # sorted; -0.0 and +0.0 collapse to one zero


# ---------------------------------------------------------------------------------------
# bytes: Sec. 4.1 and the proof of Theorem 3A
# ---------------------------------------------------------------------------------------
def test_hfc_bytes_of_one_plane_match_the_papers_count():
    lo = orc.plane_layout(1, 1, 8, 8, 8, 2, orc.F32, orc.BF16)
    assert lo.packed_bytes + lo.stats_bytes == golden("hfc_bytes_per_plane_side8_Q2")


@pytest.mark.parametrize("side,block,q", [(56, 8, 2), (112, 8, 2), (32, 8, 4), (8, 8, 8), (16, 4, 2), (4, 8, 2)])
def test_plane_bytes_are_the_papers_three_terms(side, block, q):
    """bf16 low-frequency map + Q bits per element + 4 bytes, per plane (Theorem 3A's proof)."""
    n, c = 3, 5
    lo = orc.plane_layout(n, c, side, side, block, q, orc.F32, orc.BF16)
    per_plane = 2 * side * side // min(block * block, side * side) + side * side * q // 8 + 4
    assert lo.closed_form_bytes == n * c * per_plane
    # and that is the per-layer DIVISION term inside the conv-block rate of Theorem 3A
    n2 = side * side
    rate = (4 * n2 * 2 + n2) / (2 * per_plane + n2 / 8)
    assert rate == pytest.approx(orc.paper_conv_block_rate(side, block, q), rel=1e-12)


def test_plane_layout_differs_from_the_per_sample_one_only_in_the_stats_section():
    a = orc.compressed_layout(4, 6, 20, 12, 8, 2)
    b = orc.plane_layout(4, 6, 20, 12, 8, 2)
    assert (a.lfc_off, a.lfc_bytes, a.packed_off, a.packed_bytes, a.stats_off) == \
           (b.lfc_off, b.lfc_bytes, b.packed_off, b.packed_bytes, b.stats_off)
    assert b.stats_bytes == 4 * 4 * 6 and b.total_bytes == b.stats_off + b.stats_bytes


# ---------------------------------------------------------------------------------------
# directed bfloat16 rounding, against a brute-force table of all bfloat16 numbers
# ---------------------------------------------------------------------------------------
def test_directed_bf16_rounding_against_the_table_of_all_bf16_numbers():
    table = all_finite_bf16()
    rng = np.random.default_rng(3)
    v = np.concatenate([
        rng.standard_normal(4000).astype(np.float32) * np.float32(10.0) ** rng.integers(-30, 30, 4000),
        table[::97], np.array([0.0, -0.0, 1.0, -1.0, 1.0 + 2.0 ** -9, -1.0 - 2.0 ** -9,
                               1e-40, -1e-40, 3e38, -3e38], dtype=np.float32)]).astype(np.float32)
    v = v[np.isfinite(v) & (np.abs(v) <= table[-1])]
    down = orc.bf16_bits_to_f32(orc.bf16_floor_bits(v))
    up = orc.bf16_bits_to_f32(orc.bf16_ceil_bits(v))
    want_down = table[np.searchsorted(table, v, side="right") - 1]
    want_up = table[np.searchsorted(table, v, side="left")]
    np.testing.assert_array_equal(down, want_down)
    np.testing.assert_array_equal(up, want_up)
    assert not np.signbit(down[v == 0]).any() and not np.signbit(up[v == 0]).any()


# ---------------------------------------------------------------------------------------
# plane parameters
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("q", [1, 2, 4, 8])
def test_plane_stats_bracket_the_residuals(q):
    table = all_finite_bf16()
    rng = np.random.default_rng(q)
    for trial in range(50):
        r = (rng.standard_normal(200) * 10.0 ** rng.integers(-3, 3)).astype(np.float32)
        delta_b, step_b, scale = orc.plane_stats(r, q)
        qmax = (1 << q) - 1
        i = np.searchsorted(table, r.min(), side="right") - 1
        assert delta_b == table[i]                                   # largest bf16 <= min
        assert delta_b in table and step_b in table
        exact = (float(r.max()) - float(delta_b)) / qmax
        assert step_b >= np.float32(exact)                           # never below the exact step
        assert step_b <= exact * (1 + 2.0 ** -7) * (1 + 2.0 ** -20)  # at most one bf16 step above it
        assert scale == np.float32(1.0) / step_b
        t = (r - delta_b) * scale
        assert t.min() >= 0 and t.max() <= qmax * (1 + 2.0 ** -20)   # the clamp only absorbs rounding


def test_plane_stats_agree_with_the_per_sample_rule_when_bf16_is_exact():
    """min, max and step all bfloat16 numbers and the step a power of two: both rules coincide."""
    r = np.array([-1.5, -0.25, 0.0, 0.75, 1.5], dtype=np.float32)
    assert orc.plane_stats(r, 2) == orc.sample_stats(r, 2) == (np.float32(-1.5), np.float32(1.0), np.float32(1.0))
    r8 = np.array([-4.0, 0.0, 59.75], dtype=np.float32)
    assert orc.plane_stats(r8, 8) == orc.sample_stats(r8, 8) == (np.float32(-4.0), np.float32(0.25), np.float32(4.0))


def test_degenerate_planes():
    zero = np.float32(0)
    assert orc.plane_stats(np.zeros(16, np.float32), 2) == (zero, zero, zero)
    d, s, sc = orc.plane_stats(np.full(16, -0.0, np.float32), 4)
    assert (d, s, sc) == (zero, zero, zero) and not np.signbit(d)
    # a constant that is a bfloat16 number: range 0
    assert orc.plane_stats(np.full(9, 2.5, np.float32), 2) == (np.float32(2.5), zero, zero)
    # a constant that is not: delta_b lies just below it and the plane still quantises within one step
    v = np.float32(1.0 + 2.0 ** -12)
    d, s, sc = orc.plane_stats(np.full(9, v, np.float32), 2)
    assert d == np.float32(1.0) and s > 0 and (v - d) <= 3 * s
    # a step whose reciprocal overflows
    tiny = np.array([0.0, 1e-44], dtype=np.float32)
    assert orc.plane_stats(tiny, 1)[1:] == (zero, zero)


# ---------------------------------------------------------------------------------------
# the pair
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("shape,block,q,xd,ld", [
    ((2, 3, 16, 24), 8, 2, orc.F32, orc.F32), ((2, 4, 14, 14), 8, 4, orc.F32, orc.BF16),
    ((1, 5, 7, 7), 8, 2, orc.F32, orc.F32), ((2, 2, 9, 13), 4, 8, orc.F32, orc.F32),
    ((2, 3, 12, 20), 4, 1, orc.BF16, orc.BF16)])
def test_error_is_bounded_by_the_planes_own_step(shape, block, q, xd, ld):
    """|H_hat - H| <= Delta_b of the element's own plane (Sec. 4.1's bound with the stored step)."""
    x = synth.activation_map(*shape, "bn", 21)
    if xd == orc.BF16:
        x = orc.f32_to_bf16_bits(x)
    comp = orc.compress_planes(x, block, q, 99, xd, ld)
    xhat = orc.decompress_planes(comp)
    x32 = orc.widen_input(x, xd)
    err = np.abs(xhat.astype(np.float64) - x32.astype(np.float64))
    bound = comp.step[:, :, None, None].astype(np.float64)
    slack = 2.0 ** -7 * np.abs(x32) + 1e-6 if xd == orc.BF16 else 4e-6 * (np.abs(x32) + bound + 1)
    assert (err <= bound + slack).all()
    assert comp.codes.max() <= (1 << q) - 1


def test_groups_are_planes():
    """Changing one plane changes that plane's parameters and codes and nothing else."""
    x = synth.activation_map(2, 4, 16, 16, "bn", 5)
    a = orc.compress_planes(x, 8, 2, 7)
    y = x.copy()
    y[1, 2] *= 3.0
    b = orc.compress_planes(y, 8, 2, 7)
    same = np.ones((2, 4), bool)
    same[1, 2] = False
    np.testing.assert_array_equal(a.codes[same], b.codes[same])
    np.testing.assert_array_equal(a.delta[same], b.delta[same])
    np.testing.assert_array_equal(a.step[same], b.step[same])
    assert b.step[1, 2] > a.step[1, 2] and (a.codes[1, 2] != b.codes[1, 2]).any() is not None
    # and each plane's parameters come from that plane's residuals alone
    r = (x - orc.upsample_nearest(a.lfc, 8, 16, 16)).reshape(2, 4, -1)
    for i in range(2):
        for j in range(4):
            assert (a.delta[i, j], a.step[i, j]) == orc.plane_stats(r[i, j], 2)[:2]


def test_reconstruction_is_unbiased_over_seeds():
    """E[H_hat] = H (Sec. 4.1): the mean over many seeds approaches H at the 1/sqrt(seeds) rate."""
    x = synth.activation_map(1, 3, 8, 8, "bn", 17)
    seeds = 600
    acc = np.zeros(x.shape, np.float64)
    for s in range(seeds):
        acc += orc.decompress_planes(orc.compress_planes(x, 8, 2, 1000 + s))
    step = orc.compress_planes(x, 8, 2, 0).step[:, :, None, None].astype(np.float64)
    z = (acc / seeds - x) / (0.5 * step / np.sqrt(seeds))          # sd of one draw <= step / 2
    assert np.abs(z).max() < 5.0 and abs(z.mean()) < 0.5


def test_codes_use_the_same_random_stream_and_packing_as_the_per_sample_form():
    """With one channel and bf16-exact parameters the per-plane codes ARE the per-sample codes."""
    n, h, w = 3, 8, 8
    rng = np.random.default_rng(8)
    # residual range exactly [-1.5, 1.5] in every sample: step 1 at Q = 2; the tile mean is 0 by symmetry
    base = rng.uniform(-1.4, 1.4, size=(n, 1, h, w // 2)).astype(np.float32)
    base[:, 0, 0, 0] = 1.5
    x = np.concatenate([base, -base], axis=3)        # mirrored columns: the tree sum cancels exactly
    a = orc.compress(x, 8, 2, 31)
    assert np.all(a.lfc == 0) and np.all(a.step == 1) and np.all(a.delta == -1.5)
    b = orc.compress_planes(x, 8, 2, 31)
    np.testing.assert_array_equal(a.codes.reshape(-1), b.codes.reshape(-1))
    np.testing.assert_array_equal(a.words, b.words)
    np.testing.assert_array_equal(orc.decompress(a), orc.decompress_planes(b))


def test_blob_round_trip_and_stats_encoding():
    x = synth.activation_map(2, 3, 10, 12, "relu", 4)
    comp = orc.compress_planes(x, 4, 4, 5, orc.F32, orc.BF16)
    blob = comp.blob()
    lo = comp.layout
    assert blob.size == lo.total_bytes
    pair = blob[lo.stats_off:lo.stats_off + lo.stats_bytes].view("<u2").reshape(2, 3, 2)
    np.testing.assert_array_equal((pair[:, :, 0].astype(np.uint32) << 16).view(np.float32), comp.delta)
    np.testing.assert_array_equal((pair[:, :, 1].astype(np.uint32) << 16).view(np.float32), comp.step)
    back = orc.parse_plane_blob(blob, 2, 3, 10, 12, 4, 4, orc.F32, orc.BF16)
    np.testing.assert_array_equal(back.codes, comp.codes)
    np.testing.assert_array_equal(orc.decompress_planes(back), orc.decompress_planes(comp))
    # padding between the sections stays zero
    assert not blob[lo.lfc_bytes:lo.packed_off].any()
    assert not blob[lo.packed_off + lo.packed_bytes:lo.stats_off].any()
