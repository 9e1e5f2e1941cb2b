"""Parity of the per-plane form (one bfloat16 (delta, Delta) pair per (sample, channel) plane; Sec. 4.1 byte
count, proof of Theorem 3A) with the CPU checker, through the C ABI.  Exact equality throughout: stored
low-frequency values, the bfloat16 pairs, every packed word, the whole blob, the reconstruction.
"""
import numpy as np
import pytest
import torch

from oracle import division_oracle as orc
from paper_2208_04187_b200 import binding, build, synth

pytestmark = pytest.mark.gpu

GENERAL = binding.DIV_FLAG_FORCE_TWO_PASS


@pytest.fixture(scope="module", autouse=True)
def built_library():
    build.build()
    binding.lib()


def to_device(x_np, x_dtype):
    t = torch.from_numpy(x_np)
    if x_dtype == "bf16":
        t = t.view(torch.bfloat16)
    return t.cuda()


def to_host_f32(t, x_dtype):
    if x_dtype == "bf16":
        return orc.bf16_bits_to_f32(t.view(torch.int16).cpu().numpy().view(np.uint16))
    return t.cpu().numpy()


def make_input(shape, kind, seed, x_dtype):
    x = synth.activation_map(*shape, kind, seed)
    return orc.f32_to_bf16_bits(x) if x_dtype == "bf16" else x


def assert_parity(x_np, block, qbits, seed, x_dtype="f32", lfc_dtype="f32", flags=0, expect_fused=None):
    n, c, h, w = x_np.shape
    ref = orc.compress_planes(x_np, block, qbits, seed, x_dtype, lfc_dtype)
    codec = binding.PlaneGroupCodec(n, c, h, w, block, qbits, x_dtype, lfc_dtype)
    if expect_fused is not None:
        assert codec.plan(flags).fused == expect_fused
    lo = codec.layout
    assert (lo.total_bytes, lo.closed_form_bytes, lo.stats_off, lo.stats_bytes, lo.workspace_bytes) == \
           (ref.layout.total_bytes, ref.layout.closed_form_bytes, ref.layout.stats_off, ref.layout.stats_bytes, 0)
    codec.blob.fill_(0xA5)                       # stale bytes must not leak into the packed words
    codec.blob[lo.lfc_bytes:lo.packed_off] = 0   # (the padding between sections is never written)
    codec.blob[lo.packed_off + lo.packed_bytes:lo.stats_off] = 0
    codec.compress(to_device(x_np, x_dtype), seed=seed, flags=flags)
    xhat = codec.decompress()
    torch.cuda.synchronize()
    got = orc.parse_plane_blob(codec.blob.cpu().numpy(), n, c, h, w, block, qbits, x_dtype, lfc_dtype)
    np.testing.assert_array_equal(got.lfc, ref.lfc, err_msg="low-frequency values")
    np.testing.assert_array_equal(got.delta, ref.delta, err_msg="delta_b")
    np.testing.assert_array_equal(got.step, ref.step, err_msg="Delta_b")
    bad = np.flatnonzero(got.words != ref.words)
    assert bad.size == 0, f"{bad.size} of {ref.words.size} packed words differ, first at {bad[:5]}"
    np.testing.assert_array_equal(codec.blob.cpu().numpy(), ref.blob(), err_msg="blob bytes")
    np.testing.assert_array_equal(to_host_f32(xhat, x_dtype), orc.decompress_planes(ref), err_msg="reconstruction")
    return codec


# shapes the strip kernel takes: W % 4 == 0, B in {4, 8}, Q in {2, 4, 8}; ragged rows and column tiles included
STRIP = [
    ((2, 3, 16, 16), 8, 2, "f32", "f32"), ((3, 5, 56, 56), 8, 2, "f32", "f32"), ((2, 2, 112, 112), 8, 2, "f32", "f32"),
    ((2, 7, 28, 28), 8, 4, "f32", "bf16"), ((2, 3, 20, 12), 8, 8, "f32", "f32"), ((3, 4, 13, 20), 4, 2, "bf16", "bf16"),
    ((2, 600, 4, 4), 4, 2, "f32", "f32"), ((1, 1, 8, 8), 8, 2, "f32", "f32"), ((2, 9, 30, 36), 8, 4, "bf16", "f32"),
    ((1, 3, 128, 128), 8, 2, "f32", "f32"), ((5, 11, 8, 24), 4, 8, "f32", "bf16"), ((2, 130, 8, 8), 8, 2, "f32", "f32"),
    ((1, 3, 1, 4), 4, 2, "f32", "f32"),          # 12 elements: the last packed word is partial
]
# shapes the small-plane kernel takes: any width, padded tile row of at most 32 columns, sample size a multiple of 4
SMALL_PLANE = [
    ((2, 8, 14, 14), 8, 2, "f32", "f32"), ((3, 16, 7, 7), 8, 2, "f32", "f32"), ((2, 4, 9, 13), 4, 4, "f32", "f32"),
    ((2, 40, 7, 7), 8, 4, "bf16", "bf16"), ((1, 4, 6, 10), 3, 2, "bf16", "f32"), ((2, 3, 12, 20), 12, 2, "f32", "bf16"),
    ((130, 12, 14, 14), 8, 8, "f32", "f32"), ((5, 100, 7, 7), 8, 2, "f32", "bf16"), ((2, 6, 30, 30), 16, 2, "f32", "f32"),
    ((3, 700, 2, 6), 4, 2, "f32", "f32"),
]
# shapes only the general kernel takes (sample size not a multiple of 4, other block sizes, Q = 1, wide odd planes)
GENERAL_ONLY = [
    ((2, 3, 7, 7), 8, 2, "f32", "f32"), ((2, 5, 7, 7), 8, 2, "f32", "f32"), ((2, 3, 9, 13), 4, 4, "f32", "f32"),
    ((1, 4, 16, 16), 8, 1, "f32", "f32"), ((2, 3, 13, 50), 8, 2, "f32", "bf16"), ((3, 3, 5, 5), 16, 8, "bf16", "bf16"),
    ((1, 2, 160, 160), 8, 2, "f32", "f32"), ((2, 2, 3, 1), 2, 1, "f32", "f32"), ((1, 8, 6, 10), 64, 1, "bf16", "f32"),
]


@pytest.mark.parametrize("shape,block,q,xd,ld", STRIP)
@pytest.mark.parametrize("kind", ["bn", "relu"])
def test_strip_kernel_matches_the_checker(shape, block, q, xd, ld, kind):
    assert_parity(make_input(shape, kind, 31, xd), block, q, 77, xd, ld, expect_fused=1)


@pytest.mark.parametrize("shape,block,q,xd,ld", SMALL_PLANE)
@pytest.mark.parametrize("kind", ["bn", "relu"])
def test_small_plane_kernel_matches_the_checker(shape, block, q, xd, ld, kind):
    codec = assert_parity(make_input(shape, kind, 34, xd), block, q, 80, xd, ld, expect_fused=2)
    assert codec.plan().decompress_fast == 2


@pytest.mark.parametrize("shape,block,q,xd,ld", STRIP + SMALL_PLANE + GENERAL_ONLY)
def test_general_kernel_matches_the_checker(shape, block, q, xd, ld):
    assert_parity(make_input(shape, "bn", 32, xd), block, q, 78, xd, ld, flags=GENERAL, expect_fused=0)


@pytest.mark.parametrize("shape,block,q,xd,ld", GENERAL_ONLY)
def test_default_path_on_shapes_outside_the_special_kernels(shape, block, q, xd, ld):
    assert_parity(make_input(shape, "relu", 33, xd), block, q, 79, xd, ld, expect_fused=0)


def test_degenerate_planes_store_a_zero_step():
    x = synth.activation_map(2, 4, 16, 16, "bn", 5)
    x[0, 1] = 0.0              # all-zero plane
    x[1, 2] = 3.25             # constant plane: residual 0
    x[1, 3, :8] = 1.0          # constant tiles
    x[1, 3, 8:] = -2.0
    for flags in (0, GENERAL):
        codec = assert_parity(x, 8, 2, 5, flags=flags)
        got = orc.parse_plane_blob(codec.blob.cpu().numpy(), 2, 4, 16, 16, 8, 2)
        assert got.step[0, 1] == 0 and got.step[1, 2] == 0 and got.step[1, 3] == 0
        assert not got.codes[0, 1].any() and not got.codes[1, 2].any()
    # the same on planes of the small-plane kernel
    y = synth.activation_map(2, 4, 14, 14, "bn", 5)
    y[0, 1] = 0.0
    y[1, 2] = 3.25
    assert_parity(y, 8, 2, 5, expect_fused=2)


def test_extreme_magnitudes():
    x = synth.activation_map(2, 3, 16, 16, "bn", 6)
    x[0, 0] *= 1e30
    x[0, 1] *= 1e-30
    x[1, 0] *= 1e-42           # subnormal residuals
    x[1, 1, 0, 0] = 1.5e38
    x[1, 1, 0, 1] = -1.5e38    # range close to the largest fp32 number, reciprocal of the step subnormal
    for flags in (0, GENERAL):
        assert_parity(x, 8, 2, 9, flags=flags)
    assert_parity(x[:, :2, :14, :14].copy(), 8, 2, 9, expect_fused=2)


def test_outputs_do_not_depend_on_the_kernel():
    x = synth.activation_map(3, 6, 24, 16, "relu", 8)
    a = binding.PlaneGroupCodec(3, 6, 24, 16, 8, 2)
    b = binding.PlaneGroupCodec(3, 6, 24, 16, 8, 2)
    xd = torch.from_numpy(x).cuda()
    a.compress(xd, seed=3)
    b.compress(xd, seed=3, flags=GENERAL)
    torch.cuda.synchronize()
    assert torch.equal(a.blob, b.blob)


def test_argument_checks():
    desc = binding.make_desc(2, 3, 16, 16, 8, 2)
    lo = binding.div_planegroup_bytes(desc)
    x = torch.zeros(2, 3, 16, 16, device="cuda")
    blob = torch.zeros(int(lo.total_bytes), dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.DivisionError) as e:
        binding.div_planegroup_compress(desc, x.data_ptr(), blob.data_ptr(), int(lo.total_bytes) - 1, 0)
    assert e.value.status == binding.DIV_ERR_CAPACITY
    with pytest.raises(binding.DivisionError) as e:
        binding.div_planegroup_compress(desc, x.data_ptr() + 4, blob.data_ptr(), int(lo.total_bytes), 0)
    assert e.value.status == binding.DIV_ERR_ALIGN
    with pytest.raises(binding.DivisionError) as e:
        binding.div_planegroup_compress(desc, x.data_ptr(), blob.data_ptr(), int(lo.total_bytes), 0, flags=2)
    assert e.value.status == binding.DIV_ERR_PARAM
    with pytest.raises(binding.DivisionError) as e:
        binding.div_planegroup_decompress(desc, blob.data_ptr(), int(lo.total_bytes) - 1, x.data_ptr())
    assert e.value.status == binding.DIV_ERR_CAPACITY


@pytest.mark.parametrize("cfg", [1, 2, 3])
def test_benchmark_shaped_maps(cfg):
    """Maps of the workload configurations at their full spatial size and dtype; two samples and up to 24
    channels of each are checked whole against the checker (planes are independent of one another)."""
    seen = set()
    for spec in synth.config_specs(cfg):
        key = (spec.h, spec.w, spec.block, spec.qbits, spec.x_dtype)
        if key in seen:
            continue
        seen.add(key)
        x = synth.activation_map(2, min(spec.c, 24), spec.h, spec.w, spec.kind, 40 + cfg)
        if spec.x_dtype == "bf16":
            x = orc.f32_to_bf16_bits(x)
        assert_parity(x, spec.block, spec.qbits, 11, spec.x_dtype, spec.lfc_dtype)
