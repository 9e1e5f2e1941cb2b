"""Parity of the CUDA library with the CPU checker, element by element, through the C ABI.

The bar (stated, not derived): packed codes, stored low-frequency values, (delta, Delta) and the
reconstruction are compared for EXACT equality -- both sides take every floating-point decision in
fp32 with the same operation order, so nothing is left to a tolerance.  (The looser acceptance bound
of the task -- off-by-one codes within 1 ulp of a rounding threshold at a rate <= 1e-6, 1e-6 / 1e-2
relative reconstruction error for fp32 / bf16 -- is therefore met with margin.)
"""
import numpy as np
import pytest
import torch

from oracle import division_oracle as orc
from paper_2208_04187_b200 import binding, build, synth

pytestmark = pytest.mark.gpu

TWO_PASS = binding.DIV_FLAG_FORCE_TWO_PASS
# the three single-launch kernels for W % 4 == 0: each flag set leaves exactly one of them in line
LAGGED = binding.DIV_FLAG_NO_STRIP_KERNEL | binding.DIV_FLAG_NO_STAGED_KERNEL
RING = binding.DIV_FLAG_NO_LAGGED_KERNEL | binding.DIV_FLAG_NO_STAGED_KERNEL
STAGED = binding.DIV_FLAG_NO_STRIP_KERNEL | binding.DIV_FLAG_NO_LAGGED_KERNEL
NO_SPECIAL = STAGED | binding.DIV_FLAG_NO_STAGED_KERNEL                     # small-plane kernels, else general ring
PLANES_PAIR = NO_SPECIAL | binding.DIV_FLAG_TWO_LAUNCH_PLANES               # the small-plane pair instead of the fused kernel
NO_STRIP = NO_SPECIAL | binding.DIV_FLAG_NO_PLANE_KERNELS                   # general ring, else two-pass


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


def split_blob(blob_np, lo, lfc_dtype):
    raw = blob_np[lo.lfc_off:lo.lfc_off + lo.lfc_bytes]
    lfc = raw.view("<f4").astype(np.float32) if lfc_dtype == "f32" else orc.bf16_bits_to_f32(raw.view("<u2"))
    words = blob_np[lo.packed_off:lo.packed_off + lo.packed_bytes].view("<u4")
    stats = blob_np[lo.stats_off:lo.stats_off + lo.stats_bytes].view("<f4").reshape(-1, 2)
    return lfc, words, stats


def run_gpu(x_np, block, qbits, seed, x_dtype="f32", lfc_dtype="f32", flags=0):
    n, c, h, w = x_np.shape
    codec = binding.Codec(n, c, h, w, block, qbits, x_dtype, lfc_dtype)
    xd = to_device(x_np, x_dtype)
    codec.compress(xd, seed=seed, flags=flags)
    xhat = codec.decompress()
    torch.cuda.synchronize()
    assert codec.device_status() == binding.DIV_OK
    return codec, codec.blob.cpu().numpy(), to_host_f32(xhat, x_dtype)


def assert_full_parity(x_np, block, qbits, seed, x_dtype="f32", lfc_dtype="f32", flags=0):
    ref = orc.compress(x_np, block, qbits, seed, x_dtype, lfc_dtype)
    codec, blob, xhat = run_gpu(x_np, block, qbits, seed, x_dtype, lfc_dtype, flags)
    lfc, words, stats = split_blob(blob, codec.layout, lfc_dtype)
    np.testing.assert_array_equal(lfc, ref.lfc.reshape(-1), err_msg="low-frequency values")
    np.testing.assert_array_equal(stats[:, 0], ref.delta, err_msg="delta")
    np.testing.assert_array_equal(stats[:, 1], ref.step, err_msg="Delta")
    bad = np.flatnonzero(words != ref.words)
    assert bad.size == 0, f"{bad.size} of {words.size} packed words differ, first at {bad[:5]}"
    np.testing.assert_array_equal(xhat, orc.decompress(ref), err_msg="reconstruction")
    return codec


# ----------------------------------------------------------------------------------------------
# small cases: several tiles, ragged tails, every Q, both dtypes, both compress paths
# ----------------------------------------------------------------------------------------------
SMALL = [
    # n, c, h, w, block, q, x_dtype, lfc_dtype
    (1, 2, 3, 3, 2, 2, "f32", "f32"),
    (1, 1, 1, 1, 8, 2, "f32", "f32"),
    (3, 5, 7, 9, 4, 1, "f32", "f32"),
    (2, 3, 5, 6, 1, 8, "f32", "f32"),
    (2, 16, 7, 7, 8, 2, "f32", "f32"),
    (2, 8, 14, 14, 8, 2, "f32", "f32"),
    (2, 4, 28, 28, 8, 2, "f32", "bf16"),
    (3, 4, 32, 32, 8, 2, "f32", "f32"),
    (2, 4, 32, 32, 8, 4, "f32", "f32"),
    (2, 4, 32, 32, 8, 8, "f32", "f32"),
    (2, 4, 32, 32, 8, 1, "f32", "f32"),
    (2, 4, 32, 32, 4, 2, "f32", "f32"),
    (2, 3, 40, 24, 16, 2, "f32", "f32"),
    (2, 2, 64, 48, 32, 4, "f32", "f32"),
    (2, 3, 36, 30, 12, 2, "f32", "f32"),
    (2, 3, 36, 54, 18, 2, "f32", "f32"),
    (2, 2, 70, 70, 64, 2, "f32", "f32"),
    (2, 3, 4, 4, 8, 2, "f32", "f32"),
    (2, 8, 32, 32, 8, 2, "bf16", "bf16"),
    (2, 8, 16, 16, 4, 4, "bf16", "bf16"),
    (2, 8, 14, 14, 8, 2, "bf16", "f32"),
    (3, 7, 5, 3, 4, 2, "bf16", "bf16"),
    (5, 2, 33, 17, 12, 2, "f32", "f32"),
    (1, 3, 112, 112, 8, 2, "f32", "f32"),
    # samples of at least 8 units of 32 strips: the lagged kernel takes these
    (3, 16, 32, 32, 8, 2, "f32", "f32"),
    (2, 24, 28, 28, 8, 2, "f32", "bf16"),
    (2, 32, 16, 16, 4, 4, "bf16", "bf16"),
    (2, 16, 32, 32, 8, 4, "f32", "f32"),
    (2, 16, 32, 32, 8, 8, "bf16", "f32"),
    (3, 20, 24, 40, 4, 2, "f32", "f32"),
    (2, 9, 36, 20, 8, 2, "f32", "f32"),
    (5, 11, 12, 52, 8, 2, "bf16", "bf16"),
    # small planes of odd width: the pair of plane kernels
    (3, 12, 14, 14, 8, 2, "f32", "f32"),
    (2, 20, 7, 7, 8, 2, "f32", "bf16"),
    (2, 8, 14, 14, 8, 4, "bf16", "bf16"),
    (2, 4, 13, 9, 4, 2, "f32", "f32"),
    (3, 4, 21, 27, 16, 8, "f32", "f32"),
    (2, 8, 7, 7, 4, 2, "bf16", "f32"),
    (1, 4, 30, 10, 8, 2, "f32", "f32"),
]


def small_input(n, c, h, w, x_dtype, seed):
    x = synth.activation_map(n, c, h, w, "relu" if seed % 2 else "bn", 9000 + seed)
    return synth.to_bf16_bits(x) if x_dtype == "bf16" else x


@pytest.mark.parametrize("case", SMALL, ids=lambda c: "x".join(map(str, c)))
@pytest.mark.parametrize("flags", [0, RING, LAGGED, STAGED, NO_SPECIAL, PLANES_PAIR, NO_STRIP, TWO_PASS],
                         ids=["default", "strip_ring", "lagged", "staged", "planes", "planes_pair", "general_ring", "two_pass"])
def test_small_cases_match_the_checker(case, flags):
    n, c, h, w, block, q, xd, ld = case
    x = small_input(n, c, h, w, xd, seed=n + c + h + w + block + q)
    assert_full_parity(x, block, q, seed=1234567, x_dtype=xd, lfc_dtype=ld, flags=flags)


def planes_shape(case):
    n, c, h, w, block, q, xd, ld = case
    b = min(block, max(h, w))
    p2 = 1
    while p2 < b:
        p2 *= 2
    wb = -(-w // b)
    return q in (2, 4, 8) and p2 in (4, 8, 16) and wb * p2 <= 32 and (c * h * w) % 4 == 0 and h * w <= 8192


def test_fused_path_is_taken_where_expected():
    """Guards against silently testing only the general kernels."""
    fused = {case: binding.div_plan_query(binding.make_desc(*case)).fused for case in SMALL}
    lagged = {case: binding.div_plan_query(binding.make_desc(*case), LAGGED).fused for case in SMALL}
    staged = {case: binding.div_plan_query(binding.make_desc(*case), STAGED).fused for case in SMALL}
    special = {case: binding.div_plan_query(binding.make_desc(*case), NO_SPECIAL).fused for case in SMALL}
    for case in SMALL:
        n, c, h, w, block, q, xd, ld = case
        strip_shape = w % 4 == 0 and min(block, max(h, w)) in (4, 8) and q in (2, 4, 8)
        if strip_shape:
            # narrow planes (W <= 32 for B = 8) take the fused small-plane kernel by default, wider ones a strip kernel
            assert fused[case] == (7 if planes_shape(case) else 2) and lagged[case] == 3, case
            # bulk copies need every sample, plane and band to start on a 16-byte boundary
            sx = 4 if xd == "f32" else 2
            b = min(block, max(h, w))
            aligned = (c * h * w * sx) % 16 == 0 and (h * w * sx) % 16 == 0 and (b * w * sx) % 16 == 0
            assert staged[case] == (6 if aligned else (7 if planes_shape(case) else 1)), case
        elif planes_shape(case):
            assert fused[case] == 7 and lagged[case] == 7 and staged[case] == 7, case
            assert binding.div_plan_query(binding.make_desc(*case), PLANES_PAIR).fused == 4, case
        else:
            assert fused[case] in (0, 1) and lagged[case] == fused[case] and staged[case] == fused[case], case
        assert special[case] == (7 if planes_shape(case) else binding.div_plan_query(binding.make_desc(*case), NO_STRIP).fused), case
    assert sum(1 for c in SMALL if fused[c] == 2) >= 2
    assert sum(1 for c in SMALL if binding.div_plan_query(binding.make_desc(*c), RING).fused == 2) >= 12
    assert sum(1 for c in SMALL if staged[c] == 6) >= 12
    assert sum(1 for c in SMALL if fused[c] == 7) >= 15
    assert sum(1 for c in SMALL if special[c] == 7) >= 12
    assert fused[(2, 4, 32, 32, 8, 1, "f32", "f32")] == 1          # Q = 1: general ring kernel
    assert fused[(2, 8, 14, 14, 8, 2, "f32", "f32")] == 7
    assert fused[(2, 16, 7, 7, 8, 2, "f32", "f32")] == 7
    assert fused[(2, 3, 40, 24, 16, 2, "f32", "f32")] == 7
    assert binding.div_plan_query(binding.make_desc(3, 4, 32, 32, 8, 2), NO_STRIP).fused == 1
    assert fused[(1, 2, 3, 3, 2, 2, "f32", "f32")] == 0          # sample is not a whole number of words
    assert fused[(2, 2, 70, 70, 64, 2, "f32", "f32")] == 0        # block wider than a warp
    for spec in synth.config2() + synth.config1() + synth.config3():
        d = binding.make_desc(*spec.shape, spec.block, spec.qbits, spec.x_dtype, spec.lfc_dtype)
        nbytes = spec.numel * (4 if spec.x_dtype == "f32" else 2)
        first = 6 if (nbytes >= 56 * 2 ** 20 and spec.block == 8) else (3 if nbytes >= 20 * 2 ** 20 else 2)
        narrow = planes_shape((*spec.shape, spec.block, spec.qbits, spec.x_dtype, spec.lfc_dtype))
        if narrow and nbytes < 56 * 2 ** 20 and not (spec.x_dtype == "bf16" and nbytes >= 32 * 2 ** 20):
            first = 7
        assert binding.div_plan_query(d).fused == (first if spec.w % 4 == 0 else 7), spec.label()
        assert binding.div_plan_query(d, LAGGED).fused == (3 if spec.w % 4 == 0 else 7), spec.label()
        assert binding.div_plan_query(d, RING).fused == (2 if spec.w % 4 == 0 else 7), spec.label()
        assert binding.div_plan_query(d, STAGED).fused == (6 if spec.w % 4 == 0 else 7), spec.label()
        assert binding.div_plan_query(d).decompress_fast == (1 if spec.w % 4 == 0 else 2)


def test_decompress_reads_a_checker_blob():
    """The two directions are independent: the GPU decodes a buffer the CPU checker wrote."""
    for (shape, block, q, xd, ld) in [((2, 4, 28, 28), 8, 2, "f32", "f32"), ((2, 6, 14, 14), 8, 4, "bf16", "bf16"),
                                      ((3, 5, 7, 9), 4, 1, "f32", "bf16")]:
        x = small_input(*shape, xd, seed=5)
        ref = orc.compress(x, block, q, 77, xd, ld)
        codec = binding.Codec(*shape, block, q, xd, ld)
        codec.blob.copy_(torch.from_numpy(ref.blob()))
        xhat = to_host_f32(codec.decompress(), xd)
        np.testing.assert_array_equal(xhat, orc.decompress(ref))


def test_degenerate_inputs():
    # constant tensor: residual identically zero, Delta = 0, exact reconstruction
    x = np.full((2, 4, 16, 16), 1.7, dtype=np.float32)
    for flags in (0, RING, LAGGED, STAGED, TWO_PASS):
        codec, blob, xhat = run_gpu(x, 8, 2, 3, flags=flags)
        lfc, words, stats = split_blob(blob, codec.layout, "f32")
        assert not words.any() and not stats.any()
        np.testing.assert_array_equal(xhat, x)
    # all zeros, and B = 1
    assert_full_parity(np.zeros((2, 4, 16, 16), dtype=np.float32), 8, 2, 0)
    x = small_input(2, 4, 8, 8, "f32", 3)
    codec = assert_full_parity(x, 1, 2, 0)
    # large magnitudes and denormal-scale values stay finite and in parity
    assert_full_parity(small_input(2, 4, 16, 16, "f32", 4) * np.float32(1e30), 8, 2, 0)
    assert_full_parity(small_input(2, 4, 16, 16, "f32", 5) * np.float32(1e-35), 8, 2, 0)


def test_same_seed_same_bytes_other_seed_other_codes():
    spec = synth.config0()[0]
    x = synth.make_input(spec)
    xd = to_device(x, "f32")
    codec = binding.Codec(*spec.shape, spec.block, spec.qbits)
    a = codec.compress(xd, seed=9).clone()
    b = codec.compress(xd, seed=9).clone()
    c = codec.compress(xd, seed=10).clone()
    t = codec.compress(xd, seed=9, flags=TWO_PASS).clone()
    torch.cuda.synchronize()
    assert torch.equal(a, b) and torch.equal(a, t)
    lo = codec.layout
    la, wa, sa = split_blob(a.cpu().numpy(), lo, "f32")
    lc, wc, sc = split_blob(c.cpu().numpy(), lo, "f32")
    np.testing.assert_array_equal(la, lc)
    np.testing.assert_array_equal(sa, sc)
    assert (wa != wc).mean() > 0.5


@pytest.mark.parametrize("flags", [RING, LAGGED, STAGED, NO_SPECIAL], ids=["strip_ring", "lagged", "staged", "planes_fused"])
def test_a_wait_that_cannot_end_gives_up_and_reports_it(flags):
    """Failure detection without a fault: the kernel waits for arrivals that never come, its 2 ms limit
    runs out, it records the timeout in the status word and returns; the context stays usable."""
    import ctypes
    spec = synth.config0()[0]
    if flags == NO_SPECIAL:
        spec = synth.TensorSpec(0, 0, 8, 64, 14, 14, "relu", "f32", "f32", 8, 2)      # a small-plane map
    x = to_device(synth.make_input(spec), "f32")
    codec = binding.Codec(*spec.shape, spec.block, spec.qbits)
    assert codec.plan(flags).fused == {RING: 2, LAGGED: 3, STAGED: 6, NO_SPECIAL: 7}[flags]
    st = binding.lib().div_debug_compress_starved(
        ctypes.byref(codec.desc), ctypes.c_void_p(x.data_ptr()), ctypes.c_void_p(codec.blob.data_ptr()), codec.blob.numel(),
        ctypes.c_void_p(codec.workspace.data_ptr()), codec.workspace.numel(), 0, ctypes.c_void_p(binding.current_stream_handle()),
        flags, 2_000_000)
    assert st == binding.DIV_OK
    torch.cuda.synchronize()
    assert codec.device_status() == binding.DIV_ERR_TIMEOUT
    # the next ordinary call on the same buffers works and is correct
    ref = orc.compress(synth.make_input(spec), spec.block, spec.qbits, 5)
    codec.compress(x, seed=5, flags=flags)
    torch.cuda.synchronize()
    assert codec.device_status() == binding.DIV_OK
    _, words, _ = split_blob(codec.blob.cpu().numpy(), codec.layout, "f32")
    np.testing.assert_array_equal(words, ref.words)


def test_guard_bands_stay_untouched():
    """Sentinel bytes around every output buffer survive both calls (no out-of-bounds write)."""
    for case in [(2, 8, 14, 14, 8, 2, "f32", "f32"), (3, 4, 32, 32, 8, 2, "f32", "f32"), (3, 5, 7, 9, 4, 1, "f32", "f32"),
                 (2, 8, 32, 32, 8, 2, "bf16", "bf16")]:
        n, c, h, w, block, q, xd, ld = case
        for flags in (0, RING, LAGGED, STAGED, NO_SPECIAL, PLANES_PAIR, NO_STRIP, TWO_PASS):
            x = small_input(n, c, h, w, xd, seed=7)
            codec = binding.Codec(n, c, h, w, block, q, xd, ld)
            pad = 4096
            total = int(codec.layout.total_bytes)
            big = torch.full((total + 2 * pad,), 0xA5, dtype=torch.uint8, device="cuda")
            inner = big[pad:pad + total]
            codec.compress(to_device(x, xd), seed=1, flags=flags, blob=inner)
            nbytes = x.size * (4 if xd == "f32" else 2)
            out_big = torch.full((nbytes + 2 * pad,), 0x5A, dtype=torch.uint8, device="cuda")
            out = out_big[pad:pad + nbytes].view(binding.torch_dtype(xd)).view(n, c, h, w)
            codec.decompress(blob=inner, out=out)
            torch.cuda.synchronize()
            assert bool((big[:pad] == 0xA5).all()) and bool((big[pad + total:] == 0xA5).all())
            assert bool((out_big[:pad] == 0x5A).all()) and bool((out_big[pad + nbytes:] == 0x5A).all())
            lo = codec.layout
            gap1 = inner[lo.lfc_off + lo.lfc_bytes:lo.packed_off]
            gap2 = inner[lo.packed_off + lo.packed_bytes:lo.stats_off]
            assert bool((gap1 == 0xA5).all()) and bool((gap2 == 0xA5).all())


# ----------------------------------------------------------------------------------------------
# the five workload configurations at full size
# ----------------------------------------------------------------------------------------------
def assert_sampled_parity(spec, seed, sample_ids, flags=0):
    """Compress the whole tensor on the GPU; the checker recomputes whole samples of it (samples are
    independent units: per-sample statistics, random stream keyed by the sample's index)."""
    x = synth.make_input(spec)
    codec, blob, xhat = run_gpu(x, spec.block, spec.qbits, seed, spec.x_dtype, spec.lfc_dtype, flags)
    lfc, words, stats = split_blob(blob, codec.layout, spec.lfc_dtype)
    chw = spec.c * spec.h * spec.w
    hb, wb = orc.grid_shape(spec.h, spec.w, spec.block)
    tps = spec.c * hb * wb
    wps = chw * spec.qbits // 32
    assert chw * spec.qbits % 32 == 0
    for i in sample_ids:
        ref = orc.compress(x[i:i + 1], spec.block, spec.qbits, seed, spec.x_dtype, spec.lfc_dtype, first_sample=i)
        np.testing.assert_array_equal(lfc[i * tps:(i + 1) * tps], ref.lfc.reshape(-1), err_msg=f"lfc, sample {i}")
        np.testing.assert_array_equal(stats[i], [ref.delta[0], ref.step[0]], err_msg=f"stats, sample {i}")
        bad = np.flatnonzero(words[i * wps:(i + 1) * wps] != ref.words)
        assert bad.size == 0, f"sample {i}: {bad.size} of {wps} packed words differ"
        np.testing.assert_array_equal(xhat[i:i + 1], orc.decompress(ref), err_msg=f"reconstruction, sample {i}")
    # properties that hold at any size: every sample reconstructs within one quantisation step
    x32 = orc.widen_input(x, spec.x_dtype)
    err = np.abs(xhat - x32).reshape(spec.n, -1).max(axis=1)
    slack = 2.0 ** -7 * np.abs(x32).reshape(spec.n, -1).max(axis=1) if spec.x_dtype == "bf16" else 1e-6
    assert np.all(err <= stats[:, 1] * (1 + 1e-5) + slack)
    assert np.all(stats[:, 1] > 0)


def test_config0_full():
    spec = synth.config0()[0]
    x = synth.make_input(spec)
    for flags in (0, RING, LAGGED, STAGED, NO_SPECIAL, NO_STRIP, TWO_PASS):
        assert_full_parity(x, spec.block, spec.qbits, 0, flags=flags)


@pytest.mark.parametrize("spec", synth.config1(), ids=lambda s: s.label())
def test_config1_resnet18_cifar(spec):
    x = synth.make_input(spec)
    assert_full_parity(x, spec.block, spec.qbits, 0)


@pytest.mark.parametrize("spec", synth.config2(), ids=lambda s: s.label())
def test_config2_resnet50_imagenet(spec):
    # the two 205 MB maps (the kernel the benchmark's roofline figure is about): every sample against the checker
    assert_sampled_parity(spec, 0, range(spec.n) if spec.index < 2 else [0, 31, 63])


@pytest.mark.parametrize("flags,code", [(0, 6), (LAGGED, 3), (RING, 2)], ids=["staged", "lagged", "strip_ring"])
def test_full_size_output_does_not_depend_on_timing(flags, code):
    """The single-launch kernels hand out work by timing (claim counters, whoever closes a chunk last); the output
    must not depend on it: the same call twice on a full-size map gives byte-identical blobs."""
    spec = synth.config2()[1]
    x = to_device(synth.make_input(spec), spec.x_dtype)
    codec = binding.Codec(*spec.shape, spec.block, spec.qbits)
    assert codec.plan(flags).fused == code
    first = codec.compress(x, seed=3, flags=flags).clone()
    second = codec.compress(x, seed=3, flags=flags).clone()
    third = codec.compress(x.clone(), seed=3, flags=flags)
    torch.cuda.synchronize()
    assert codec.device_status() == binding.DIV_OK
    assert torch.equal(first, second) and torch.equal(first, third)


def test_block_sum_order_on_every_path():
    """A tile on which the documented summation order (trees down the rows of each column, then across the columns),
    the rows-first order and a running sum round differently in fp32, planted among ordinary tiles."""
    big = np.float32(2.0 ** 24)
    tile = np.zeros((8, 8), dtype=np.float32)
    tile[:4, 0] = [1, big, 1, -big]
    tile[:4, 1] = [1, 0, 1, 0]
    x = small_input(3, 16, 32, 32, "f32", 8)
    x[0, 0, 0:8, 0:8] = tile
    x[1, 7, 8:16, 24:32] = tile
    x[2, 15, 24:32, 16:24] = tile.T
    for flags in (0, RING, LAGGED, STAGED, NO_SPECIAL, NO_STRIP, TWO_PASS):
        codec = assert_full_parity(x, 8, 2, seed=5, flags=flags)
        lfc, _, _ = split_blob(codec.blob.cpu().numpy(), codec.layout, "f32")
        assert lfc.reshape(3, 16, 4, 4)[0, 0, 0, 0] == np.float32(3.0 / 64.0)


def test_config2_other_paths_on_one_tensor():
    assert_sampled_parity(synth.config2()[2], 0, [0, 63], flags=TWO_PASS)
    assert_sampled_parity(synth.config2()[2], 0, [0, 63], flags=NO_STRIP)
    assert_sampled_parity(synth.config2()[2], 0, [0, 63], flags=LAGGED)
    assert_sampled_parity(synth.config2()[2], 0, [0, 63], flags=RING)
    assert_sampled_parity(synth.config2()[2], 0, [0, 63], flags=STAGED)
    assert_sampled_parity(synth.config2()[3], 0, [0, 63], flags=PLANES_PAIR)
    assert_sampled_parity(synth.config2()[4], 0, [0, 63], flags=PLANES_PAIR)
    assert_sampled_parity(synth.config2()[0], 0, [17], flags=RING)


@pytest.mark.parametrize("spec", synth.config3(), ids=lambda s: s.label())
def test_config3_wrn_bf16(spec):
    assert_sampled_parity(spec, 0, [0, 77, 127])


@pytest.mark.parametrize("spec", synth.config4(), ids=lambda s: s.label())
def test_config4_densenet_sweep(spec):
    assert_sampled_parity(spec, 0, [0, 63])
