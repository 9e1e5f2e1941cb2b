"""div_compress_static: the compress call for callers that cannot allocate device memory.

Some users of this library run where a device allocation is off limits at the moment they compress (inside
another framework's callback, with the memory budget already handed out, or in a loop that must not pay for
a device-synchronising cudaMalloc).  For them the library carries its own fixed scratch array.  These tests
call that entry point through the C ABI several times in a row, on maps that take each of the single-launch
compress kernels, and check every result against the CPU checker and, byte for byte, against what the
ordinary div_compress writes for the same input and seed (the bar of the other parity tests): the fixed
array's stale contents from one call (claim counters, arrival counts, published parameters) must not leak
into the next.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import division_oracle as orc
from paper_2208_04187_b200 import binding, build, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built_library():
    build.build()
    binding.lib()


def _reference_blob(x, desc_args, seed):
    codec = binding.Codec(*desc_args)
    codec.compress(x, seed=seed)
    torch.cuda.synchronize()
    assert codec.device_status() == binding.DIV_OK
    return codec, codec.blob.clone()


def _sections(blob, lo):
    return (blob[lo.lfc_off:lo.lfc_off + lo.lfc_bytes], blob[lo.packed_off:lo.packed_off + lo.packed_bytes],
            blob[lo.stats_off:lo.stats_off + lo.stats_bytes])


def _assert_equals_checker(blob, layout, x_np, block, qbits, seed, samples):
    """The blob's sections for the given samples equal what the CPU checker computes for them."""
    n, c, h, w = x_np.shape
    host = blob.cpu().numpy()
    lfc = host[layout.lfc_off:layout.lfc_off + layout.lfc_bytes].view("<f4")
    words = host[layout.packed_off:layout.packed_off + layout.packed_bytes].view("<u4")
    stats = host[layout.stats_off:layout.stats_off + layout.stats_bytes].view("<f4").reshape(-1, 2)
    hb, wb = orc.grid_shape(h, w, block)
    tps, wps = c * hb * wb, c * h * w * qbits // 32
    for i in samples:
        ref = orc.compress(x_np[i:i + 1], block, qbits, seed, first_sample=i)
        np.testing.assert_array_equal(lfc[i * tps:(i + 1) * tps], ref.lfc.reshape(-1))
        np.testing.assert_array_equal(stats[i], [ref.delta[0], ref.step[0]])
        np.testing.assert_array_equal(words[i * wps:(i + 1) * wps], ref.words)


def test_static_scratch_matches_the_checker_and_div_compress_on_calls_in_a_row():
    stream = binding.current_stream_handle()
    # four maps of different shapes, one per compress path that keeps state in the scratch, so that every call
    # finds another kernel's leftovers in the shared array
    cases = [
        ("strip ring kernel", synth.activation_map(8, 16, 64, 64, "relu", 4246), 8, 2, 2),           # planes too wide for the small-plane kernel
        ("fused small-plane kernel", synth.activation_map(5, 24, 14, 14, "relu", 4242), 8, 2, 7),
        ("lagged kernel", synth.activation_map(8, 64, 112, 112, "relu", 4243), 8, 2, 3),             # 25.7 MB
        ("staged kernel", synth.activation_map(20, 64, 112, 112, "relu", 4244), 8, 2, 6),            # 64.2 MB
    ]
    prepared = []
    for name, x_np, block, qbits, plan_code in cases:
        args = (*x_np.shape, block, qbits)
        x = torch.from_numpy(x_np).cuda()
        codec, want = _reference_blob(x, args, seed=11)
        assert codec.plan().fused == plan_code, name
        prepared.append((name, x_np, x, codec, want, block, qbits))

    # back to back on one stream: every map, then every map again in reverse order
    order = list(range(len(prepared))) + list(reversed(range(len(prepared))))
    outputs = []
    for i in order:
        name, x_np, x, codec, want, block, qbits = prepared[i]
        got = torch.full_like(want, 0xEE)
        binding.div_compress_static(codec.desc, x.data_ptr(), got.data_ptr(), got.numel(), 11, stream)
        outputs.append((i, got))
    torch.cuda.synchronize()
    assert binding.div_read_static_status(stream) == binding.DIV_OK

    for i, got in outputs:
        name, x_np, x, codec, want, block, qbits = prepared[i]
        for g, w in zip(_sections(got, codec.layout), _sections(want, codec.layout)):
            assert torch.equal(g, w), name
        n = x_np.shape[0]
        _assert_equals_checker(got, codec.layout, x_np, block, qbits, 11, sorted({0, n // 2, n - 1}))
    # and the result decodes like any other blob
    name, x_np, x, codec, want, block, qbits = prepared[0]
    xhat = codec.decompress(blob=outputs[-1][1])
    xref = codec.decompress(blob=want)
    torch.cuda.synchronize()
    assert torch.equal(xhat, xref)


def test_static_status_word_is_readable_through_its_accessor():
    """The device-side status of a static call (a bounded wait that ran out would show here) can be read without
    knowing where the library keeps its array; bad arguments are refused."""
    stream = binding.current_stream_handle()
    spec = synth.config0()[0]
    x_np = synth.make_input(spec)
    x = torch.from_numpy(x_np).cuda()
    codec = binding.Codec(*spec.shape, spec.block, spec.qbits)
    got = torch.zeros_like(codec.blob)
    binding.div_compress_static(codec.desc, x.data_ptr(), got.data_ptr(), got.numel(), 5, stream)
    torch.cuda.synchronize()
    assert binding.div_read_static_status(stream) == binding.DIV_OK
    _assert_equals_checker(got, codec.layout, x_np, spec.block, spec.qbits, 5, range(spec.n))
    out = ctypes.c_int32(-1)
    assert binding.lib().div_read_static_status(None, None) == binding.DIV_ERR_NULL
    assert binding.lib().div_read_static_status(ctypes.c_void_p(stream), ctypes.byref(out)) == binding.DIV_OK and out.value == 0


def test_static_scratch_refuses_more_samples_than_it_has_slots_for():
    L = binding.lib()
    n = binding.DIV_STATIC_MAX_SAMPLES + 1
    d = binding.make_desc(n, 1, 8, 8, 8, 2)
    lo = binding.div_compressed_bytes(d)
    x = torch.zeros((n, 1, 8, 8), device="cuda")
    blob = torch.zeros(int(lo.total_bytes), dtype=torch.uint8, device="cuda")
    st = L.div_compress_static(ctypes.byref(d), ctypes.c_void_p(x.data_ptr()), ctypes.c_void_p(blob.data_ptr()),
                               blob.numel(), 0, None)
    assert st == binding.DIV_ERR_CAPACITY
    with pytest.raises(binding.DivisionError):
        binding.div_compress_static(d, x.data_ptr(), blob.data_ptr(), blob.numel(), 0)
    # the largest count it accepts works
    d2 = binding.make_desc(binding.DIV_STATIC_MAX_SAMPLES, 1, 8, 8, 8, 2)
    lo2 = binding.div_compressed_bytes(d2)
    x2 = torch.rand((binding.DIV_STATIC_MAX_SAMPLES, 1, 8, 8), device="cuda")
    blob2 = torch.zeros(int(lo2.total_bytes), dtype=torch.uint8, device="cuda")
    binding.div_compress_static(d2, x2.data_ptr(), blob2.data_ptr(), blob2.numel(), 3)
    codec = binding.Codec(binding.DIV_STATIC_MAX_SAMPLES, 1, 8, 8, 8, 2)
    codec.compress(x2, seed=3)
    torch.cuda.synchronize()
    lo = codec.layout
    assert torch.equal(blob2[lo.packed_off:lo.packed_off + lo.packed_bytes], codec.blob[lo.packed_off:lo.packed_off + lo.packed_bytes])
    assert torch.equal(blob2[lo.stats_off:], codec.blob[lo.stats_off:])
