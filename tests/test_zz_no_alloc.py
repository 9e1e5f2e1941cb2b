"""div_compress_static: the compress call for callers that cannot allocate device memory.

Some users of this library run where a device allocation is off limits at the moment they compress (inside
another framework's callback, with the memory budget already handed out, or in a loop that must not pay for
a device-synchronising cudaMalloc).  For them the library carries its own fixed scratch array.  This test
calls that entry point through the C ABI twice in a row and checks that each result equals, byte for byte,
what the ordinary div_compress writes for the same input and seed (the bar of the other parity tests), and
that the fixed array's stale contents from the first call do not leak into the second.

The file name sorts last on purpose: a run that stops at the first failure has then run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

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


def test_static_scratch_matches_div_compress_on_two_calls_in_a_row():
    stream = binding.current_stream_handle()
    # two different maps, so that the second call finds the first call's leftovers in the shared array
    spec_a = synth.config0()[0]                                   # 8 x 64 x 32 x 32, strip ring kernel
    xa = torch.from_numpy(synth.make_input(spec_a)).cuda()
    xb = torch.from_numpy(synth.activation_map(5, 24, 14, 14, "relu", 4242)).cuda()   # general ring kernel
    args_a = (*spec_a.shape, spec_a.block, spec_a.qbits)
    args_b = (5, 24, 14, 14, 8, 2)
    codec_a, want_a = _reference_blob(xa, args_a, seed=11)
    codec_b, want_b = _reference_blob(xb, args_b, seed=12)

    got_a = torch.full_like(want_a, 0xEE)
    got_b = torch.full_like(want_b, 0xEE)
    got_a2 = torch.full_like(want_a, 0xEE)
    # back to back on one stream: a, b, a again
    binding.div_compress_static(codec_a.desc, xa.data_ptr(), got_a.data_ptr(), got_a.numel(), 11, stream)
    binding.div_compress_static(codec_b.desc, xb.data_ptr(), got_b.data_ptr(), got_b.numel(), 12, stream)
    binding.div_compress_static(codec_a.desc, xa.data_ptr(), got_a2.data_ptr(), got_a2.numel(), 11, stream)
    torch.cuda.synchronize()

    def sections(blob, layout):
        lo = layout
        return (blob[lo.lfc_off:lo.lfc_off + lo.lfc_bytes], blob[lo.packed_off:lo.packed_off + lo.packed_bytes],
                blob[lo.stats_off:lo.stats_off + lo.stats_bytes])

    for got, want, codec in ((got_a, want_a, codec_a), (got_b, want_b, codec_b), (got_a2, want_a, codec_a)):
        for g, w in zip(sections(got, codec.layout), sections(want, codec.layout)):
            assert torch.equal(g, w)
    # and the result decodes like any other blob
    xhat = codec_a.decompress(blob=got_a2)
    xref = codec_a.decompress(blob=want_a)
    torch.cuda.synchronize()
    assert torch.equal(xhat, xref)


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
