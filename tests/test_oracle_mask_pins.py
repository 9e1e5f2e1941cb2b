"""Pins of the checker's ReLU / dropout operators with a packed 1-bit mask (the paper's appendix algorithms
"Relu operator" and "Dropout operator"; N^2/8 bytes per plane in the proof of Theorem 3A).  No GPU needed."""
import numpy as np
import pytest
import torch

from oracle import division_oracle as orc
from paper_2208_04187_b200 import synth


def test_mask_bytes_are_one_bit_per_element():
    """Theorem 3A's proof: a ReLU operator caches N^2 bits = N^2/8 bytes per plane."""
    for side in (8, 16, 56, 112):
        assert orc.mask_bytes(side * side) == side * side // 8
    assert orc.mask_bytes(1) == 4 and orc.mask_bytes(32) == 4 and orc.mask_bytes(33) == 8 and orc.mask_bytes(49) == 8


def test_relu_forward_is_the_library_relu_and_little_endian_packbits():
    x = synth.activation_map(2, 3, 9, 13, "bn", 3)
    x[0, 0, 0, :4] = [0.0, -0.0, 1e-45, -1e-45]
    out, words = orc.relu_forward(x)
    np.testing.assert_array_equal(out, torch.relu(torch.from_numpy(x)).numpy().reshape(-1))
    bits = (x.reshape(-1) > 0).astype(np.uint8)
    ref = np.packbits(np.concatenate([bits, np.zeros(-bits.size % 32, np.uint8)]), bitorder="little").view("<u4")
    np.testing.assert_array_equal(words, ref)
    assert words.size * 4 == orc.mask_bytes(x.size)
    assert not np.signbit(out[x.reshape(-1) <= 0]).any()          # masked positions are +0.0


def test_relu_backward_is_autograd_of_the_library_relu():
    x = synth.activation_map(2, 4, 7, 7, "bn", 5)
    g = synth.activation_map(2, 4, 7, 7, "bn", 6)
    xt = torch.from_numpy(x).requires_grad_(True)
    torch.relu(xt).backward(torch.from_numpy(g))
    _, words = orc.relu_forward(x)
    np.testing.assert_array_equal(orc.mask_backward(words, g), xt.grad.numpy().reshape(-1))


def test_relu_on_bf16_bit_patterns():
    x = orc.f32_to_bf16_bits(synth.activation_map(1, 3, 8, 8, "bn", 7))
    out, words = orc.relu_forward(x, orc.BF16)
    x32 = orc.bf16_bits_to_f32(x).reshape(-1)
    np.testing.assert_array_equal(out, np.maximum(x32, 0))
    np.testing.assert_array_equal(orc.unpack_mask(words, x32.size), (x32 > 0))


def test_dropout_mask_follows_the_random_stream_and_the_threshold():
    x = np.ones(1 << 16, np.float32)
    seed = 77
    fields = np.array([orc.divrng_fields(seed, 0, np.array([i], dtype=np.uint64))[0] for i in range(0, 4096, 37)])
    for thr in (0, 1, 16384, 32768, 65535, 65536):
        out, words = orc.dropout_forward(x, seed, thr)
        v = orc.unpack_mask(words, x.size)
        np.testing.assert_array_equal(out, v.astype(np.float32))            # no rescaling: kept values pass unchanged
        np.testing.assert_array_equal(v[0:4096:37], fields >= thr)          # element by element against the stream
        keep = v.mean()
        p = thr / 65536.0
        assert abs(keep - (1 - p)) <= 4 * np.sqrt(max(p * (1 - p), 1e-12) / x.size) + 1e-12
    assert orc.dropout_forward(x, seed, 0)[1].tolist() == [0xFFFFFFFF] * (x.size // 32)
    assert not orc.dropout_forward(x, seed, 65536)[1].any()
    with pytest.raises(ValueError):
        orc.dropout_forward(x, seed, 65537)


def test_dropout_backward_passes_the_gradient_where_the_forward_kept_the_value():
    x = synth.activation_map(1, 2, 10, 10, "bn", 8)
    g = synth.activation_map(1, 2, 10, 10, "bn", 9)
    out, words = orc.dropout_forward(x, 5, 20000)
    gin = orc.mask_backward(words, g)
    kept = out != 0
    np.testing.assert_array_equal(gin[kept], g.reshape(-1)[kept])
    dropped = orc.unpack_mask(words, x.size) == 0
    assert not gin[dropped].any() and not out[dropped].any()


def test_mask_round_trip_with_a_ragged_tail():
    rng = np.random.default_rng(1)
    for total in (1, 31, 32, 33, 49, 1000):
        v = rng.integers(0, 2, total).astype(np.uint8)
        words = orc.pack_mask(v)
        assert words.size * 4 == orc.mask_bytes(total)
        np.testing.assert_array_equal(orc.unpack_mask(words, total), v)
        if total % 32:
            assert words[-1] >> (total % 32) == 0                           # unused high bits stay zero
