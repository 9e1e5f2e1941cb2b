"""Parity of the ReLU / dropout mask operators (the paper's appendix algorithms "Relu operator" and "Dropout
operator") with the CPU checker, through the C ABI: outputs, packed masks and gradients for exact equality."""
import numpy as np
import pytest
import torch

from oracle import division_oracle as orc
from paper_2208_04187_b200 import binding, build

pytestmark = pytest.mark.gpu

TOTALS = [1, 7, 8, 9, 31, 32, 33, 49, 2047, 2048, 2049, 64 * 49, 100003, 3 * 112 * 112 * 5 + 5]


@pytest.fixture(scope="module", autouse=True)
def built_library():
    build.build()
    binding.lib()


def host_values(total, seed, dtype):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal(total).astype(np.float32)
    x[rng.integers(0, total, max(1, total // 10))] = 0.0
    x[rng.integers(0, total, max(1, total // 10))] = -0.0
    return orc.f32_to_bf16_bits(x) if dtype == "bf16" else x


def to_device(a, dtype):
    t = torch.from_numpy(a)
    return (t.view(torch.bfloat16) if dtype == "bf16" else t).cuda()


def to_host(t, dtype):
    return t.view(torch.int16).cpu().numpy().view(np.uint16) if dtype == "bf16" else t.cpu().numpy()


def as_f32(a, dtype):
    return orc.bf16_bits_to_f32(a) if dtype == "bf16" else a


def mask_buffer(total):
    nbytes = binding.div_mask_bytes(total)
    assert nbytes == orc.mask_bytes(total)
    return torch.full((nbytes + 16,), 0xA5, dtype=torch.uint8, device="cuda"), nbytes   # guard bytes behind it


@pytest.mark.parametrize("total", TOTALS)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_relu_forward_and_backward(total, dtype):
    x = host_values(total, 3, dtype)
    g = host_values(total, 4, dtype)
    ref_y, ref_words = orc.relu_forward(x, dtype)
    xd, gd = to_device(x, dtype), to_device(g, dtype)
    yd, gind = torch.empty_like(xd), torch.empty_like(gd)
    mask, nbytes = mask_buffer(total)
    s = torch.cuda.current_stream().cuda_stream
    binding.div_relu_forward(xd.data_ptr(), yd.data_ptr(), mask.data_ptr(), nbytes, total, dtype, s)
    binding.div_mask_backward(mask.data_ptr(), nbytes, gd.data_ptr(), gind.data_ptr(), total, dtype, s)
    torch.cuda.synchronize()
    m = mask.cpu().numpy()
    np.testing.assert_array_equal(m[:nbytes].view("<u4"), ref_words)
    assert (m[nbytes:] == 0xA5).all()
    y = to_host(yd, dtype)
    np.testing.assert_array_equal(as_f32(y, dtype), ref_y)
    assert not np.signbit(as_f32(y, dtype)).any()                    # masked positions are +0.0
    np.testing.assert_array_equal(as_f32(to_host(gind, dtype), dtype), orc.mask_backward(ref_words, g, dtype))
    # in place
    binding.div_relu_forward(xd.data_ptr(), xd.data_ptr(), mask.data_ptr(), nbytes, total, dtype, s)
    binding.div_mask_backward(mask.data_ptr(), nbytes, gd.data_ptr(), gd.data_ptr(), total, dtype, s)
    torch.cuda.synchronize()
    assert torch.equal(xd, yd) and torch.equal(gd, gind)


@pytest.mark.parametrize("total", TOTALS)
@pytest.mark.parametrize("thr", [0, 1, 6554, 32768, 65535, 65536])
def test_dropout_forward(total, thr):
    dtype = "f32" if thr % 2 == 0 else "bf16"
    x = host_values(total, 5, dtype)
    ref_y, ref_words = orc.dropout_forward(x, 991, thr, dtype)
    xd = to_device(x, dtype)
    yd = torch.empty_like(xd)
    mask, nbytes = mask_buffer(total)
    binding.div_dropout_forward(xd.data_ptr(), yd.data_ptr(), mask.data_ptr(), nbytes, total, 991, thr, dtype,
                                torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    m = mask.cpu().numpy()
    np.testing.assert_array_equal(m[:nbytes].view("<u4"), ref_words)
    assert (m[nbytes:] == 0xA5).all()
    got = as_f32(to_host(yd, dtype), dtype)
    # kept values pass unchanged (a kept -0.0 keeps its sign), dropped ones are +0.0
    np.testing.assert_array_equal(got.view(np.uint32), ref_y.view(np.uint32))


def test_full_size_map_sampled():
    """The 64x64x112x112 map of the benchmark set: whole mask compared, values on a sample of positions."""
    total = 64 * 64 * 112 * 112
    x = torch.randn(total, device="cuda")
    y = torch.empty_like(x)
    mask, nbytes = mask_buffer(total)
    s = torch.cuda.current_stream().cuda_stream
    binding.div_relu_forward(x.data_ptr(), y.data_ptr(), mask.data_ptr(), nbytes, total, "f32", s)
    torch.cuda.synchronize()
    xh = x.cpu().numpy()
    ref_y, ref_words = orc.relu_forward(xh)
    np.testing.assert_array_equal(mask.cpu().numpy()[:nbytes].view("<u4"), ref_words)
    idx = np.random.default_rng(0).integers(0, total, 200000)
    np.testing.assert_array_equal(y.cpu().numpy()[idx], ref_y[idx])
    binding.div_dropout_forward(x.data_ptr(), y.data_ptr(), mask.data_ptr(), nbytes, total, 17, 13107, "f32", s)
    torch.cuda.synchronize()
    _, ref_words = orc.dropout_forward(xh, 17, 13107)
    np.testing.assert_array_equal(mask.cpu().numpy()[:nbytes].view("<u4"), ref_words)


def test_argument_checks():
    x = torch.zeros(64, device="cuda")
    mask = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.DivisionError) as e:
        binding.div_relu_forward(x.data_ptr(), x.data_ptr(), mask.data_ptr(), 4, 64)
    assert e.value.status == binding.DIV_ERR_CAPACITY
    with pytest.raises(binding.DivisionError) as e:
        binding.div_relu_forward(x.data_ptr() + 4, x.data_ptr(), mask.data_ptr(), 8, 32)
    assert e.value.status == binding.DIV_ERR_ALIGN
    with pytest.raises(binding.DivisionError) as e:
        binding.div_dropout_forward(x.data_ptr(), x.data_ptr(), mask.data_ptr(), 8, 64, 0, 65537)
    assert e.value.status == binding.DIV_ERR_PARAM
    with pytest.raises(binding.DivisionError) as e:
        binding.div_mask_backward(mask.data_ptr(), 4, x.data_ptr(), x.data_ptr(), 64)
    assert e.value.status == binding.DIV_ERR_CAPACITY
    with pytest.raises(binding.DivisionError) as e:
        binding.div_relu_forward(x.data_ptr(), x.data_ptr(), mask.data_ptr(), 8, 0)
    assert e.value.status == binding.DIV_ERR_SHAPE
