"""The autograd glue (Algorithm 1): what the backward pass receives is the checker's reconstruction of what the
forward pass saved; the mask operators are exact; a whole network trains through it."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import division_oracle as orc
from paper_2208_04187_b200 import autograd as dv
from paper_2208_04187_b200 import binding, build, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built_library():
    build.build()
    binding.lib()


class Probe(torch.autograd.Function):
    """Saves its input and hands the backward pass's view of it to the test."""
    seen = []

    @staticmethod
    def forward(ctx, x):
        ctx.save_for_backward(x)
        return x * 2.0

    @staticmethod
    def backward(ctx, g):
        (x,) = ctx.saved_tensors
        Probe.seen.append(x.detach().clone())
        return g * 2.0


@pytest.mark.parametrize("shape,q,per_plane", [((4, 8, 32, 32), 2, False), ((3, 16, 14, 14), 4, False),
                                               ((4, 8, 32, 32), 2, True), ((2, 64, 256), 8, False)])
def test_backward_sees_the_checkers_reconstruction(shape, q, per_plane):
    if len(shape) == 4:
        x_np = synth.activation_map(*shape, "bn", 3)
    else:
        x_np = np.random.default_rng(3).standard_normal(shape).astype(np.float32)
    leaf = torch.from_numpy(x_np).cuda().requires_grad_(True)
    Probe.seen.clear()
    with dv.DivisionCache(block=8, qbits=q, seed=41, min_elems=1, per_plane=per_plane) as cache:
        act = leaf * 1.0                      # a non-leaf activation map
        y = Probe.apply(act)
    y.sum().backward()
    assert cache.maps == 1 and cache.records[0][0] == 41
    if len(shape) == 3:
        ref = orc.decompress_1d(orc.compress_1d(x_np, 8, q, 41))
        closed = orc.compressed_layout(shape[0], shape[1], 1, shape[2], 8, q).closed_form_bytes
    elif per_plane:
        ref = orc.decompress_planes(orc.compress_planes(x_np, 8, q, 41))
        closed = orc.plane_layout(*shape, 8, q).closed_form_bytes
    else:
        ref = orc.decompress(orc.compress(x_np, 8, q, 41))
        closed = orc.compressed_layout(*shape, 8, q).closed_form_bytes
    np.testing.assert_array_equal(Probe.seen[0].cpu().numpy(), ref)
    assert cache.raw_bytes == x_np.nbytes and cache.cached_bytes == closed
    np.testing.assert_array_equal(leaf.grad.cpu().numpy(), np.full(shape, 2.0, np.float32))


def test_parameters_small_tensors_and_integer_tensors_are_left_alone():
    w = torch.randn(8, 8, 3, 3, device="cuda", requires_grad=True)
    x = torch.randn(2, 8, 16, 16, device="cuda", requires_grad=True)
    with dv.DivisionCache(min_elems=1 << 20) as cache:
        y = F.conv2d(x * 1.0, w, padding=1)
        z, _ = F.max_pool2d(y, 2, return_indices=True)
    z.sum().backward()
    assert cache.maps == 0 and w.grad is not None


def test_mask_operators_are_exact():
    x = torch.randn(3, 5, 17, 19, device="cuda", requires_grad=True)
    g = torch.randn_like(x)
    y = dv.DivisionReLU()(x)
    y.backward(g)
    x2 = x.detach().clone().requires_grad_(True)
    y2 = torch.relu(x2)
    y2.backward(g)
    assert torch.equal(y, y2) and torch.equal(x.grad, x2.grad)
    drop = dv.DivisionDropout(0.25, seed=5)
    x3 = x.detach().clone().requires_grad_(True)
    y3 = drop(x3)
    y3.backward(g)
    ref_y, words = orc.dropout_forward(x.detach().cpu().numpy(), 6, 16384)
    np.testing.assert_array_equal(y3.detach().cpu().numpy().reshape(-1), ref_y)
    np.testing.assert_array_equal(x3.grad.cpu().numpy().reshape(-1), orc.mask_backward(words, g.cpu().numpy()))
    drop.eval()
    assert drop(x3) is x3


def test_a_residual_network_trains_through_the_cache():
    """Forward results are untouched (compression only changes what the backward pass reads); with Q = 8 the
    gradients stay close to the exact ones; the cached bytes follow the closed form."""
    import torchvision
    torch.manual_seed(0)
    model = torchvision.models.resnet18(weights=None, num_classes=10).cuda().train()
    ref_model = torchvision.models.resnet18(weights=None, num_classes=10).cuda().train()
    ref_model.load_state_dict(model.state_dict())
    dv.to_division_modules(model)
    x = torch.randn(8, 3, 64, 64, device="cuda")
    out_ref = ref_model(x)
    out_ref.square().mean().backward()
    with dv.DivisionCache(block=8, qbits=8, min_elems=1024) as cache:
        out = model(x)
    out.square().mean().backward()
    assert torch.allclose(out, out_ref, rtol=1e-5, atol=1e-6)
    assert cache.maps > 30 and cache.raw_bytes / cache.cached_bytes > 3.0
    num = den1 = den2 = 0.0
    for (_, p), (_, r) in zip(model.named_parameters(), ref_model.named_parameters()):
        assert p.grad is not None and torch.isfinite(p.grad).all()
        num += float((p.grad * r.grad).sum())
        den1 += float(p.grad.square().sum())
        den2 += float(r.grad.square().sum())
    assert num / (den1 * den2) ** 0.5 > 0.98


def test_cache_reads_back_device_status_and_raises_on_a_recorded_timeout():
    """Every compress call of the cache has a scratch slice of its own; the first decompress of the backward pass
    reads their status words back.  A timeout is planted by hand in one slice (no kernel is made to wait)."""
    x_np = synth.activation_map(4, 8, 32, 32, "bn", 5)
    leaf = torch.from_numpy(x_np).cuda().requires_grad_(True)
    with dv.DivisionCache(block=8, qbits=2, seed=1, min_elems=1) as cache:
        a = Probe.apply(leaf * 1.0)
        b = Probe.apply(a * 1.0)
    assert cache.maps == 2 and len(cache._slices) == 2
    assert cache._slices[0] != cache._slices[1]                 # no scratch is shared between the two calls
    cache.check()                                               # both status words are DIV_OK
    Probe.seen.clear()
    b.sum().backward()
    assert len(Probe.seen) == 2

    with dv.DivisionCache(block=8, qbits=2, seed=1, min_elems=1) as cache2:
        y = Probe.apply(leaf * 1.0)
    ci, off = cache2._slices[0]
    torch.cuda.synchronize()
    cache2._arena[ci][0].view(torch.int32)[off // 4] = binding.DIV_ERR_TIMEOUT
    with pytest.raises(binding.DivisionError) as err:
        y.sum().backward()
    assert err.value.status == binding.DIV_ERR_TIMEOUT
