"""Selection rule of the autograd glue (which saved tensors are cached in compressed form); no GPU needed."""
import torch

from paper_2208_04187_b200 import autograd as dv


def test_only_activation_maps_are_selected():
    ok = dict(is_cuda=True, is_param_like=False, min_elems=1 << 14)
    assert dv.should_compress((64, 64, 56, 56), torch.float32, **ok)
    assert dv.should_compress((32, 512, 768), torch.bfloat16, **ok)                       # 1-D map
    assert not dv.should_compress((64, 64, 56, 56), torch.float32, is_cuda=False, is_param_like=False, min_elems=1)
    assert not dv.should_compress((64, 64, 3, 3), torch.float32, is_cuda=True, is_param_like=True, min_elems=1)   # a weight
    assert not dv.should_compress((64, 64, 56, 56), torch.int64, **ok)                    # pooling indices
    assert not dv.should_compress((64, 64, 56, 56), torch.float16, **ok)
    assert not dv.should_compress((64, 1000), torch.float32, **ok)                        # 2-D: not an activation map
    assert not dv.should_compress((2, 3, 8, 8), torch.float32, **ok)                      # below min_elems
    assert not dv.should_compress((2, 3, 4, 8, 8), torch.float32, is_cuda=True, is_param_like=False, min_elems=1)  # 3-D maps


def test_module_conversion_replaces_relu_only():
    m = torch.nn.Sequential(torch.nn.Conv2d(3, 4, 3), torch.nn.ReLU(inplace=True),
                            torch.nn.Sequential(torch.nn.BatchNorm2d(4), torch.nn.ReLU()))
    dv.to_division_modules(m)
    kinds = [type(x).__name__ for x in m.modules()]
    assert kinds.count("DivisionReLU") == 2 and "ReLU" not in kinds and "Conv2d" in kinds and "BatchNorm2d" in kinds
    assert dv.DivisionDropout(0.1).drop_threshold == 6554
