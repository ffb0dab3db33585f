"""Layer fusion: first-layer convolution + bias + ReLU + 3x3/2 max-pool in one kernel, against the two
separate kernels (bit for bit) and against the oracle's convolution followed by the oracle's max-pool."""
import numpy as np
import pytest
import torch

import oracle
import paper_2012_00596_b200 as npas
from paper_2012_00596_b200 import inputs
from util import TOL_BF16, dev, floored_rel_err, host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("kw", [
    dict(N=2, H=32, W=32, K=64, keep=49),                    # 16x16 conv output -> 8x8 pooled
    dict(N=1, H=34, W=30, K=32, keep=20),                    # punched, odd conv height (17 x 15 -> 9 x 8)
    dict(N=3, H=64, W=64, K=64, keep=49),
    dict(N=1, H=224, W=224, K=64, keep=49),                  # the ImageNet first layer: 112x112 -> 56x56
])
def test_fused_first_layer_and_maxpool(kw):
    c = inputs.conv_case(C=3, Mb=16, Nb=3, R=7, S=7, stride=2, pad=3, dtype="bf16", act="normal", w_sigma=0.1,
                         seed=701, **kw)
    x, w = dev(c.x, "bf16"), dev(c.w, "bf16")
    blob = npas.pack_bp(w, c.tap_mask, c.Mb, c.Nb)
    bias = dev(c.bias)
    ws = npas.workspace()
    y = npas.conv2d_bp(x, blob, bias, stride=2, pad=3, relu=True, ws=ws)
    two = npas.maxpool2d(y, 3, 2, 1)
    n0 = npas.launch_count()
    one = npas.conv2d_bp_maxpool(x, blob, bias, stride=2, pad=3, relu=True, ws=ws)
    assert npas.launch_count() - n0 == 1                      # one kernel
    npas.check_device_status(ws)
    assert one.shape == two.shape and torch.equal(one, two)   # a maximum is exact: same bits as the two kernels
    assert torch.equal(one, npas.conv2d_bp_maxpool(x, blob, bias, stride=2, pad=3, relu=True, ws=ws))
    conv = oracle.conv2d_bp(c.x, c.w, c.tap_mask, Mb=c.Mb, Nb=c.Nb, stride=2, pad=3, bias=c.bias, relu=True)
    ref = oracle.maxpool2d(conv, R=3, stride=2, pad=1)
    assert floored_rel_err(host(one), ref) < TOL_BF16


def test_fusion_declines_what_it_does_not_cover():
    c = inputs.conv_case(N=1, H=32, W=32, C=3, K=32, Mb=16, Nb=3, R=7, S=7, stride=2, pad=3, keep=49, dtype="bf16", seed=702)
    x, w = dev(c.x, "bf16"), dev(c.w, "bf16")
    blob = npas.pack_bp(w, c.tap_mask, c.Mb, c.Nb)
    for kwargs in (dict(relu=False), dict(pool=(2, 2, 0)), dict(pool=(3, 1, 1))):
        with pytest.raises(npas.NpasError) as e:
            npas.conv2d_bp_maxpool(x, blob, dev(c.bias), stride=2, pad=3, **{"relu": True, **kwargs})
        assert e.value.code == 8
    c2 = inputs.conv_case(N=1, H=14, W=14, C=64, K=64, Mb=16, Nb=8, keep=3, dtype="bf16", seed=703)      # not a first layer
    blob2 = npas.pack_bp(dev(c2.w, "bf16"), c2.tap_mask, 16, 8)
    with pytest.raises(npas.NpasError) as e:
        npas.conv2d_bp_maxpool(dev(c2.x, "bf16"), blob2, dev(c2.bias), relu=True)
    assert e.value.code == 8
