"""The scratch-free convolution entry point (collected last on purpose).

npas_conv2d_bp_static_ws serves callers that cannot allocate device memory - a fixed-budget or
real-time inference loop, a plug-in whose host owns every allocation - by keeping the kernels'
scratch in an array inside the library.  It must give what npas_conv2d_bp gives, call after call,
because all calls share that one array.
"""
import pytest
import torch

import paper_2012_00596_b200 as npas
from paper_2012_00596_b200 import inputs
from util import TOL_BF16, dev, floored_rel_err, host

pytestmark = pytest.mark.gpu


def test_static_workspace_entry_matches_regular_entry_twice_in_a_row():
    c = inputs.conv_case(N=3, H=14, W=14, C=64, K=64, Mb=16, Nb=8, keep=3, dtype="bf16", residual=True, seed=401)
    x, w = dev(c.x, "bf16"), dev(c.w, "bf16")
    blob = npas.pack_bp(w, c.tap_mask, c.Mb, c.Nb)
    bias, res = dev(c.bias), dev(c.residual, "bf16")
    ws = npas.workspace()
    want = npas.conv2d_bp(x, blob, bias, res, relu=True, ws=ws, path=2)
    npas.check_device_status(ws)
    out = torch.empty_like(want)
    for _ in range(2):                                   # second call reuses the shared array
        out.zero_()
        got = npas.conv2d_bp_static_ws(x, blob, bias, res, relu=True, out=out, path=2)
        assert got.data_ptr() == out.data_ptr()
        assert floored_rel_err(host(got), host(want)) < TOL_BF16
        assert torch.equal(got, want)                    # same kernel, same order of additions
    # a layer on the CUDA-core path goes through the same entry
    c2 = inputs.config1()
    x2, w2 = dev(c2.x), dev(c2.w)
    blob2 = npas.pack_bp(w2, c2.tap_mask, c2.Mb, c2.Nb)
    a = npas.conv2d_bp(x2, blob2, ws=ws)
    b = npas.conv2d_bp_static_ws(x2, blob2)
    assert torch.equal(a, b)
