"""The scratch-free convolution entry point (collected last on purpose).

npas_conv2d_bp_static_ws serves callers that cannot allocate device memory - a fixed-budget or
real-time inference loop, a plug-in whose host owns every allocation - by keeping the kernels'
scratch in an array inside the library.  It must give what npas_conv2d_bp gives, call after call,
because all calls share that one array.
"""
import pytest
import torch

import oracle
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
    ref = oracle.conv2d_bp(c.x, c.w, c.tap_mask, Mb=c.Mb, Nb=c.Nb, bias=c.bias, residual=c.residual, relu=True)
    out = torch.empty_like(want)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for _ in range(2):                                   # second call reuses the shared array
        out.zero_()
        got = npas.conv2d_bp_static_ws(x, blob, bias, res, relu=True, out=out, path=2)
        assert got.data_ptr() == out.data_ptr()
        assert floored_rel_err(host(got), ref) < TOL_BF16      # against the oracle
        assert torch.equal(got, want)                    # same kernel, same order of additions
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before   # the entry point took no device memory
    # a layer on the CUDA-core path goes through the same entry
    c2 = inputs.config1()
    x2, w2 = dev(c2.x), dev(c2.w)
    blob2 = npas.pack_bp(w2, c2.tap_mask, c2.Mb, c2.Nb)
    a = npas.conv2d_bp(x2, blob2, ws=ws)
    b = npas.conv2d_bp_static_ws(x2, blob2)
    assert torch.equal(a, b)


def test_static_workspace_entry_reports_a_device_side_error_and_recovers():
    """A blob that breaks its descriptor's promise is reported by the kernel through the shared array
    (NPAS_ERR_BLOB), and the next call, which clears the array first, is clean again."""
    c = inputs.conv_case(N=1, H=14, W=14, C=64, K=64, Mb=16, Nb=16, keep=3, dtype="bf16", seed=402)
    x, w = dev(c.x, "bf16"), dev(c.w, "bf16")
    blob = npas.pack_bp(w, c.tap_mask, c.Mb, c.Nb)
    bias = dev(c.bias)
    blob.desc.max_taps = 1                               # the blob keeps three taps per block
    with pytest.raises(npas.NpasError) as e:
        npas.conv2d_bp_static_ws(x, blob, bias, relu=True, path=8)
    assert e.value.code == 6
    blob.desc.max_taps = 3
    got = npas.conv2d_bp_static_ws(x, blob, bias, relu=True, path=8)
    ref = oracle.conv2d_bp(c.x, c.w, c.tap_mask, Mb=c.Mb, Nb=c.Nb, bias=c.bias, relu=True)
    assert floored_rel_err(host(got), ref) < TOL_BF16
    # a refused call enqueues nothing and reports the refusal
    c2 = inputs.conv_case(N=1, H=14, W=14, C=64, K=32, Mb=16, Nb=16, keep=3, dtype="bf16", seed=403)
    blob2 = npas.pack_bp(dev(c2.w, "bf16"), c2.tap_mask, c2.Mb, c2.Nb)
    with pytest.raises(npas.NpasError) as e:
        npas.conv2d_bp_static_ws(x, blob2, None, relu=True, path=7)      # 32 filters: outside the pair kernel
    assert e.value.code == 8
