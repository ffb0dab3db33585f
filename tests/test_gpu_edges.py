"""Degenerate and extreme inputs: a layer with nothing kept, one-pixel images, one-row GEMMs, the largest
kernel the format allows, and sizes the calls must refuse."""
import numpy as np
import pytest
import torch

import oracle
import paper_2012_00596_b200 as npas
from paper_2012_00596_b200 import inputs
from util import TOL_BF16, TOL_F32, dev, floored_rel_err, host

pytestmark = pytest.mark.gpu


def _conv(c, path=0):
    dt = c.dtype
    blob = npas.pack_bp(dev(c.w, dt), c.tap_mask, c.Mb, c.Nb)
    ws = npas.workspace()
    y = npas.conv2d_bp(dev(c.x, dt), blob, dev(c.bias), dev(c.residual, dt), stride=c.stride, pad=c.pad, relu=c.relu, ws=ws, path=path)
    npas.check_device_status(ws)
    return y


def _conv_ref(c):
    return oracle.conv2d_bp(c.x, c.w, c.tap_mask, Mb=c.Mb, Nb=c.Nb, stride=c.stride, pad=c.pad, bias=c.bias,
                            residual=c.residual, relu=c.relu)


@pytest.mark.parametrize("path,Mb,Nb", [(1, 16, 16), (3, 16, 16), (6, 16, 16), (7, 16, 16), (8, 16, 16), (6, 1, 1)])
def test_layer_with_nothing_kept_is_bias_plus_residual(path, Mb, Nb):
    c = inputs.conv_case(N=2, H=14, W=14, C=64, K=128, Mb=Mb, Nb=Nb, keep=0, dtype="bf16", residual=True, relu=False, seed=801)
    assert not c.tap_mask.any()
    y = host(_conv(c, path))
    want = inputs.bf16_representable((c.bias[None, None, None, :].astype(np.float32) + c.residual).astype(np.float32))
    assert np.array_equal(y, want)                                   # one rounding of an exact fp32 sum
    assert floored_rel_err(y, _conv_ref(c)) < TOL_BF16


@pytest.mark.parametrize("H,W", [(1, 1), (2, 3), (1, 17)])
def test_images_smaller_than_the_kernel(H, W):
    """3x3, pad 1 on images of one or two pixels per side: most taps fall on padding."""
    for path, kw in ((0, dict(C=64, K=64, Mb=16, Nb=16)), (8, dict(C=64, K=64, Mb=16, Nb=16)), (1, dict(C=8, K=8, Mb=4, Nb=4))):
        c = inputs.conv_case(N=3, H=H, W=W, keep=5, dtype="bf16", residual=True, seed=802, **kw)
        assert floored_rel_err(host(_conv(c, path)), _conv_ref(c)) < TOL_BF16, (path, H, W)


def test_largest_kernel_the_format_allows():
    """R*S = 64 taps (8x8), every bit of the tap word in use; CUDA-core kernel, fp32."""
    c = inputs.conv_case(N=1, H=9, W=10, C=4, K=4, Mb=2, Nb=2, R=8, S=8, pad=3, keep=lambda fb, cb: 64 - 21 * (fb + cb), dtype="f32",
                         act="normal", w_sigma=0.2, seed=803)
    assert int(c.tap_mask[0, 0]) == 2 ** 64 - 1
    y = _conv(c)
    assert floored_rel_err(host(y), _conv_ref(c)) < TOL_F32
    blob = npas.pack_bp(dev(c.w), c.tap_mask, 2, 2)
    assert np.array_equal(blob.data.cpu().numpy(), oracle.pack_bp(c.w, c.tap_mask, 2, 2, "f32"))


@pytest.mark.parametrize("M", [1, 7, 129])
@pytest.mark.parametrize("path", [0, 1, 3, 5, 6])
def test_gemm_with_few_rows_and_empty_blocks(M, path):
    c = inputs.linear_case(M=M, I=128, O=256, Bo=64, Bi=64, keep_rows=lambda a, b: 0 if (a + b) % 2 else 20,
                           keep_cols=lambda a, b: 24, dtype="bf16", seed=804)
    x, w = dev(c.x, "bf16"), dev(c.w, "bf16")
    blob = npas.pack_bb(w, c.row_keep, c.col_keep, 64, 64)
    ws = npas.workspace()
    y = npas.linear_bb(x, blob, dev(c.bias), relu=True, ws=ws, path=path)
    npas.check_device_status(ws)
    ref = oracle.linear_bb(c.x, c.w, c.row_keep, c.col_keep, Bo=64, Bi=64, bias=c.bias, relu=True)
    assert floored_rel_err(host(y), ref) < TOL_BF16


def test_gemm_with_nothing_kept_is_the_bias():
    c = inputs.linear_case(M=130, I=128, O=128, Bo=64, Bi=64, keep_rows=0, keep_cols=0, dtype="bf16", relu=False, seed=805)
    blob = npas.pack_bb(dev(c.w, "bf16"), c.row_keep, c.col_keep, 64, 64)
    for path in (0, 1, 3, 5, 6):
        y = host(npas.linear_bb(dev(c.x, "bf16"), blob, dev(c.bias), relu=False, out_dtype=torch.float32, path=path))
        assert np.array_equal(y, np.broadcast_to(c.bias, y.shape)), path


def test_empty_and_oversized_problems_are_refused():
    c = inputs.conv_case(N=1, H=4, W=4, C=16, K=16, Mb=16, Nb=16, keep=3, dtype="bf16", seed=806)
    blob = npas.pack_bp(dev(c.w, "bf16"), c.tap_mask, 16, 16)
    x0 = torch.empty((0, 4, 4, 16), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(npas.NpasError) as e:
        npas.conv2d_bp(x0, blob)                                      # empty batch
    assert e.value.code == 2
    with pytest.raises(npas.NpasError) as e:                          # image smaller than the kernel without padding
        npas.conv2d_bp(dev(c.x[:, :2, :2], "bf16"), blob, pad=0)
    assert e.value.code == 2
    # weight tensors beyond what 32-bit blob offsets address are refused by the size call
    import ctypes
    from paper_2012_00596_b200 import binding as B
    lib = npas.load()
    d = B.BpDesc(16384, 16384, 3, 3, 16, 16, B.BF16, B.BF16, 9)
    size = ctypes.c_size_t(0)
    tm = np.zeros(4, dtype=np.uint64)
    assert lib.npas_pack_bp_size(ctypes.byref(d), tm.ctypes.data_as(ctypes.c_void_p), ctypes.byref(size)) == 2
