"""The other pruning schemes as special cases of block-punched pruning (paper Sec. 3: unstructured =
blocks of 1 x 1, coarse-grained = one block for the whole tensor; Sec. 2.1: pattern-based = 1 x 1 blocks
whose tap sets come from a small pattern library, plus whole kernels removed), on the tensor-core path."""
import numpy as np
import pytest
import torch

import oracle
import paper_2012_00596_b200 as npas
from paper_2012_00596_b200 import inputs
from util import TOL_BF16, dev, floored_rel_err, host

pytestmark = pytest.mark.gpu


def _run(c, path=0):
    x, w = dev(c.x, "bf16"), dev(c.w, "bf16")
    blob = npas.pack_bp(w, c.tap_mask, c.Mb, c.Nb)
    assert np.array_equal(blob.data.cpu().numpy(), oracle.pack_bp(c.w, c.tap_mask, c.Mb, c.Nb, "bf16"))
    ws = npas.workspace()
    kid = npas.conv2d_bp_kernel(c.x.shape, blob, stride=c.stride, pad=c.pad, relu=c.relu, bias=c.bias is not None,
                                residual=c.residual is not None, path=path)
    y = npas.conv2d_bp(x, blob, dev(c.bias), dev(c.residual, "bf16"), stride=c.stride, pad=c.pad, relu=c.relu, ws=ws, path=path)
    npas.check_device_status(ws)
    return y, kid


def _ref(c):
    return oracle.conv2d_bp(c.x, c.w, c.tap_mask, Mb=c.Mb, Nb=c.Nb, stride=c.stride, pad=c.pad, bias=c.bias,
                            residual=c.residual, relu=c.relu)


def test_pattern_library_is_eight_four_tap_patterns_with_the_centre():
    lib = inputs.PATTERN_LIBRARY
    assert len(set(lib)) == 8 and all(bin(p).count("1") == 4 and (p >> 4) & 1 and p < 512 for p in lib)


@pytest.mark.parametrize("kw", [dict(N=2, H=14, W=14, C=32, K=32), dict(N=1, H=28, W=28, C=64, K=128, stride=2)])
def test_pattern_based_pruning_on_tensor_cores(kw):
    c = inputs.pattern_case(residual=True, seed=601, **kw)
    counts = np.array([bin(int(v)).count("1") for v in c.tap_mask.ravel()])
    assert set(counts) == {0, 4} and 0.1 < np.mean(counts == 0) < 0.4
    y, kid = _run(c)
    assert kid in (6, 7)                                   # a tcgen05 kernel, not the CUDA-core one
    assert floored_rel_err(host(y), _ref(c)) < TOL_BF16
    y1, kid1 = _run(c, path=1)                              # and the CUDA-core kernel agrees
    assert kid1 == 1 and floored_rel_err(host(y1), _ref(c)) < TOL_BF16


def test_unstructured_pruning_is_one_by_one_blocks():
    """Each kernel keeps its own arbitrary number of taps (0 to 9)."""
    c = inputs.conv_case(N=2, H=14, W=14, C=32, K=48, Mb=1, Nb=1, keep=lambda fb, cb: (7 * fb + 3 * cb) % 10, dtype="bf16",
                         residual=True, seed=602)
    y, kid = _run(c)
    assert kid == 6 and floored_rel_err(host(y), _ref(c)) < TOL_BF16


@pytest.mark.parametrize("path", [0, 6, 8])
def test_coarse_grained_pruning_is_one_block_for_the_whole_tensor(path):
    """One block = the whole layer: the same four taps are cut everywhere, i.e. a convolution with a reduced
    kernel shape.  The dense-image kernel skips the cut taps through the tap union, the kept-pairs kernel
    never sees them."""
    c = inputs.conv_case(N=4, H=14, W=14, C=64, K=64, Mb=64, Nb=64, keep=5, dtype="bf16", residual=True, seed=603)
    assert c.tap_mask.shape == (1, 1)
    y, kid = _run(c, path=path)
    assert kid == (6 if path == 0 else path)
    ref = _ref(c)
    assert floored_rel_err(host(y), ref) < TOL_BF16
    # equals the dense convolution of the weights with the cut taps zeroed (library routine, fp64)
    m = oracle.bp_element_mask(c.tap_mask, 64, 64, 3, 3, 64, 64)
    t = torch.nn.functional.conv2d(torch.from_numpy(c.x.astype(np.float64)).permute(0, 3, 1, 2),
                                   torch.from_numpy((c.w * m).astype(np.float64)).permute(0, 3, 1, 2), torch.from_numpy(c.bias.astype(np.float64)),
                                   padding=1).permute(0, 2, 3, 1).numpy()
    assert np.allclose(np.maximum(t + c.residual, 0.0), ref, rtol=1e-10, atol=1e-10)
