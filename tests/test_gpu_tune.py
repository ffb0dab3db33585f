"""Auto-tuning entry points: the returned (path, variant) runs, matches the oracle and is not slower
than the automatic choice on the standard workloads."""
import numpy as np
import pytest
import torch

import oracle
import paper_2012_00596_b200 as npas
from paper_2012_00596_b200 import inputs
from util import TOL_BF16, dev, floored_rel_err, host

pytestmark = pytest.mark.gpu


def _time_us(f, reps=20):
    # the oracle's CPU time before this call lets the GPU clocks drop: run for a while first, and take the
    # better of two measurements
    for _ in range(200):
        f()
    torch.cuda.synchronize()
    return min(_time_once(f, reps), _time_once(f, reps))


def _time_once(f, reps):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        f()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / reps


@pytest.mark.parametrize("name", ["config2", "config5_16x16_3", "config5_32x32_2", "stack_3x3_s2"])
def test_tuned_conv_plan_is_valid_and_not_slower(name):
    c = {"config2": lambda: inputs.config2(),
         "config5_16x16_3": lambda: inputs.config5(16, 16, 3, N=16),
         "config5_32x32_2": lambda: inputs.config5(32, 32, 2, N=16),
         "stack_3x3_s2": lambda: inputs.conv_case(N=16, H=28, W=28, C=256, K=256, Mb=16, Nb=8, keep=3, stride=2, seed=5)}[name]()
    x, w = dev(c.x, "bf16"), dev(c.w, "bf16")
    blob = npas.pack_bp(w, c.tap_mask, c.Mb, c.Nb)
    bias = dev(c.bias)
    ws = npas.workspace()
    y = torch.empty((c.N, c.P, c.Q, c.K), dtype=torch.bfloat16, device="cuda")
    path, variant, us = npas.tune_conv2d_bp(x, blob, bias, stride=c.stride, pad=c.pad, relu=c.relu, out=y, ws=ws, reps=20)
    assert path in npas.CONV_KERNELS and us > 0
    # the plan is what the kernel query accepts, and running it gives the layer's result
    assert npas.conv2d_bp_kernel(c.x.shape, blob, stride=c.stride, pad=c.pad, relu=c.relu, bias=bias is not None,
                                 path=path, variant=variant) == path
    y.zero_()
    npas.conv2d_bp(x, blob, bias, stride=c.stride, pad=c.pad, relu=c.relu, out=y, ws=ws, path=path, variant=variant)
    npas.check_device_status(ws)
    rng = inputs.rng_for(78)
    pts = np.stack([rng.integers(0, c.N, 3000), rng.integers(0, c.P, 3000), rng.integers(0, c.Q, 3000),
                    rng.integers(0, c.K, 3000)], axis=1).astype(np.int32)
    ref = oracle.conv2d_bp(c.x, c.w, c.tap_mask, Mb=c.Mb, Nb=c.Nb, stride=c.stride, pad=c.pad, bias=c.bias, relu=c.relu,
                           points=pts)
    assert floored_rel_err(host(y)[pts[:, 0], pts[:, 1], pts[:, 2], pts[:, 3]], ref) < TOL_BF16
    t_plan = _time_us(lambda: npas.conv2d_bp(x, blob, bias, stride=c.stride, pad=c.pad, relu=c.relu, out=y, ws=ws, path=path,
                                             variant=variant))
    t_auto = _time_us(lambda: npas.conv2d_bp(x, blob, bias, stride=c.stride, pad=c.pad, relu=c.relu, out=y, ws=ws))
    assert t_plan <= 1.25 * t_auto, (path, variant, t_plan, t_auto)      # eager launches: allow timing noise


def test_tuned_linear_plan_is_valid_and_not_slower():
    c = inputs.config3()
    x, w = dev(c.x, "bf16"), dev(c.w, "bf16")
    blob = npas.pack_bb(w, c.row_keep, c.col_keep, c.Bo, c.Bi)
    bias = dev(c.bias)
    ws = npas.workspace()
    y = torch.empty((c.M, c.O), dtype=torch.bfloat16, device="cuda")
    path, variant, us = npas.tune_linear_bb(x, blob, bias, relu=True, out=y, ws=ws, reps=20)
    assert path in npas.LINEAR_KERNELS and path != 1 and us > 0
    assert npas.linear_bb_kernel(c.M, blob, relu=True, bias=True, path=path, variant=variant) == path
    y.zero_()
    npas.linear_bb(x, blob, bias, relu=True, out=y, ws=ws, path=path, variant=variant)
    npas.check_device_status(ws)
    ref = oracle.linear_bb(c.x, c.w, c.row_keep, c.col_keep, Bo=c.Bo, Bi=c.Bi, bias=c.bias, relu=True)
    assert floored_rel_err(host(y), ref) < TOL_BF16
    t_plan = _time_us(lambda: npas.linear_bb(x, blob, bias, relu=True, out=y, ws=ws, path=path, variant=variant))
    t_auto = _time_us(lambda: npas.linear_bb(x, blob, bias, relu=True, out=y, ws=ws))
    assert t_plan <= 1.25 * t_auto, (path, variant, t_plan, t_auto)


def test_tuner_rejects_bad_arguments_without_launching():
    c = inputs.conv_case(N=1, H=14, W=14, C=64, K=64, Mb=16, Nb=8, keep=3, dtype="bf16", seed=501)
    x, w = dev(c.x, "bf16"), dev(c.w, "bf16")
    blob = npas.pack_bp(w, c.tap_mask, c.Mb, c.Nb)
    n0 = npas.launch_count()
    with pytest.raises(npas.NpasError) as e:
        npas.tune_conv2d_bp(x, blob, reps=0)
    assert e.value.code == 2 and npas.launch_count() == n0
