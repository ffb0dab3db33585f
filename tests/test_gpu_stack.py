"""ResNet-50-topology stack: every layer of the CUDA path against the fp64 oracle, each layer fed
the bf16 input (and shortcut) that the CUDA path itself produced, so errors do not compound."""
import numpy as np
import pytest
import torch

import oracle
import paper_2012_00596_b200 as npas
from paper_2012_00596_b200 import inputs
from paper_2012_00596_b200.resnet50 import Resnet50Stack
from util import TOL_BF16, floored_rel_err, host

pytestmark = pytest.mark.gpu


def oracle_layer(lay, x, res, points=None):
    """x [N,H,W,C] float64 (NHWC), res like the output or None; returns the full output or the points."""
    if lay.kind == "pw":
        xs = x[:, ::lay.stride, ::lay.stride, :]
        n, h, w, c = xs.shape
        r2 = None if res is None else res.reshape(n * h * w, lay.Cout)
        pts = None
        if points is not None:      # (n, p, q, k) -> (row, column)
            pts = np.stack([(points[:, 0] * h + points[:, 1]) * w + points[:, 2], points[:, 3]], axis=1).astype(np.int32)
        y = oracle.linear_bb(np.ascontiguousarray(xs).reshape(n * h * w, c), lay.w, lay.row_keep, lay.col_keep, Bo=64, Bi=64,
                             bias=lay.bias, residual=r2, relu=lay.relu, points=pts)
        return y if points is not None else y.reshape(n, h, w, lay.Cout)
    Mb, Nb = inputs.STACK_BLOCKS[lay.kind]
    pad = 3 if lay.kind == "stem" else 1
    return oracle.conv2d_bp(x, lay.w, lay.tap_mask, Mb=Mb, Nb=Nb, stride=lay.stride, pad=pad, bias=lay.bias,
                            residual=res, relu=lay.relu, points=points)


def f64(t):
    return None if t is None else t.to(torch.float32).cpu().numpy().astype(np.float64)


def test_small_stack_every_layer_in_full():
    H, N = 64, 2
    layers = inputs.config4(H=H)
    net = Resnet50Stack(layers)
    x = torch.from_numpy(inputs.config4_input(N, H)).cuda().to(torch.bfloat16)
    y, seen, pooled = net.forward(x, keep=True)
    net.check()
    assert tuple(y.shape) == (N, 2, 2, 2048) and len(seen) == 53
    assert np.array_equal(host(pooled), oracle.maxpool2d(f64(seen[0][2]), R=3, stride=2, pad=1))
    worst = 0.0
    for lay, (xin, res, out) in zip(layers, seen):
        ref = oracle_layer(lay, f64(xin), f64(res))
        err = floored_rel_err(host(out), ref)
        worst = max(worst, err)
        assert err < TOL_BF16, (lay.name, err)
        rms = float(np.sqrt(np.mean(ref ** 2)))
        assert 1e-3 < rms < 1e3, (lay.name, rms)          # the activation scale stays in bf16's comfortable range
    assert torch.equal(y, net.forward(x))                  # run-to-run determinism of the whole chain


def test_full_size_stack_sampled_points():
    H, N, n_pts = 224, 64, 3000
    layers = inputs.config4(H=H)
    net = Resnet50Stack(layers)
    x = torch.from_numpy(inputs.config4_input(N, H)).cuda().to(torch.bfloat16)
    y, seen, _ = net.forward(x, keep=True)
    net.check()
    assert tuple(y.shape) == (N, 7, 7, 2048)
    rng = inputs.rng_for(404)
    for lay, (xin, res, out) in zip(layers, seen):
        n, p, q, k = out.shape
        pts = np.stack([rng.integers(0, n, n_pts), rng.integers(0, p, n_pts), rng.integers(0, q, n_pts),
                        rng.integers(0, k, n_pts)], axis=1).astype(np.int32)
        ref = oracle_layer(lay, f64(xin), f64(res), points=pts)
        got = host(out)[pts[:, 0], pts[:, 1], pts[:, 2], pts[:, 3]]
        rms = float(np.sqrt(np.mean(ref ** 2))) + 1e-30
        err = float(np.max(np.abs(got - ref) / (np.abs(ref) + 1e-3 * rms)))
        assert err < TOL_BF16, (lay.name, err)


def test_small_stack_on_tuned_plans_every_layer_in_full():
    """Every layer on the kernel and tile shape the library's tuner measured fastest for it: the plan cache has an
    entry per distinct layer shape, survives a JSON round trip, and every layer still matches the oracle."""
    H, N = 64, 2
    layers = inputs.config4(H=H)
    net = Resnet50Stack(layers)
    x = torch.from_numpy(inputs.config4_input(N, H)).cuda().to(torch.bfloat16)
    plans = net.tune(x, reps=3)
    net.check()
    assert len(plans.plans) >= 20 and all(v[0] > 0 and v[2] > 0 for v in plans.plans.values())
    net.plans = npas.PlanCache.from_json(plans.to_json())
    y, seen, _ = net.forward(x, keep=True)
    net.check()
    for lay, (xin, res, out) in zip(layers, seen):
        assert floored_rel_err(host(out), oracle_layer(lay, f64(xin), f64(res))) < TOL_BF16, lay.name
    assert torch.equal(y, net.forward(x))
