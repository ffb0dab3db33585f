"""Pins for the CPU oracle's block-punched convolution (CPU only).

Each test pins the oracle to something other than itself: a hand-worked example, an
independently written brute force, torch's fp64 conv2d, closed forms and the special cases the
paper names (Sec. 3: unstructured = 1x1 blocks, coarse-grained = whole-tensor block; Sec. 4:
1x1 kernels are a plain GEMM).
"""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2012_00596_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def brute_force_conv(x, w, tap_mask, Mb, Nb, stride, pad, bias=None, residual=None, relu=False):
    """Input-stationary scatter form: every (input pixel, kept tap) pushes into the outputs it
    feeds.  Written independently of the oracle: other loop order, mask looked up per block."""
    N, H, W, C = x.shape
    K, R, S, _ = w.shape
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    y = np.zeros((N, P, Q, K))
    for fb in range(K // Mb):
        for cb in range(C // Nb):
            kept = [t for t in range(R * S) if (int(tap_mask[fb, cb]) >> t) & 1]
            for t in kept:
                r, s = divmod(t, S)
                for n in range(N):
                    for h in range(H):
                        for v in range(W):
                            ph, pv = h + pad - r, v + pad - s
                            if ph % stride or pv % stride:
                                continue
                            p, q = ph // stride, pv // stride
                            if not (0 <= p < P and 0 <= q < Q):
                                continue
                            for f in range(Mb):
                                for c in range(Nb):
                                    y[n, p, q, fb * Mb + f] += float(x[n, h, v, cb * Nb + c]) * \
                                        float(w[fb * Mb + f, r, s, cb * Nb + c])
    if bias is not None:
        y += np.asarray(bias, dtype=np.float64)
    if residual is not None:
        y += residual
    if relu:
        y = np.maximum(y, 0)
    return y


def torch_masked_dense(x, w, m, stride, pad, bias=None):
    xt = torch.from_numpy(np.asarray(x, dtype=np.float64)).permute(0, 3, 1, 2)
    wt = torch.from_numpy(np.asarray(w, dtype=np.float64) * m).permute(0, 3, 1, 2)
    b = None if bias is None else torch.from_numpy(np.asarray(bias, dtype=np.float64))
    y = torch.nn.functional.conv2d(xt, wt, b, stride=stride, padding=pad)
    return y.permute(0, 2, 3, 1).numpy()


def test_worked_example_from_golden_file():
    rows = [l for l in open(os.path.join(GOLD, "conv_bp_worked_example.txt")) if not l.startswith("#")]
    expect = np.array([[float(v) for v in r.split()] for r in rows if r.strip()])
    x = np.arange(1, 10, dtype=np.float64).reshape(1, 3, 3, 1)
    w = np.arange(1, 10, dtype=np.float64).reshape(1, 3, 3, 1)
    tm = np.array([[(1 << 0) | (1 << 4) | (1 << 8)]], dtype=np.uint64)
    y = oracle.conv2d_bp(x, w, tm, Mb=1, Nb=1)
    assert np.array_equal(y[0, :, :, 0], expect)


@pytest.mark.parametrize("stride,pad,R", [(1, 1, 3), (2, 1, 3), (1, 0, 3), (1, 2, 5), (2, 0, 1)])
def test_against_brute_force_tiny(stride, pad, R):
    c = inputs.conv_case(N=2, H=5, W=6, C=4, K=4, R=R, S=R, stride=stride, pad=pad, Mb=2, Nb=2,
                         keep=lambda fb, cb: (fb * 2 + cb) % (R * R + 1), dtype="f32",
                         act="normal", w_sigma=1.0, residual=True, seed=11 + R)
    y = oracle.conv2d_bp(c.x, c.w, c.tap_mask, Mb=2, Nb=2, stride=stride, pad=pad, bias=c.bias,
                         residual=c.residual, relu=True)
    yb = brute_force_conv(c.x, c.w, c.tap_mask, 2, 2, stride, pad, c.bias, c.residual, True)
    np.testing.assert_allclose(y, yb, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("stride", [1, 2])
def test_equals_library_dense_conv_of_masked_weights(stride):
    c = inputs.conv_case(N=2, H=9, W=7, C=16, K=24, Mb=8, Nb=4, keep=3, dtype="f32",
                         act="normal", w_sigma=0.5, stride=stride, seed=5)
    m = oracle.bp_element_mask(c.tap_mask, c.K, c.C, 3, 3, 8, 4)
    y = oracle.conv2d_bp(c.x, c.w, c.tap_mask, Mb=8, Nb=4, stride=stride, pad=1, bias=c.bias)
    np.testing.assert_allclose(y, torch_masked_dense(c.x, c.w, m, stride, 1, c.bias),
                               rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("tap", range(9))
def test_shifted_delta_closed_form(tap):
    """W[k,r0,s0,c] = delta_kc with only tap (r0,s0) kept: Y is X shifted by (r0-pad, s0-pad)
    with a zero border - pins cross-correlation (no flip), padding side and index order."""
    r0, s0 = divmod(tap, 3)
    rng = inputs.rng_for(3)
    x = rng.standard_normal((1, 5, 6, 4))
    w = np.zeros((4, 3, 3, 4))
    for k in range(4):
        w[k, r0, s0, k] = 1.0
    w += 7.0 * (np.arange(9).reshape(1, 3, 3, 1) != tap)     # junk on pruned taps must not leak
    tm = np.full((2, 2), 1 << tap, dtype=np.uint64)
    y = oracle.conv2d_bp(x, w, tm, Mb=2, Nb=2)
    xp = np.pad(x, ((0, 0), (1, 1), (1, 1), (0, 0)))
    expect = xp[:, r0:r0 + 5, s0:s0 + 6, :]
    assert np.array_equal(y, expect)


def test_mask_structure_invariant():
    """All Mb*Nb kernels of a block have the same tap support (paper Sec. 3)."""
    rng = inputs.rng_for(9)
    tm = inputs.draw_tap_masks(rng, 3, 4, 9, lambda fb, cb: (fb + cb) % 10)
    m = oracle.bp_element_mask(tm, 12, 8, 3, 3, 4, 2)
    for fb in range(3):
        for cb in range(4):
            blk = m[fb * 4:(fb + 1) * 4, :, :, cb * 2:(cb + 1) * 2]        # [Mb,3,3,Nb]
            ref = blk[0, :, :, 0]
            assert all(np.array_equal(blk[f, :, :, c], ref) for f in range(4) for c in range(2))
            assert int(ref.sum()) == bin(int(tm[fb, cb])).count("1")
            for t in range(9):
                assert ref[t // 3, t % 3] == ((int(tm[fb, cb]) >> t) & 1)


def test_special_case_whole_tensor_block_is_reduced_tap_conv():
    c = inputs.conv_case(N=1, H=6, W=6, C=4, K=6, Mb=6, Nb=4, keep=4, dtype="f32", act="normal",
                         w_sigma=1.0, bias=False, seed=21)
    y = oracle.conv2d_bp(c.x, c.w, c.tap_mask, Mb=6, Nb=4)
    taps = [t for t in range(9) if (int(c.tap_mask[0, 0]) >> t) & 1]
    xp = np.pad(c.x.astype(np.float64), ((0, 0), (1, 1), (1, 1), (0, 0)))
    expect = np.zeros_like(y)
    for t in taps:
        r, s = divmod(t, 3)
        expect += np.einsum("nhwc,kc->nhwk", xp[:, r:r + 6, s:s + 6, :], c.w[:, r, s, :].astype(np.float64))
    np.testing.assert_allclose(y, expect, rtol=1e-12, atol=1e-12)


def test_special_case_1x1_blocks_is_arbitrary_per_kernel_mask():
    c = inputs.conv_case(N=1, H=5, W=5, C=3, K=4, Mb=1, Nb=1, keep=lambda fb, cb: (3 * fb + cb) % 10,
                         dtype="f32", act="normal", w_sigma=1.0, seed=22)
    m = np.zeros((4, 3, 3, 3))
    for k in range(4):
        for ch in range(3):
            for t in range(9):
                m[k, t // 3, t % 3, ch] = (int(c.tap_mask[k, ch]) >> t) & 1
    y = oracle.conv2d_bp(c.x, c.w, c.tap_mask, Mb=1, Nb=1, bias=c.bias)
    np.testing.assert_allclose(y, torch_masked_dense(c.x, c.w, m, 1, 1, c.bias), rtol=1e-12, atol=1e-12)


def test_all_taps_kept_is_dense_conv():
    c = inputs.conv_case(N=1, H=6, W=5, C=8, K=8, Mb=4, Nb=4, keep=9, dtype="f32", act="normal",
                         w_sigma=1.0, seed=23)
    y = oracle.conv2d_bp(c.x, c.w, c.tap_mask, Mb=4, Nb=4, bias=c.bias)
    np.testing.assert_allclose(y, torch_masked_dense(c.x, c.w, np.ones_like(c.w), 1, 1, c.bias),
                               rtol=1e-12, atol=1e-12)


def test_centre_tap_only_equals_full_keep_linear_equals_matmul():
    """A 3x3 layer that keeps only the centre tap is a 1x1 CONV, i.e. a GEMM (paper Sec. 4)."""
    c = inputs.conv_case(N=2, H=4, W=4, C=8, K=8, Mb=4, Nb=4, keep=0, dtype="f32", act="normal",
                         w_sigma=1.0, seed=24)
    tm = np.full((2, 2), 1 << 4, dtype=np.uint64)
    y = oracle.conv2d_bp(c.x, c.w, tm, Mb=4, Nb=4, bias=c.bias)
    x2 = c.x.reshape(-1, 8)
    w2 = c.w[:, 1, 1, :]
    full = np.full((2, 2), (1 << 4) - 1, dtype=np.uint64)
    yl = oracle.linear_bb(x2, w2, full, full, Bo=4, Bi=4, bias=c.bias)
    ym = x2.astype(np.float64) @ w2.astype(np.float64).T + c.bias.astype(np.float64)
    np.testing.assert_allclose(y.reshape(-1, 8), yl, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(yl, ym, rtol=1e-13, atol=1e-13)


def test_linearity_tap_decomposition_and_zero_tap_pruning():
    c = inputs.conv_case(N=1, H=6, W=6, C=8, K=8, Mb=4, Nb=2, keep=4, dtype="f32", act="normal",
                         w_sigma=1.0, bias=False, seed=25)
    kw = dict(Mb=4, Nb=2)
    w2 = inputs.rng_for(26).standard_normal(c.w.shape)
    y1 = oracle.conv2d_bp(c.x, c.w, c.tap_mask, **kw)
    y2 = oracle.conv2d_bp(c.x, w2, c.tap_mask, **kw)
    y12 = oracle.conv2d_bp(c.x, c.w.astype(np.float64) + w2, c.tap_mask, **kw)
    np.testing.assert_allclose(y12, y1 + y2, rtol=1e-12, atol=1e-12)
    parts = np.zeros_like(y1)
    for t in range(9):
        parts += oracle.conv2d_bp(c.x, c.w, c.tap_mask & np.uint64(1 << t), **kw)
    np.testing.assert_allclose(parts, y1, rtol=1e-12, atol=1e-12)
    # pruning a tap whose weights are already zero changes nothing
    wz = c.w.copy()
    wz[:, 0, 0, :] = 0
    ya = oracle.conv2d_bp(c.x, wz, c.tap_mask, **kw)
    yb = oracle.conv2d_bp(c.x, wz, c.tap_mask & ~np.uint64(1), **kw)
    assert np.array_equal(ya, yb)


def test_points_api_matches_full_and_relu_bias_residual():
    c = inputs.conv_case(N=2, H=6, W=6, C=8, K=8, Mb=4, Nb=4, keep=3, dtype="bf16", residual=True,
                         seed=27)
    kw = dict(Mb=4, Nb=4, bias=c.bias, residual=c.residual, relu=True)
    y = oracle.conv2d_bp(c.x, c.w, c.tap_mask, **kw)
    lin = oracle.conv2d_bp(c.x, c.w, c.tap_mask, Mb=4, Nb=4)
    np.testing.assert_allclose(y, np.maximum(lin + c.bias.astype(np.float64) + c.residual, 0), atol=1e-13)
    pts = np.array([[0, 0, 0, 0], [1, 5, 5, 7], [1, 2, 3, 4], [0, 5, 0, 3]], dtype=np.int32)
    yp = oracle.conv2d_bp(c.x, c.w, c.tap_mask, points=pts, **kw)
    assert np.array_equal(yp, y[pts[:, 0], pts[:, 1], pts[:, 2], pts[:, 3]])


def test_kept_mac_count_formula():
    c = inputs.config1()
    m = oracle.bp_element_mask(c.tap_mask, c.K, c.C, 3, 3, c.Mb, c.Nb)
    assert c.kept_macs() == c.N * c.P * c.Q * int(m.sum())
    assert c.kept_macs() == 16 * 16 * 32 * 32 * 3
