"""Block-punched convolution: CUDA kernels vs the fp64 oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
import paper_2012_00596_b200 as npas
from paper_2012_00596_b200 import inputs
from dispatch_table import CONV_AUTO, CONV_CASES, CONV_TAKES, UNSUPPORTED
from util import TOL_BF16, TOL_F32, dev, floored_rel_err, host

pytestmark = pytest.mark.gpu


def run_case(c, path=0, out_dtype=None, variant=0):
    dt = c.dtype
    x, w = dev(c.x, dt), dev(c.w, dt)
    blob = npas.pack_bp(w, c.tap_mask, c.Mb, c.Nb)
    bias = dev(c.bias)
    res = dev(c.residual, dt if out_dtype is None else "f32")
    ws = npas.workspace()
    y = npas.conv2d_bp(x, blob, bias, res, stride=c.stride, pad=c.pad, relu=c.relu, out_dtype=out_dtype, ws=ws,
                       path=path, variant=variant)
    npas.check_device_status(ws)
    return y


def kernel_of(c, path=0):
    """Which kernel the call would run (host-side query, same descriptor as run_case builds)."""
    blob = npas.pack_bp(dev(c.w, c.dtype), c.tap_mask, c.Mb, c.Nb)
    return npas.conv2d_bp_kernel(c.x.shape, blob, stride=c.stride, pad=c.pad, relu=c.relu, bias=c.bias is not None,
                                 residual=c.residual is not None, path=path)


def oracle_case(c):
    return oracle.conv2d_bp(c.x, c.w, c.tap_mask, Mb=c.Mb, Nb=c.Nb, stride=c.stride, pad=c.pad, bias=c.bias,
                            residual=c.residual, relu=c.relu)


def test_config1_fp32():
    c = inputs.config1()
    y = run_case(c)
    assert y.dtype == torch.float32 and tuple(y.shape) == (1, 16, 16, 32)
    assert floored_rel_err(host(y), oracle_case(c)) < TOL_F32


@pytest.mark.parametrize("kw", [
    dict(N=2, H=9, W=7, C=16, K=24, Mb=8, Nb=4, keep=3, stride=2),
    dict(N=1, H=8, W=8, C=12, K=10, Mb=5, Nb=3, keep=lambda fb, cb: (fb + cb) % 10),
    dict(N=1, H=6, W=6, C=8, K=8, Mb=1, Nb=1, keep=lambda fb, cb: (3 * fb + cb) % 10),
    dict(N=3, H=5, W=11, C=8, K=16, Mb=16, Nb=8, keep=4, R=5, S=5, pad=2),
    dict(N=1, H=10, W=10, C=16, K=16, Mb=8, Nb=16, keep=1, R=1, S=1, pad=0, stride=2),
])
def test_simt_fp32_geometries(kw):
    c = inputs.conv_case(dtype="f32", act="normal", w_sigma=0.3, residual=True, seed=201, **kw)
    y = run_case(c)
    assert floored_rel_err(host(y), oracle_case(c)) < TOL_F32


@pytest.mark.parametrize("path", sorted(CONV_TAKES))
@pytest.mark.parametrize("idx", range(len(CONV_CASES)))
def test_bf16_forced_paths_match_oracle(idx, path):
    """Every (case, forced kernel) pair of the committed table: listed pairs must match the oracle, the
    others must be declined by the query and by the call.  No skips."""
    c = inputs.conv_case(dtype="bf16", residual=True, seed=202, **CONV_CASES[idx])
    if idx not in CONV_TAKES[path]:
        with pytest.raises(npas.NpasError) as e:
            kernel_of(c, path)
        assert e.value.code == UNSUPPORTED
        with pytest.raises(npas.NpasError) as e:
            run_case(c, path=path)
        assert e.value.code == UNSUPPORTED
        return
    assert kernel_of(c, path) == path
    y = run_case(c, path=path)
    assert y.dtype == torch.bfloat16
    assert floored_rel_err(host(y), oracle_case(c)) < TOL_BF16


@pytest.mark.parametrize("idx", range(len(CONV_CASES)))
def test_bf16_automatic_choice_matches_oracle(idx):
    c = inputs.conv_case(dtype="bf16", residual=True, seed=202, **CONV_CASES[idx])
    assert kernel_of(c, 0) == CONV_AUTO[idx]
    assert floored_rel_err(host(run_case(c)), oracle_case(c)) < TOL_BF16


@pytest.mark.parametrize("path", [1, 5])
@pytest.mark.parametrize("kw", [
    dict(N=2, H=32, W=32, K=64, keep=49),                    # dense first layer, tiles span several rows
    dict(N=1, H=33, W=30, K=32, keep=20),                    # punched, odd height, ragged last tile
    dict(N=1, H=224, W=224, K=64, keep=49),                  # the ImageNet stem shape
])
def test_three_channel_first_layer(kw, path):
    c = inputs.conv_case(C=3, Mb=16, Nb=3, R=7, S=7, stride=2, pad=3, dtype="bf16", act="normal", w_sigma=0.1,
                         seed=207, **kw)
    y = run_case(c, path=path)
    assert floored_rel_err(host(y), oracle_case(c)) < TOL_BF16


def test_bf16_no_bias_no_relu_f32_out():
    c = inputs.conv_case(N=2, H=14, W=14, C=64, K=64, Mb=16, Nb=8, keep=3, dtype="bf16", bias=False, relu=False, seed=203)
    for path in (1, 3, 6):
        y = run_case(c, path=path, out_dtype=torch.float32)
        assert y.dtype == torch.float32
        assert floored_rel_err(host(y), oracle_case(c)) < 2e-3


def test_filter_block_without_any_kept_tap_gives_bias_only():
    c = inputs.conv_case(N=1, H=14, W=14, C=32, K=48, Mb=16, Nb=8, keep=lambda fb, cb: 0 if fb == 1 else 3,
                         dtype="bf16", relu=False, seed=204)
    ref = oracle_case(c)
    for path in (1, 3, 6):
        y = host(run_case(c, path=path))
        assert floored_rel_err(y, ref) < TOL_BF16
        assert np.array_equal(y[..., 16:32], np.broadcast_to(inputs.bf16_representable(c.bias[16:32]), y[..., 16:32].shape))


@pytest.mark.parametrize("kw", [
    dict(N=3, H=14, W=14, C=64, K=128, Mb=16, Nb=8, keep=3),                     # 6 tiles: three pairs, 64 filters per CTA
    dict(N=1, H=7, W=7, C=64, K=256, Mb=16, Nb=16, keep=3),                      # one tile: the peer CTA has none of its own
    dict(N=5, H=14, W=14, C=192, K=256, Mb=32, Nb=16, keep=2),                   # three 64-channel blocks
    dict(N=40, H=14, W=14, C=64, K=128, Mb=16, Nb=8, keep=3),                    # more items than pairs: accumulators alternate
    dict(N=48, H=14, W=14, C=64, K=256, Mb=16, Nb=8, keep=lambda fb, cb: (fb + 2 * cb) % 10),
    dict(N=9, H=28, W=28, C=64, K=384, Mb=16, Nb=16, keep=3, stride=2),          # strided, three filter sets of 128
    dict(N=2, H=9, W=9, C=64, K=128, Mb=16, Nb=8, keep=1, R=1, S=1, pad=0),      # 1x1 layer
    dict(N=2, H=14, W=14, C=64, K=128, Mb=128, Nb=64, keep=3),                   # whole-layer block: six taps skipped everywhere
    dict(N=2, H=56, W=56, C=64, K=128, Mb=16, Nb=16, keep=4),                    # two image rows per tile
    dict(N=1, H=6, W=126, C=64, K=128, Mb=16, Nb=8, keep=3),                     # widest image the tile takes
    dict(N=3, H=15, W=13, C=64, K=128, Mb=16, Nb=16, keep=4, stride=2),          # strided by phases: odd H and W
    dict(N=2, H=56, W=56, C=128, K=128, Mb=16, Nb=8, keep=3, stride=2),          # strided by phases: four output rows per tile
    dict(N=2, H=14, W=14, C=64, K=128, Mb=16, Nb=8, keep=9, stride=2),           # strided by phases: the whole 7x7 output in one tile
    dict(N=5, H=7, W=7, C=128, K=256, Mb=16, Nb=8, keep=3),                      # two 7x7 images per tile, the last tile holds one
    dict(N=64, H=7, W=7, C=64, K=512, Mb=16, Nb=8, keep=3),                      # two images per tile, one item per pair
    dict(N=7, H=4, W=4, C=64, K=128, Mb=16, Nb=16, keep=4),                      # four 4x4 images per tile
    dict(N=3, H=5, W=7, C=64, K=64, Mb=16, Nb=8, keep=9),                        # two 5x7 images per tile, every tap, 64 filters
    dict(N=9, H=8, W=8, C=64, K=128, Mb=16, Nb=8, keep=5, stride=2),             # by phases: five 4x4 outputs per tile
    dict(N=5, H=13, W=13, C=64, K=128, Mb=16, Nb=8, keep=9, stride=2),           # by phases: two 7x7 outputs per tile, odd input
])
def test_cta_pair_kernel_matches_oracle(kw):
    c = inputs.conv_case(dtype="bf16", residual=True, seed=208, **kw)
    y = run_case(c, path=7)
    ref = oracle_case(c)
    assert floored_rel_err(host(y), ref) < TOL_BF16
    assert torch.equal(y, run_case(c, path=7))                                   # run-to-run determinism


@pytest.mark.parametrize("stride", [1, 2])
def test_cta_pair_kernel_declines_25_taps(stride):
    c = inputs.conv_case(N=2, H=12, W=12, C=64, K=128, Mb=16, Nb=8, keep=5, R=5, S=5, pad=2, stride=stride, dtype="bf16",
                         residual=True, seed=208)
    with pytest.raises(npas.NpasError) as e:
        run_case(c, path=7)
    assert e.value.code == UNSUPPORTED


@pytest.mark.parametrize("shape", [(128, 1), (128, 2), (256, 1), (256, 2)])
@pytest.mark.parametrize("kw", [
    dict(N=21, H=14, W=14, C=128, K=256, Mb=16, Nb=8, keep=3),                   # 42 tiles: the last item lacks tiles
    dict(N=100, H=14, W=14, C=64, K=256, Mb=16, Nb=16, keep=2, stride=2),        # more items than CTA pairs
])
def test_cta_pair_kernel_every_item_shape(kw, shape):
    """Filters per item (128 or 256) x position tiles per CTA (1 or 2), each forced through the call
    descriptor's `variant`."""
    c = inputs.conv_case(dtype="bf16", residual=True, seed=209, **kw)
    if kw.get("stride", 1) == 2 and shape[1] == 2:
        # by phases a CTA stages four slabs per position tile: two tiles do not fit in shared memory
        with pytest.raises(npas.NpasError) as e:
            run_case(c, path=7, variant=shape[0] | (shape[1] << 16))
        assert e.value.code == UNSUPPORTED
        return
    y = run_case(c, path=7, variant=shape[0] | (shape[1] << 16))
    assert floored_rel_err(host(y), oracle_case(c)) < TOL_BF16


@pytest.mark.parametrize("kw", [
    dict(N=1, H=28, W=28, C=64, K=96, Mb=16, Nb=16, keep=3),                     # group of two blocks (96 = 3 x 32 filters)
    dict(N=2, H=7, W=7, C=128, K=64, Mb=32, Nb=32, keep=5),                      # two chunks per channel block
    dict(N=1, H=12, W=12, C=64, K=64, Mb=64, Nb=64, keep=2),                     # one block per group, four chunks per block
    dict(N=3, H=7, W=7, C=64, K=512, Mb=16, Nb=16, keep=9),                      # dense: every run spans its whole segment
    dict(N=2, H=14, W=14, C=64, K=256, Mb=16, Nb=16, keep=lambda fb, cb: (fb * 3 + cb) % 10),   # 0..9 taps, empty blocks
    dict(N=2, H=14, W=14, C=32, K=256, Mb=16, Nb=16, keep=1),
    dict(N=1, H=28, W=28, C=96, K=64, Mb=32, Nb=32, keep=3),                     # six chunks: stages of two
    dict(N=1, H=56, W=56, C=16, K=16, Mb=16, Nb=16, keep=4),                     # a single chunk (one stager set)
    dict(N=1, H=6, W=126, C=32, K=32, Mb=16, Nb=16, keep=3),                     # widest image the tile takes
    dict(N=5, H=9, W=13, C=48, K=128, Mb=16, Nb=16, keep=5, R=3, S=5, pad=1),    # 15 taps, three chunks
    dict(N=2, H=9, W=9, C=32, K=64, Mb=16, Nb=16, keep=1, R=1, S=1, pad=0),      # 1x1 layer
    dict(N=40, H=14, W=14, C=32, K=512, Mb=16, Nb=32, keep=2),                   # several tiles per CTA, two groups
    dict(N=2, H=14, W=14, C=64, K=256, Mb=128, Nb=16, keep=4),                   # two blocks of 128 filters per group
])
def test_kept_runs_kernel_matches_oracle(kw):
    """The kernel that multiplies kept (block, tap) pairs only (path 8)."""
    c = inputs.conv_case(dtype="bf16", residual=True, seed=210, **kw)
    y = run_case(c, path=8)
    assert floored_rel_err(host(y), oracle_case(c)) < TOL_BF16
    assert torch.equal(y, run_case(c, path=8))                                  # run-to-run determinism


def test_workspace_sized_by_the_query_runs_the_layer():
    """npas_conv2d_bp_workspace tells how much scratch a layer's call can use; a buffer of that size is accepted."""
    c = inputs.conv_case(N=2, H=14, W=14, C=64, K=64, Mb=16, Nb=16, keep=3, dtype="bf16", residual=True, seed=212)
    x, w = dev(c.x, "bf16"), dev(c.w, "bf16")
    blob = npas.pack_bp(w, c.tap_mask, c.Mb, c.Nb)
    ws = npas.conv2d_bp_workspace(c.x.shape, blob, pad=c.pad, relu=c.relu, bias=True, residual=True)
    assert ws.numel() >= npas.binding.WORKSPACE_BYTES and int(ws.max()) == 0
    y = npas.conv2d_bp(x, blob, dev(c.bias), dev(c.residual, "bf16"), pad=c.pad, relu=c.relu, ws=ws)
    npas.check_device_status(ws)
    assert floored_rel_err(host(y), oracle_case(c)) < TOL_BF16


@pytest.mark.parametrize("path", [3, 6, 7])
def test_config2_full_size_each_tensor_kernel(path):
    c = inputs.config2()
    assert floored_rel_err(host(run_case(c, path=path)), oracle_case(c)) < TOL_BF16


def test_broken_tap_promise_is_reported_not_computed():
    """max_taps in the descriptor is a promise the kept-pairs kernel sizes its weight slots by; a blob with
    more kept taps per block must come back as NPAS_ERR_BLOB through the status words, without a fault."""
    c = inputs.conv_case(N=1, H=14, W=14, C=64, K=64, Mb=16, Nb=16, keep=3, dtype="bf16", seed=205)
    x, w = dev(c.x, "bf16"), dev(c.w, "bf16")
    blob = npas.pack_bp(w, c.tap_mask, c.Mb, c.Nb)
    assert blob.desc.max_taps == 3
    blob.desc.max_taps = 1
    ws = npas.workspace()
    npas.conv2d_bp(x, blob, dev(c.bias), relu=True, ws=ws, path=8)
    with pytest.raises(npas.NpasError) as e:
        npas.check_device_status(ws)
    assert e.value.code == 6
    npas.check_device_status(ws)                 # the words were cleared
    blob.desc.max_taps = 0                       # no promise: sized for all taps
    y = npas.conv2d_bp(x, blob, dev(c.bias), relu=True, ws=ws, path=8)
    npas.check_device_status(ws)
    assert floored_rel_err(host(y), oracle_case(c)) < TOL_BF16


def test_config2_full_size():
    c = inputs.config2()
    y = run_case(c)
    ref = oracle_case(c)
    assert tuple(y.shape) == (32, 14, 14, 256)
    assert floored_rel_err(host(y), ref) < TOL_BF16
    # run-to-run determinism (no atomics in the accumulation)
    y2 = run_case(c)
    assert torch.equal(y, y2)


@pytest.mark.parametrize("taps", [1, 2, 3, 5, 9])
@pytest.mark.parametrize("Mb,Nb", [(4, 4), (8, 8), (16, 16), (32, 32)])
def test_config5_full_size_sampled(Mb, Nb, taps):
    """All twenty points of the 64x28x28x512 -> 512 sweep at full size, on sampled outputs the oracle computes
    one by one: the automatic choice, both dense-image kernels and (blocks of 16 and 32) the kept-pairs kernel."""
    c = inputs.config5(Mb, Nb, taps)
    rng = inputs.rng_for(77)
    pts = np.stack([rng.integers(0, 64, 4000), rng.integers(0, 28, 4000), rng.integers(0, 28, 4000),
                    rng.integers(0, 512, 4000)], axis=1).astype(np.int32)
    pts[:8] = [[0, 0, 0, 0], [63, 27, 27, 511], [0, 27, 0, 255], [63, 0, 27, 256], [31, 3, 4, 15], [31, 4, 3, 16],
               [1, 0, 0, 511], [62, 27, 27, 0]]
    ref = oracle.conv2d_bp(c.x, c.w, c.tap_mask, Mb=Mb, Nb=Nb, points=pts)
    x, w = dev(c.x, "bf16"), dev(c.w, "bf16")
    blob = npas.pack_bp(w, c.tap_mask, Mb, Nb)
    ws = npas.workspace()
    y = torch.empty((64, 28, 28, 512), dtype=torch.bfloat16, device="cuda")
    for path in (0, 6, 7) + ((8,) if Mb >= 16 else ()):
        y.zero_()
        npas.conv2d_bp(x, blob, None, None, relu=False, out=y, ws=ws, path=path)
        npas.check_device_status(ws)
        got = host(y)[pts[:, 0], pts[:, 1], pts[:, 2], pts[:, 3]]
        assert floored_rel_err(got, ref) < TOL_BF16, path
    if Mb < 16:
        with pytest.raises(npas.NpasError) as e:
            npas.conv2d_bp(x, blob, None, None, relu=False, out=y, ws=ws, path=8)
        assert e.value.code == UNSUPPORTED
