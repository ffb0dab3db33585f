"""Block-based pruned GEMM: CUDA kernels vs the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2012_00596_b200 as npas
from paper_2012_00596_b200 import inputs
from dispatch_table import LINEAR_AUTO, LINEAR_CASES, LINEAR_TAKES, UNSUPPORTED
from util import TOL_BF16, TOL_F32, dev, floored_rel_err, host

pytestmark = pytest.mark.gpu


def run_case(c, path=0, out_dtype=None):
    x, w = dev(c.x, c.dtype), dev(c.w, c.dtype)
    blob = npas.pack_bb(w, c.row_keep, c.col_keep, c.Bo, c.Bi)
    ws = npas.workspace()
    y = npas.linear_bb(x, blob, dev(c.bias), relu=c.relu, out_dtype=out_dtype, ws=ws, path=path)
    npas.check_device_status(ws)
    return y


def oracle_case(c):
    return oracle.linear_bb(c.x, c.w, c.row_keep, c.col_keep, Bo=c.Bo, Bi=c.Bi, bias=c.bias, relu=c.relu)


@pytest.mark.parametrize("kw", [
    dict(M=37, I=48, O=40, Bo=8, Bi=16, keep_rows=3, keep_cols=5),
    dict(M=130, I=64, O=64, Bo=64, Bi=64, keep_rows=lambda a, b: 17, keep_cols=lambda a, b: 9),
    dict(M=5, I=12, O=9, Bo=3, Bi=4, keep_rows=lambda a, b: (a + b) % 4, keep_cols=lambda a, b: (a * 2 + b) % 5),
])
def test_simt_fp32(kw):
    c = inputs.linear_case(dtype="f32", w_sigma=0.3, seed=301, **kw)
    assert floored_rel_err(host(run_case(c)), oracle_case(c)) < TOL_F32


@pytest.mark.parametrize("path", sorted(LINEAR_TAKES))
@pytest.mark.parametrize("idx", range(len(LINEAR_CASES) - 1))
def test_bf16_forced_paths_match_oracle(idx, path):
    """Every (case, forced kernel) pair of the committed table; pairs not listed must be declined."""
    c = inputs.linear_case(dtype="bf16", seed=302, **LINEAR_CASES[idx])
    if idx not in LINEAR_TAKES[path]:
        with pytest.raises(npas.NpasError) as e:
            run_case(c, path=path)
        assert e.value.code == UNSUPPORTED
        return
    y = run_case(c, path=path)
    assert y.dtype == torch.bfloat16
    assert floored_rel_err(host(y), oracle_case(c)) < TOL_BF16


@pytest.mark.parametrize("idx", range(len(LINEAR_CASES)))
def test_bf16_automatic_choice(idx):
    c = inputs.linear_case(dtype="bf16", seed=302, **LINEAR_CASES[idx])
    blob = npas.pack_bb(dev(c.w, "bf16"), c.row_keep, c.col_keep, c.Bo, c.Bi)
    assert npas.linear_bb_kernel(c.M, blob, relu=c.relu, bias=True) == LINEAR_AUTO[idx]
    assert floored_rel_err(host(run_case(c)), oracle_case(c)) < TOL_BF16


@pytest.mark.parametrize("path", sorted(LINEAR_TAKES))
@pytest.mark.parametrize("out_dtype", [None, torch.float32])
def test_residual_epilogue(path, out_dtype):
    c = inputs.linear_case(dtype="bf16", seed=304, **LINEAR_CASES[6])
    assert 6 in LINEAR_TAKES[path]
    ydt = torch.bfloat16 if out_dtype is None else out_dtype
    res = (torch.randn(300, 256, generator=torch.Generator().manual_seed(5)) * 2).to(ydt)
    x, w = dev(c.x, c.dtype), dev(c.w, c.dtype)
    blob = npas.pack_bb(w, c.row_keep, c.col_keep, c.Bo, c.Bi)
    ws = npas.workspace()
    y = npas.linear_bb(x, blob, dev(c.bias), res.cuda(), relu=True, out_dtype=out_dtype, ws=ws, path=path)
    npas.check_device_status(ws)
    ref = oracle.linear_bb(c.x, c.w, c.row_keep, c.col_keep, Bo=c.Bo, Bi=c.Bi, bias=c.bias,
                           residual=res.to(torch.float64).numpy(), relu=True)
    assert floored_rel_err(host(y), ref) < TOL_BF16


@pytest.mark.parametrize("path", [5, 6])
@pytest.mark.parametrize("with_res", [False, True])
@pytest.mark.parametrize("I,O", [(64, 256), (128, 512), (256, 128)])
def test_many_tiles_per_cta_epilogue_ring(I, O, with_res, path):
    """More output tiles than SMs, so that every CTA walks several tiles and the ring of epilogue
    slots (residual slabs in, output slabs out) wraps; the last row tile is ragged."""
    M = 148 * 128 * 2 + 77
    c = inputs.linear_case(M=M, I=I, O=O, Bo=64, Bi=64, keep_rows=32, keep_cols=32, dtype="bf16", seed=305)
    res = (torch.randn(M, O, generator=torch.Generator().manual_seed(7)) * 2).to(torch.bfloat16) if with_res else None
    x, w = dev(c.x, c.dtype), dev(c.w, c.dtype)
    blob = npas.pack_bb(w, c.row_keep, c.col_keep, c.Bo, c.Bi)
    ws = npas.workspace()
    y = npas.linear_bb(x, blob, dev(c.bias), res.cuda() if with_res else None, relu=True, ws=ws, path=path)
    npas.check_device_status(ws)
    ref = oracle.linear_bb(c.x, c.w, c.row_keep, c.col_keep, Bo=c.Bo, Bi=c.Bi, bias=c.bias,
                           residual=res.to(torch.float64).numpy() if with_res else None, relu=True)
    assert floored_rel_err(host(y), ref) < TOL_BF16
    y2 = npas.linear_bb(x, blob, dev(c.bias), res.cuda() if with_res else None, relu=True, ws=ws, path=path)
    assert torch.equal(y, y2)


def test_subsample2d_is_a_strided_pixel_copy():
    x = torch.randn(3, 9, 7, 64, generator=torch.Generator().manual_seed(6)).to(torch.bfloat16).cuda()
    y = npas.subsample2d(x, 2)
    assert torch.equal(y, x[:, ::2, ::2, :].contiguous())


def test_row_block_with_no_kept_column_gives_bias_only():
    c = inputs.linear_case(M=130, I=128, O=128, Bo=64, Bi=64, keep_rows=8, keep_cols=lambda a, b: 0 if a == 0 else 8,
                           dtype="bf16", relu=False, seed=303)
    ref = oracle_case(c)
    for path in (1, 3, 5):
        y = host(run_case(c, path=path, out_dtype=torch.float32))
        assert floored_rel_err(y, ref) < 2e-3
        assert np.array_equal(y[:, :64], np.broadcast_to(c.bias[:64], y[:, :64].shape))


@pytest.mark.parametrize("path", [0, 3, 5, 6])
def test_config3_full_size(path):
    c = inputs.config3()
    y = run_case(c, path=path)
    assert tuple(y.shape) == (3136, 2048)
    assert floored_rel_err(host(y), oracle_case(c)) < TOL_BF16
    assert torch.equal(y, run_case(c, path=path))
