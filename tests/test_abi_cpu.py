"""CPU-only checks of the C-ABI library: it loads, exports what the header declares, and its
host-side logic (sizes, argument validation) behaves - no kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2012_00596_b200 as npas
from paper_2012_00596_b200 import binding, build, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def test_exports_every_declared_symbol(lib):
    hdr = open(os.path.join(ROOT, "include", "npas.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(npas_[a-z0-9_]+)\s*\(", hdr))
    assert len(declared) >= 16
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(binding.EXPORTS)


def test_status_strings_and_version(lib):
    assert lib.npas_abi_version() == 1
    seen = {npas.status_string(c) for c in range(11)}
    assert len(seen) == 11 and npas.status_string(0) == "ok"
    assert npas.status_string(99) == "unknown status"


@pytest.mark.parametrize("Mb,Nb,dt", [(8, 4, 0), (16, 8, 1), (16, 16, 1), (32, 32, 1)])
def test_pack_bp_size_matches_oracle_blob(lib, Mb, Nb, dt):
    K, C = 2 * Mb, 3 * Nb
    c = inputs.conv_case(N=1, H=4, W=4, C=C, K=K, Mb=Mb, Nb=Nb, keep=lambda fb, cb: (fb + 2 * cb) % 10, seed=3)
    d = binding.BpDesc(K, C, 3, 3, Mb, Nb, 0, dt)
    size = ctypes.c_size_t(0)
    tm = np.ascontiguousarray(c.tap_mask)
    assert lib.npas_pack_bp_size(ctypes.byref(d), tm.ctypes.data_as(ctypes.c_void_p), ctypes.byref(size)) == 0
    assert size.value == oracle.pack_bp(c.w, c.tap_mask, Mb, Nb, "f32" if dt == 0 else "bf16").size


def test_pack_bb_size_matches_oracle_blob(lib):
    c = inputs.linear_case(M=1, I=128, O=192, Bo=64, Bi=64, keep_rows=lambda a, b: 5 * a + b,
                           keep_cols=lambda a, b: 7 * b + a + 1, seed=4)
    d = binding.BbDesc(192, 128, 64, 64, 0, 1)
    size = ctypes.c_size_t(0)
    rk, ck = np.ascontiguousarray(c.row_keep), np.ascontiguousarray(c.col_keep)
    assert lib.npas_pack_bb_size(ctypes.byref(d), rk.ctypes.data_as(ctypes.c_void_p),
                                 ck.ctypes.data_as(ctypes.c_void_p), ctypes.byref(size)) == 0
    assert size.value == oracle.pack_bb(c.w, c.row_keep, c.col_keep, 64, 64, "bf16").size


def test_host_side_argument_errors(lib):
    size = ctypes.c_size_t(0)
    tm = np.zeros(4, dtype=np.uint64)
    bad = binding.BpDesc(30, 32, 3, 3, 8, 4, 0, 0)            # K % Mb != 0
    assert lib.npas_pack_bp_size(ctypes.byref(bad), tm.ctypes.data_as(ctypes.c_void_p), ctypes.byref(size)) == 2
    ok = binding.BpDesc(32, 32, 3, 3, 8, 4, 0, 0)
    assert lib.npas_pack_bp_size(ctypes.byref(ok), None, ctypes.byref(size)) == 1
    assert lib.npas_pack_bp_size(None, tm.ctypes.data_as(ctypes.c_void_p), ctypes.byref(size)) == 1
    widen = binding.BpDesc(32, 32, 3, 3, 8, 4, 1, 0)           # bf16 in, f32 packed
    assert lib.npas_pack_bp_size(ctypes.byref(widen), tm.ctypes.data_as(ctypes.c_void_p), ctypes.byref(size)) == 3
    big = binding.BbDesc(256, 256, 128, 64, 0, 0)              # Bo > 64
    assert lib.npas_pack_bb_size(ctypes.byref(big), tm.ctypes.data_as(ctypes.c_void_p),
                                 tm.ctypes.data_as(ctypes.c_void_p), ctypes.byref(size)) == 2
    # compute calls reject bad arguments before touching the device
    cd = binding.ConvDesc(1, 8, 8, 32, 32, 3, 3, 1, 1, 0, 0, 0, 0, 0, 0)
    null = ctypes.c_void_p(0)
    p16, p8 = ctypes.c_void_p(4096), ctypes.c_void_p(4104)
    n256 = ctypes.c_size_t(256)
    assert lib.npas_conv2d_bp(ctypes.byref(cd), ctypes.byref(ok), null, p16, null, null, p16, p16, n256, null) == 1
    assert lib.npas_conv2d_bp(ctypes.byref(cd), ctypes.byref(ok), p8, p16, null, null, ctypes.c_void_p(8192), p16, n256, null) == 4
    assert lib.npas_conv2d_bp(ctypes.byref(cd), ctypes.byref(ok), p16, p16, null, null, ctypes.c_void_p(8192), p16,
                              ctypes.c_size_t(8), null) == 7
    cd_bad = binding.ConvDesc(1, 8, 8, 16, 32, 3, 3, 1, 1, 0, 0, 0, 0, 0, 0)   # C differs from the blob's
    assert lib.npas_conv2d_bp(ctypes.byref(cd_bad), ctypes.byref(ok), p16, p16, null, null, ctypes.c_void_p(8192),
                              p16, n256, null) == 2
    cd_tc = binding.ConvDesc(1, 8, 8, 32, 32, 3, 3, 1, 1, 0, 0, 0, 0, 0, 2)    # tcgen05 forced on an fp32 layer
    assert lib.npas_conv2d_bp(ctypes.byref(cd_tc), ctypes.byref(ok), p16, p16, null, null, ctypes.c_void_p(8192),
                              p16, n256, null) == 8
    ld = binding.LinearDesc(4, 64, 64, 0, 1, 0, 0, 0, 0)       # f32 in, bf16 out
    bb = binding.BbDesc(64, 64, 16, 16, 0, 0)
    assert lib.npas_linear_bb(ctypes.byref(ld), ctypes.byref(bb), p16, p16, null, null, ctypes.c_void_p(8192), p16, n256,
                              null) == 3
    ld_res = binding.LinearDesc(4, 64, 64, 1, 1, 0, 0, 1, 0)   # residual announced but not passed
    bb16 = binding.BbDesc(64, 64, 16, 16, 1, 1)
    assert lib.npas_linear_bb(ctypes.byref(ld_res), ctypes.byref(bb16), p16, p16, null, null, ctypes.c_void_p(8192), p16,
                              n256, null) == 1
    assert lib.npas_subsample2d(1, 8, 8, 12, 2, 2, p16, ctypes.c_void_p(8192), null) == 2   # 24-byte pixels
    assert lib.npas_subsample2d(1, 8, 8, 16, 2, 3, p16, ctypes.c_void_p(8192), null) == 3
