"""CPU oracle (test infrastructure, never a product path).

fp64 restatement of block-punched convolution and block-based pruned GEMM (paper Sec. 3) in
plain C (``npas_oracle.c``), plus a numpy restatement of the packed-weight formats
(``packers.py``).  Only the tests, the smoke check and the benchmark's CPU-baseline leg import
this package; it imports nothing from the CUDA library.

Every function here is pinned by CPU tests against brute force, library routines, closed forms
and structural invariants; none is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "npas_oracle.c")
_LIB_PATH = os.path.join(_HERE, "_build", "libnpas_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over output rows) and return the library path."""
    os.makedirs(os.path.dirname(_LIB_PATH), exist_ok=True)
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(_SRC)):
        return _LIB_PATH
    tmp = _LIB_PATH + f".tmp{os.getpid()}"
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99",
                           "-o", tmp, _SRC])
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def _ptr(a, ty=ctypes.c_double):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ty))


def conv2d_bp(x, w, tap_mask, *, Mb, Nb, stride=1, pad=1, bias=None, residual=None, relu=False,
              points=None):
    """Block-punched convolution by definition (paper Sec. 3), fp64.

    x [N,H,W,C], w [K,R,S,C] dense and unmasked, tap_mask [K/Mb, C/Nb] uint64 (bit r*S+s = kept).
    Returns y [N,P,Q,K] float64, or the values at ``points`` ([n,4] int32 rows n,p,q,k).
    """
    lib = _load()
    x, w, bias, residual = _f64(x), _f64(w), _f64(bias), _f64(residual)
    N, H, W, C = x.shape
    K, R, S, C2 = w.shape
    assert C2 == C
    tm = np.ascontiguousarray(tap_mask, dtype=np.uint64)
    assert tm.shape == (K // Mb, C // Nb)
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    args = [N, H, W, C, K, R, S, stride, pad, Mb, Nb, _ptr(x), _ptr(w),
            _ptr(tm, ctypes.c_uint64), _ptr(bias), _ptr(residual), int(bool(relu))]
    if points is None:
        y = np.empty((N, P, Q, K), dtype=np.float64)
        rc = lib.oracle_conv2d_bp(*args, _ptr(y))
    else:
        idx = np.ascontiguousarray(points, dtype=np.int32)
        y = np.empty((idx.shape[0],), dtype=np.float64)
        rc = lib.oracle_conv2d_bp_points(*args, _ptr(idx, ctypes.c_int32),
                                         ctypes.c_int64(idx.shape[0]), _ptr(y))
    if rc != 0:
        raise ValueError("oracle_conv2d_bp: bad geometry")
    return y


def linear_bb(x, w, row_keep, col_keep, *, Bo, Bi, bias=None, residual=None, relu=False, points=None):
    """Block-based pruned GEMM by definition (paper Sec. 3), fp64.

    x [M,I], w [O,I] dense and unmasked, row_keep/col_keep [O/Bo, I/Bi] uint64 bitsets;
    residual [M,O] (a shortcut branch) is added before the activation.
    Returns y [M,O] float64, or the values at ``points`` ([n,2] int32 rows m,o).
    """
    lib = _load()
    x, w, bias, residual = _f64(x), _f64(w), _f64(bias), _f64(residual)
    M, I = x.shape
    O, I2 = w.shape
    assert I2 == I and (residual is None or residual.shape == (M, O))
    rk = np.ascontiguousarray(row_keep, dtype=np.uint64)
    ck = np.ascontiguousarray(col_keep, dtype=np.uint64)
    assert rk.shape == (O // Bo, I // Bi) and ck.shape == rk.shape
    args = [M, I, O, Bo, Bi, _ptr(x), _ptr(w), _ptr(rk, ctypes.c_uint64),
            _ptr(ck, ctypes.c_uint64), _ptr(bias), _ptr(residual), int(bool(relu))]
    if points is None:
        y = np.empty((M, O), dtype=np.float64)
        rc = lib.oracle_linear_bb(*args, _ptr(y))
    else:
        idx = np.ascontiguousarray(points, dtype=np.int32)
        y = np.empty((idx.shape[0],), dtype=np.float64)
        rc = lib.oracle_linear_bb_points(*args, _ptr(idx, ctypes.c_int32),
                                         ctypes.c_int64(idx.shape[0]), _ptr(y))
    if rc != 0:
        raise ValueError("oracle_linear_bb: bad geometry")
    return y


def maxpool2d(x, *, R=3, stride=2, pad=1):
    lib = _load()
    x = _f64(x)
    N, H, W, C = x.shape
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - R) // stride + 1
    y = np.empty((N, P, Q, C), dtype=np.float64)
    lib.oracle_maxpool2d(N, H, W, C, R, stride, pad, _ptr(x), _ptr(y))
    return y


def prune_bp(w, *, Mb, Nb, keep):
    """One-shot magnitude pruning, block-punched (paper Sec. 5.2): per block keep the `keep` taps with
    the largest sum of squares.  w [K,R,S,C] -> tap bitsets [K/Mb, C/Nb] uint64."""
    lib = _load()
    w = _f64(w)
    K, R, S, C = w.shape
    tm = np.zeros((K // Mb, C // Nb), dtype=np.uint64)
    if lib.oracle_prune_bp(K, C, R, S, Mb, Nb, _ptr(w), int(keep), _ptr(tm, ctypes.c_uint64)) != 0:
        raise ValueError("oracle_prune_bp: bad geometry")
    return tm


def prune_bp_global(w, *, Mb, Nb, n_keep):
    """One-shot magnitude pruning to a layer-wide budget (paper Sec. 5.2, rates of Table 1): of all
    (block, tap) groups of the layer keep the ``n_keep`` with the largest sum of squares, ties to the
    lower group index.  w [K,R,S,C] -> tap bitsets [K/Mb, C/Nb] uint64 (counts differ between blocks)."""
    lib = _load()
    w = _f64(w)
    K, R, S, C = w.shape
    tm = np.zeros((K // Mb, C // Nb), dtype=np.uint64)
    if lib.oracle_prune_bp_global(K, C, R, S, Mb, Nb, _ptr(w), ctypes.c_int64(int(n_keep)), _ptr(tm, ctypes.c_uint64)) != 0:
        raise ValueError("oracle_prune_bp_global: bad geometry")
    return tm


def prune_bb(w, *, Bo, Bi, keep_rows, keep_cols):
    """One-shot magnitude pruning, block-based (paper Sec. 5.2): per block keep the rows and the columns
    with the largest sum of squares.  w [O,I] -> (row bitsets, column bitsets) [O/Bo, I/Bi] uint64."""
    lib = _load()
    w = _f64(w)
    O, I = w.shape
    rk = np.zeros((O // Bo, I // Bi), dtype=np.uint64)
    ck = np.zeros_like(rk)
    if lib.oracle_prune_bb(O, I, Bo, Bi, _ptr(w), int(keep_rows), int(keep_cols), _ptr(rk, ctypes.c_uint64),
                           _ptr(ck, ctypes.c_uint64)) != 0:
        raise ValueError("oracle_prune_bb: bad geometry")
    return rk, ck


from .packers import (bp_element_mask, bb_element_mask, pack_bp, unpack_bp, pack_bb,  # noqa: E402
                      unpack_bb, f32_to_bf16_bits)
