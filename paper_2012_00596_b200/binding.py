"""ctypes binding over libnpas.so: argument marshalling only, every step runs in the CUDA kernels.

The function names mirror the C ABI (include/npas.h).  Tensors are torch CUDA tensors used purely
as device buffers; calls are enqueued on torch's current stream.  There is no CPU fallback: when
the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnpas.so")
WORKSPACE_BYTES = 256
F32, BF16 = 0, 1
_lib = None


class NpasError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {status_string(code)} (npas_status {code})")
        self.code = code


class BpDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("K", "C", "R", "S", "Mb", "Nb", "w_in", "w_packed", "max_taps")]


class BbDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("O", "I", "Bo", "Bi", "w_in", "w_packed", "max_cols")]


class ConvDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("N", "H", "W", "C", "K", "R", "S", "stride", "pad", "x_dtype",
                                              "y_dtype", "relu", "has_bias", "has_residual", "path", "variant")]


class LinearDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("M", "I", "O", "x_dtype", "y_dtype", "relu", "has_bias", "has_residual", "path",
                                              "variant")]


EXPORTS = ["npas_status_string", "npas_abi_version", "npas_mask_bp_from_dense", "npas_mask_bb_from_dense",
           "npas_pack_bp_size", "npas_pack_bp", "npas_unpack_bp", "npas_pack_bb_size", "npas_pack_bb",
           "npas_unpack_bb", "npas_conv2d_bp", "npas_linear_bb", "npas_blob_check",
           "npas_check_device_status", "npas_launch_count", "npas_maxpool2d", "npas_conv2d_bp_static_ws",
           "npas_subsample2d", "npas_prune_bp_magnitude", "npas_prune_bb_magnitude",
           "npas_conv2d_bp_workspace", "npas_linear_bb_workspace", "npas_conv2d_bp_kernel", "npas_linear_bb_kernel",
           "npas_tune_conv2d_bp", "npas_tune_linear_bb", "npas_prune_bp_global_workspace", "npas_prune_bp_magnitude_global", "npas_conv2d_bp_maxpool"]


def load() -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built (there is no other code path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} is missing: build it with paper_2012_00596_b200/build.py")
        lib = ctypes.CDLL(LIB_PATH)
        for name in EXPORTS:
            getattr(lib, name)
        lib.npas_status_string.restype = ctypes.c_char_p
        lib.npas_status_string.argtypes = [ctypes.c_int]
        lib.npas_abi_version.restype = ctypes.c_uint32
        lib.npas_launch_count.restype = ctypes.c_uint64
        for name in EXPORTS[2:]:
            if name == "npas_launch_count":
                continue
            getattr(lib, name).restype = ctypes.c_int
        _lib = lib
    return _lib


def status_string(code: int) -> str:
    return load().npas_status_string(int(code)).decode()


def launch_count() -> int:
    return int(load().npas_launch_count())


def _check(code: int, what: str):
    if code != 0:
        raise NpasError(code, what)


def _p(t):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _torch_dt(code: int):
    return torch.float32 if code == F32 else torch.bfloat16


def _mask_to_device(mask, device) -> torch.Tensor:
    """uint64 bitsets (numpy or tensor) -> contiguous int64 CUDA tensor holding the same bits."""
    if isinstance(mask, torch.Tensor):
        return mask.to(device=device, dtype=torch.int64).contiguous()
    return torch.from_numpy(np.ascontiguousarray(mask, dtype=np.uint64).view(np.int64)).to(device)


def mask_to_numpy(mask: torch.Tensor) -> np.ndarray:
    return mask.cpu().numpy().view(np.uint64)


@dataclass
class BpBlob:
    data: torch.Tensor          # uint8 device buffer holding the blob
    desc: BpDesc


@dataclass
class BbBlob:
    data: torch.Tensor
    desc: BbDesc


def workspace(device="cuda") -> torch.Tensor:
    """Zeroed device scratch for the compute calls (holds the device status words)."""
    return torch.zeros(WORKSPACE_BYTES, dtype=torch.uint8, device=device)


# ---------------------------------------------------------------------------- packers ----------

def pack_bp(w: torch.Tensor, tap_mask, Mb: int, Nb: int, packed_dtype=None) -> BpBlob:
    """npas_pack_bp: dense KRSC weights + per-block tap bitsets -> blob (on w's device)."""
    lib = load()
    assert w.is_cuda and w.is_contiguous() and w.dim() == 4
    K, R, S, C = w.shape
    w_in = _dt(w)
    w_packed = w_in if packed_dtype is None else (_dt(torch.empty(0, dtype=packed_dtype)))
    host = np.ascontiguousarray(mask_to_numpy(tap_mask) if isinstance(tap_mask, torch.Tensor) else tap_mask,
                                dtype=np.uint64)
    live = (1 << (R * S)) - 1
    max_taps = max((bin(int(v) & live).count("1") for v in host.ravel()), default=0)
    d = BpDesc(K, C, R, S, Mb, Nb, w_in, w_packed, max(1, max_taps))
    size = ctypes.c_size_t(0)
    _check(lib.npas_pack_bp_size(ctypes.byref(d), host.ctypes.data_as(ctypes.c_void_p), ctypes.byref(size)),
           "npas_pack_bp_size")
    dev_mask = _mask_to_device(host, w.device)
    blob = torch.empty(size.value, dtype=torch.uint8, device=w.device)
    _check(lib.npas_pack_bp(ctypes.byref(d), _p(w), _p(dev_mask), _p(blob), ctypes.c_size_t(size.value),
                            _stream()), "npas_pack_bp")
    return BpBlob(blob, d)


def unpack_bp(blob: BpBlob):
    """npas_unpack_bp -> (masked dense weights in the blob's dtype [K,R,S,C], tap_mask int64 [nFB,nCB])."""
    lib = load()
    d = blob.desc
    w = torch.empty((d.K, d.R, d.S, d.C), dtype=_torch_dt(d.w_packed), device=blob.data.device)
    tm = torch.empty((d.K // d.Mb, d.C // d.Nb), dtype=torch.int64, device=blob.data.device)
    _check(lib.npas_unpack_bp(ctypes.byref(d), _p(blob.data), ctypes.c_size_t(blob.data.numel()), _p(w), _p(tm),
                              _stream()), "npas_unpack_bp")
    return w, tm


def pack_bb(w: torch.Tensor, row_keep, col_keep, Bo: int, Bi: int, packed_dtype=None) -> BbBlob:
    lib = load()
    assert w.is_cuda and w.is_contiguous() and w.dim() == 2
    O, I = w.shape
    w_in = _dt(w)
    w_packed = w_in if packed_dtype is None else (_dt(torch.empty(0, dtype=packed_dtype)))
    rk = np.ascontiguousarray(mask_to_numpy(row_keep) if isinstance(row_keep, torch.Tensor) else row_keep, dtype=np.uint64)
    ck = np.ascontiguousarray(mask_to_numpy(col_keep) if isinstance(col_keep, torch.Tensor) else col_keep, dtype=np.uint64)
    live = (1 << Bi) - 1
    max_cols = max((bin(int(v) & live).count("1") for v in ck.ravel()), default=0)
    d = BbDesc(O, I, Bo, Bi, w_in, w_packed, max(1, max_cols))
    size = ctypes.c_size_t(0)
    _check(lib.npas_pack_bb_size(ctypes.byref(d), rk.ctypes.data_as(ctypes.c_void_p),
                                 ck.ctypes.data_as(ctypes.c_void_p), ctypes.byref(size)), "npas_pack_bb_size")
    drk, dck = _mask_to_device(rk, w.device), _mask_to_device(ck, w.device)
    blob = torch.empty(size.value, dtype=torch.uint8, device=w.device)
    _check(lib.npas_pack_bb(ctypes.byref(d), _p(w), _p(drk), _p(dck), _p(blob), ctypes.c_size_t(size.value),
                            _stream()), "npas_pack_bb")
    return BbBlob(blob, d)


def unpack_bb(blob: BbBlob):
    lib = load()
    d = blob.desc
    dev = blob.data.device
    w = torch.empty((d.O, d.I), dtype=_torch_dt(d.w_packed), device=dev)
    rk = torch.empty((d.O // d.Bo, d.I // d.Bi), dtype=torch.int64, device=dev)
    ck = torch.empty_like(rk)
    _check(lib.npas_unpack_bb(ctypes.byref(d), _p(blob.data), ctypes.c_size_t(blob.data.numel()), _p(w), _p(rk),
                              _p(ck), _stream()), "npas_unpack_bb")
    return w, rk, ck


def prune_bp_magnitude(w: torch.Tensor, Mb: int, Nb: int, keep_taps: int) -> torch.Tensor:
    """npas_prune_bp_magnitude: dense KRSC weights -> per-block tap bitsets (int64 tensor on the device)."""
    lib = load()
    assert w.is_cuda and w.is_contiguous() and w.dim() == 4
    K, R, S, C = w.shape
    d = BpDesc(K, C, R, S, Mb, Nb, _dt(w), _dt(w), 0)
    tm = torch.empty((K // Mb, C // Nb), dtype=torch.int64, device=w.device)
    _check(lib.npas_prune_bp_magnitude(ctypes.byref(d), _p(w), int(keep_taps), _p(tm), _stream()), "npas_prune_bp_magnitude")
    return tm


def prune_bp_magnitude_global(w: torch.Tensor, Mb: int, Nb: int, *, rate: float = None, n_keep: int = None) -> torch.Tensor:
    """npas_prune_bp_magnitude_global: keep the ``n_keep`` highest-scoring (block, tap) groups of the whole
    layer (``rate``: n_keep = round(groups / rate), e.g. 2.5 or 7); tap bitsets as an int64 device tensor."""
    lib = load()
    assert w.is_cuda and w.is_contiguous() and w.dim() == 4 and (rate is None) != (n_keep is None)
    K, R, S, C = w.shape
    d = BpDesc(K, C, R, S, Mb, Nb, _dt(w), _dt(w), 0)
    groups = (K // Mb) * (C // Nb) * R * S
    if n_keep is None:
        n_keep = int(np.floor(groups / float(rate) + 0.5))
    size = ctypes.c_size_t(0)
    _check(lib.npas_prune_bp_global_workspace(ctypes.byref(d), ctypes.byref(size)), "npas_prune_bp_global_workspace")
    ws = torch.empty(size.value, dtype=torch.uint8, device=w.device)
    tm = torch.empty((K // Mb, C // Nb), dtype=torch.int64, device=w.device)
    _check(lib.npas_prune_bp_magnitude_global(ctypes.byref(d), _p(w), ctypes.c_int64(int(n_keep)), _p(tm), _p(ws),
                                              ctypes.c_size_t(size.value), _stream()), "npas_prune_bp_magnitude_global")
    return tm


def prune_bb_magnitude(w: torch.Tensor, Bo: int, Bi: int, keep_rows: int, keep_cols: int):
    """npas_prune_bb_magnitude: dense [O,I] weights -> (row bitsets, column bitsets), int64 tensors on the device."""
    lib = load()
    assert w.is_cuda and w.is_contiguous() and w.dim() == 2
    O, I = w.shape
    d = BbDesc(O, I, Bo, Bi, _dt(w), _dt(w), 0)
    rk = torch.empty((O // Bo, I // Bi), dtype=torch.int64, device=w.device)
    ck = torch.empty_like(rk)
    _check(lib.npas_prune_bb_magnitude(ctypes.byref(d), _p(w), int(keep_rows), int(keep_cols), _p(rk), _p(ck), _stream()),
           "npas_prune_bb_magnitude")
    return rk, ck


def mask_bp_from_dense(dense_mask: torch.Tensor, Mb: int, Nb: int) -> torch.Tensor:
    """npas_mask_bp_from_dense: uint8 [K,R,S,C] 0/1 mask -> tap bitsets; raises on a bad structure."""
    lib = load()
    K, R, S, C = dense_mask.shape
    d = BpDesc(K, C, R, S, Mb, Nb, F32, F32)
    m = dense_mask.to(torch.uint8).contiguous()
    tm = torch.empty((K // Mb, C // Nb), dtype=torch.int64, device=m.device)
    viol = torch.zeros(1, dtype=torch.int32, device=m.device)
    _check(lib.npas_mask_bp_from_dense(ctypes.byref(d), _p(m), _p(tm), _p(viol), _stream()),
           "npas_mask_bp_from_dense")
    return tm


def mask_bb_from_dense(dense_mask: torch.Tensor, Bo: int, Bi: int):
    lib = load()
    O, I = dense_mask.shape
    d = BbDesc(O, I, Bo, Bi, F32, F32)
    m = dense_mask.to(torch.uint8).contiguous()
    rk = torch.empty((O // Bo, I // Bi), dtype=torch.int64, device=m.device)
    ck = torch.empty_like(rk)
    viol = torch.zeros(1, dtype=torch.int32, device=m.device)
    _check(lib.npas_mask_bb_from_dense(ctypes.byref(d), _p(m), _p(rk), _p(ck), _p(viol), _stream()),
           "npas_mask_bb_from_dense")
    return rk, ck


def blob_check(blob) -> None:
    lib = load()
    bp = ctypes.byref(blob.desc) if isinstance(blob, BpBlob) else None
    bb = ctypes.byref(blob.desc) if isinstance(blob, BbBlob) else None
    _check(lib.npas_blob_check(bp, bb, _p(blob.data), ctypes.c_size_t(blob.data.numel()), _stream()),
           "npas_blob_check")


# ---------------------------------------------------------------------------- compute ----------

def conv2d_bp(x: torch.Tensor, blob: BpBlob, bias=None, residual=None, *, stride=1, pad=1, relu=False,
              out_dtype=None, out=None, ws=None, path=0, variant=0) -> torch.Tensor:
    """npas_conv2d_bp on NHWC x; returns NHWC y (allocated here unless ``out`` is given)."""
    lib = load()
    assert x.is_cuda and x.is_contiguous() and x.dim() == 4
    N, H, W, C = x.shape
    d = blob.desc
    P = (H + 2 * pad - d.R) // stride + 1
    Q = (W + 2 * pad - d.S) // stride + 1
    ydt = x.dtype if out_dtype is None else out_dtype
    if out is None:
        out = torch.empty((N, P, Q, d.K), dtype=ydt, device=x.device)
    if ws is None:
        ws = workspace(x.device)
    cd = ConvDesc(N, H, W, C, d.K, d.R, d.S, stride, pad, _dt(x), _dt(out), int(bool(relu)),
                  int(bias is not None), int(residual is not None), path, variant)
    _check(lib.npas_conv2d_bp(ctypes.byref(cd), ctypes.byref(d), _p(x), _p(blob.data), _p(bias), _p(residual),
                              _p(out), _p(ws), ctypes.c_size_t(ws.numel()), _stream()), "npas_conv2d_bp")
    return out


def linear_bb(x: torch.Tensor, blob: BbBlob, bias=None, residual=None, *, relu=False, out_dtype=None, out=None,
              ws=None, path=0, variant=0) -> torch.Tensor:
    lib = load()
    assert x.is_cuda and x.is_contiguous() and x.dim() == 2
    M, I = x.shape
    d = blob.desc
    ydt = x.dtype if out_dtype is None else out_dtype
    if out is None:
        out = torch.empty((M, d.O), dtype=ydt, device=x.device)
    if ws is None:
        ws = workspace(x.device)
    if residual is not None:
        assert residual.is_cuda and residual.is_contiguous() and residual.shape == out.shape and residual.dtype == out.dtype
    ld = LinearDesc(M, I, d.O, _dt(x), _dt(out), int(bool(relu)), int(bias is not None), int(residual is not None), path,
                    variant)
    _check(lib.npas_linear_bb(ctypes.byref(ld), ctypes.byref(d), _p(x), _p(blob.data), _p(bias), _p(residual), _p(out),
                              _p(ws), ctypes.c_size_t(ws.numel()), _stream()), "npas_linear_bb")
    return out


def subsample2d(x: torch.Tensor, stride: int) -> torch.Tensor:
    """Y[n,p,q,:] = X[n, p*stride, q*stride, :] (the input of a strided 1x1 convolution run as a GEMM)."""
    lib = load()
    assert x.is_cuda and x.is_contiguous() and x.dim() == 4
    N, H, W, C = x.shape
    y = torch.empty((N, (H - 1) // stride + 1, (W - 1) // stride + 1, C), dtype=x.dtype, device=x.device)
    _check(lib.npas_subsample2d(N, H, W, C, stride, x.element_size(), _p(x), _p(y), _stream()), "npas_subsample2d")
    return y


def check_device_status(ws: torch.Tensor) -> None:
    """Synchronises and raises NpasError(NPAS_ERR_TIMEOUT) if a kernel gave up on a bounded wait."""
    lib = load()
    detail = ctypes.c_int32(0)
    code = lib.npas_check_device_status(_p(ws), _stream(), ctypes.byref(detail))
    if code != 0:
        raise NpasError(code, f"device status (detail 0x{detail.value:x})")


def maxpool2d(x: torch.Tensor, R=3, stride=2, pad=1) -> torch.Tensor:
    lib = load()
    N, H, W, C = x.shape
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - R) // stride + 1
    y = torch.empty((N, P, Q, C), dtype=x.dtype, device=x.device)
    _check(lib.npas_maxpool2d(N, H, W, C, R, stride, pad, _p(x), _p(y), _stream()), "npas_maxpool2d")
    return y


def conv2d_bp_maxpool(x: torch.Tensor, blob: BpBlob, bias=None, *, stride=1, pad=1, relu=True, pool=(3, 2, 1), out=None,
                      ws=None, path=0) -> torch.Tensor:
    """npas_conv2d_bp_maxpool: convolution + bias + ReLU + max-pool fused in one kernel; returns the pooled
    NHWC tensor.  Raises NpasError(8) where no kernel has the fused epilogue (run the two calls then)."""
    lib = load()
    assert x.is_cuda and x.is_contiguous() and x.dim() == 4
    N, H, W, C = x.shape
    d = blob.desc
    P = (H + 2 * pad - d.R) // stride + 1
    Q = (W + 2 * pad - d.S) // stride + 1
    pr, ps, pp = pool
    PP, PQ = (P + 2 * pp - pr) // ps + 1, (Q + 2 * pp - pr) // ps + 1
    if out is None:
        out = torch.empty((N, PP, PQ, d.K), dtype=x.dtype, device=x.device)
    if ws is None:
        ws = workspace(x.device)
    cd = ConvDesc(N, H, W, C, d.K, d.R, d.S, stride, pad, _dt(x), _dt(out), int(bool(relu)), int(bias is not None), 0, path, 0)
    _check(lib.npas_conv2d_bp_maxpool(ctypes.byref(cd), ctypes.byref(d), pr, ps, pp, _p(x), _p(blob.data), _p(bias), _p(out),
                                      _p(ws), ctypes.c_size_t(ws.numel()), _stream()), "npas_conv2d_bp_maxpool")
    return out


def conv2d_bp_static_ws(x: torch.Tensor, blob: BpBlob, bias=None, residual=None, *, stride=1, pad=1, relu=False,
                        out_dtype=None, out=None, path=0, check=True) -> torch.Tensor:
    """npas_conv2d_bp_static_ws: same result as ``conv2d_bp`` without caller-provided scratch.

    For callers that may not allocate device memory (fixed-budget or real-time inference loops,
    plug-ins whose host owns all allocations): the library's own 256-byte device array takes the
    place of the workspace.  ``out`` is still the caller's (this helper allocates it only when it
    is not passed).  With ``check`` the call synchronises and raises on a device-side time-out.
    """
    lib = load()
    assert x.is_cuda and x.is_contiguous() and x.dim() == 4
    N, H, W, C = x.shape
    d = blob.desc
    P = (H + 2 * pad - d.R) // stride + 1
    Q = (W + 2 * pad - d.S) // stride + 1
    if out is None:
        out = torch.empty((N, P, Q, d.K), dtype=x.dtype if out_dtype is None else out_dtype, device=x.device)
    cd = ConvDesc(N, H, W, C, d.K, d.R, d.S, stride, pad, _dt(x), _dt(out), int(bool(relu)),
                  int(bias is not None), int(residual is not None), path, 0)
    status = ctypes.c_int32(0)
    _check(lib.npas_conv2d_bp_static_ws(ctypes.byref(cd), ctypes.byref(d), _p(x), _p(blob.data), _p(bias),
                                        _p(residual), _p(out), ctypes.byref(status) if check else None, _stream()),
           "npas_conv2d_bp_static_ws")
    return out


# ---------------------------------------------------------------------------- kernel choice ----

CONV_KERNELS = {1: "conv_bp_simt_kernel", 3: "conv_bp_tc_kernel", 5: "conv_stem_kernel", 6: "conv_bp_dn_kernel",
                7: "conv_bp_d2_kernel", 8: "conv_bp_kr_kernel"}
LINEAR_KERNELS = {1: "linear_bb_simt_kernel", 3: "linear_bb_tc_kernel", 5: "linear_bb_dn_kernel", 6: "linear_bb_d2_kernel"}


def conv2d_bp_kernel(x_shape, blob: BpBlob, *, stride=1, pad=1, dtype=torch.bfloat16, out_dtype=None, relu=False,
                     bias=False, residual=False, path=0, variant=0) -> int:
    """npas_conv2d_bp_kernel: id of the kernel the call would run (host only; raises NpasError(8) when the
    requested path declines the geometry)."""
    lib = load()
    N, H, W, C = x_shape
    d = blob.desc
    t = torch.empty(0, dtype=dtype)
    to = t if out_dtype is None else torch.empty(0, dtype=out_dtype)
    cd = ConvDesc(N, H, W, C, d.K, d.R, d.S, stride, pad, _dt(t), _dt(to), int(bool(relu)), int(bool(bias)),
                  int(bool(residual)), path, variant)
    kid = ctypes.c_int32(0)
    _check(lib.npas_conv2d_bp_kernel(ctypes.byref(cd), ctypes.byref(d), ctypes.byref(kid)), "npas_conv2d_bp_kernel")
    return kid.value


def conv2d_bp_workspace(x_shape, blob: BpBlob, *, stride=1, pad=1, dtype=torch.bfloat16, out_dtype=None, relu=False,
                        bias=False, residual=False, path=0, variant=0, device="cuda") -> torch.Tensor:
    """npas_conv2d_bp_workspace: zeroed device scratch of the size the call can use for this layer (the status
    words, plus room for the partial sums of a split last round where the kept-pairs kernel runs)."""
    lib = load()
    N, H, W, C = x_shape
    d = blob.desc
    t = torch.empty(0, dtype=dtype)
    to = t if out_dtype is None else torch.empty(0, dtype=out_dtype)
    cd = ConvDesc(N, H, W, C, d.K, d.R, d.S, stride, pad, _dt(t), _dt(to), int(bool(relu)), int(bool(bias)),
                  int(bool(residual)), path, variant)
    n = ctypes.c_size_t(0)
    _check(lib.npas_conv2d_bp_workspace(ctypes.byref(cd), ctypes.byref(d), ctypes.byref(n)), "npas_conv2d_bp_workspace")
    return torch.zeros(max(n.value, WORKSPACE_BYTES), dtype=torch.uint8, device=device)


def linear_bb_kernel(M: int, blob: BbBlob, *, dtype=torch.bfloat16, out_dtype=None, relu=False, bias=False,
                     residual=False, path=0, variant=0) -> int:
    lib = load()
    d = blob.desc
    t = torch.empty(0, dtype=dtype)
    to = t if out_dtype is None else torch.empty(0, dtype=out_dtype)
    ld = LinearDesc(M, d.I, d.O, _dt(t), _dt(to), int(bool(relu)), int(bool(bias)), int(bool(residual)), path, variant)
    kid = ctypes.c_int32(0)
    _check(lib.npas_linear_bb_kernel(ctypes.byref(ld), ctypes.byref(d), ctypes.byref(kid)), "npas_linear_bb_kernel")
    return kid.value


def tune_conv2d_bp(x: torch.Tensor, blob: BpBlob, bias=None, residual=None, *, stride=1, pad=1, relu=False,
                   out=None, ws=None, reps=10):
    """npas_tune_conv2d_bp: times every kernel / tile shape that takes the layer on these buffers and returns
    (path, variant, microseconds) of the fastest; pass the first two to ``conv2d_bp``."""
    lib = load()
    N, H, W, C = x.shape
    d = blob.desc
    P = (H + 2 * pad - d.R) // stride + 1
    Q = (W + 2 * pad - d.S) // stride + 1
    if out is None:
        out = torch.empty((N, P, Q, d.K), dtype=x.dtype, device=x.device)
    if ws is None:
        ws = workspace(x.device)
    cd = ConvDesc(N, H, W, C, d.K, d.R, d.S, stride, pad, _dt(x), _dt(out), int(bool(relu)),
                  int(bias is not None), int(residual is not None), 0, 0)
    path, variant, us = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_float(0)
    _check(lib.npas_tune_conv2d_bp(ctypes.byref(cd), ctypes.byref(d), _p(x), _p(blob.data), _p(bias), _p(residual),
                                   _p(out), _p(ws), ctypes.c_size_t(ws.numel()), int(reps), ctypes.byref(path),
                                   ctypes.byref(variant), ctypes.byref(us), _stream()), "npas_tune_conv2d_bp")
    return path.value, variant.value, us.value


def tune_linear_bb(x: torch.Tensor, blob: BbBlob, bias=None, residual=None, *, relu=False, out=None, ws=None, reps=10):
    lib = load()
    M, I = x.shape
    d = blob.desc
    if out is None:
        out = torch.empty((M, d.O), dtype=x.dtype, device=x.device)
    if ws is None:
        ws = workspace(x.device)
    ld = LinearDesc(M, I, d.O, _dt(x), _dt(out), int(bool(relu)), int(bias is not None), int(residual is not None), 0, 0)
    path, variant, us = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_float(0)
    _check(lib.npas_tune_linear_bb(ctypes.byref(ld), ctypes.byref(d), _p(x), _p(blob.data), _p(bias), _p(residual),
                                   _p(out), _p(ws), ctypes.c_size_t(ws.numel()), int(reps), ctypes.byref(path),
                                   ctypes.byref(variant), ctypes.byref(us), _stream()), "npas_tune_linear_bb")
    return path.value, variant.value, us.value


class PlanCache:
    """Tuned (path, variant) pairs keyed by what the choice depends on: the call geometry, the block
    sizes and the mask statistic the kernels plan with (largest kept count of a block).  Plain JSON on
    disk, so a tuning run on one process serves later ones on the same GPU model."""

    def __init__(self):
        self.plans = {}

    @staticmethod
    def conv_key(x_shape, blob: BpBlob, stride, pad, relu, has_bias, has_residual) -> str:
        d = blob.desc
        return "conv:" + ",".join(str(int(v)) for v in (*x_shape, d.K, d.R, d.S, d.Mb, d.Nb, d.max_taps, stride, pad,
                                                         relu, has_bias, has_residual))

    @staticmethod
    def linear_key(M, blob: BbBlob, relu, has_bias, has_residual) -> str:
        d = blob.desc
        return "linear:" + ",".join(str(int(v)) for v in (M, d.I, d.O, d.Bo, d.Bi, d.max_cols, relu, has_bias, has_residual))

    def get(self, key: str):
        v = self.plans.get(key)
        return None if v is None else (int(v[0]), int(v[1]))

    def put(self, key: str, path: int, variant: int, us: float) -> None:
        self.plans[key] = [int(path), int(variant), round(float(us), 3)]

    def to_json(self) -> str:
        import json
        return json.dumps({"version": 1, "plans": self.plans}, sort_keys=True)

    @classmethod
    def from_json(cls, text: str) -> "PlanCache":
        import json
        obj = json.loads(text)
        if obj.get("version") != 1 or not isinstance(obj.get("plans"), dict):
            raise ValueError("not a plan cache")
        c = cls()
        for k, v in obj["plans"].items():
            if not (isinstance(v, list) and len(v) == 3):
                raise ValueError(f"bad plan entry {k!r}")
            c.plans[str(k)] = [int(v[0]), int(v[1]), float(v[2])]
        return c
