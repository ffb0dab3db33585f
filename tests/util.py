"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

TOL_BF16 = 1e-2   # bf16 inputs, fp32 accumulation, one output rounding
TOL_F32 = 1e-5    # fp32 path


def floored_rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max |g - o| / (|o| + 1e-3 * rms(o)): element-wise relative error with a small floor."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref * ref))) if ref.size else 0.0
    if ref.size == 0:
        return 0.0
    return float(np.max(np.abs(got - ref) / (np.abs(ref) + 1e-3 * rms + 1e-30)))


def dev(a, dtype="f32"):
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def host(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy()
