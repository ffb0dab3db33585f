"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle harness.

This module holds no arithmetic of the method itself: it only draws random tensors and
random block masks with the shapes and value distributions of the workloads, so that the
CUDA path and the oracle can be fed the very same arrays.  Random numbers come from numpy's
counter-based Philox generator keyed by an explicit seed.  Rounding of drawn values to
bf16-representable floats is delegated to torch's own cast (a library routine).

Mask conventions (paper Sec. 3, "Block-punched Pruning" / "Block-based Pruning"):
  * block-punched: ``tap_mask[fb, cb]`` is a uint64 bitset, bit ``t = r*S + s`` set when kernel
    position (r, s) is KEPT in the block of filters ``fb*Mb..`` and channels ``cb*Nb..``.
  * block-based:   ``row_keep[bo, bi]`` / ``col_keep[bo, bi]`` are uint64 bitsets of the rows
    (outputs) and columns (inputs) KEPT inside block (bo, bi) of the weight matrix.
"""
from __future__ import annotations

import dataclasses
import numpy as np

BASE_SEED = 20120596 * 10


def rng_for(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=int(seed)))


def bf16_representable(a: np.ndarray) -> np.ndarray:
    """fp32 array whose every value is exactly representable in bf16 (torch's RNE cast)."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    return t.to(torch.bfloat16).to(torch.float32).numpy()


def as_bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 view of the upper halves of bf16-representable fp32 values (no rounding)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    assert not np.any(bits & np.uint32(0xFFFF)), "values are not bf16-representable"
    return (bits >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def draw_tap_masks(rng, n_fb: int, n_cb: int, n_taps: int, keep) -> np.ndarray:
    """One random tap subset per block, by partial Fisher-Yates, blocks in (fb, cb) order.

    ``keep`` is an int (same count in every block) or a callable ``(fb, cb) -> count``.
    """
    out = np.zeros((n_fb, n_cb), dtype=np.uint64)
    for fb in range(n_fb):
        for cb in range(n_cb):
            k = keep(fb, cb) if callable(keep) else int(keep)
            perm = list(range(n_taps))
            bits = 0
            for i in range(k):
                j = i + int(rng.integers(0, n_taps - i))
                perm[i], perm[j] = perm[j], perm[i]
                bits |= 1 << perm[i]
            out[fb, cb] = np.uint64(bits)
    return out


def draw_keep_sets(rng, n_bo: int, n_bi: int, size: int, keep) -> np.ndarray:
    """Random ``keep``-of-``size`` subsets as uint64 bitsets, one per block."""
    return draw_tap_masks(rng, n_bo, n_bi, size, keep)


@dataclasses.dataclass
class ConvCase:
    N: int; H: int; W: int; C: int; K: int; R: int; S: int
    stride: int; pad: int; Mb: int; Nb: int
    dtype: str                      # "f32" | "bf16"
    relu: bool
    x: np.ndarray                   # [N,H,W,C] fp32 (bf16-representable when dtype == "bf16")
    w: np.ndarray                   # [K,R,S,C] fp32 dense, unmasked
    tap_mask: np.ndarray            # [K/Mb, C/Nb] uint64
    bias: np.ndarray | None         # [K] fp32
    residual: np.ndarray | None = None

    @property
    def P(self): return (self.H + 2 * self.pad - self.R) // self.stride + 1

    @property
    def Q(self): return (self.W + 2 * self.pad - self.S) // self.stride + 1

    def kept_macs(self) -> int:
        pops = sum(bin(int(v)).count("1") for v in self.tap_mask.ravel())
        return self.N * self.P * self.Q * pops * self.Mb * self.Nb

    def algorithmic_bytes(self) -> int:
        """Activations once + outputs once + packed values and indices once + bias."""
        es = 4 if self.dtype == "f32" else 2
        pops = sum(bin(int(v)).count("1") for v in self.tap_mask.ravel())
        b = self.x.size * es + self.N * self.P * self.Q * self.K * es
        b += pops * self.Mb * self.Nb * es + pops * 4 + (self.tap_mask.size + 1) * 4
        if self.bias is not None:
            b += self.K * 4
        if self.residual is not None:
            b += self.residual.size * es
        return b


@dataclasses.dataclass
class LinearCase:
    M: int; I: int; O: int; Bo: int; Bi: int
    dtype: str
    relu: bool
    x: np.ndarray                   # [M,I]
    w: np.ndarray                   # [O,I] dense, unmasked
    row_keep: np.ndarray            # [O/Bo, I/Bi] uint64
    col_keep: np.ndarray            # [O/Bo, I/Bi] uint64
    bias: np.ndarray | None

    def kept_macs(self) -> int:
        tot = 0
        for r, c in zip(self.row_keep.ravel(), self.col_keep.ravel()):
            tot += bin(int(r)).count("1") * bin(int(c)).count("1")
        return self.M * tot

    def algorithmic_bytes(self) -> int:
        es = 4 if self.dtype == "f32" else 2
        kept = self.kept_macs() // self.M
        b = self.x.size * es + self.M * self.O * es + kept * es
        b += self.row_keep.size * (self.Bo + self.Bi + 2 + 4)
        if self.bias is not None:
            b += self.O * 4
        return b


def conv_case(*, N, H, W, C, K, R=3, S=3, stride=1, pad=1, Mb, Nb, keep, dtype="bf16",
              act="relu_normal", w_sigma=0.02, bias=True, relu=True, residual=False,
              seed=0) -> ConvCase:
    rng = rng_for(seed)
    x = rng.standard_normal((N, H, W, C), dtype=np.float32)
    if act == "relu_normal":
        x = np.maximum(x, 0.0)
    elif act == "half_normal":
        x = np.abs(x)
    elif act != "normal":
        raise ValueError(act)
    w = (rng.standard_normal((K, R, S, C), dtype=np.float32) * np.float32(w_sigma))
    b = (rng.standard_normal((K,), dtype=np.float32) * np.float32(0.1)) if bias else None
    tm = draw_tap_masks(rng, K // Mb, C // Nb, R * S, keep)
    res = None
    if residual:
        P = (H + 2 * pad - R) // stride + 1
        Q = (W + 2 * pad - S) // stride + 1
        res = rng.standard_normal((N, P, Q, K), dtype=np.float32)
    if dtype == "bf16":
        x, w = bf16_representable(x), bf16_representable(w)
        if res is not None:
            res = bf16_representable(res)
    return ConvCase(N, H, W, C, K, R, S, stride, pad, Mb, Nb, dtype, relu, x, w, tm, b, res)


# 3x3 kernel patterns of four taps (pattern-based pruning, paper Sec. 2.1): the centre tap plus three
# neighbours.  Eight patterns: the centre with three of the four edge neighbours, and the centre with
# two adjacent edge neighbours and the corner between them.  Tap index = r*3 + s.
PATTERN_LIBRARY = tuple(
    [sum(1 << t for t in (4, *[e for e in (1, 3, 5, 7) if e != skip])) for skip in (1, 3, 5, 7)] +
    [sum(1 << t for t in (4, a, b, c)) for (a, b, c) in ((1, 3, 0), (1, 5, 2), (7, 3, 6), (7, 5, 8))])


def pattern_case(*, N, H, W, C, K, removed=0.25, dtype="bf16", seed=0, **kw) -> ConvCase:
    """A 3x3 layer under pattern-based pruning: every kernel (one filter x one channel, i.e. blocks of
    1 x 1) keeps one of the eight four-tap patterns, drawn at random, and a fraction ``removed`` of the
    kernels is cut entirely (connectivity pruning)."""
    c = conv_case(N=N, H=H, W=W, C=C, K=K, Mb=1, Nb=1, keep=0, dtype=dtype, seed=seed, **kw)
    rng = rng_for(seed + 1000)
    pick = rng.integers(0, len(PATTERN_LIBRARY), size=(K, C))
    gone = rng.random((K, C)) < removed
    tm = np.array(PATTERN_LIBRARY, dtype=np.uint64)[pick]
    tm[gone] = 0
    c.tap_mask = tm
    return c


def linear_case(*, M, I, O, Bo=64, Bi=64, keep_rows, keep_cols, dtype="bf16", w_sigma=0.02,
                bias=True, relu=True, seed=0) -> LinearCase:
    rng = rng_for(seed)
    x = np.maximum(rng.standard_normal((M, I), dtype=np.float32), 0.0)
    w = rng.standard_normal((O, I), dtype=np.float32) * np.float32(w_sigma)
    b = (rng.standard_normal((O,), dtype=np.float32) * np.float32(0.1)) if bias else None
    rk = draw_keep_sets(rng, O // Bo, I // Bi, Bo, keep_rows)
    ck = draw_keep_sets(rng, O // Bo, I // Bi, Bi, keep_cols)
    if dtype == "bf16":
        x, w = bf16_representable(x), bf16_representable(w)
    return LinearCase(M, I, O, Bo, Bi, dtype, relu, x, w, rk, ck, b)


# ---- the five workload recipes (shapes and distributions of the evaluation configs) ----------

def config1(seed=BASE_SEED + 1) -> ConvCase:
    """fp32 3x3 CONV, 1x16x16x32 -> 32, Mb=8 x Nb=4, 3 of 9 taps, half-normal input, no bias."""
    return conv_case(N=1, H=16, W=16, C=32, K=32, Mb=8, Nb=4, keep=3, dtype="f32",
                     act="half_normal", w_sigma=0.05, bias=False, relu=False, seed=seed)


def config2(seed=BASE_SEED + 2, N=32) -> ConvCase:
    """bf16 3x3 CONV, ResNet-50 stage-3 shape 32x14x14x256 -> 256, Mb=16 x Nb=8, 3 of 9 taps."""
    return conv_case(N=N, H=14, W=14, C=256, K=256, Mb=16, Nb=8, keep=3, dtype="bf16",
                     act="relu_normal", w_sigma=0.02, bias=True, relu=True, seed=seed)


def config3(seed=BASE_SEED + 3, M=64 * 7 * 7) -> LinearCase:
    """bf16 block-based GEMM 3136x512 -> 2048, 64x64 blocks keeping 16 rows x 16 cols."""
    return linear_case(M=M, I=512, O=2048, Bo=64, Bi=64, keep_rows=16, keep_cols=16,
                       dtype="bf16", w_sigma=0.02, bias=True, relu=True, seed=seed)


def config5(Mb=16, Nb=16, taps=3, seed=BASE_SEED + 5, N=64, H=28, C=512, K=512) -> ConvCase:
    """bf16 3x3 CONV sweep point, 64x28x28x512 -> 512, no bias / ReLU."""
    return conv_case(N=N, H=H, W=H, C=C, K=K, Mb=Mb, Nb=Nb, keep=taps, dtype="bf16",
                     act="relu_normal", w_sigma=0.02, bias=False, relu=False,
                     seed=seed + 100 * Mb + taps)


# ---- ResNet-50 topology stack (v1.5: the stride sits on the 3x3 of the first bottleneck) ------
@dataclasses.dataclass
class StackLayer:
    name: str
    kind: str                       # "stem" | "conv3" (block-punched 3x3) | "pw" (block-based 1x1)
    Cin: int; Cout: int
    H_in: int                       # input height = width
    stride: int
    relu: bool
    src: int                        # index of the layer whose output is this layer's input (-1: network input / pool)
    res: int                        # index of the layer whose output is added before the activation, or -1
    w: np.ndarray | None = None     # [K,R,S,C] (stem, conv3) or [O,I] (pw), bf16-representable fp32
    bias: np.ndarray | None = None
    tap_mask: np.ndarray | None = None
    row_keep: np.ndarray | None = None
    col_keep: np.ndarray | None = None

    @property
    def H_out(self) -> int:
        return (self.H_in - 1) // self.stride + 1

    def kept_macs_per_image(self) -> int:
        px = self.H_out * self.H_out
        if self.kind == "pw":
            kept = sum(bin(int(r)).count("1") * bin(int(c)).count("1")
                       for r, c in zip(self.row_keep.ravel(), self.col_keep.ravel()))
            return px * kept
        Mb, Nb = STACK_BLOCKS[self.kind]
        pops = sum(bin(int(v)).count("1") for v in self.tap_mask.ravel())
        return px * pops * Mb * min(Nb, self.Cin)

    def algorithmic_bytes_per_image(self) -> int:
        """bf16 activations in once + out once (+ residual once); weights and bias are per batch."""
        b = self.H_in * self.H_in * self.Cin * 2 // (self.stride * self.stride if self.kind == "pw" else 1)
        b += self.H_out * self.H_out * self.Cout * 2 * (2 if self.res >= 0 else 1)
        return b

    def weight_bytes(self) -> int:
        if self.kind == "pw":
            kept = sum(bin(int(r)).count("1") * bin(int(c)).count("1")
                       for r, c in zip(self.row_keep.ravel(), self.col_keep.ravel()))
            return kept * 2 + self.row_keep.size * (64 + 64 + 6) + self.Cout * 4
        Mb, Nb = STACK_BLOCKS[self.kind]
        pops = sum(bin(int(v)).count("1") for v in self.tap_mask.ravel())
        return pops * Mb * min(Nb, self.Cin) * 2 + pops * 4 + self.tap_mask.size * 4 + self.Cout * 4


STACK_BLOCKS = {"stem": (16, 3), "conv3": (16, 8)}      # (Mb, Nb); the stem keeps all 49 taps


def resnet50_topology(H: int = 224):
    """The 53 convolutions of the ResNet-50 body as (name, kind, Cin, Cout, H_in, stride, relu, src, res)."""
    L = []
    L.append(("stem", "stem", 3, 64, H, 2, True, -1, -1))
    h = ((H - 1) // 2 + 1 - 1) // 2 + 1          # after the 7x7/2 stem and the 3x3/2 max-pool
    cin, prev = 64, -2                            # -2: the max-pool output
    for stage, (width, blocks) in enumerate([(64, 3), (128, 4), (256, 6), (512, 3)]):
        for b in range(blocks):
            s = 2 if (b == 0 and stage > 0) else 1
            tag = f"s{stage + 1}b{b + 1}"
            block_in = prev
            L.append((tag + ".reduce", "pw", cin, width, h, 1, True, block_in, -1)); i_red = len(L) - 1
            L.append((tag + ".conv3", "conv3", width, width, h, s, True, i_red, -1)); i_c3 = len(L) - 1
            h_out = (h - 1) // s + 1
            if b == 0:
                L.append((tag + ".proj", "pw", cin, 4 * width, h, s, False, block_in, -1)); shortcut = len(L) - 1
            else:
                shortcut = block_in
            L.append((tag + ".expand", "pw", width, 4 * width, h_out, 1, True, i_c3, shortcut)); prev = len(L) - 1
            cin, h = 4 * width, h_out
    return L


def config4(seed=BASE_SEED + 4, H: int = 224, gain: float = 0.5):
    """ResNet-50-topology stack, random-init: 3x3 block-punched (16x8, 3 of 9 taps), 1x1 block-based
    (64x64 blocks keeping 32 rows x 32 columns), dense 7x7 stem.  Weights N(0, 2 / kept fan-in), the
    last 1x1 of every bottleneck and the projections scaled by ``gain`` so that the activation scale
    stays bounded through the residual additions; bias N(0, 0.01^2)."""
    rng = rng_for(seed)
    layers = []
    for (name, kind, cin, cout, h, s, relu, src, res) in resnet50_topology(H):
        lay = StackLayer(name, kind, cin, cout, h, s, relu, src, res)
        if kind == "pw":
            lay.row_keep = draw_keep_sets(rng, cout // 64, cin // 64, 64, 32)
            lay.col_keep = draw_keep_sets(rng, cout // 64, cin // 64, 64, 32)
            sigma = np.sqrt(2.0 / (cin / 2)) * (gain if (res >= 0 or not relu) else 1.0)
            w = rng.standard_normal((cout, cin), dtype=np.float32) * np.float32(sigma)
        else:
            Mb, Nb = STACK_BLOCKS[kind]
            R = 7 if kind == "stem" else 3
            keep = R * R if kind == "stem" else 3
            lay.tap_mask = draw_tap_masks(rng, cout // Mb, cin // Nb, R * R, keep)
            sigma = np.sqrt(2.0 / (cin * keep))
            w = rng.standard_normal((cout, R, R, cin), dtype=np.float32) * np.float32(sigma)
        lay.w = bf16_representable(w)
        lay.bias = rng.standard_normal((cout,), dtype=np.float32) * np.float32(0.01)
        layers.append(lay)
    return layers


def config4_input(N: int, H: int = 224, seed=BASE_SEED + 4) -> np.ndarray:
    """Network input [N,H,H,3] ~ N(0,1), bf16-representable."""
    return bf16_representable(rng_for(seed + 1000).standard_normal((N, H, H, 3), dtype=np.float32))
