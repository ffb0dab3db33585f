"""ResNet-50-topology stack of pruned convolutions run through the C-ABI library.

Every 3x3 convolution is block-punched, every 1x1 convolution is a block-based pruned GEMM over the
pixels (paper Sec. 3: a 1x1 CONV layer is a matrix product), the 7x7 stem is dense (all taps kept),
shortcut additions and ReLU are fused into the producing layer's epilogue.  The class only packs the
weights and sequences the library calls; all arithmetic runs in the CUDA kernels.
"""
from __future__ import annotations

import torch

from . import binding as npas
from .inputs import STACK_BLOCKS, StackLayer


class Resnet50Stack:
    def __init__(self, layers: list[StackLayer], device="cuda"):
        self.layers = layers
        self.device = torch.device(device)
        self.blobs, self.biases = [], []
        for lay in layers:
            w = torch.from_numpy(lay.w).to(self.device).to(torch.bfloat16)
            if lay.kind == "pw":
                self.blobs.append(npas.pack_bb(w, lay.row_keep, lay.col_keep, 64, 64))
            else:
                Mb, Nb = STACK_BLOCKS[lay.kind]
                self.blobs.append(npas.pack_bp(w, lay.tap_mask, Mb, Nb))
            self.biases.append(torch.from_numpy(lay.bias).to(self.device))
        self.ws = npas.workspace(self.device)
        self.fuse_pool = True          # stem + max-pool as one fused call (False: the two separate kernels)
        self.plans = npas.PlanCache()  # measured (kernel, tile shape) per layer; empty = the library's own choice
        self._tuning = 0               # > 0: repetitions per candidate while tune() walks the stack

    def tune(self, x: torch.Tensor, reps: int = 20) -> "npas.PlanCache":
        """One pass over the stack on input x in which every layer asks the library's tuner (it times each kernel
        and tile shape that takes the layer, on the tensors the layer really sees) and keeps the answer; later
        passes run every layer on its measured choice.  Returns the plan cache (JSON-serialisable)."""
        self.plans = npas.PlanCache()
        self._tuning = int(reps)
        try:
            self.forward(x)
        finally:
            self._tuning = 0
        return self.plans

    def run_layer(self, i: int, x: torch.Tensor, res: torch.Tensor | None, out: torch.Tensor | None = None):
        """Layer i on NHWC input x (and the shortcut tensor res, if the layer adds one)."""
        lay = self.layers[i]
        if lay.kind == "pw":
            if lay.stride != 1:
                x = npas.subsample2d(x, lay.stride)
            n, h, w_, c = x.shape
            r2 = None if res is None else res.view(n * h * w_, lay.Cout)
            o2 = None if out is None else out.view(n * h * w_, lay.Cout)
            x2 = x.view(n * h * w_, c)
            key = npas.PlanCache.linear_key(n * h * w_, self.blobs[i], lay.relu, True, r2 is not None)
            if self._tuning:
                pth, var, us = npas.tune_linear_bb(x2, self.blobs[i], self.biases[i], r2, relu=lay.relu, ws=self.ws, reps=self._tuning)
                self.plans.put(key, pth, var, us)
            pth, var = self.plans.get(key) or (0, 0)
            y = npas.linear_bb(x2, self.blobs[i], self.biases[i], r2, relu=lay.relu, out=o2, ws=self.ws, path=pth, variant=var)
            return y.view(n, h, w_, lay.Cout)
        pad = 3 if lay.kind == "stem" else 1
        key = npas.PlanCache.conv_key(tuple(x.shape), self.blobs[i], lay.stride, pad, lay.relu, True, res is not None)
        if self._tuning:
            pth, var, us = npas.tune_conv2d_bp(x, self.blobs[i], self.biases[i], res, stride=lay.stride, pad=pad, relu=lay.relu,
                                               ws=self.ws, reps=self._tuning)
            self.plans.put(key, pth, var, us)
        pth, var = self.plans.get(key) or (0, 0)
        return npas.conv2d_bp(x, self.blobs[i], self.biases[i], res, stride=lay.stride, pad=pad, relu=lay.relu,
                              out=out, ws=self.ws, path=pth, variant=var)

    def forward(self, x: torch.Tensor, keep: bool = False):
        """x [N,H,W,3] bf16 -> [N,H/32,W/32,2048].  With ``keep`` also returns, per layer, the tuple
        (input, shortcut or None, output) the layer actually saw, for layer-by-layer checks."""
        outs: dict[int, torch.Tensor] = {}
        seen = []
        for i, lay in enumerate(self.layers):
            if lay.src == -1:
                xin = x
            elif lay.src == -2:
                xin = outs[-2]
            else:
                xin = outs[lay.src]
            res = outs[lay.res] if lay.res >= 0 else (outs[-2] if lay.res == -2 else None)
            if lay.kind == "stem" and not keep and self.fuse_pool:
                # first layer + ReLU + max-pool in one kernel: the 112x112 intermediate is never written
                outs[-2] = npas.conv2d_bp_maxpool(xin, self.blobs[i], self.biases[i], stride=lay.stride, pad=3, relu=lay.relu,
                                                  ws=self.ws)
                continue
            y = self.run_layer(i, xin, res)
            outs[i] = y
            if keep:
                seen.append((xin, res, y))
            if lay.kind == "stem":
                outs[-2] = npas.maxpool2d(y, 3, 2, 1)
            # drop tensors no later layer reads
            if not keep:
                last_use = {}
                for j in range(i + 1, len(self.layers)):
                    for s in (self.layers[j].src, self.layers[j].res):
                        last_use[s] = j
                for k in [k for k in outs if k not in last_use and k != i]:
                    del outs[k]
        npas_out = outs[len(self.layers) - 1]
        return (npas_out, seen, outs.get(-2)) if keep else npas_out

    def check(self):
        npas.check_device_status(self.ws)
