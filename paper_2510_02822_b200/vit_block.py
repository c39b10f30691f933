"""One ViT encoder block around the mixed GEMMs (Sec. 6: 4- or 8-bit integer computation for the linear
layers, 16-bit floating point for normalisation, attention and GELU; Sec. 7: model latency against
the low-bit ratio).

    python -m paper_2510_02822_b200.vit_block [--model vitb|deits|vitl] [--batch 64] [--iters 20]

The four linears (QKV, proj, fc1, fc2) run through the library: fp16 activations -> prologue
(Eq. 1 + bit-lowering) -> mixed GEMM with fp16 output.  Everything between them (layer norm,
softmax attention, GELU, residual adds) is NOT part of the method's hot path and runs as stock
PyTorch fp16 operators, as the paper runs them in fp16; they are here only so that the share of the
quantized linears in a block's latency can be measured.  Random-init weights, seeded activations; each linear's activation scale,
extraction positions and group order are calibrated on the block's own activations with the device
calibration kernels.
Prints the block latency and the time of the four quantized linears per ratio.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch
import torch.nn.functional as F

from . import binding as fx
from . import calib, inputs

DIMS = {"deits": (384, 6), "vitb": (768, 12), "vitl": (1024, 16)}


class Block:
    def __init__(self, model: str, batch: int, dev, seed: int = 11000):
        D, heads = DIMS[model]
        self.D, self.heads, self.batch, self.T = D, heads, batch, 197
        self.M = batch * self.T
        self.dev = dev
        shapes = [("qkv", D, 3 * D), ("proj", D, D), ("fc1", D, 4 * D), ("fc2", 4 * D, D)]
        self.layers = {}
        for i, (name, K, N) in enumerate(shapes):
            c = inputs.vit_linear(f"blk_{name}", 256, K, N, 16, seed=seed + i)   # weights and calibration rows only
            perm, xs = calib.static_preparation(calib.quantize_reference(torch.from_numpy(c.Xcal), c.x_scale), torch.from_numpy(c.Wq), 16)
            L = fx.Layer(torch.from_numpy(c.Wq).to(dev), torch.from_numpy(c.w_scale).to(dev), torch.from_numpy(c.bias).to(dev), perm, xs, 16)
            slab = torch.empty(self.M * K + 16, dtype=torch.uint8, device=dev)
            Y = torch.empty((self.M, N), dtype=torch.float16, device=dev)
            self.layers[name] = [L, c.x_scale, slab, Y, torch.from_numpy(c.Wq).to(dev)]
        x = inputs.normal(seed, 50, self.M * D).reshape(self.M, D)
        self.x = torch.from_numpy(x.astype(np.float16)).to(dev)
        self.ln = [torch.ones(D, dtype=torch.float16, device=dev), torch.zeros(D, dtype=torch.float16, device=dev)]
        self.gemm_events = []
        self.calibrating = True
        self.forward()           # scales, positions and group order from the block's own activations
        self.calibrating = False
        torch.cuda.synchronize()

    def set_ratio(self, ratio: float):
        for L, *_ in self.layers.values():
            L.set_lowbit_ratio(ratio)

    def linear(self, name: str, x16: torch.Tensor, timed: bool = False):
        """fp16 activations -> Eq. 1 + bit-lowering -> mixed GEMM -> fp16 (two library launches)."""
        L, x_scale, slab, Y, Wq = self.layers[name]
        if self.calibrating:
            # activation scale (absmax / 127), static extraction positions and greedy group order (device kernels),
            # then the handle is laid out again for them
            x_scale = float(np.float32(float(x16.abs().max()) / 127.0))
            perm, xs, _info = calib.static_preparation_device(x16, x_scale, Wq, 16)
            L.set_group_perm(Wq, perm, xs)
            self.layers[name][1] = x_scale
        if timed:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
        fx.flexiq_quantize_lower(L.h, x16, fx.DTYPE_F16, self.M, x_scale, 0, slab, None)
        fx.flexiq_mixed_gemm(L.h, slab, None, None, self.M, x_scale, 1.0, fx.OUT_DEQUANT_F16, Y)
        if timed:
            e1.record()
            self.gemm_events.append((e0, e1))
        return Y

    def forward(self, timed: bool = False):
        B, T, D, H = self.batch, self.T, self.D, self.heads
        x = self.x
        h = F.layer_norm(x, (D,), self.ln[0], self.ln[1])
        qkv = self.linear("qkv", h, timed).view(B, T, 3, H, D // H).permute(2, 0, 3, 1, 4)
        a = F.scaled_dot_product_attention(qkv[0], qkv[1], qkv[2])
        a = a.transpose(1, 2).reshape(self.M, D).contiguous()
        x = x + self.linear("proj", a, timed)
        h = F.layer_norm(x, (D,), self.ln[0], self.ln[1])
        h = F.gelu(self.linear("fc1", h, timed))
        return x + self.linear("fc2", h, timed)

    def close(self):
        for L, *_ in self.layers.values():
            L.close()


def measure(block: Block, iters: int):
    out = []
    for ratio in (0.0, 0.25, 0.5, 0.75, 1.0):
        block.set_ratio(ratio)
        for _ in range(3):
            y = block.forward()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            y = block.forward()
        e1.record()
        torch.cuda.synchronize()
        block_us = e0.elapsed_time(e1) / iters * 1e3
        block.gemm_events = []
        for _ in range(iters):
            block.forward(timed=True)
        torch.cuda.synchronize()
        lin_us = sum(a.elapsed_time(b) for a, b in block.gemm_events) / iters * 1e3
        out.append({"ratio": ratio, "block_us": round(block_us, 1), "quantized_linears_us": round(lin_us, 1),
                    "share": round(lin_us / block_us, 3), "finite": bool(torch.isfinite(y).all())})
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--model", default="vitb", choices=sorted(DIMS))
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--iters", type=int, default=20)
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    block = Block(args.model, args.batch, dev)
    print(json.dumps({"model": args.model, "batch": args.batch, "rows": block.M, "what": "one encoder block: library linears (prologue + mixed GEMM, fp16 out), "
                      "stock fp16 layer norm / attention / GELU around them"}), flush=True)
    for row in measure(block, args.iters):
        print(json.dumps(row), flush=True)
    fx.flexiq_check_status()
    block.close()


if __name__ == "__main__":
    main()
