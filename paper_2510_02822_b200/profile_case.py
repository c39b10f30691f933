"""Runs one layer shape of the benchmark configurations a few times, for profilers.

    python -m paper_2510_02822_b200.profile_case --layer vitb_qkv --ratio 0.5 --iters 3
    python -m paper_2510_02822_b200.profile_case --layer vitb_fc2 --aux reorder       # residual reorder of the layer's input
    python -m paper_2510_02822_b200.profile_case --layer vitb_fc2 --aux distance      # squared-distance reduction (selection fitness)

Prints the average device time of the prologue and of the mixed GEMM (CUDA events on the
launching stream).  Layers: vitb_{qkv,proj,fc1,fc2}, vitl_{...}, deits_{...} (append
@<batch> to change the batch, e.g. deits_fc1@8), rn50_<name> from the ResNet-50 list.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as fx
from . import calib, inputs


def make_case(name: str):
    batch = None
    if "@" in name:
        name, b = name.split("@")
        batch = int(b)
    fam, layer = name.split("_", 1)
    if fam in ("vitb", "vitl", "deits"):
        table = {"vitb": inputs.VIT_B_LAYERS, "vitl": inputs.VIT_L_LAYERS, "deits": inputs.DEIT_S_LAYERS}[fam]
        i = [n for n, _, _ in table].index(layer)
        _, K, N = table[i]
        batch = batch or {"vitb": 64, "vitl": 128, "deits": 1}[fam]
        if fam == "deits":
            return inputs.ranged_linear(name, batch * 197, K, N, 16, seed=4000 + i), False
        return inputs.vit_linear(name, batch * 197, K, N, 16, seed=2000 + i), False
    if fam == "rn50":
        i = [n for n, *_ in inputs.RESNET50_CONVS].index(layer)
        _, H, C, Co, R = inputs.RESNET50_CONVS[i]
        return inputs.resnet_conv(name, batch or 32, H, C, Co, R, 16, seed=3000 + i), True
    raise SystemExit(f"unknown layer {name}")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layer", default="vitb_qkv")
    ap.add_argument("--ratio", type=float, default=0.5)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    ap.add_argument("--path", default="masked", choices=["masked", "packed"])
    ap.add_argument("--out", default="i8", choices=["i8", "f32", "i32", "f16", "bf16"])
    ap.add_argument("--dynamic", action="store_true", help="run-time extraction positions (Sec. 4.1): the prologue finds them from the call's own values")
    ap.add_argument("--aux", default="", choices=["", "reorder", "calib", "distance"], help="run an auxiliary kernel on the layer's input instead: the residual reorder operator, the calibration range kernels, or the squared-distance reduction (on the int8 view of the input and a shifted copy)")
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    c, is_conv = make_case(args.layer)
    qcal = calib.quantize_reference(torch.from_numpy(c.Xcal), c.x_scale)
    perm, x_shift = calib.static_preparation(qcal, torch.from_numpy(c.Wq), c.G, conv=is_conv)
    L = fx.Layer(torch.from_numpy(c.Wq).to(dev), torch.from_numpy(c.w_scale).to(dev), torch.from_numpy(c.bias).to(dev),
                 perm, x_shift, c.G, conv=(c.stride, c.pad) if is_conv else None)
    L.set_lowbit_path(fx.LOWBIT_PACKED_U4 if args.path == "packed" else fx.LOWBIT_MASKED_I8)
    L.set_lowbit_ratio(args.ratio)
    X = torch.from_numpy(c.X).to(dev)
    mode = {"i8": fx.OUT_REQUANT_I8, "f32": fx.OUT_DEQUANT_F32, "i32": fx.OUT_ACC_I32, "f16": fx.OUT_DEQUANT_F16,
            "bf16": fx.OUT_DEQUANT_BF16}[args.out]
    M = X.numel() // L.K
    stream = torch.cuda.current_stream()
    if args.aux:
        Xq = X.reshape(-1, L.K)
        lo = torch.empty(L.K, dtype=torch.int32, device=dev)
        hi = torch.empty(L.K, dtype=torch.int32, device=dev)
        Yr = torch.empty_like(Xq)
        if args.aux == "distance":
            A8 = Xq.view(torch.int8).reshape(-1)
            B8 = torch.roll(A8, 16)
            d_out = torch.zeros(1, dtype=torch.int64, device=dev)

        def aux():
            if args.aux == "distance":
                fx.flexiq_sq_distance_i8(A8, B8, d_out)
            elif args.aux == "reorder":
                L.reorder_channels(Xq, fx.REORDER_TO_SLAB, Y=Yr)
            else:
                fx.flexiq_calib_channel_ranges(Xq, fx._dtype_code(Xq), Xq.shape[0], L.K, c.x_scale, False, lo, hi)

        for _ in range(args.warmup):
            aux()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(args.iters):
            aux()
        e1.record(stream)
        torch.cuda.synchronize()
        t = e0.elapsed_time(e1) / args.iters
        moved = Xq.numel() * Xq.element_size() * (1 if args.aux == "calib" else 2)
        print(f"{args.layer} {args.aux}: {t * 1e3:.1f} us, {moved / t / 1e6:.0f} GB/s")
        L.close()
        return

    def mixed(x4, x8):
        if is_conv:
            return L.mixed_conv(x4, x8, c.Nb, c.H, c.W, c.x_scale, c.y_scale, mode, Y=Ybuf, x_shift=shifts)
        return L.mixed_gemm(x4, x8, M, c.x_scale, c.y_scale, mode, Y=Ybuf, x_shift=shifts)

    x4, x8, shifts = L.quantize_lower(X, c.x_scale, dynamic=args.dynamic)
    slabs = (x4, x8)
    Ybuf = None
    Ybuf = mixed(x4, x8)
    ops = 2.0 * Ybuf.numel() * (c.R * c.S * c.C if is_conv else c.K)
    for _ in range(args.warmup):
        L.quantize_lower(X, c.x_scale, dynamic=args.dynamic, slabs=slabs)
        mixed(x4, x8)
    # back-to-back launches: the queue stays full, so launch latency is hidden
    e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    torch.cuda.synchronize()
    e[0].record(stream)
    for _ in range(args.iters):
        L.quantize_lower(X, c.x_scale, dynamic=args.dynamic, slabs=slabs)
    e[1].record(stream)
    for _ in range(args.iters):
        mixed(x4, x8)
    e[2].record(stream)
    torch.cuda.synchronize()
    fx.flexiq_check_status()
    tp = e[0].elapsed_time(e[1]) / args.iters
    tg = e[1].elapsed_time(e[2]) / args.iters
    print(f"{args.layer} ratio={args.ratio} path={args.path}{' dynamic positions' if args.dynamic else ''}: prologue {tp * 1e3:.1f} us, mixed kernel {tg * 1e3:.1f} us, "
          f"{ops / tg / 1e9:.1f} TOPS")
    L.close()


if __name__ == "__main__":
    main()
