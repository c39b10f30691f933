"""Ratio sweeps over the benchmark configurations (one GPU).

    python -m paper_2510_02822_b200.sweep --config 2            # ViT-B linears, M = 12608
    python -m paper_2510_02822_b200.sweep --config 3            # ResNet-50 convolutions, batch 32
    python -m paper_2510_02822_b200.sweep --config 4 --cold     # DeiT-S small batch, L2 flushed between calls
    python -m paper_2510_02822_b200.sweep --config 4 --stack    # DeiT-S 12-block stack, one CUDA graph per replica, cold and warm
    python -m paper_2510_02822_b200.sweep --config 5            # ViT-L stack, ratio switched between passes

Prints one JSON line per (layer, ratio): device time of the prologue and of the mixed kernel
(CUDA events on the launching stream), TOPS = 2*M*N*K / t and algorithmic GB/s of the mixed kernel.
Warm numbers come from back-to-back launches (--graph: captured in a CUDA graph and replayed, which
removes the host time between launches that dominates small shapes); --cold flushes L2 (writes a 256 MB buffer) before
every timed launch and times each launch on its own.
"""
from __future__ import annotations

import argparse
import json
import time

import numpy as np
import torch

from . import binding as fx
from . import calib, inputs

RATIOS = [0.0, 0.25, 0.5, 0.75, 1.0]


def _layer_for(case, dev, is_conv, path):
    qcal = calib.quantize_reference(torch.from_numpy(case.Xcal), case.x_scale)
    perm, x_shift = calib.static_preparation(qcal, torch.from_numpy(case.Wq), case.G, conv=is_conv)
    L = fx.Layer(torch.from_numpy(case.Wq).to(dev), torch.from_numpy(case.w_scale).to(dev), torch.from_numpy(case.bias).to(dev),
                 perm, x_shift, case.G, conv=(case.stride, case.pad) if is_conv else None)
    L.set_lowbit_path(path)
    return L


def _alg_bytes(case, is_conv, ratio, Mout):
    K = case.C if is_conv else case.K
    N = case.Cout if is_conv else case.N
    taps = case.R * case.S if is_conv else 1
    n_low = round(ratio * (K // case.G))
    rho = n_low * case.G / K
    Min = case.Nb * case.H * case.W if is_conv else case.M
    return Min * K * (1 - rho / 2) + taps * K * N * (1 - rho / 2) + n_low * N + 8 * N + Mout * N


def _say(quiet, obj):
    if not quiet:
        print(json.dumps(obj), flush=True)


def time_case(case, is_conv, dev, path, iters, cold, flush, graph=False, ratios=None, quiet=False):
    L = _layer_for(case, dev, is_conv, path)
    X = torch.from_numpy(case.X).to(dev)
    stream = torch.cuda.current_stream()
    rows = []
    for r in (RATIOS if ratios is None else ratios):
        L.set_lowbit_ratio(r)
        x4, x8, _ = L.quantize_lower(X, case.x_scale)

        def mixed(Y=None):
            if is_conv:
                return L.mixed_conv(x4, x8, case.Nb, case.H, case.W, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8, Y=Y)
            return L.mixed_gemm(x4, x8, case.M, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8, Y=Y)

        Y = mixed()
        Mout = Y.numel() // Y.shape[-1]
        K = case.C if is_conv else case.K
        ops = 2.0 * Y.numel() * (case.R * case.S * K if is_conv else K)
        for _ in range(3):
            L.quantize_lower(X, case.x_scale)
            mixed(Y)
        torch.cuda.synchronize()
        if cold:
            tp = tg = 0.0
            for _ in range(iters):
                e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
                flush.add_(1)
                e[0].record(stream)
                L.quantize_lower(X, case.x_scale)
                e[1].record(stream)
                flush.add_(1)
                e[2].record(stream)
                mixed(Y)
                e[3].record(stream)
                torch.cuda.synchronize()
                tp += e[0].elapsed_time(e[1])
                tg += e[2].elapsed_time(e[3])
            tp, tg = tp / iters, tg / iters
        elif graph:
            # the launches are captured once and replayed: no host time between them
            times = []
            for body in (lambda: L.quantize_lower(X, case.x_scale), lambda: mixed(Y)):
                g = torch.cuda.CUDAGraph()
                side = torch.cuda.Stream()
                side.wait_stream(stream)
                with torch.cuda.stream(side):
                    with torch.cuda.graph(g, stream=side):
                        for _ in range(iters):
                            body()
                torch.cuda.synchronize()
                g.replay()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(5):
                    g.replay()
                e1.record(stream)
                torch.cuda.synchronize()
                times.append(e0.elapsed_time(e1) / (5 * iters))
            tp, tg = times
        else:
            e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            e[0].record(stream)
            for _ in range(iters):
                L.quantize_lower(X, case.x_scale)
            e[1].record(stream)
            for _ in range(iters):
                mixed(Y)
            e[2].record(stream)
            torch.cuda.synchronize()
            tp, tg = e[0].elapsed_time(e[1]) / iters, e[1].elapsed_time(e[2]) / iters
        rows.append({"layer": case.name, "ratio": r, "path": "packed" if path else "masked", "cold": bool(cold), "graph": bool(graph),
                     "prologue_us": round(tp * 1e3, 2), "mixed_us": round(tg * 1e3, 2),
                     "mixed_tops": round(ops / tg / 1e9, 1), "mixed_alg_gbs": round(_alg_bytes(case, is_conv, r, Mout) / tg / 1e6, 1),
                     "ops": ops, "alg_bytes": _alg_bytes(case, is_conv, r, Mout)})
        _say(quiet, rows[-1])
    fx.flexiq_check_status()
    L.close()
    return rows


def run_stack(dev, batch, iters, quiet=False):
    """ViT-L/16 stack of linears: every layer's prologue + mixed GEMM in sequence, the ratio switched
    between passes with flexiq_set_lowbit_ratio (no re-packing, no re-allocation).  Also: the mixed GEMM
    alone per layer shape (the 24 blocks' layers of that shape in turn, so that no weights stay in L2), and
    the device time of a ratio switch.  The activations are a seeded block of M / 8 rows repeated eight times
    (the time does not depend on the values; drawing 130 million numbers on the host would take longer than
    the measurement).  Returns the rows it prints."""
    M = batch * 197
    out = []
    layers, meta = [], []
    t0 = time.time()
    Xs = {}
    for blk in range(24):
        for i, (name, K, N) in enumerate(inputs.VIT_L_LAYERS):
            c = inputs.vit_linear(f"vitl_b{blk}_{name}", 256, K, N, 16, seed=5000 + blk * 4 + i)  # 256 rows: weights + calibration only
            perm, xs = calib.static_preparation(calib.quantize_reference(torch.from_numpy(c.Xcal), c.x_scale), torch.from_numpy(c.Wq), 16)
            L = fx.Layer(torch.from_numpy(c.Wq).to(dev), torch.from_numpy(c.w_scale).to(dev), torch.from_numpy(c.bias).to(dev), perm, xs, 16)
            layers.append(L)
            meta.append((K, N, c.x_scale, c.y_scale))
            if K not in Xs:
                rows_drawn = (M + 7) // 8
                big = inputs.vit_linear("x", rows_drawn, K, 16, 16, seed=5900 + K)
                Xs[K] = torch.from_numpy(big.X).to(dev).repeat(8, 1)[:M].contiguous()
    slabs = {K: (torch.empty(M * K + 16, dtype=torch.uint8, device=dev), torch.empty(M * K + 16, dtype=torch.int8, device=dev)) for K in Xs}
    Ys = {N: torch.empty((M, N), dtype=torch.int8, device=dev) for N in {n for _, n, _, _ in meta}}
    _say(quiet, {"setup_s": round(time.time() - t0, 1), "layers": len(layers), "M": M})
    ops = sum(2.0 * M * K * N for K, N, _, _ in meta)
    stream = torch.cuda.current_stream()

    def one_pass():
        for L, (K, N, xs, ys) in zip(layers, meta):
            x4, x8 = slabs[K]
            fx.flexiq_quantize_lower(L.h, Xs[K], fx.DTYPE_F32, M, xs, 0, x4, x8)
            fx.flexiq_mixed_gemm(L.h, x4, x8, None, M, xs, ys, fx.OUT_REQUANT_I8, Ys[N])

    one_pass()
    torch.cuda.synchronize()
    # up and down again, so that a drift of the clocks over the run does not read as a trend over the ratio
    acc = {}
    for ratio in (0.0, 0.5, 1.0, 1.0, 0.5, 0.0):
        t_sw = time.perf_counter()
        for L in layers:
            L.set_lowbit_ratio(ratio)
        switch_us = (time.perf_counter() - t_sw) * 1e6
        one_pass()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(iters):
            one_pass()
        e1.record(stream)
        torch.cuda.synchronize()
        acc.setdefault(ratio, []).append((e0.elapsed_time(e1) / iters, switch_us))
    for ratio in (0.0, 0.5, 1.0):
        ms = sum(m for m, _ in acc[ratio]) / len(acc[ratio])
        switch_us = sum(u for _, u in acc[ratio]) / len(acc[ratio])
        out.append({"config": 5, "ratio": ratio, "pass_ms": round(ms, 3), "pass_ms_up_down": [round(m, 3) for m, _ in acc[ratio]],
                    "pass_tops_prologue_plus_gemm": round(ops / ms / 1e9, 1),
                    "ratio_switch_host_us_all_96_layers": round(switch_us, 1)})
        _say(quiet, out[-1])
    # the mixed GEMM alone, per layer shape and ratio: slabs written once, then the 24 layers of the shape in turn
    for si, (name, K, N) in enumerate(inputs.VIT_L_LAYERS):
        same = [L for i, L in enumerate(layers) if i % 4 == si]
        xs, ys = meta[si][2], meta[si][3]
        for ratio in (0.0, 0.5, 1.0):
            for L in same:
                L.set_lowbit_ratio(ratio)
            x4, x8 = slabs[K]
            fx.flexiq_quantize_lower(same[0].h, Xs[K], fx.DTYPE_F32, M, xs, 0, x4, x8)
            for L in same:
                fx.flexiq_layer_set_slab_check(L.h, False)   # one slab (same group order is not required for timing) feeds all 24
                fx.flexiq_mixed_gemm(L.h, x4, x8, None, M, xs, ys, fx.OUT_REQUANT_I8, Ys[N])
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(iters):
                for L in same:
                    fx.flexiq_mixed_gemm(L.h, x4, x8, None, M, xs, ys, fx.OUT_REQUANT_I8, Ys[N])
            e1.record(stream)
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) / (iters * len(same)) * 1e3
            out.append({"config": 5, "gemm_only": name, "K": K, "N": N, "ratio": ratio, "us": round(us, 2),
                        "tops": round(2.0 * M * K * N / us / 1e6, 1)})
            _say(quiet, out[-1])
        for L in same:
            fx.flexiq_layer_set_slab_check(L.h, True)
    # Device time of a ratio switch: everything flexiq_layer_sync_ratio enqueues for the 96 layers, captured in one
    # CUDA graph and replayed (launched from the host the 96 calls take longer than their kernels run).  At 0 / 50 /
    # 100 % max_4bit_ch is a multiple of the K block in every layer, so nothing is enqueued at all; 30 % falls
    # inside a block.  In a running model the write rides in the next prologue launch instead.
    for frm, to in ((0.0, 0.5), (0.5, 1.0), (1.0, 0.3), (0.3, 0.0)):
        t_sw = time.perf_counter()
        for L in layers:
            L.set_lowbit_ratio(to)
        host_us = (time.perf_counter() - t_sw) * 1e6
        moved = sum(N * 128 for K, N, _, _ in meta if (oracle_free_n_low(to, K // 16) * 16) % 128 != 0)
        dev_us = 0.0
        if moved:
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    for L in layers:
                        L.sync_ratio()
            torch.cuda.synchronize()
            g.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(5):
                g.replay()
            e1.record(stream)
            torch.cuda.synchronize()
            dev_us = e0.elapsed_time(e1) / 5 * 1e3
        out.append({"config": 5, "switch": f"{frm} -> {to}", "device_us_all_96_layers": round(dev_us, 1), "kernels_enqueued": 96 if moved else 0,
                    "host_us_all_96_layers": round(host_us, 1), "weight_bytes_written": moved})
        _say(quiet, out[-1])
    fx.flexiq_check_status()
    for L in layers:
        L.close()
    return out


def oracle_free_n_low(ratio, n_g):
    """Number of low-bit groups the library derives from a ratio (same rounding rule), for reporting only."""
    import math
    return max(0, min(n_g, math.ceil(float(np.float32(ratio)) * n_g - 1e-4)))


def run_deit_stack(dev, batch, replicas, iters, quiet=False):
    """DeiT-S stack of linears (12 blocks x 4 layers = 48 layer instances, each with its own weights,
    input and output) captured in ONE CUDA graph per replica; `replicas` distinct copies of the whole
    stack are replayed in turn so that nothing a replay touches is still in L2 from the previous time
    (cold), then one replica is replayed alone (warm).  Reports time per pass and the algorithmic GB/s
    (fp32 input + slab written and read + weights + int8 output) at ratios 0 / 0.5 / 1."""
    M = batch * 197
    stacks, total_bytes = [], 0
    t0 = time.time()
    base = {}
    for i, (name, K, N) in enumerate(inputs.DEIT_S_LAYERS):
        c = inputs.ranged_linear(f"deits_{name}", M, K, N, 16, seed=4000 + i)
        perm, xs = calib.static_preparation(calib.quantize_reference(torch.from_numpy(c.Xcal), c.x_scale), torch.from_numpy(c.Wq), 16)
        base[name] = (c, perm, xs)
    for rep_i in range(replicas):
        inst = []
        for blk in range(12):
            for name, K, N in inputs.DEIT_S_LAYERS:
                c, perm, xs = base[name]
                # distinct memory per instance (the values may repeat: only the addresses matter for the caches)
                L = fx.Layer(torch.from_numpy(c.Wq).to(dev), torch.from_numpy(c.w_scale).to(dev), torch.from_numpy(c.bias).to(dev), perm, xs, 16)
                X = torch.from_numpy(c.X).to(dev)
                x4 = torch.empty(M * K + 16, dtype=torch.uint8, device=dev)
                Y = torch.empty((M, N), dtype=torch.int8, device=dev)
                inst.append((L, c, X, x4, Y))
                total_bytes += int(2.5 * K * N) + M * K * 5 + M * N  # w8, w8m, w4; X fp32 + slab; Y
        stacks.append(inst)
    alg = sum(c.M * c.K * 4 + 2 * c.M * c.K + c.K * c.N + 8 * c.N + c.M * c.N for _, c, _, _, _ in stacks[0])
    out = [{"setup_s": round(time.time() - t0, 1), "replicas": replicas, "instances": replicas * 48, "M": M,
            "resident_MB": round(total_bytes / 1e6, 1), "algorithmic_MB_per_pass": round(alg / 1e6, 2)}]
    _say(quiet, out[-1])
    stream = torch.cuda.current_stream()

    def one_pass(inst):
        for L, c, X, x4, Y in inst:
            fx.flexiq_quantize_lower(L.h, X, fx.DTYPE_F32, c.M, c.x_scale, 0, x4, None)
            fx.flexiq_mixed_gemm(L.h, x4, None, None, c.M, c.x_scale, c.y_scale, fx.OUT_REQUANT_I8, Y)

    for ratio in (0.0, 0.5, 1.0):
        graphs = []
        for inst in stacks:
            for L, *_ in inst:
                L.set_lowbit_ratio(ratio)
            one_pass(inst)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    one_pass(inst)
            graphs.append(g)
        torch.cuda.synchronize()
        res = {}
        for label, order in (("cold", list(range(replicas))), ("warm", [0] * replicas)):
            for gi in order:
                graphs[gi].replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(iters):
                for gi in order:
                    graphs[gi].replay()
            e1.record(stream)
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) / (iters * len(order)) * 1e3
            res[label] = {"pass_us": round(us, 1), "us_per_layer": round(us / 48, 2), "alg_gbs": round(alg / us / 1e3, 1)}
        out.append({"config": 4, "protocol": "48-layer graph per replica", "batch": batch, "ratio": ratio, **res})
        _say(quiet, out[-1])
        del graphs
    fx.flexiq_check_status()
    for inst in stacks:
        for L, *_ in inst:
            L.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--iters", type=int, default=30)
    ap.add_argument("--cold", action="store_true")
    ap.add_argument("--graph", action="store_true", help="capture the launches in a CUDA graph and time its replay")
    ap.add_argument("--path", default="masked", choices=["masked", "packed"])
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--stack", action="store_true", help="config 4: 12-block DeiT-S stack in one CUDA graph, rotating replicas (cold) and one replica (warm)")
    ap.add_argument("--replicas", type=int, default=0)
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    path = fx.LOWBIT_PACKED_U4 if args.path == "packed" else fx.LOWBIT_MASKED_I8
    flush = torch.zeros(64 * 1024 * 1024, dtype=torch.int32, device=dev) if args.cold else None
    if args.config == 1:
        time_case(inputs.config1(), False, dev, path, args.iters, args.cold, flush, args.graph)
    elif args.config == 2:
        for c in inputs.config2(args.batch or 64):
            time_case(c, False, dev, path, args.iters, args.cold, flush, args.graph)
    elif args.config == 3:
        for c in inputs.config3(args.batch or 32):
            time_case(c, True, dev, path, args.iters, args.cold, flush, args.graph)
    elif args.config == 4 and args.stack:
        b = args.batch or 1
        run_deit_stack(dev, b, args.replicas or (10 if b == 1 else 4), max(2, args.iters // 10))
    elif args.config == 4:
        for c in inputs.config4(args.batch or 1):
            time_case(c, False, dev, path, args.iters, args.cold, flush, args.graph)
    elif args.config == 5:
        run_stack(dev, args.batch or 128, max(1, args.iters // 10))


if __name__ == "__main__":
    main()
