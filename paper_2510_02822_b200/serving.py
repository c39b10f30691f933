"""Serving experiment on the GPU (Sec. 8): request queue + run-time ratio controller around the
stack of quantized linears of a transformer.

    python -m paper_2510_02822_b200.serving [--model vitb|deits] [--max-batch 1] [--requests 4000]
                                            [--service measured|paper-shaped] [--live] [--no-graphs]

1. profile: the time of one pass over the model's 48 quantized linear layers (prologue + mixed GEMM
   per layer, through the library, ratio set by flexiq_set_lowbit_ratio) per level (0/25/50/75/100 %)
   and batch size 1 .. max_batch; each (level, batch) pass is one CUDA graph that is complete in itself
   (it holds the write of the ratio-dependent weight block where its ratio needs one), so the graphs replay in any order.  `--service paper-shaped` replaces the measured table by one that
   falls with the ratio as the paper's GPU does (1.43x faster at 100 % than at 0 %), to exercise the
   controller where the hardware gives it something to trade; it is labelled as such in the output.
2. latency against request rate: Poisson arrivals at 100 .. 3000 requests/s through
   flexiq_serving_simulate at each fixed level: median and 90th-percentile response time.
3. fluctuating rate (peak = 3 x minimum): fixed lowest level, fixed highest level and the controller
   (profiled latency = step 2's 90th percentile, threshold = twice the unloaded latency).
4. `--live`: the fluctuating trace again, but every dispatched batch really runs on the GPU at the
   controller's level and the clock of the queue advances by the measured time of that batch.

Everything is synthetic: random-init 8-bit layers of the model's shapes, seeded request traces.
"""
from __future__ import annotations

import argparse
import json
import time

import numpy as np
import torch

from . import binding as fx
from . import calib, inputs

LEVELS = 5


class Stack:
    """The 12 x 4 quantized linears of a ViT-style encoder, each with its own weights and buffers."""

    def __init__(self, model: str, max_batch: int, dev, use_graphs: bool = True):
        layers = {"vitb": inputs.VIT_B_LAYERS, "deits": inputs.DEIT_S_LAYERS}[model]
        make = inputs.vit_linear if model == "vitb" else inputs.ranged_linear
        self.max_rows = max_batch * 197
        self.inst = []
        for i, (name, K, N) in enumerate(layers):
            c = make(f"{model}_{name}", self.max_rows, K, N, 16, seed=7000 + i)
            perm, xs = calib.static_preparation(calib.quantize_reference(torch.from_numpy(c.Xcal), c.x_scale), torch.from_numpy(c.Wq), 16)
            for _blk in range(12):
                L = fx.Layer(torch.from_numpy(c.Wq).to(dev), torch.from_numpy(c.w_scale).to(dev), torch.from_numpy(c.bias).to(dev), perm, xs, 16)
                X = torch.from_numpy(c.X).to(dev)
                slab = torch.empty(self.max_rows * K + 16, dtype=torch.uint8, device=dev)
                Y = torch.empty((self.max_rows, N), dtype=torch.int8, device=dev)
                self.inst.append((L, c, X, slab, Y))
        # block order: qkv, proj, fc1, fc2 of block 0, then block 1, ...
        self.inst = [self.inst[k * 12 + b] for b in range(12) for k in range(len(layers))]
        self.level = -1
        self.graphs = {}
        self.use_graphs = use_graphs

    def set_level(self, level: int):
        """Run-time ratio switch: one host integer per layer (flexiq_layer_sync_ratio below is kept as a no-cost
        precaution: a captured graph writes the ratio-dependent weight block itself)."""
        if level != self.level:
            for L, *_ in self.inst:
                L.set_lowbit_ratio(level / (LEVELS - 1))
                if self.use_graphs:
                    L.sync_ratio()
            self.level = level

    def launch(self, batch: int):
        rows = batch * 197
        for L, c, X, slab, Y in self.inst:
            fx.flexiq_quantize_lower(L.h, X, fx.DTYPE_F32, rows, c.x_scale, 0, slab, None)
            fx.flexiq_mixed_gemm(L.h, slab, None, None, rows, c.x_scale, c.y_scale, fx.OUT_REQUANT_I8, Y)

    def run(self, batch: int):
        """One pass at the level in force: 96 host launches, or the replay of the graph of (level, batch)."""
        if not self.use_graphs:
            return self.launch(batch)
        g = self.graphs.get((self.level, batch))
        if g is None:
            self.launch(batch)  # per-call scale vectors and tensor maps are made outside the capture
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    self.launch(batch)
            torch.cuda.current_stream().wait_stream(side)
            self.graphs[(self.level, batch)] = g
        g.replay()

    def timed(self, level: int, batch: int) -> float:
        """Seconds of one pass, switch of the ratio included, measured with CUDA events."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        self.set_level(level)
        self.run(batch)
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1) * 1e-3


def profile_service(stack: Stack, max_batch: int, reps: int) -> np.ndarray:
    table = np.zeros((LEVELS, max_batch))
    for _ in range(20):  # clocks, caches, first-call set-up
        stack.timed(0, 1)
    for level in range(LEVELS):
        for b in range(1, max_batch + 1):
            for _ in range(3):  # the graph is captured on the first pass
                stack.timed(level, b)
            table[level, b - 1] = float(np.median([stack.timed(level, b) for _ in range(reps)]))
    return table


def paper_shaped(table: np.ndarray) -> np.ndarray:
    """Level 0's measured times, scaled down linearly with the ratio to 1 / 1.43 at 100 % (Sec. 8)."""
    f = np.array([1.0 - (1.0 - 1.0 / 1.43) * l / (LEVELS - 1) for l in range(LEVELS)])
    return table[0][None, :] * f[:, None]


def stats(resp: np.ndarray) -> dict:
    return {"median_ms": round(float(np.median(resp)) * 1e3, 3), "p90_ms": round(float(np.percentile(resp, 90)) * 1e3, 3)}


def latency_vs_rate(service, max_batch, rates, n_req, seed=100):
    med = np.zeros((LEVELS, len(rates)))
    p90 = np.zeros((LEVELS, len(rates)))
    for j, rate in enumerate(rates):
        arr = inputs.poisson_arrivals(seed + j, rate, n_req)
        for level in range(LEVELS):
            resp, _ = fx.flexiq_serving_simulate(None, level, arr, service, max_batch)
            med[level, j] = np.median(resp)
            p90[level, j] = np.percentile(resp, 90)
    return med, p90


def per_second(arr, resp, lvl, duration):
    out = []
    for s in range(int(duration)):
        m = (arr >= s) & (arr < s + 1)
        if m.any():
            out.append({"t": s, "rate": int(m.sum()), "median_ms": round(float(np.median(resp[m])) * 1e3, 3),
                        "mean_level": round(float(lvl[m].mean()), 2)})
    return out


def live(stack: Stack, ctrl: fx.Controller, arr: np.ndarray, max_batch: int, window: float):
    """The queue of flexiq_serving_simulate with the service time of each batch measured on the GPU."""
    n = arr.size
    resp = np.zeros(n)
    lvl = np.zeros(n, dtype=np.int32)
    level = ctrl.level
    free_at = last = 0.0
    i = 0
    while i < n:
        start = max(free_at, arr[i])
        b = 1
        while i + b < n and b < max_batch and arr[i + b] <= start:
            b += 1
        if start - last >= window:
            cnt = int(np.searchsorted(arr, start, side="right") - np.searchsorted(arr, start - window, side="right"))
            level = ctrl.update(cnt / window)
            last = start
        done = start + stack.timed(level, b)
        resp[i:i + b] = done - arr[i:i + b]
        lvl[i:i + b] = level
        free_at = done
        i += b
    return resp, lvl


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--model", default="vitb", choices=["vitb", "deits"])
    ap.add_argument("--max-batch", type=int, default=1)
    ap.add_argument("--requests", type=int, default=4000)
    ap.add_argument("--reps", type=int, default=7)
    ap.add_argument("--service", default="measured", choices=["measured", "paper-shaped"])
    ap.add_argument("--duration", type=float, default=12.0)
    ap.add_argument("--live", action="store_true")
    ap.add_argument("--no-graphs", action="store_true", help="96 host launches per pass instead of one CUDA graph per (level, batch)")
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    t0 = time.time()
    stack = Stack(args.model, args.max_batch, dev, use_graphs=not args.no_graphs)
    measured = profile_service(stack, args.max_batch, args.reps)
    service = paper_shaped(measured) if args.service == "paper-shaped" else measured
    print(json.dumps({"step": "profile", "model": args.model, "layers": len(stack.inst), "setup_s": round(time.time() - t0, 1),
                      "service_table": args.service, "launch": "host launches" if args.no_graphs else "one CUDA graph per (level, batch)",
                      "pass_ms[level][batch]": [[round(v * 1e3, 4) for v in row] for row in service]}), flush=True)

    rates = [100.0, 250.0, 500.0, 750.0, 1000.0, 1250.0, 1500.0, 1750.0, 2000.0, 2500.0, 3000.0]
    med, p90 = latency_vs_rate(service, args.max_batch, rates, args.requests)
    for level in range(LEVELS):
        print(json.dumps({"step": "latency_vs_rate", "ratio": level / (LEVELS - 1), "rates": rates,
                          "median_ms": [round(v * 1e3, 3) for v in med[level]], "p90_ms": [round(v * 1e3, 3) for v in p90[level]]}), flush=True)

    # fluctuating trace: the peak is three times the minimum; the peak sits at 90 % of what the lowest ratio can serve
    cap0 = args.max_batch / service[0, args.max_batch - 1]
    peak = 0.9 * cap0 if args.service == "measured" else 1.15 * cap0
    arr = inputs.fluctuating_arrivals(200, peak / 3.0, peak, args.duration / 2.0, args.duration)
    threshold = 2.0 * float(service[0, 0])
    window = 0.25
    out = {"step": "fluctuating", "rate_min": round(peak / 3, 1), "rate_max": round(peak, 1), "requests": int(arr.size),
           "threshold_ms": round(threshold * 1e3, 3), "window_s": window}
    for name, level in (("fixed_0", 0), ("fixed_100", LEVELS - 1)):
        resp, lvl = fx.flexiq_serving_simulate(None, level, arr, service, args.max_batch)
        out[name] = stats(resp)
    ctrl = fx.Controller(np.array(rates), p90, threshold, window)
    resp, lvl = fx.flexiq_serving_simulate(ctrl, 0, arr, service, args.max_batch)
    out["controller"] = {**stats(resp), "mean_ratio": round(float(lvl.mean()) / (LEVELS - 1), 3),
                         "switches": int(np.count_nonzero(np.diff(lvl)))}
    print(json.dumps(out), flush=True)
    print(json.dumps({"step": "fluctuating_per_second", "controller": per_second(arr, resp, lvl, args.duration)}), flush=True)
    ctrl.close()

    if args.live:
        ctrl = fx.Controller(np.array(rates), p90, threshold, window)
        t1 = time.time()
        resp, lvl = live(stack, ctrl, arr, args.max_batch, window)
        print(json.dumps({"step": "live", "what": "every batch ran on the GPU at the controller's level; queue clock advanced by its measured time",
                          "wall_s": round(time.time() - t1, 1), **stats(resp), "mean_ratio": round(float(lvl.mean()) / (LEVELS - 1), 3),
                          "switches": int(np.count_nonzero(np.diff(lvl)))}), flush=True)
        ctrl.close()
    fx.flexiq_check_status()


if __name__ == "__main__":
    main()
