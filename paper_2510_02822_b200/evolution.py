"""Evolutionary selection of low-bitwidth channel groups on the GPU (Sec. 4.2, Algorithm 1).

The genetic operators run in the library on the host (flexiq_evo_init, flexiq_evo_next_generation);
the fitness of a chromosome is measured with the hot path itself: every layer of a chain of
quantized linears is created with the chromosome's selected groups first in its group order and
K_lo = their number, the chain runs (prologue + mixed GEMM per layer, int8 between layers) and
flexiq_sq_distance_i8 gives the exact squared distance of the last layer's outputs from those of
the 8-bit chain.  One handle per layer serves every chromosome: flexiq_layer_set_group_perm lays it
out again for the next selection without allocating or synchronising.

    python -m paper_2510_02822_b200.evolution [--model deits|vitb] [--blocks 2] [--batch 4]
                                              [--population 16] [--generations 10] [--ratios 0.25 0.5 0.75]

searches nested selections for the given ratios on a synthetic chain of that model's linears and
reports, per ratio, the distance of the greedy per-layer selection, of the best chromosome, and
the time per generation.  Everything is synthetic: random-init 8-bit layers, seeded inputs; the
distance to the 8-bit chain stands in for the paper's distance between soft labels.
"""
from __future__ import annotations

import argparse
import json
import time

import numpy as np
import torch

from . import binding as fx
from . import calib, inputs


def selection_perm(flags_layer):
    """Group order for a selection: the selected groups (index order), then the others."""
    f = np.asarray(flags_layer).astype(bool)
    idx = np.arange(f.size, dtype=np.int32)
    return np.concatenate([idx[f], idx[~f]]).astype(np.int32), int(f.sum())


class ChainFitness:
    """Distance of a chain of quantized linears under a selection from the 8-bit chain.

    layers[l] = dict(Wq [K, N] int8, w_scale, bias, x_scale, y_scale, G, sx_group [K/G]); layer l + 1
    takes layer l's int8 output as its quantized input (x_scale of l + 1 = y_scale of l)."""

    def __init__(self, layers, X, dev):
        self.dev = dev
        self.layers = layers
        self.M = X.shape[0]
        self.groups = [L["Wq"].shape[0] // L["G"] for L in layers]
        self.off = np.concatenate([[0], np.cumsum(self.groups)]).astype(int)
        self.X = torch.from_numpy(np.ascontiguousarray(X)).to(dev)
        self.dev_params = [(torch.from_numpy(L["Wq"]).to(dev), torch.from_numpy(L["w_scale"]).to(dev), torch.from_numpy(L["bias"]).to(dev))
                           for L in layers]
        self.slab = [torch.empty(self.M * L["Wq"].shape[0] + 16, dtype=torch.uint8, device=dev) for L in layers]
        self.Y = [torch.empty((self.M, L["Wq"].shape[1]), dtype=torch.int8, device=dev) for L in layers]
        self.handles = [None] * len(layers)
        self.current = [None] * len(layers)
        self.created = 0
        self.evaluated = 0
        self.Y8 = self.outputs(np.zeros(int(self.off[-1]), dtype=np.uint8)).clone()

    def _layer(self, l, flags_layer):
        """The handle of layer l laid out for this selection: one handle per layer, re-laid out in place
        (flexiq_layer_set_group_perm: no allocation, no synchronisation) when the selection changes."""
        key = bytes(np.asarray(flags_layer, dtype=np.uint8))
        h = self.handles[l]
        if key != self.current[l]:
            perm, n_low = selection_perm(flags_layer)
            Wq, ws, b = self.dev_params[l]
            xs = np.asarray(self.layers[l]["sx_group"], dtype=np.uint8)
            if h is None:
                h = self.handles[l] = fx.Layer(Wq, ws, b, perm, xs, self.layers[l]["G"])
            else:
                h.set_group_perm(Wq, perm, xs)
            h.set_lowbit_ratio(n_low / self.groups[l])
            self.current[l] = key
            self.created += 1
        return h

    def outputs(self, flags):
        """int8 outputs of the last layer under the selection `flags` (device tensor, reused by the next call)."""
        src, dtype = self.X, fx.DTYPE_F32
        for l, L in enumerate(self.layers):
            h = self._layer(l, flags[self.off[l]:self.off[l + 1]])
            fx.flexiq_quantize_lower(h.h, src, dtype, self.M, L["x_scale"], 0, self.slab[l], None)
            fx.flexiq_mixed_gemm(h.h, self.slab[l], None, None, self.M, L["x_scale"], L["y_scale"], fx.OUT_REQUANT_I8, self.Y[l])
            src, dtype = self.Y[l], fx.DTYPE_I8
        self.evaluated += 1
        return self.Y[-1]

    def distances(self, pop):
        """Exact squared distances of every chromosome of `pop` (one device synchronisation in all)."""
        out = torch.zeros(len(pop), dtype=torch.int64, device=self.dev)
        for i, c in enumerate(pop):
            fx.flexiq_sq_distance_i8(self.outputs(np.asarray(c, dtype=np.uint8)), self.Y8, out[i:i + 1])
        return [int(v) for v in out.cpu().tolist()]

    def close(self):
        for h in self.handles:
            if h is not None:
                h.close()
        self.handles = [None] * len(self.layers)
        self.current = [None] * len(self.layers)


def search(fit: ChainFitness, score, per_layer_target, N, k, r, rate_bp, generations, seed, locked=None):
    """Algorithm 1: returns (best flags, its distance, best distance per generation, seconds per generation)."""
    groups = fit.groups
    pop, target = fx.flexiq_evo_init(groups, score, per_layer_target, N, seed, locked)
    history, secs = [], []
    for g in range(generations):
        t0 = time.time()
        dist = fit.distances(pop)
        history.append(min(dist))
        pop = fx.flexiq_evo_next_generation(pop, dist, groups, score, target, k, r, rate_bp, seed, g, locked)
        secs.append(time.time() - t0)
    dist = fit.distances(pop)
    history.append(min(dist))
    best = min(range(len(dist)), key=lambda i: (dist[i], i))
    return pop[best].copy(), dist[best], history, secs


def nested_search(fit: ChainFitness, score, ratios, N, k, r, rate_bp, generations, seed):
    """Selections for ascending ratios, each keeping the groups of the one before (the nesting that
    lets one stored order serve every ratio); returns the per-ratio results and, per layer, the group
    order: groups by the first ratio that selected them (then index), never-selected groups last."""
    locked = None
    first = np.full(int(fit.off[-1]), len(ratios), dtype=np.int32)
    results = []
    for t, ratio in enumerate(sorted(ratios)):
        tgt = [int(np.ceil(ratio * g - 1e-4)) for g in fit.groups]
        flags, dist, hist, secs = search(fit, score, tgt, N, k, r, rate_bp, generations, seed + t, locked)
        first = np.where((flags == 1) & (first == len(ratios)), t, first)
        locked = flags.copy()
        results.append(dict(ratio=ratio, flags=flags, distance=dist, history=hist, seconds=secs))
    perms = []
    for l in range(len(fit.groups)):
        f = first[fit.off[l]:fit.off[l + 1]]
        perms.append(np.argsort(f, kind="stable").astype(np.int32))
    return results, perms


def synthetic_chain(model: str, blocks: int, batch: int, G: int = 16, seed: int = 9000):
    """fc1 -> fc2 pairs of the model's MLPs chained `blocks` times (K -> 4K -> K -> ...), scales chained,
    static activation positions and error scores from the 8-bit chain's own activations."""
    table = {"deits": (384, 1536), "vitb": (768, 3072)}[model]
    dims = [table[0]]
    for _ in range(blocks):
        dims += [table[1], table[0]]
    M = batch * 197
    layers, X0 = [], None
    for l in range(len(dims) - 1):
        c = inputs.ranged_linear(f"evo_{model}_{l}", M, dims[l], dims[l + 1], G, seed=seed + l, group_structured=True)
        if X0 is None:
            X0 = c.X
        layers.append(dict(Wq=c.Wq, w_scale=c.w_scale, bias=c.bias, x_scale=c.x_scale, y_scale=c.y_scale, G=G,
                           sx_group=np.zeros(dims[l] // G, np.uint8)))
    for l in range(len(layers) - 1):
        layers[l + 1]["x_scale"] = layers[l]["y_scale"]
    return layers, X0


def calibrate_chain(layers, X, dev):
    """Static positions and error scores of every layer from the 8-bit chain's activations (device calibration)."""
    scores = []
    src = torch.from_numpy(np.ascontiguousarray(X)).to(dev)
    for i, L in enumerate(layers):
        Wq = torch.from_numpy(L["Wq"]).to(dev)
        _perm, xs, info = calib.static_preparation_device(src, L["x_scale"], Wq, L["G"])
        score = info["score"].cpu().numpy()
        L["sx_group"] = xs
        scores += [int(v) for v in score]
        ident = np.arange(L["Wq"].shape[0] // L["G"], dtype=np.int32)
        h = fx.Layer(Wq, torch.from_numpy(L["w_scale"]).to(dev), torch.from_numpy(L["bias"]).to(dev), ident, xs, L["G"])
        M = src.shape[0]
        slab = torch.empty(M * L["Wq"].shape[0] + 16, dtype=torch.uint8, device=dev)
        Y = torch.empty((M, L["Wq"].shape[1]), dtype=torch.int8, device=dev)
        fx.flexiq_quantize_lower(h.h, src, fx.DTYPE_I8 if src.dtype == torch.int8 else fx.DTYPE_F32, M, L["x_scale"], 0, slab, None)
        # output scale of the 8-bit chain: absmax of the de-quantized outputs (nothing saturates), which is
        # also the next layer's input scale
        Yf = torch.empty((M, L["Wq"].shape[1]), dtype=torch.float32, device=dev)
        fx.flexiq_mixed_gemm(h.h, slab, None, None, M, L["x_scale"], 1.0, fx.OUT_DEQUANT_F32, Yf)
        L["y_scale"] = float(np.float32(float(Yf.abs().max()) / 127.0))
        fx.flexiq_mixed_gemm(h.h, slab, None, None, M, L["x_scale"], L["y_scale"], fx.OUT_REQUANT_I8, Y)
        torch.cuda.synchronize()
        h.close()
        src = Y
        if i + 1 < len(layers):
            layers[i + 1]["x_scale"] = L["y_scale"]
    return scores


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--model", default="deits", choices=["deits", "vitb"])
    ap.add_argument("--blocks", type=int, default=2)
    ap.add_argument("--batch", type=int, default=4)
    ap.add_argument("--population", type=int, default=16)
    ap.add_argument("--elites", type=int, default=2)
    ap.add_argument("--parents", type=int, default=8)
    ap.add_argument("--mutation-bp", type=int, default=100)
    ap.add_argument("--generations", type=int, default=10)
    ap.add_argument("--ratios", type=float, nargs="+", default=[0.25, 0.5, 0.75])
    ap.add_argument("--seed", type=int, default=1)
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    layers, X = synthetic_chain(args.model, args.blocks, args.batch)
    score = calibrate_chain(layers, X, dev)
    fit = ChainFitness(layers, X, dev)
    print(json.dumps({"step": "setup", "model": args.model, "layers": len(layers), "rows": int(X.shape[0]),
                      "groups_per_layer": fit.groups, "flags": int(fit.off[-1])}), flush=True)
    t0 = time.time()
    results, perms = nested_search(fit, score, args.ratios, args.population, args.elites, args.parents, args.mutation_bp,
                                   args.generations, args.seed)
    for res in results:
        per_layer = [float(res["flags"][fit.off[l]:fit.off[l + 1]].mean()) for l in range(len(fit.groups))]
        print(json.dumps({"step": "ratio", "ratio": res["ratio"], "greedy_or_first_generation_best": res["history"][0],
                          "best": res["distance"], "gain": round(1.0 - res["distance"] / max(1, res["history"][0]), 4),
                          "history": res["history"], "per_layer_ratio": [round(v, 3) for v in per_layer],
                          "s_per_generation": round(float(np.mean(res["seconds"])), 4)}), flush=True)
    print(json.dumps({"step": "done", "wall_s": round(time.time() - t0, 2), "chromosomes_evaluated": fit.evaluated,
                      "layer_layouts": fit.created}), flush=True)
    # the stored group order serves every ratio: check the nesting on the first layer
    for t in range(1, len(results)):
        assert np.all(results[t]["flags"] >= results[t - 1]["flags"])
    fit.close()
    fx.flexiq_check_status()


if __name__ == "__main__":
    main()
