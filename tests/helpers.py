"""Shared test plumbing: oracle-side preparation of a case and expected results."""
from __future__ import annotations

import numpy as np

import oracle


def prepare_linear(case, x_shift_override=None):
    """Static preparation with the oracle: calibration ranges -> positions -> greedy order."""
    qcal = oracle.quantize(case.Xcal, case.x_scale)
    lo, hi = oracle.channel_ranges(qcal)
    sx_group = oracle.static_positions(lo, hi, case.G)
    if x_shift_override is not None:
        sx_group = np.asarray(x_shift_override, np.uint8)
    perm, _ = oracle.greedy_order(lo, hi, oracle.weight_absmax_linear(case.Wq), case.G)
    sw = oracle.weight_positions_linear(case.Wq, case.G, perm)
    return perm, sx_group, sx_group[perm].copy(), sw


def prepare_conv(case, x_shift_override=None):
    qcal = oracle.quantize(case.Xcal, case.x_scale).reshape(-1, case.C)
    lo, hi = oracle.channel_ranges(qcal)
    sx_group = oracle.static_positions(lo, hi, case.G)
    if x_shift_override is not None:
        sx_group = np.asarray(x_shift_override, np.uint8)
    perm, _ = oracle.greedy_order(lo, hi, oracle.weight_absmax_conv(case.Wq), case.G)
    sw = oracle.weight_positions_conv(case.Wq, case.G, perm)
    return perm, sx_group, sx_group[perm].copy(), sw


def masked_slab(X4_packed, G, sx_slab, n_low):
    """int8 form of the packed low-bit slab: nibble value << position (for the MASKED path)."""
    M = X4_packed.shape[0]
    K_lo = n_low * G
    b = X4_packed[:, :K_lo // 2]
    lo = (b & 15).astype(np.int16)
    hi = (b >> 4).astype(np.int16)
    lo = np.where(lo > 7, lo - 16, lo)
    hi = np.where(hi > 7, hi - 16, hi)
    v = np.empty((M, K_lo), np.int16)
    v[:, 0::2] = lo
    v[:, 1::2] = hi
    sh = np.repeat(sx_slab[:n_low].astype(np.int16), G)[None, :]
    return (v << sh).astype(np.int8)


def with_guard(torch, shape, dtype, device, guard=256):
    """A tensor surrounded by poisoned guard bands; returns (view, check())."""
    n = int(np.prod(shape))
    esz = torch.empty(0, dtype=dtype).element_size()
    raw = torch.full((guard + n * esz + guard,), 0x5A, dtype=torch.uint8, device=device)
    view = raw[guard:guard + n * esz].view(dtype).view(*shape)

    def check():
        assert bool((raw[:guard] == 0x5A).all()) and bool((raw[guard + n * esz:] == 0x5A).all()), "guard band overwritten"
    return view, check


def tiny_stack(seed=50, M=48, dims=(64, 96, 64), G=16, small=False):
    """A short chain of quantized linears for the selection search: layer dicts (scales chained, static
    positions from the 8-bit chain's own activations), the fp32 input, groups per layer and the 8-bit
    chain's int8 outputs (plain integer matmuls).  small=True: every value fits four bits."""
    from paper_2510_02822_b200 import inputs
    layers, X0 = [], None
    K = dims[0]
    for l, N in enumerate(dims[1:] + (dims[-1],)):
        c = inputs.ranged_linear(f"evo{l}", M, K, N, G, seed=seed + l, group_structured=True)
        Wq = np.clip(c.Wq, -7, 7) if small else c.Wq
        if X0 is None:
            X0 = c.X * (np.float32(0.05) if small else np.float32(1.0))
        layers.append(dict(Wq=Wq, w_scale=c.w_scale, bias=c.bias, x_scale=c.x_scale, y_scale=c.y_scale, G=G,
                           sx_group=np.zeros(K // G, np.uint8)))
        K = N
    # chain the scales: a layer's output scale is the next layer's input scale
    for l in range(len(layers) - 1):
        layers[l + 1]["x_scale"] = layers[l]["y_scale"]
    q = oracle.quantize(X0, layers[0]["x_scale"])
    for L in layers:  # static positions from the 8-bit chain's own activations
        lo, hi = oracle.channel_ranges(q)
        L["sx_group"] = np.zeros_like(oracle.static_positions(lo, hi, G)) if small else oracle.static_positions(lo, hi, G)
        acc = q.astype(np.int64) @ L["Wq"].astype(np.int64)
        q = oracle.epilogue_i8(acc.astype(np.int32), L["x_scale"], L["w_scale"], L["bias"], L["y_scale"])
    return layers, X0, [L["Wq"].shape[0] // G for L in layers], q
