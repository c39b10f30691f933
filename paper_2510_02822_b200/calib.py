"""Offline preparation that feeds the hot path (host side, runs once per layer).

From a calibration batch: per-channel ranges of the quantized activations, the static
extraction position of every channel group (Sec. 4.1), the error-estimation score
(activation range x largest weight range, Sec. 4.2) and the greedy nested group order
whose prefixes are the low-bit sets of every ratio (Sec. 4.2 / Sec. 5).  Written with
torch tensor ops; it is independent of the test oracle.
"""
from __future__ import annotations

import numpy as np
import torch


def quantize_reference(x: torch.Tensor, scale: float) -> torch.Tensor:
    """Eq. 1 on the host (calibration only): fp32 division, round-half-even, clip."""
    s = torch.tensor(scale, dtype=torch.float32)
    return torch.clamp(torch.round(x.to(torch.float32) / s), -128, 127).to(torch.int8)


def _used_bits(lo: torch.Tensor, hi: torch.Tensor) -> torch.Tensor:
    # magnitude bits needed for [lo, hi]: bit length of hi and of ~lo
    m = torch.maximum(hi.clamp(min=0), (-lo - 1).clamp(min=0)).to(torch.int64)
    bits = torch.zeros_like(m)
    for b in range(8):
        bits = torch.where(m >= (1 << b), torch.full_like(m, b + 1), bits)
    return bits


def static_preparation(Xcal_q: torch.Tensor, Wq: torch.Tensor, G: int, conv: bool = False):
    """Returns (group_perm int32 [n_g], x_shift uint8 [n_g] per ORIGINAL group).

    Xcal_q: int8 calibration activations [..., C]; Wq: int8 [K, N] (linear) or
    [Cout, R, S, Cin] (conv)."""
    C = Xcal_q.shape[-1]
    q = Xcal_q.reshape(-1, C).to(torch.int32)
    lo = q.min(0).values.clamp(max=0)
    hi = q.max(0).values.clamp(min=0)
    bits = _used_bits(lo, hi).reshape(-1, G).max(1).values
    x_shift = (bits - 3).clamp(min=0).to(torch.uint8)
    w = Wq.to(torch.int32).abs()
    wmax = w.reshape(-1, C).max(0).values if conv else w.max(1).values
    score = (torch.maximum(hi, -lo).to(torch.int64) * wmax.to(torch.int64)).reshape(-1, G).max(1).values
    perm = torch.sort(score, stable=True).indices.to(torch.int32)
    return np.ascontiguousarray(perm.numpy()), np.ascontiguousarray(x_shift.numpy())


def permute_outputs_for_next(Wq: torch.Tensor, w_scale: torch.Tensor, bias, next_perm, next_G: int, conv: bool = False):
    """Moves the next layer's channel reordering offline into this layer (Sec. 5): returns this
    layer's weights, scales and bias with the output channels in the next layer's slab order, so
    that output channel n of the permuted layer is slab channel n of the next one.

    Wq: int8 [K, N] (linear) or [Cout, R, S, Cin] (conv); next_perm: the next layer's group order."""
    cols = torch.cat([torch.arange(int(g) * next_G, (int(g) + 1) * next_G) for g in next_perm]).to(Wq.device)
    Wp = Wq.index_select(0 if conv else 1, cols).contiguous()
    return Wp, w_scale.index_select(0, cols).contiguous(), None if bias is None else bias.index_select(0, cols).contiguous()


def static_preparation_device(Xcal: torch.Tensor, x_scale: float, Wq: torch.Tensor, G: int, conv: bool = False, batches: int = 1,
                              coverage: float | None = None):
    """The same preparation with the library's calibration kernels, on device tensors.

    Xcal: calibration activations [..., C] (fp32 / fp16 / bf16 / int8) on the GPU; Wq as in
    static_preparation, on the GPU.  The rows are fed in `batches` accumulating calls.
    coverage (e.g. 0.99): channel ranges that cover that share of each channel's calibration values
    (per-channel histograms, equal tails dropped) instead of the exact min / max.
    Returns (group_perm, x_shift, info) with info = {lo, hi, wmax, score, unused_hist} (torch tensors)."""
    from . import binding as fx
    dev = Xcal.device
    C = Xcal.shape[-1]
    X2 = Xcal.reshape(-1, C)
    lo = torch.empty(C, dtype=torch.int32, device=dev)
    hi = torch.empty(C, dtype=torch.int32, device=dev)
    rows = X2.shape[0]
    step = (rows + batches - 1) // batches
    hist = torch.empty((C, 256), dtype=torch.int32, device=dev) if coverage is not None else None
    for b in range(batches):
        part = X2[b * step:(b + 1) * step]
        if coverage is None:
            fx.flexiq_calib_channel_ranges(part, fx._dtype_code(part), part.shape[0], C, x_scale, b > 0, lo, hi)
        else:
            fx.flexiq_calib_channel_histogram(part, fx._dtype_code(part), part.shape[0], C, x_scale, b > 0, hist)
    if coverage is not None:
        fx.flexiq_calib_ranges_from_histogram(hist, C, int(rows * (1.0 - coverage) / 2.0), lo, hi)
    wmax = torch.empty(C, dtype=torch.int32, device=dev)
    if conv:
        fx.flexiq_calib_weight_absmax(Wq, True, C, Wq.shape[0], Wq.shape[1] * Wq.shape[2], wmax)
    else:
        fx.flexiq_calib_weight_absmax(Wq, False, C, Wq.shape[1], 1, wmax)
    n_g = C // G
    perm = torch.empty(n_g, dtype=torch.int32, device=dev)
    x_shift = torch.empty(n_g, dtype=torch.uint8, device=dev)
    score = torch.empty(n_g, dtype=torch.int64, device=dev)
    hist = torch.empty(5, dtype=torch.int32, device=dev)
    fx.flexiq_calib_prepare(lo, hi, wmax, C, G, perm, x_shift, score, hist)
    info = {"lo": lo, "hi": hi, "wmax": wmax, "score": score, "unused_hist": hist}
    return np.ascontiguousarray(perm.cpu().numpy()), np.ascontiguousarray(x_shift.cpu().numpy()), info
