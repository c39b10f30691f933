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
