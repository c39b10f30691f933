"""The allocation-free dynamic prologue (flexiq_quantize_lower_dynamic_noalloc).

Some callers cannot call cudaMalloc where they run the prologue (a stream being captured into
a CUDA graph, an allocator hook, a serving loop that owns no spare device memory), so they
cannot provide the scratch words the regular dynamic-position call needs.  The entry point
tested here uses a fixed array inside the library instead.  It must give exactly the slabs and
positions of the regular entry point -- and of the CPU oracle -- on two calls in a row (the array keeps the previous
call's contents, so the second call proves that it is cleared), and it must refuse layers
with more channel groups than the array holds.

Collected last on purpose: a failure here cannot hide a failure of any other test.
"""
import numpy as np
import pytest
import torch

import helpers
import oracle
from paper_2510_02822_b200 import binding as fx
from paper_2510_02822_b200 import inputs

pytestmark = pytest.mark.gpu


def _perm(case, G):
    return np.random.default_rng(case.K).permutation(case.K // G).astype(np.int32)


def _layer(case, dev, G):
    n_g = case.K // G
    perm = _perm(case, G)
    return fx.Layer(torch.from_numpy(case.Wq).to(dev), torch.from_numpy(case.w_scale).to(dev), None, perm,
                    np.zeros(n_g, np.uint8), G)


def _run(L, case, X, entry, dev):
    """Slabs and positions written by one call of `entry` (buffers pre-filled with a pattern)."""
    M, K = case.M, case.K
    x4 = torch.full((M * K + 16,), 0xA5, dtype=torch.uint8, device=dev)
    x8 = torch.full((M * K + 16,), 0x5A, dtype=torch.uint8, device=dev).view(torch.int8)
    shifts = torch.full((K // L.G,), 0xEE, dtype=torch.uint8, device=dev)
    if entry == "regular":
        scratch = torch.full((K // L.G,), -1, dtype=torch.int32, device=dev)  # dirty on purpose: the call clears it
        fx.flexiq_quantize_lower(L.h, X, fx.DTYPE_F32, M, case.x_scale, 1, x4, x8, shifts, scratch)
    else:
        fx.flexiq_quantize_lower_dynamic_noalloc(L.h, X, fx.DTYPE_F32, M, case.x_scale, x4, x8, shifts)
    torch.cuda.synchronize()
    return x4.cpu().numpy(), x8.cpu().numpy(), shifts.cpu().numpy()


@pytest.mark.parametrize("path", [fx.LOWBIT_MASKED_I8, fx.LOWBIT_PACKED_U4])
def test_noalloc_entry_point_matches_regular_entry_point_twice(path):
    dev = torch.device("cuda:0")
    big = inputs.ranged_linear("na_big", 301, 384, 32, 16, seed=91, group_structured=True)     # wide ranges
    small = inputs.ranged_linear("na_small", 77, 384, 32, 16, seed=92, group_structured=True)  # then small values:
    small.X = (small.X * 0.01).astype(np.float32)                                              # stale OR bits would show
    L = _layer(big, dev, 16)
    L.set_lowbit_path(path)
    L.set_lowbit_ratio(0.75)
    for case in (big, small):  # two calls in a row through the new entry point
        X = torch.from_numpy(case.X).to(dev)
        ref = _run(L, case, X, "regular", dev)
        got = _run(L, case, X, "noalloc", dev)
        for r, g in zip(ref, got):
            assert np.array_equal(r, g)
        # and against the oracle: positions from the OR over the call's own values, slabs lowered with them
        M, K, G = case.M, case.K, 16
        perm = _perm(big, G)
        q = oracle.quantize(case.X, case.x_scale)
        sx = oracle.dynamic_positions(q, G, perm)
        assert np.array_equal(got[2], sx)
        nl = oracle.n_low(0.75, K // G)
        e4, e8 = oracle.make_slabs(q, G, perm, sx, nl)
        if path == fx.LOWBIT_MASKED_I8:
            slab = got[0][:M * K].reshape(M, K).view(np.int8)
            assert np.array_equal(slab[:, :nl * G], helpers.masked_slab(e4, G, sx, nl))
            assert np.array_equal(slab[:, nl * G:], e8)
        else:
            pitch = fx.flexiq_x4_pitch(L.h, nl * G)
            assert np.array_equal(got[0][:M * pitch].reshape(M, pitch)[:, :nl * G // 2], e4[:, :nl * G // 2])
            assert np.array_equal(got[1][:M * (K - nl * G)].reshape(M, K - nl * G), e8)
    # the second input is much smaller, so its positions must be smaller too (nothing left over)
    assert _run(L, small, torch.from_numpy(small.X).to(dev), "noalloc", dev)[2].max() <= 1
    L.close()


def test_noalloc_entry_point_rejects_layers_beyond_its_scratch():
    dev = torch.device("cuda:0")
    K, N, G = 4112 * 16, 16, 16  # 4112 groups > 4096
    Wq = torch.zeros((K, N), dtype=torch.int8, device=dev)
    L = fx.Layer(Wq, torch.ones(N, device=dev), None, np.arange(K // G, dtype=np.int32), None, G)
    X = torch.zeros((2, K), device=dev)
    x4, x8 = L.alloc_slabs(2)
    shifts = torch.zeros(K // G, dtype=torch.uint8, device=dev)
    with pytest.raises(fx.FlexiqError) as e:
        fx.flexiq_quantize_lower_dynamic_noalloc(L.h, X, fx.DTYPE_F32, 2, 1.0, x4, x8, shifts)
    assert e.value.code == fx.ERR_INVALID_ARG and "4096" in str(e.value)
    L.close()
