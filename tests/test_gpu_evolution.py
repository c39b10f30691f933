"""Evolutionary selection on the GPU (Sec. 4.2, Algorithm 1): the distance kernel against numpy
integers, the chain fitness against the oracle's, and a whole search, generation by generation."""
import numpy as np
import pytest
import torch

import helpers
from oracle import evolution as ev
from paper_2510_02822_b200 import binding as fx
from paper_2510_02822_b200 import evolution as gpu_ev
from paper_2510_02822_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    return torch.device("cuda:0")


@pytest.mark.parametrize("n", [0, 1, 15, 16, 17, 4101, 1000003, 40 * 1024 * 1024 + 7])
def test_sq_distance_is_exact(dev, n):
    a = (inputs.uniform(60, 0, n) * 256).astype(np.int64) - 128
    b = (inputs.uniform(60, 1, n) * 256).astype(np.int64) - 128
    if n > 2:
        a[0], b[0] = -128, 127      # the largest difference
        a[n - 1], b[n - 1] = 127, -128
    A = torch.from_numpy(a.astype(np.int8)).to(dev)
    B = torch.from_numpy(b.astype(np.int8)).to(dev)
    out = torch.full((1,), -5, dtype=torch.int64, device=dev)
    fx.flexiq_sq_distance_i8(A, B, out)
    assert int(out.item()) == int(((a - b) ** 2).sum())


def test_chain_fitness_matches_oracle(dev):
    layers, X, groups, y8 = helpers.tiny_stack(M=200, dims=(128, 192, 96))
    fit = gpu_ev.ChainFitness(layers, X, dev)
    assert fit.groups == groups
    assert np.array_equal(fit.Y8.cpu().numpy(), y8)
    pop = ev.init_population(groups, [int(v * 500) for v in inputs.uniform(61, 0, sum(groups))], [g // 2 for g in groups], 6, seed=3)
    pop.append([1] * sum(groups))
    want = [ev.sq_distance(ev.stack_forward(layers, X, c, groups), y8) for c in pop]
    assert fit.distances(pop) == want
    assert min(want) > 0
    fit.close()
    fx.flexiq_check_status()


def test_search_matches_oracle_generation_by_generation(dev):
    layers, X, groups, y8 = helpers.tiny_stack(seed=70, M=96, dims=(96, 128, 64))
    score = [int(v * 3000) for v in inputs.uniform(62, 0, sum(groups))]
    tgt = [max(1, g // 2) for g in groups]
    N, k, r, bp, gens, seed = 8, 2, 4, 1500, 5, 17

    def fitness(flags):
        return ev.sq_distance(ev.stack_forward(layers, X, flags, groups), y8)

    want_flags, want_dist, want_hist = ev.run(fitness, groups, score, tgt, N, k, r, bp, gens, seed)
    fit = gpu_ev.ChainFitness(layers, X, dev)
    flags, dist, hist, _ = gpu_ev.search(fit, score, tgt, N, k, r, bp, gens, seed)
    assert hist == want_hist
    assert dist == want_dist and flags.tolist() == want_flags
    assert all(b <= a for a, b in zip(hist, hist[1:]))
    fit.close()
    fx.flexiq_check_status()


def test_nested_search_keeps_smaller_selections(dev):
    layers, X, groups, y8 = helpers.tiny_stack(seed=80, M=64, dims=(128, 128, 128))
    score = [int(v * 3000) for v in inputs.uniform(63, 0, sum(groups))]
    fit = gpu_ev.ChainFitness(layers, X, dev)
    results, perms = gpu_ev.nested_search(fit, score, [0.25, 0.5, 0.75], 6, 2, 3, 1000, 3, seed=5)
    off = np.concatenate([[0], np.cumsum(groups)])
    for a, b in zip(results, results[1:]):
        assert np.all(b["flags"] >= a["flags"])
    for res in results:
        assert int(res["flags"].sum()) == sum(int(np.ceil(res["ratio"] * g - 1e-4)) for g in groups)
    # the stored order serves every ratio: the groups selected at a ratio are a prefix of the layer's order
    for l, perm in enumerate(perms):
        assert sorted(perm.tolist()) == list(range(groups[l]))
        for res in results:
            sel = set(np.flatnonzero(res["flags"][off[l]:off[l + 1]]).tolist())
            assert set(perm[:len(sel)].tolist()) == sel
    fit.close()


def test_relayout_in_place_matches_a_fresh_layer(dev):
    """flexiq_layer_set_group_perm: the handle laid out again for another order and other static
    positions computes what the oracle computes for that order, at the ratio that was in force."""
    import oracle
    case = inputs.ranged_linear("relay", 260, 256, 176, 16, seed=91, group_structured=True)
    perm_a, sxg, _, _ = helpers.prepare_linear(case)
    L = fx.Layer(torch.from_numpy(case.Wq).to(dev), torch.from_numpy(case.w_scale).to(dev), torch.from_numpy(case.bias).to(dev), perm_a, sxg, case.G)
    L.set_lowbit_ratio(0.5)
    X = torch.from_numpy(case.X).to(dev)
    Wq = torch.from_numpy(case.Wq).to(dev)
    x4, x8 = L.alloc_slabs(case.M)
    Y = torch.empty((case.M, case.N), dtype=torch.int8, device=dev)
    q = oracle.quantize(case.X, case.x_scale)
    n_g = case.K // case.G
    orders = [perm_a, np.arange(n_g, dtype=np.int32)[::-1].copy(), np.roll(np.arange(n_g, dtype=np.int32), 5)]
    shifts = [sxg, np.minimum(sxg + 1, 4).astype(np.uint8), sxg]
    for ratio in (0.5, 0.25, 1.0):
        L.set_lowbit_ratio(ratio)
        for perm, xs in zip(orders, shifts):
            L.set_group_perm(Wq, perm, xs)
            fx.flexiq_quantize_lower(L.h, X, fx.DTYPE_F32, case.M, case.x_scale, 0, x4, x8)
            fx.flexiq_mixed_gemm(L.h, x4, x8, None, case.M, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8, Y)
            sw = oracle.weight_positions_linear(case.Wq, case.G, perm)
            acc = oracle.mixed_gemm_acc(q, case.Wq, case.G, perm, xs[perm].copy(), sw, oracle.n_low(ratio, n_g))
            assert np.array_equal(Y.cpu().numpy(), oracle.epilogue_i8(acc, case.x_scale, case.w_scale, case.bias, case.y_scale))
    with pytest.raises(fx.FlexiqError):
        L.set_group_perm(Wq, np.zeros(n_g, dtype=np.int32))
    fx.flexiq_check_status()
    L.close()


def test_relayout_in_place_conv_and_fused_tables(dev):
    """The same for a convolution handle, and for the chunk tables a producer layer uses when it writes
    this layer's slab directly (fused boundary): they follow the new order too."""
    import oracle
    case = inputs.resnet_conv("relay_c", 2, 14, 128, 64, 3, seed=93)
    perm_a, sxg, _, _ = helpers.prepare_conv(case)
    L = fx.Layer(torch.from_numpy(case.Wq).to(dev), torch.from_numpy(case.w_scale).to(dev), torch.from_numpy(case.bias).to(dev),
                 perm_a, sxg, case.G, conv=(case.stride, case.pad))
    Wq = torch.from_numpy(case.Wq).to(dev)
    X = torch.from_numpy(case.X).to(dev)
    q = oracle.quantize(case.X, case.x_scale)
    n_g = case.C // case.G
    perm_b = np.roll(np.arange(n_g, dtype=np.int32)[::-1].copy(), 3)
    for perm in (perm_b, perm_a):
        L.set_group_perm(Wq, perm, sxg)
        L.set_lowbit_ratio(0.5)
        x4, x8, _ = L.quantize_lower(X, case.x_scale)
        y = L.mixed_conv(x4, x8, case.Nb, case.H, case.W, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8)
        sw = oracle.weight_positions_conv(case.Wq, case.G, perm)
        acc = oracle.mixed_conv_acc(q, case.Wq, case.stride, case.pad, case.G, perm, sxg[perm].copy(), sw, oracle.n_low(0.5, n_g))
        assert np.array_equal(y.cpu().numpy(), oracle.epilogue_i8(acc, case.x_scale, case.w_scale, case.bias, case.y_scale))
    L.close()
    # producer -> consumer chain: the consumer is laid out again, the producer's epilogue follows its new tables
    a = inputs.ranged_linear("relay_a", 200, 128, 192, 16, seed=94, group_structured=True)
    b = inputs.ranged_linear("relay_b", 200, 192, 96, 16, seed=95, group_structured=True)
    pa, sa, sas, swa = helpers.prepare_linear(a)
    pb, sb, _, _ = helpers.prepare_linear(b)
    LA = fx.Layer(torch.from_numpy(a.Wq).to(dev), torch.from_numpy(a.w_scale).to(dev), torch.from_numpy(a.bias).to(dev), pa, sa, 16)
    LB = fx.Layer(torch.from_numpy(b.Wq).to(dev), torch.from_numpy(b.w_scale).to(dev), torch.from_numpy(b.bias).to(dev), pb, sb, 16)
    WB = torch.from_numpy(b.Wq).to(dev)
    XA = torch.from_numpy(a.X).to(dev)
    qa = oracle.quantize(a.X, a.x_scale)
    next_scale = a.y_scale
    for perm in (pb, np.arange(192 // 16, dtype=np.int32)[::-1].copy()):
        LB.set_group_perm(WB, perm, sb)
        for L_, r in ((LA, 0.5), (LB, 0.5)):
            L_.set_lowbit_ratio(r)
        x4, x8, _ = LA.quantize_lower(XA, a.x_scale)
        slab = LA.mixed_gemm_to_slab(x4, x8, a.M, a.x_scale, LB, next_scale)
        yb = LB.mixed_gemm(slab, None, a.M, next_scale, b.y_scale, fx.OUT_REQUANT_I8)
        acc_a = oracle.mixed_gemm_acc(qa, a.Wq, 16, pa, sas, swa, oracle.n_low(0.5, 128 // 16))
        qb = oracle.epilogue_i8(acc_a, a.x_scale, a.w_scale, a.bias, next_scale)
        swb = oracle.weight_positions_linear(b.Wq, 16, perm)
        acc_b = oracle.mixed_gemm_acc(qb, b.Wq, 16, perm, sb[perm].copy(), swb, oracle.n_low(0.5, 192 // 16))
        assert np.array_equal(yb.cpu().numpy(), oracle.epilogue_i8(acc_b, next_scale, b.w_scale, b.bias, b.y_scale))
    fx.flexiq_check_status()
    LA.close()
    LB.close()
