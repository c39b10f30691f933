"""GPU parity on seeded random shapes: linear layers and convolutions with random sizes, group sizes,
ratios, positions and output modes, on both low-bit paths, against the oracle (bit-exact)."""
import numpy as np
import pytest
import torch

import helpers
import oracle
from paper_2510_02822_b200 import binding as fx
from paper_2510_02822_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    return torch.device("cuda:0")


@pytest.mark.parametrize("seed", range(12))
def test_random_linear(dev, seed):
    rng = np.random.default_rng(1000 + seed)
    G = int(rng.choice([16, 32, 64]))
    K = G * int(rng.integers(1, 24))
    N = 16 * int(rng.integers(1, 40))
    M = int(rng.integers(1, 900))
    case = inputs.ranged_linear("r", M, K, N, G, seed=seed, group_structured=True)
    shifts = rng.integers(0, 5, K // G).astype(np.uint8)
    perm, sxg, sxs, sw = helpers.prepare_linear(case, shifts)
    q = oracle.quantize(case.X, case.x_scale)
    X = torch.from_numpy(case.X).to(dev)
    for path in (fx.LOWBIT_MASKED_I8, fx.LOWBIT_PACKED_U4):
        L = fx.Layer(torch.from_numpy(case.Wq).to(dev), torch.from_numpy(case.w_scale).to(dev), torch.from_numpy(case.bias).to(dev), perm, sxg, G)
        L.set_lowbit_path(path)
        for ratio in rng.choice([0.0, 0.25, 0.5, 0.75, 1.0], 2, replace=False):
            L.set_lowbit_ratio(float(ratio))
            nl = oracle.n_low(float(ratio), K // G)
            x4, x8, _ = L.quantize_lower(X, case.x_scale)
            acc = oracle.mixed_gemm_acc(q, case.Wq, G, perm, sxs, sw, nl)
            assert np.array_equal(L.mixed_gemm(x4, x8, M, case.x_scale, case.y_scale, fx.OUT_ACC_I32).cpu().numpy(), acc)
            assert np.array_equal(L.mixed_gemm(x4, x8, M, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8).cpu().numpy(),
                                  oracle.epilogue_i8(acc, case.x_scale, case.w_scale, case.bias, case.y_scale))
        L.close()
    fx.flexiq_check_status()


@pytest.mark.parametrize("seed", range(8))
def test_random_conv(dev, seed):
    rng = np.random.default_rng(2000 + seed)
    C = 16 * int(rng.choice([1, 2, 4, 6, 8, 12, 16]))
    Cout = 16 * int(rng.integers(1, 20))
    R = int(rng.choice([1, 3]))
    stride = int(rng.choice([1, 2])) if R == 3 else 1
    H = int(rng.integers(5, 30))
    Nb = int(rng.integers(1, 4))
    case = inputs.resnet_conv("r", Nb, H, C, Cout, R, seed=seed, stride=stride)
    shifts = rng.integers(0, 5, C // case.G).astype(np.uint8)
    perm, sxg, sxs, sw = helpers.prepare_conv(case, shifts)
    q = oracle.quantize(case.X, case.x_scale)
    X = torch.from_numpy(case.X).to(dev)
    L = fx.Layer(torch.from_numpy(case.Wq).to(dev), torch.from_numpy(case.w_scale).to(dev), torch.from_numpy(case.bias).to(dev), perm, sxg, case.G,
                 conv=(case.stride, case.pad))
    for ratio in rng.choice([0.0, 0.25, 0.5, 0.75, 1.0], 2, replace=False):
        L.set_lowbit_ratio(float(ratio))
        nl = oracle.n_low(float(ratio), C // case.G)
        x4, x8, _ = L.quantize_lower(X, case.x_scale)
        acc = oracle.mixed_conv_acc(q, case.Wq, case.stride, case.pad, case.G, perm, sxs, sw, nl)
        assert np.array_equal(L.mixed_conv(x4, x8, Nb, H, H, case.x_scale, case.y_scale, fx.OUT_ACC_I32).cpu().numpy(), acc)
        got = L.mixed_conv(x4, x8, Nb, H, H, case.x_scale, case.y_scale, fx.OUT_DEQUANT_F32).cpu().numpy()
        exp = oracle.epilogue_f32(acc, case.x_scale, case.w_scale, case.bias)
        assert np.all(np.abs(got - exp) <= 1e-6 * np.abs(exp))
    L.close()
    fx.flexiq_check_status()


@pytest.mark.parametrize("tile", [(0, 0), (1, 64), (1, 128), (2, 128)])
@pytest.mark.parametrize("M,K,N,G", [(1, 1296, 176, 16), (300, 2304, 96, 64), (700, 1056, 240, 32)])
def test_one_long_k_tile_per_cta(dev, tile, M, K, N, G):
    """Few narrow tiles and many K blocks: each CTA has one tile, and its two MMA warps share the tile's K
    blocks into accumulators of their own, which the epilogue adds.  Every output mode reads both."""
    case = inputs.ranged_linear("s", M, K, N, G, seed=K + N, group_structured=True)
    perm, sxg, sxs, sw = helpers.prepare_linear(case)
    q = oracle.quantize(case.X, case.x_scale)
    X = torch.from_numpy(case.X).to(dev)
    L = fx.Layer(torch.from_numpy(case.Wq).to(dev), torch.from_numpy(case.w_scale).to(dev), torch.from_numpy(case.bias).to(dev), perm, sxg, G)
    fx.flexiq_force_tile(*tile)
    try:
        for ratio in (0.0, 0.5, 1.0):
            L.set_lowbit_ratio(ratio)
            x4, x8, _ = L.quantize_lower(X, case.x_scale)
            acc = oracle.mixed_gemm_acc(q, case.Wq, G, perm, sxs, sw, oracle.n_low(ratio, K // G))
            assert np.array_equal(L.mixed_gemm(x4, x8, M, case.x_scale, case.y_scale, fx.OUT_ACC_I32).cpu().numpy(), acc)
            assert np.array_equal(L.mixed_gemm(x4, x8, M, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8).cpu().numpy(),
                                  oracle.epilogue_i8(acc, case.x_scale, case.w_scale, case.bias, case.y_scale))
            assert np.array_equal(L.mixed_gemm(x4, x8, M, case.x_scale, case.y_scale, fx.OUT_DEQUANT_F32).cpu().numpy(),
                                  oracle.epilogue_f32(acc, case.x_scale, case.w_scale, case.bias))
            y16 = L.mixed_gemm(x4, x8, M, case.x_scale, case.y_scale, fx.OUT_DEQUANT_F16).cpu().numpy()
            assert np.array_equal(y16.view(np.uint16), oracle.epilogue_f16(acc, case.x_scale, case.w_scale, case.bias).view(np.uint16))
    finally:
        fx.flexiq_force_tile(0, 0)
    L.close()
    fx.flexiq_check_status()
