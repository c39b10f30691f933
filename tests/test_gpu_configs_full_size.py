"""GPU parity at the stated size of every benchmark configuration, in the launch configuration the
benchmark uses (automatic tile choice, default low-bit path unless named): the CUDA library through its
C ABI against the CPU oracle, bit-exact.  Where the oracle cannot afford the whole output (the ViT
linears) it computes sampled rows -- every 97th or 197th row, the ragged last tile, a stretch inside a
tile -- and the rest is covered by a property that holds at any size (identical results run to run)."""
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


def _linear_layer(case, dev, path=fx.LOWBIT_MASKED_I8):
    perm, sxg, sxs, sw = helpers.prepare_linear(case)
    L = fx.Layer(torch.from_numpy(case.Wq).to(dev), torch.from_numpy(case.w_scale).to(dev),
                 torch.from_numpy(case.bias).to(dev), perm, sxg, case.G)
    L.set_lowbit_path(path)
    return L, perm, sxs, sw


def _sample_rows(M, step):
    return np.unique(np.concatenate([np.arange(0, M, step), np.arange(M - 70, M), np.arange(120, 136)])).astype(np.int64)


def _check_sampled(L, case, X, rows, q_rows, perm, sxs, sw, ratio, modes=(fx.OUT_ACC_I32, fx.OUT_REQUANT_I8)):
    L.set_lowbit_ratio(ratio)
    nl = oracle.n_low(ratio, case.K // case.G)
    x4, x8, _ = L.quantize_lower(X, case.x_scale)
    acc_e = oracle.mixed_gemm_acc(q_rows, case.Wq, case.G, perm, sxs, sw, nl)
    for mode in modes:
        Y = L.mixed_gemm(x4, x8, case.M, case.x_scale, case.y_scale, mode)
        torch.cuda.synchronize()
        fx.flexiq_check_status()
        got = Y[torch.from_numpy(rows).to(Y.device)].cpu().numpy()
        if mode == fx.OUT_ACC_I32:
            assert np.array_equal(got, acc_e), f"accumulators differ at ratio {ratio}"
        else:
            assert np.array_equal(got, oracle.epilogue_i8(acc_e, case.x_scale, case.w_scale, case.bias, case.y_scale)), \
                f"int8 outputs differ at ratio {ratio}"
    return acc_e


# ---------------------------------------------------------------- configuration 2: ViT-B/16, batch 64
@pytest.mark.parametrize("layer", [1, 2])
def test_vit_b_proj_and_fc1_full_size(dev, layer):
    name, K, N = inputs.VIT_B_LAYERS[layer]
    case = inputs.vit_linear(f"cfg2_{name}", 64 * 197, K, N, 16, seed=2000 + layer)
    L, perm, sxs, sw = _linear_layer(case, dev)
    X = torch.from_numpy(case.X).to(dev)
    rows = _sample_rows(case.M, 97)
    q_rows = oracle.quantize(case.X[rows], case.x_scale)
    for r in inputs.RATIOS:
        _check_sampled(L, case, X, rows, q_rows, perm, sxs, sw, r)
    L.close()


def test_vit_b_packed_path_full_size(dev):
    """The packed 4-bit slabs at the size the packed path is timed at (M = 12608), on the proj layer."""
    name, K, N = inputs.VIT_B_LAYERS[1]
    case = inputs.vit_linear(f"cfg2_{name}", 64 * 197, K, N, 16, seed=2001)
    L, perm, sxs, sw = _linear_layer(case, dev, path=fx.LOWBIT_PACKED_U4)
    X = torch.from_numpy(case.X).to(dev)
    rows = _sample_rows(case.M, 97)
    q_rows = oracle.quantize(case.X[rows], case.x_scale)
    for r in (0.25, 0.5, 1.0):
        _check_sampled(L, case, X, rows, q_rows, perm, sxs, sw, r)
        # the packed slab itself, on the sampled rows
        nl = oracle.n_low(r, K // 16)
        e4, e8 = oracle.make_slabs(q_rows, 16, perm, sxs, nl)
        x4, x8 = L.alloc_slabs(case.M)
        pitch = fx.flexiq_x4_pitch(L.h, nl * 16)
        ridx = torch.from_numpy(rows).to(dev)
        g4 = x4[:case.M * pitch].view(case.M, pitch)[ridx].cpu().numpy()
        assert np.array_equal(g4[:, :nl * 8], e4[:, :nl * 8])
        if K - nl * 16:
            assert np.array_equal(x8[:case.M * (K - nl * 16)].view(case.M, -1)[ridx].cpu().numpy(), e8)
    L.close()


# ---------------------------------------------------------------- configuration 3: ResNet-50 convolutions, batch 32
@pytest.mark.parametrize("idx", range(8))
def test_resnet50_convs_batch_32(dev, idx):
    """All eight convolution shapes of the configuration at batch 32: whole outputs against the oracle
    (accumulators and int8), two ratios each, one of which splits a K block between low and 8-bit groups."""
    name, H, C, Co, R = inputs.RESNET50_CONVS[idx]
    case = inputs.resnet_conv(f"cfg3_{name}", 32, H, C, Co, R, 16, seed=3000 + idx)
    perm, sxg, sxs, sw = helpers.prepare_conv(case)
    L = fx.Layer(torch.from_numpy(case.Wq).to(dev), torch.from_numpy(case.w_scale).to(dev), torch.from_numpy(case.bias).to(dev),
                 perm, sxg, case.G, conv=(case.stride, case.pad))
    X = torch.from_numpy(case.X).to(dev)
    q = oracle.quantize(case.X, case.x_scale)
    for r in (0.25, 1.0):
        L.set_lowbit_ratio(r)
        nl = oracle.n_low(r, C // 16)
        x4, x8, _ = L.quantize_lower(X, case.x_scale)
        acc = L.mixed_conv(x4, x8, case.Nb, H, H, case.x_scale, case.y_scale, fx.OUT_ACC_I32)
        y8 = L.mixed_conv(x4, x8, case.Nb, H, H, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8)
        torch.cuda.synchronize()
        fx.flexiq_check_status()
        acc_e = oracle.mixed_conv_acc(q, case.Wq, case.stride, case.pad, case.G, perm, sxs, sw, nl)
        assert np.array_equal(acc.cpu().numpy(), acc_e), f"{name}: accumulators differ at ratio {r}"
        assert np.array_equal(y8.cpu().numpy(), oracle.epilogue_i8(acc_e, case.x_scale, case.w_scale, case.bias, case.y_scale))
    L.close()


# ---------------------------------------------------------------- configuration 4: DeiT-S at batch 8
def test_deit_small_batch_8_all_layers(dev):
    """M = 1576 rows, the four DeiT-S linears, every ratio, both low-bit paths (the packed slab at half the bytes
    is the configuration's subject); whole outputs."""
    for case in inputs.config4(batch=8):
        for path in (fx.LOWBIT_MASKED_I8, fx.LOWBIT_PACKED_U4):
            L, perm, sxs, sw = _linear_layer(case, dev, path=path)
            X = torch.from_numpy(case.X).to(dev)
            q = oracle.quantize(case.X, case.x_scale)
            rows = np.arange(case.M, dtype=np.int64)
            for r in inputs.RATIOS:
                _check_sampled(L, case, X, rows, q, perm, sxs, sw, r)
            L.close()


# ---------------------------------------------------------------- configuration 5: ViT-L/16, batch 128, ratio switched at run time
@pytest.mark.parametrize("layer", [0, 1, 2])
def test_vit_l_qkv_proj_fc1_full_size(dev, layer):
    name, K, N = inputs.VIT_L_LAYERS[layer]
    case = inputs.vit_linear(f"cfg5_{name}", 128 * 197, K, N, 16, seed=5000 + layer)
    L, perm, sxs, sw = _linear_layer(case, dev)
    X = torch.from_numpy(case.X).to(dev)
    rows = _sample_rows(case.M, 197)
    q_rows = oracle.quantize(case.X[rows], case.x_scale)
    for r in (0.0, 0.5, 1.0):
        _check_sampled(L, case, X, rows, q_rows, perm, sxs, sw, r, modes=(fx.OUT_REQUANT_I8,))
    L.close()


def test_vit_l_ratio_walk_on_one_handle(dev):
    """Sec. 7 run-time ratio adjustment: ONE handle (fc2, K = 4096, M = 25216) driven 0 -> 0.5 -> 1.0 -> 0.5 -> 0
    -> 0.3 (a boundary inside a K block) with prologue + GEMM after every switch; then one CUDA graph per ratio,
    captured once and replayed in scrambled order, each replay checked against the oracle at its ratio."""
    name, K, N = inputs.VIT_L_LAYERS[3]
    case = inputs.vit_linear(f"cfg5_{name}", 128 * 197, K, N, 16, seed=5003)
    L, perm, sxs, sw = _linear_layer(case, dev)
    X = torch.from_numpy(case.X).to(dev)
    rows = _sample_rows(case.M, 197)
    ridx = torch.from_numpy(rows).to(dev)
    q_rows = oracle.quantize(case.X[rows], case.x_scale)
    want = {}
    for r in (0.0, 0.5, 1.0, 0.5, 0.0, 0.3):
        acc_e = _check_sampled(L, case, X, rows, q_rows, perm, sxs, sw, r, modes=(fx.OUT_REQUANT_I8,))
        want[r] = oracle.epilogue_i8(acc_e, case.x_scale, case.w_scale, case.bias, case.y_scale)
    # one graph per ratio: prologue + GEMM, each with slabs and output of its own
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graphs = {}
    with torch.cuda.stream(side):
        for r in (0.0, 0.3, 0.5, 1.0):
            L.set_lowbit_ratio(r)
            x4 = torch.empty(case.M * K + 16, dtype=torch.uint8, device=dev)
            Y = torch.empty((case.M, N), dtype=torch.int8, device=dev)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                fx.flexiq_quantize_lower(L.h, X, fx.DTYPE_F32, case.M, case.x_scale, 0, x4, None)
                fx.flexiq_mixed_gemm(L.h, x4, None, None, case.M, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8, Y)
            graphs[r] = (g, Y, x4)
    torch.cuda.synchronize()
    for r in (1.0, 0.0, 0.5, 0.3, 0.0, 1.0, 0.3, 0.5):
        g, Y, _ = graphs[r]
        Y.zero_()
        L.set_lowbit_ratio(r)
        L.sync_ratio()
        g.replay()
        torch.cuda.synchronize()
        fx.flexiq_check_status()
        assert np.array_equal(Y[ridx].cpu().numpy(), want[r]), f"graph replay at ratio {r}"
    L.close()
