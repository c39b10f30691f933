"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the
same seeded inputs.  Integer results (slabs, int32 accumulators, int8 outputs) must be
bit-exact; dequantized fp32 outputs within 1e-6 relative."""
import numpy as np
import pytest
import torch

import helpers
import oracle
from paper_2510_02822_b200 import binding as fx
from paper_2510_02822_b200 import inputs

pytestmark = pytest.mark.gpu
F32_RTOL = 1e-6


@pytest.fixture(scope="module")
def dev():
    return torch.device("cuda:0")


def _layer(case, dev, perm, sx_group, conv=False, path=fx.LOWBIT_MASKED_I8):
    L = fx.Layer(torch.from_numpy(case.Wq).to(dev), torch.from_numpy(case.w_scale).to(dev),
                 torch.from_numpy(case.bias).to(dev), perm, sx_group, case.G,
                 conv=(case.stride, case.pad) if conv else None)
    L.set_lowbit_path(path)
    return L


def _check_outputs(L, case, x4, x8, acc_e, dev, conv=False, x_shift=None):
    shape = acc_e.shape
    for mode, dt in ((fx.OUT_ACC_I32, torch.int32), (fx.OUT_REQUANT_I8, torch.int8), (fx.OUT_DEQUANT_F32, torch.float32),
                     (fx.OUT_DEQUANT_F16, torch.float16), (fx.OUT_DEQUANT_BF16, torch.bfloat16)):
        Y, guard_ok = helpers.with_guard(torch, shape, dt, dev)
        if conv:
            L.mixed_conv(x4, x8, case.Nb, case.H, case.W, case.x_scale, case.y_scale, mode, Y=Y, x_shift=x_shift)
        else:
            L.mixed_gemm(x4, x8, shape[0], case.x_scale, case.y_scale, mode, Y=Y, x_shift=x_shift)
        torch.cuda.synchronize()
        fx.flexiq_check_status()
        guard_ok()
        if mode == fx.OUT_DEQUANT_BF16:
            # 16-bit patterns: both sides round the same fp32 value to nearest even
            assert np.array_equal(Y.view(torch.int16).cpu().numpy().view(np.uint16),
                                  oracle.epilogue_bf16_bits(acc_e, case.x_scale, case.w_scale, case.bias))
            continue
        got = Y.cpu().numpy()
        if mode == fx.OUT_DEQUANT_F16:
            assert np.array_equal(got.view(np.uint16), oracle.epilogue_f16(acc_e, case.x_scale, case.w_scale, case.bias).view(np.uint16))
            continue
        if mode == fx.OUT_ACC_I32:
            assert np.array_equal(got, acc_e)
        elif mode == fx.OUT_REQUANT_I8:
            assert np.array_equal(got, oracle.epilogue_i8(acc_e, case.x_scale, case.w_scale, case.bias, case.y_scale))
        else:
            exp = oracle.epilogue_f32(acc_e, case.x_scale, case.w_scale, case.bias)
            assert np.all(np.abs(got - exp) <= F32_RTOL * np.abs(exp))


def _run_linear(case, dev, ratios, shifts=None, x_dtype=torch.float32, path=fx.LOWBIT_MASKED_I8, dynamic=False):
    perm, sxg, sxs, sw = helpers.prepare_linear(case, shifts)
    L = _layer(case, dev, perm, sxg, path=path)
    X = torch.from_numpy(case.X).to(dev).to(x_dtype)
    q = oracle.quantize(X.float().cpu().numpy(), case.x_scale) if x_dtype != torch.int8 else X.cpu().numpy()
    for r in ratios:
        L.set_lowbit_ratio(r)
        nl = oracle.n_low(r, case.K // case.G)
        K_lo = nl * case.G
        assert L.K_lo == K_lo
        x4, x8, shifts_dev = L.quantize_lower(X, case.x_scale, dynamic=dynamic)
        torch.cuda.synchronize()
        sx_use = sxs
        if dynamic:
            sx_use = oracle.dynamic_positions(q, case.G, perm)
            assert np.array_equal(shifts_dev.cpu().numpy(), sx_use)
        e4, e8 = oracle.make_slabs(q, case.G, perm, sx_use, nl)
        pitch = fx.flexiq_x4_pitch(L.h, K_lo)
        if path == fx.LOWBIT_MASKED_I8:
            # one slab [M][K]: the low groups as (x4 << sx), then the 8-bit groups
            assert pitch == case.K
            g = x4[:case.M * case.K].view(case.M, case.K).cpu().numpy().view(np.int8)
            if K_lo:
                assert np.array_equal(g[:, :K_lo], helpers.masked_slab(e4, case.G, sx_use, nl))
            assert np.array_equal(g[:, K_lo:], e8)
        else:
            if K_lo:
                g4 = x4[:case.M * pitch].view(case.M, pitch).cpu().numpy()
                assert np.array_equal(g4[:, :K_lo // 2], e4[:, :K_lo // 2])
            if case.K - K_lo:
                assert np.array_equal(x8[:case.M * (case.K - K_lo)].view(case.M, -1).cpu().numpy(), e8)
        acc_e = oracle.mixed_gemm_acc(q, case.Wq, case.G, perm, sx_use, sw, nl)
        _check_outputs(L, case, x4, x8, acc_e, dev, x_shift=shifts_dev)
    L.close()


def test_layer_tables(dev):
    case = inputs.ranged_linear("t", 64, 192, 80, 32, seed=1, group_structured=True)
    perm, sxg, sxs, sw = helpers.prepare_linear(case)
    L = _layer(case, dev, perm, sxg)
    sw_g = np.empty_like(sw)
    w8 = np.empty((80, 192), np.int8)
    w4 = np.empty((80, 96), np.uint8)
    fx.flexiq_layer_export(L.h, sw_g, w8, w4)
    assert np.array_equal(sw_g, sw)
    cols = np.concatenate([np.arange(g * 32, (g + 1) * 32) for g in perm])
    ws = case.Wq[cols].T.astype(np.int16)
    assert np.array_equal(w8, ws)
    sh = np.repeat(sw, 32, axis=0).T.astype(np.int16)
    n4 = (ws >> sh) & 15
    assert np.array_equal(w4, (n4[:, 0::2] | (n4[:, 1::2] << 4)).astype(np.uint8))
    L.close()


def test_config1_single_gemm_all_ratios(dev):
    _run_linear(inputs.config1(), dev, inputs.RATIOS)


def test_config1_int8_input_gives_identical_slabs(dev):
    case = inputs.config1()
    case.X = oracle.quantize(case.X, case.x_scale)  # the int8 X of the configuration
    _run_linear(case, dev, [0.5], x_dtype=torch.int8)


@pytest.mark.parametrize("M,K,N,G", [(1, 128, 16, 16), (129, 256, 48, 16), (300, 128, 272, 32), (197, 384, 384, 16),
                                     (515, 192, 144, 64), (257, 64, 64, 16), (1000, 1024, 80, 16)])
def test_ragged_shapes_with_saturating_positions(dev, M, K, N, G):
    case = inputs.ranged_linear("r", M, K, N, G, seed=M + K, group_structured=True)
    rng = np.random.default_rng(K + N)
    shifts = rng.integers(0, 5, K // G).astype(np.uint8)  # arbitrary positions: some values saturate
    _run_linear(case, dev, [0.0, 0.5, 1.0, 1.0 / (K // G)], shifts=shifts)


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_half_precision_inputs(dev, dtype):
    _run_linear(inputs.ranged_linear("h", 200, 256, 64, 16, seed=6, group_structured=True), dev, [0.5], x_dtype=dtype)


@pytest.mark.parametrize("S", [0.033, 0.0123457, 1.7e-3, 0.61, 3.3, 0.25])
def test_quantization_matches_ieee_division_near_ties(dev, S):
    # Values within a few ulps of every rounding boundary (k + 0.5) * S: the kernel's
    # reciprocal-based quotient must round exactly like the oracle's IEEE division.
    S = float(np.float32(S))
    ks = np.arange(-131, 131, dtype=np.float64) + 0.5
    base = (ks * S).astype(np.float32)
    vals = [base]
    for _ in range(4):
        vals.append(np.nextafter(vals[-1], np.float32(np.inf)))
    lo = base
    for _ in range(4):
        lo = np.nextafter(lo, np.float32(-np.inf))
        vals.append(lo)
    rng = np.random.default_rng(7)
    # ... and inputs beyond every finite quotient: Eq. 1's clip saturates them with their sign
    huge = np.array([np.inf, -np.inf, 3.0e38, -3.0e38, 1e30, -1e30], np.float32)
    x = np.concatenate(vals + [huge, rng.uniform(-140 * S, 140 * S, 4096).astype(np.float32)])
    K, G = 64, 16
    M = (x.size + K - 1) // K
    X = np.zeros((M, K), np.float32)
    X.reshape(-1)[:x.size] = x
    perm = np.arange(K // G, dtype=np.int32)
    Wq = torch.zeros((K, 16), dtype=torch.int8, device=dev)
    L = fx.Layer(Wq, torch.ones(16, device=dev), None, perm, np.zeros(K // G, np.uint8), G)
    L.set_lowbit_ratio(0.0)
    x4, x8, _ = L.quantize_lower(torch.from_numpy(X).to(dev), S)
    torch.cuda.synchronize()
    got = x4[:M * K].view(M, K).cpu().numpy().view(np.int8)  # masked path: the whole slab is in X4
    assert np.array_equal(got, oracle.quantize(X, S))
    L.close()


def test_dynamic_positions(dev):
    case = inputs.ranged_linear("dyn", 333, 384, 96, 16, seed=21, group_structured=True)
    _run_linear(case, dev, [0.5, 1.0], dynamic=True)
    case = inputs.ranged_linear("dyn2", 77, 64, 32, 32, seed=22, group_structured=True)  # fewer groups than lanes
    _run_linear(case, dev, [1.0], dynamic=True)


def test_deit_small_batch_shapes(dev):
    for case in inputs.config4(batch=1):
        _run_linear(case, dev, [0.0, 0.25, 0.5, 0.75, 1.0])


def test_empty_batch_and_argument_errors(dev):
    case = inputs.ranged_linear("e", 16, 128, 32, 16, seed=3)
    perm, sxg, sxs, sw = helpers.prepare_linear(case)
    L = _layer(case, dev, perm, sxg)
    L.set_lowbit_ratio(0.5)
    fx.flexiq_quantize_lower(L.h, None, fx.DTYPE_F32, 0, 1.0, 0, None, None)  # M == 0: no-op
    fx.flexiq_mixed_gemm(L.h, None, None, None, 0, 1.0, 1.0, fx.OUT_ACC_I32, None)
    x4, x8 = L.alloc_slabs(16)
    with pytest.raises(fx.FlexiqError) as e:
        fx.flexiq_mixed_gemm(L.h, None, x8, None, 16, 1.0, 1.0, fx.OUT_ACC_I32, x8)
    assert e.value.code == fx.ERR_INVALID_ARG
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_set_lowbit_ratio(L.h, 1.5)
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_mixed_conv(L.h, x4, x8, None, 1, 4, 4, 1.0, 1.0, fx.OUT_ACC_I32, x8)
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_mixed_gemm(L.h, x4[1:], x8, None, 16, 1.0, 1.0, fx.OUT_ACC_I32, x8)  # misaligned
    L.close()


def test_ratio_switch_is_host_only_and_nested(dev):
    case = inputs.config1()
    perm, sxg, sxs, sw = helpers.prepare_linear(case)
    L = _layer(case, dev, perm, sxg)
    seen = []
    for r in (0.0, 0.25, 0.5, 0.75, 1.0, 0.5, 0.0):
        L.set_lowbit_ratio(r)
        seen.append(L.K_lo)
    assert seen == [0, 96, 192, 288, 384, 192, 0]
    L.close()


@pytest.mark.parametrize("cg,bn", [(1, 64), (1, 128), (1, 192), (1, 256), (2, 128), (2, 192), (2, 256)])
def test_every_tile_shape(dev, cg, bn):
    fx.flexiq_force_tile(cg, bn)
    try:
        rng = np.random.default_rng(cg * 1000 + bn)
        case = inputs.ranged_linear("tile", 700, 384, 400, 16, seed=cg * 10 + bn, group_structured=True)
        _run_linear(case, dev, [0.0, 0.5, 1.0], shifts=rng.integers(0, 5, 24).astype(np.uint8))
        conv = inputs.resnet_conv("tilec", 3, 14, 128, 272, 3, seed=bn)
        _run_conv(conv, dev, [0.5])
    finally:
        fx.flexiq_force_tile(0, 0)


# ---------------------------------------------------------------- convolution
def _run_conv(case, dev, ratios, shifts=None, path=fx.LOWBIT_MASKED_I8):
    perm, sxg, sxs, sw = helpers.prepare_conv(case, shifts)
    L = _layer(case, dev, perm, sxg, conv=True, path=path)
    X = torch.from_numpy(case.X).to(dev)
    q = oracle.quantize(case.X, case.x_scale)
    for r in ratios:
        L.set_lowbit_ratio(r)
        nl = oracle.n_low(r, case.C // case.G)
        x4, x8, _ = L.quantize_lower(X, case.x_scale)
        acc_e = oracle.mixed_conv_acc(q, case.Wq, case.stride, case.pad, case.G, perm, sxs, sw, nl)
        _check_outputs(L, case, x4, x8, acc_e, dev, conv=True)
    L.close()


@pytest.mark.parametrize("Nb,H,C,Cout,R,stride", [(2, 14, 128, 64, 3, 1), (3, 28, 64, 64, 3, 1), (5, 7, 256, 128, 3, 1),
                                                  (2, 14, 128, 64, 3, 2), (2, 14, 128, 256, 1, 1), (1, 9, 192, 48, 3, 1)])
def test_conv_shapes(dev, Nb, H, C, Cout, R, stride):
    case = inputs.resnet_conv("c", Nb, H, C, Cout, R, seed=H + C, stride=stride)
    rng = np.random.default_rng(H * C)
    shifts = rng.integers(0, 5, C // case.G).astype(np.uint8)
    _run_conv(case, dev, [0.0, 0.25, 0.5, 1.0], shifts=shifts)


@pytest.mark.parametrize("Nb,H,C,Cout,R", [(3, 14, 128, 80, 3),    # 8 output rows per tile, 14 rows: a ragged second tile; 80 channels in a 128-column tile
                                          (5, 7, 64, 64, 3),      # pitch 8: one tile holds a whole image and more
                                          (2, 20, 48, 32, 3),     # fewer channels than the K block
                                          (2, 33, 64, 48, 5),     # 5 x 5 taps (the generic tap loop), pitch 64, odd height
                                          (1, 60, 32, 16, 3),     # widest image the 64-pixel pitch holds with its padding... and one K step
                                          (2, 100, 64, 64, 3),    # pitch 128: one output row per tile
                                          (2, 15, 32, 32, 3),     # W + pad == pitch: the right padding of a tile's last pixel is the
                                          (3, 31, 16, 112, 3),    # next patch row's left padding, so the patch carries one more row
                                          (4, 14, 32, 48, 5),
                                          (1, 127, 16, 32, 3),    # W + pad == 128: the widest image of the patch path, one row per tile, the extra row
                                          (1, 126, 16, 32, 5),    # the same with two pixels of padding
                                          (1, 128, 16, 32, 3)])   # one pixel too wide for it: im2col copies
def test_conv_patch_mode_edges(dev, Nb, H, C, Cout, R):
    """Stride-1 convolutions whose channels fit one K block take the patch path (one halo patch per tile, taps as row
    offsets into it): image sizes that leave unused grid columns and ragged last tiles, narrow channel counts."""
    case = inputs.resnet_conv("pm", Nb, H, C, Cout, R, seed=H + C + R)
    rng = np.random.default_rng(H * C + R)
    shifts = rng.integers(0, 5, C // case.G).astype(np.uint8)
    _run_conv(case, dev, [0.0, 0.5, 1.0], shifts=shifts)


@pytest.mark.parametrize("kind,shape", [("conv", (4, 7, 512, 256, 3)), ("conv", (2, 7, 256, 80, 3)), ("linear", (200, 2048, 256, 16)),
                                        ("linear", (130, 1536, 384, 32)), ("linear", (64, 3072, 272, 16))])
def test_small_m_long_k_shapes(dev, kind, shape):
    """Small-M, long-K layers (one narrow tile per CTA: the two MMA warps share the tile's K blocks, an accumulator
    each).  Odd numbers of K blocks, ragged M and N, every output type and several ratios (the boundary block included)."""
    if kind == "conv":
        Nb, H, C, Cout, R = shape
        case = inputs.resnet_conv("ks", Nb, H, C, Cout, R, seed=H + C + Cout)
        rng = np.random.default_rng(C + Cout)
        _run_conv(case, dev, [0.0, 0.3, 1.0], shifts=rng.integers(0, 5, C // case.G).astype(np.uint8))
    else:
        M, K, N, G = shape
        case = inputs.ranged_linear("ks", M, K, N, G, seed=M + K, group_structured=True)
        rng = np.random.default_rng(K + N)
        _run_linear(case, dev, [0.0, 0.3, 1.0], shifts=rng.integers(0, 5, K // G).astype(np.uint8))


def test_resnet50_conv_full_size_56(dev):
    # full-size 3x3 C=64 @56x56 at batch 4 (the bench runs batch 32; rows are independent)
    case = inputs.resnet_conv("c56", 4, 56, 64, 64, 3, seed=3000)
    _run_conv(case, dev, [0.0, 0.5, 1.0])


def test_resnet50_conv_full_size_7(dev):
    # 3x3, 512 -> 512 channels at 7x7, batch 32 as the sweep times it: 104 tiles, one per CTA, the two MMA
    # warps sharing each tile's 36 K blocks
    case = inputs.resnet_conv("c7", 32, 7, 512, 512, 3, seed=3007)
    _run_conv(case, dev, [0.5])


# ---------------------------------------------------------------- packed 4-bit slabs
@pytest.mark.parametrize("M,K,N,G", [(300, 384, 272, 16), (129, 256, 48, 32), (1000, 1024, 400, 16), (257, 64, 64, 16),
                                     (700, 192, 512, 64)])
def test_packed_path_linear(dev, M, K, N, G):
    case = inputs.ranged_linear("pk", M, K, N, G, seed=M + N, group_structured=True)
    rng = np.random.default_rng(M + K)
    shifts = rng.integers(0, 5, K // G).astype(np.uint8)
    _run_linear(case, dev, [0.0, 0.25, 0.5, 1.0, 1.0 / (K // G)], shifts=shifts, path=fx.LOWBIT_PACKED_U4)


def test_packed_path_config1_and_dynamic_positions(dev):
    _run_linear(inputs.config1(), dev, inputs.RATIOS, path=fx.LOWBIT_PACKED_U4)
    case = inputs.ranged_linear("pkdyn", 333, 384, 96, 16, seed=23, group_structured=True)
    _run_linear(case, dev, [0.5, 1.0], dynamic=True, path=fx.LOWBIT_PACKED_U4)


@pytest.mark.parametrize("Nb,H,C,Cout,R,stride", [(2, 14, 128, 64, 3, 1), (3, 28, 64, 64, 3, 1), (2, 14, 128, 256, 1, 1),
                                                  (2, 14, 256, 80, 3, 2)])
def test_packed_path_conv(dev, Nb, H, C, Cout, R, stride):
    case = inputs.resnet_conv("pkc", Nb, H, C, Cout, R, seed=H + C + 1, stride=stride)
    rng = np.random.default_rng(H * C + 1)
    shifts = rng.integers(0, 5, C // case.G).astype(np.uint8)
    _run_conv(case, dev, [0.25, 0.5, 1.0], shifts=shifts, path=fx.LOWBIT_PACKED_U4)


# ---------------------------------------------------------------- full-size, sampled rows
@pytest.mark.parametrize("layer", [0, 3])
def test_vit_b_full_size_sampled_rows(dev, layer):
    name, K, N = inputs.VIT_B_LAYERS[layer]
    case = inputs.vit_linear(f"cfg2_{name}", 64 * 197, K, N, 16, seed=2000 + layer)
    perm, sxg, sxs, sw = helpers.prepare_linear(case)
    L = _layer(case, dev, perm, sxg)
    X = torch.from_numpy(case.X).to(dev)
    rows = np.unique(np.concatenate([np.arange(0, case.M, 97), np.arange(case.M - 70, case.M), np.arange(120, 136)])).astype(np.int64)
    q_rows = oracle.quantize(case.X[rows], case.x_scale)
    for r in (0.0, 0.5, 1.0):
        L.set_lowbit_ratio(r)
        nl = oracle.n_low(r, K // 16)
        x4, x8, _ = L.quantize_lower(X, case.x_scale)
        acc_e = oracle.mixed_gemm_acc(q_rows, case.Wq, 16, perm, sxs, sw, nl)
        acc = L.mixed_gemm(x4, x8, case.M, case.x_scale, case.y_scale, fx.OUT_ACC_I32)
        y8 = L.mixed_gemm(x4, x8, case.M, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8)
        torch.cuda.synchronize()
        fx.flexiq_check_status()
        assert np.array_equal(acc.cpu().numpy()[rows], acc_e)
        assert np.array_equal(y8.cpu().numpy()[rows], oracle.epilogue_i8(acc_e, case.x_scale, case.w_scale, case.bias, case.y_scale))
        # property that holds at any size: results are bit-identical run to run
        acc2 = L.mixed_gemm(x4, x8, case.M, case.x_scale, case.y_scale, fx.OUT_ACC_I32)
        assert torch.equal(acc, acc2)
    L.close()


def test_vit_l_full_size_sampled_rows(dev):
    """The largest configuration (ViT-L/16, batch 128: M = 25216) at full size: fc2, K = 4096."""
    name, K, N = inputs.VIT_L_LAYERS[3]
    case = inputs.vit_linear(f"cfg5_{name}", 128 * 197, K, N, 16, seed=5003)
    perm, sxg, sxs, sw = helpers.prepare_linear(case)
    L = _layer(case, dev, perm, sxg)
    X = torch.from_numpy(case.X).to(dev)
    rows = np.unique(np.concatenate([np.arange(0, case.M, 197), np.arange(case.M - 40, case.M), np.arange(250, 262)])).astype(np.int64)
    q_rows = oracle.quantize(case.X[rows], case.x_scale)
    for r in (0.25, 1.0):
        L.set_lowbit_ratio(r)
        nl = oracle.n_low(r, K // 16)
        x4, x8, _ = L.quantize_lower(X, case.x_scale)
        acc_e = oracle.mixed_gemm_acc(q_rows, case.Wq, 16, perm, sxs, sw, nl)
        y8 = L.mixed_gemm(x4, x8, case.M, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8)
        yf = L.mixed_gemm(x4, x8, case.M, case.x_scale, case.y_scale, fx.OUT_DEQUANT_F32)
        torch.cuda.synchronize()
        fx.flexiq_check_status()
        assert np.array_equal(y8.cpu().numpy()[rows], oracle.epilogue_i8(acc_e, case.x_scale, case.w_scale, case.bias, case.y_scale))
        want = oracle.epilogue_f32(acc_e, case.x_scale, case.w_scale, case.bias)
        got = yf.cpu().numpy()[rows]
        assert np.all(np.abs(got - want) <= 1e-6 * np.maximum(1.0, np.abs(want)))
    L.close()


def test_rows_beyond_32_bit_byte_offsets(dev):
    """M * K and M * N above 2^32 bytes (4.4 million rows of 1024 channels).  The int8 input is a seeded block
    of 50,000 rows repeated -- a period that does not divide 2^32, so an offset that wrapped at 32 bits would
    land on other rows.  Every slab and output row must equal the row one period earlier (checked on the device
    for all rows); sampled rows of the first period, the rows around the 2^32-byte mark and the last rows equal
    the oracle's."""
    K, N, G, P = 1024, 1024, 16, 50_000
    M = 88 * P + 12_345
    case = inputs.vit_linear("big", P, K, N, G, seed=7000)
    perm, sxg, sxs, sw = helpers.prepare_linear(case)
    q = oracle.quantize(case.X, case.x_scale)
    L = _layer(case, dev, perm, sxg)
    X = torch.from_numpy(q).to(dev).repeat(89, 1)[:M]
    assert X.is_contiguous() and M * K > 2 ** 32
    L.set_lowbit_ratio(0.5)
    nl = oracle.n_low(0.5, K // G)
    x4, x8, _ = L.quantize_lower(X, case.x_scale)
    y8 = L.mixed_gemm(x4, x8, M, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8)
    torch.cuda.synchronize()
    fx.flexiq_check_status()
    slab = x4.view(torch.int8)[:M * K].view(M, K)
    for i in range(1, 89):
        n = min(P, M - i * P)
        assert torch.equal(y8[i * P:i * P + n], y8[:n]), f"output rows of period {i}"
        assert torch.equal(slab[i * P:i * P + n], slab[:n]), f"slab rows of period {i}"
    mark = 2 ** 32 // K
    rows = np.unique(np.concatenate([np.arange(0, P, 197), np.arange(mark - 6, mark + 6), np.arange(M - 40, M)])).astype(np.int64)
    acc_e = oracle.mixed_gemm_acc(q[rows % P], case.Wq, G, perm, sxs, sw, nl)
    got = y8[torch.from_numpy(rows).to(dev)].cpu().numpy()
    assert np.array_equal(got, oracle.epilogue_i8(acc_e, case.x_scale, case.w_scale, case.bias, case.y_scale))
    L.close()


def test_conv_beyond_32_bit_byte_offsets(dev):
    """The same for the convolution path: 22,000 images of 56 x 56 x 64 (4.4 GB in, 4.4 GB out), a seeded block
    of 7 images repeated (1,404,928 bytes: not a divisor of 2^32).  Every output image equals the image one
    period earlier; the first period, the images around the 2^32-byte mark and the last ones equal the oracle's."""
    Pd, Nb = 7, 22_000
    case = inputs.resnet_conv("bigc", Pd, 56, 64, 64, 3, seed=7100)
    perm, sxg, sxs, sw = helpers.prepare_conv(case)
    q = oracle.quantize(case.X, case.x_scale)                      # [7][56][56][64] int8
    L = _layer(case, dev, perm, sxg, conv=True)
    X = torch.from_numpy(q).to(dev).repeat(Nb // Pd + 1, 1, 1, 1)[:Nb]
    assert X.is_contiguous() and X.numel() > 2 ** 32
    L.set_lowbit_ratio(0.5)
    nl = oracle.n_low(0.5, case.C // case.G)
    x4, x8, _ = L.quantize_lower(X, case.x_scale)
    y = L.mixed_conv(x4, x8, Nb, case.H, case.W, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8)
    torch.cuda.synchronize()
    fx.flexiq_check_status()
    assert y.shape[0] == Nb and y.numel() > 2 ** 32
    for i in range(1, Nb // Pd + 1):
        n = min(Pd, Nb - i * Pd)
        if n > 0:
            assert torch.equal(y[i * Pd:i * Pd + n], y[:n]), f"images of period {i}"
    acc_e = oracle.mixed_conv_acc(q, case.Wq, case.stride, case.pad, case.G, perm, sxs, sw, nl)
    want = oracle.epilogue_i8(acc_e, case.x_scale, case.w_scale, case.bias, case.y_scale).reshape(Pd, *y.shape[1:])
    mark = 2 ** 32 // (56 * 56 * 64)
    for img in list(range(Pd)) + list(range(mark - 2, mark + 3)) + list(range(Nb - 3, Nb)):
        assert np.array_equal(y[img].cpu().numpy(), want[img % Pd]), f"image {img}"
    L.close()


@pytest.mark.parametrize("K", [240, 256, 1024])
def test_extreme_accumulators(dev, K):
    """The largest accumulator magnitudes a layer can produce (all operands at -128 / 127) survive the
    int32 -> fp32 -> int8 epilogue exactly, below and above 2^22 and 2^24."""
    M, N, G = 200, 64, 16
    case = inputs.ranged_linear("x", M, K, N, G, seed=K)
    rng = np.random.default_rng(K)
    case.Wq = np.where(rng.random((K, N)) < 0.5, -128, 127).astype(np.int8)
    case.Wq[:, 0] = -128
    case.Wq[:, 1] = 127
    sgn = np.where(rng.random((M, K)) < 0.5, -1.0, 1.0).astype(np.float32)
    sgn[0] = -1.0
    sgn[1] = 1.0
    case.X = (sgn * 200.0 * case.x_scale).astype(np.float32)  # quantizes to -128 / 127
    case.y_scale = float(np.float32(K * 128.0))
    _run_linear(case, dev, [0.0, 0.5, 1.0])


# ---------------------------------------------------------------- streams and graphs
def test_cuda_graph_replay_matches_oracle(dev):
    """Prologue + GEMM captured in a CUDA graph (nothing allocates, the launches carry their
    programmatic-dependency attributes) and replayed on new input values."""
    case = inputs.ranged_linear("g", 300, 384, 272, 16, seed=21, group_structured=True)
    perm, sxg, sxs, sw = helpers.prepare_linear(case)
    L = _layer(case, dev, perm, sxg)
    L.set_lowbit_ratio(0.5)
    nl = oracle.n_low(0.5, case.K // case.G)
    X = torch.from_numpy(case.X).to(dev)
    x4, x8 = L.alloc_slabs(case.M)
    Y = torch.empty((case.M, case.N), dtype=torch.int8, device=dev)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        fx.flexiq_quantize_lower(L.h, X, fx.DTYPE_F32, case.M, case.x_scale, 0, x4, x8)   # warm-up outside the capture
        fx.flexiq_mixed_gemm(L.h, x4, x8, None, case.M, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8, Y)
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            fx.flexiq_quantize_lower(L.h, X, fx.DTYPE_F32, case.M, case.x_scale, 0, x4, x8)
            fx.flexiq_mixed_gemm(L.h, x4, x8, None, case.M, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8, Y)
    torch.cuda.synchronize()
    for rep in range(2):
        Xn = case.X * np.float32(1.0 - 0.37 * rep)
        X.copy_(torch.from_numpy(Xn))
        Y.zero_()
        g.replay()
        torch.cuda.synchronize()
        q = oracle.quantize(Xn, case.x_scale)
        acc = oracle.mixed_gemm_acc(q, case.Wq, case.G, perm, sxs, sw, nl)
        assert np.array_equal(Y.cpu().numpy(), oracle.epilogue_i8(acc, case.x_scale, case.w_scale, case.bias, case.y_scale))
    fx.flexiq_check_status()
    L.close()


def test_graph_captured_cold_then_eager_calls_then_replays(dev):
    """Graphs captured with nothing warmed up (no earlier call at their ratio or scales), eager calls at other
    ratios and scales in between, replays in scrambled order: every graph carries the ratio-dependent weight
    block it needs, and eager calls never trust state that a replay may have rewritten."""
    case = inputs.ranged_linear("gc", 300, 384, 272, 16, seed=27, group_structured=True)
    perm, sxg, sxs, sw = helpers.prepare_linear(case)
    L = _layer(case, dev, perm, sxg)
    X = torch.from_numpy(case.X).to(dev)
    q = oracle.quantize(case.X, case.x_scale)

    def want(r, y_scale):
        acc = oracle.mixed_gemm_acc(q, case.Wq, case.G, perm, sxs, sw, oracle.n_low(r, case.K // case.G))
        return oracle.epilogue_i8(acc, case.x_scale, case.w_scale, case.bias, y_scale)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graphs = {}
    with torch.cuda.stream(side):
        for r in (0.25, 0.75, 1.0 / 3.0):   # max_4bit_ch 96, 288, 128: two fall inside a K block of 128, one on its edge
            L.set_lowbit_ratio(r)
            x4 = torch.empty(case.M * case.K + 16, dtype=torch.uint8, device=dev)
            Y = torch.empty((case.M, case.N), dtype=torch.int8, device=dev)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                fx.flexiq_quantize_lower(L.h, X, fx.DTYPE_F32, case.M, case.x_scale, 0, x4, None)
                fx.flexiq_mixed_gemm(L.h, x4, None, None, case.M, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8, Y)
            graphs[r] = (g, Y, x4)
        # a graph that holds only the GEMM, on a slab written eagerly beforehand
        L.set_lowbit_ratio(0.5)
        x4e = torch.empty(case.M * case.K + 16, dtype=torch.uint8, device=dev)
        Ye = torch.empty((case.M, case.N), dtype=torch.int8, device=dev)
        fx.flexiq_quantize_lower(L.h, X, fx.DTYPE_F32, case.M, case.x_scale, 0, x4e, None)
        side.synchronize()
        ge = torch.cuda.CUDAGraph()
        with torch.cuda.graph(ge, stream=side):
            fx.flexiq_mixed_gemm(L.h, x4e, None, None, case.M, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8, Ye)
        graphs[0.5] = (ge, Ye, x4e)
    torch.cuda.synchronize()
    ys2 = float(np.float32(case.y_scale * 1.7))
    for r in (0.75, 0.25, 0.5, 1.0 / 3.0, 0.25, 0.5, 0.75):
        # an eager call at another ratio and another output scale first
        r_e = 0.625 if r != 0.5 else 0.125
        L.set_lowbit_ratio(r_e)
        x4, x8, _ = L.quantize_lower(X, case.x_scale)
        y = L.mixed_gemm(x4, x8, case.M, case.x_scale, ys2, fx.OUT_REQUANT_I8)
        torch.cuda.synchronize()
        assert np.array_equal(y.cpu().numpy(), want(r_e, ys2)), f"eager call at {r_e}"
        g, Y, _ = graphs[r]
        Y.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(Y.cpu().numpy(), want(r, case.y_scale)), f"replay at {r}"
        # and an eager GEMM on the slab the eager prologue wrote before the replay
        y = L.mixed_gemm(x4, x8, case.M, case.x_scale, ys2, fx.OUT_REQUANT_I8)
        torch.cuda.synchronize()
        assert np.array_equal(y.cpu().numpy(), want(r_e, ys2)), f"eager GEMM after the replay at {r}"
    fx.flexiq_check_status()
    L.close()


def test_slab_written_at_another_ratio_is_refused(dev):
    """A mixed_* call on a slab buffer that the handle saw written at another max_4bit_ch returns an error instead
    of wrong values (masked path) or a read past the end of the buffer (packed path); slabs of several ratios
    prepared ahead in buffers of their own are fine; the check can be switched off."""
    case = inputs.ranged_linear("sr", 200, 256, 64, 16, seed=28, group_structured=True)
    perm, sxg, sxs, sw = helpers.prepare_linear(case)
    q = oracle.quantize(case.X, case.x_scale)
    for path in (fx.LOWBIT_MASKED_I8, fx.LOWBIT_PACKED_U4):
        L = _layer(case, dev, perm, sxg, path=path)
        X = torch.from_numpy(case.X).to(dev)
        slabs = {}
        for r in (0.25, 0.75):
            L.set_lowbit_ratio(r)
            bufs = (torch.empty(case.M * case.K + 16, dtype=torch.uint8, device=dev), torch.empty(case.M * case.K + 16, dtype=torch.int8, device=dev))
            L.quantize_lower(X, case.x_scale, slabs=bufs)
            slabs[r] = bufs
        for r_set, r_slab in ((0.25, 0.75), (0.75, 0.25), (1.0, 0.25), (0.0, 0.75)):
            L.set_lowbit_ratio(r_set)
            with pytest.raises(fx.FlexiqError) as e:
                L.mixed_gemm(*slabs[r_slab], case.M, case.x_scale, case.y_scale, fx.OUT_ACC_I32)
            assert e.value.code == fx.ERR_INVALID_ARG and "max_4bit_ch" in str(e.value)
        for r in (0.75, 0.25):   # each buffer at its own ratio, in any order
            L.set_lowbit_ratio(r)
            acc = L.mixed_gemm(*slabs[r], case.M, case.x_scale, case.y_scale, fx.OUT_ACC_I32)
            torch.cuda.synchronize()
            assert np.array_equal(acc.cpu().numpy(), oracle.mixed_gemm_acc(q, case.Wq, case.G, perm, sxs, sw, oracle.n_low(r, case.K // case.G)))
        if path == fx.LOWBIT_MASKED_I8:   # opt-out (masked slabs have the same shape at every ratio: no overrun)
            fx.flexiq_layer_set_slab_check(L.h, False)
            L.set_lowbit_ratio(0.25)
            L.mixed_gemm(*slabs[0.75], case.M, case.x_scale, case.y_scale, fx.OUT_ACC_I32)
            fx.flexiq_layer_set_slab_check(L.h, True)
        torch.cuda.synchronize()
        fx.flexiq_check_status()
        L.close()


def test_bounded_wait_expires_and_the_context_stays_usable(dev):
    """A device-side wait that nothing satisfies gives up after its limit (here a millisecond), raises the status word
    that flexiq_check_status reports as a timeout -- once -- and leaves the context usable for the next launches."""
    res = torch.zeros(3, dtype=torch.int32, device=dev)
    fx.flexiq_selftest_wait_expiry(res)
    with pytest.raises(fx.FlexiqError) as e:
        fx.flexiq_check_status()
    assert e.value.code == fx.ERR_TIMEOUT
    assert res.cpu().tolist() == [1, 0, 1]
    fx.flexiq_check_status()                       # cleared
    _run_linear(inputs.ranged_linear("after", 130, 128, 48, 16, seed=77), dev, [0.5])   # the device still computes


def test_two_layers_on_two_streams(dev):
    """Independent layer handles may run on different streams at the same time."""
    cases = [inputs.ranged_linear("a", 700, 256, 320, 16, seed=31), inputs.ranged_linear("b", 500, 512, 144, 32, seed=32)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    prepared, outs = [], []
    for c in cases:
        perm, sxg, sxs, sw = helpers.prepare_linear(c)
        L = _layer(c, dev, perm, sxg)
        L.set_lowbit_ratio(0.5)
        prepared.append((L, perm, sxs, sw, torch.from_numpy(c.X).to(dev)))
    torch.cuda.synchronize()
    for rep in range(5):
        for (L, perm, sxs, sw, X), c, st in zip(prepared, cases, streams):
            with torch.cuda.stream(st):
                x4, x8, _ = L.quantize_lower(X, c.x_scale)
                Y = L.mixed_gemm(x4, x8, c.M, c.x_scale, c.y_scale, fx.OUT_ACC_I32)
                if rep == 4:
                    outs.append(Y)
    torch.cuda.synchronize()
    for (L, perm, sxs, sw, X), c, Y in zip(prepared, cases, outs):
        q = oracle.quantize(c.X, c.x_scale)
        assert np.array_equal(Y.cpu().numpy(), oracle.mixed_gemm_acc(q, c.Wq, c.G, perm, sxs, sw, oracle.n_low(0.5, c.K // c.G)))
        L.close()
    fx.flexiq_check_status()
