"""GPU parity of the device calibration kernels against the oracle: channel ranges of the
Eq. 1-quantized calibration batch, weight ranges, static positions, error scores, greedy order,
unused-bit histogram (integers: bit-exact) and the moving-average activation range (fp32: exact)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_02822_b200 import binding as fx
from paper_2510_02822_b200 import calib, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    return torch.device("cuda:0")


def _check(case, dev, conv, batches, dtype=torch.float32):
    Xc = torch.from_numpy(case.Xcal).to(dev).to(dtype)
    perm, xs, info = calib.static_preparation_device(Xc, case.x_scale, torch.from_numpy(case.Wq).to(dev), case.G, conv=conv, batches=batches)
    C = case.Xcal.shape[-1]
    q = oracle.quantize(Xc.float().cpu().numpy().reshape(-1, C), case.x_scale)
    lo, hi = oracle.channel_ranges(q)
    assert np.array_equal(info["lo"].cpu().numpy(), lo) and np.array_equal(info["hi"].cpu().numpy(), hi)
    wmax = oracle.weight_absmax_conv(case.Wq) if conv else oracle.weight_absmax_linear(case.Wq)
    assert np.array_equal(info["wmax"].cpu().numpy(), wmax)
    assert np.array_equal(xs, oracle.static_positions(lo, hi, case.G))
    perm_e, score_e = oracle.greedy_order(lo, hi, wmax, case.G)
    assert np.array_equal(info["score"].cpu().numpy(), score_e)
    assert np.array_equal(perm, perm_e)
    assert np.array_equal(info["unused_hist"].cpu().numpy(), oracle.unused_bits_histogram(lo, hi))
    # and the host front end used elsewhere agrees with both
    perm_h, xs_h = calib.static_preparation(calib.quantize_reference(torch.from_numpy(case.Xcal).to(dtype), case.x_scale), torch.from_numpy(case.Wq), case.G, conv=conv)
    assert np.array_equal(perm_h, perm) and np.array_equal(xs_h, xs)


@pytest.mark.parametrize("K,N,G,batches", [(384, 384, 16, 1), (768, 2304, 16, 3), (3072, 768, 32, 2), (64, 16, 64, 1), (192, 80, 16, 5)])
def test_linear_calibration(dev, K, N, G, batches):
    _check(inputs.ranged_linear("c", 64, K, N, G, seed=K + N, group_structured=True), dev, False, batches)


def test_vit_outlier_channels_and_half_precision(dev):
    _check(inputs.vit_linear("v", 64, 768, 768, 16, seed=11), dev, False, 2)
    _check(inputs.ranged_linear("h", 64, 256, 64, 16, seed=12), dev, False, 1, dtype=torch.float16)
    _check(inputs.ranged_linear("b", 64, 256, 64, 16, seed=13), dev, False, 1, dtype=torch.bfloat16)


@pytest.mark.parametrize("H,C,Cout,R", [(14, 128, 64, 3), (28, 64, 256, 1), (7, 512, 512, 3)])
def test_conv_calibration(dev, H, C, Cout, R):
    _check(inputs.resnet_conv("c", 2, H, C, Cout, R, seed=H + C), dev, True, 2)


def test_wide_layer_and_ragged_window(dev):
    rng = np.random.default_rng(3)
    K = 8192 + 48  # 32 full channel windows and a partial one
    X = torch.from_numpy(rng.normal(0, 1, (40, K)).astype(np.float32)).to(dev)
    lo = torch.empty(K, dtype=torch.int32, device=dev)
    hi = torch.empty(K, dtype=torch.int32, device=dev)
    fx.flexiq_calib_channel_ranges(X, fx.DTYPE_F32, 40, K, 0.05, False, lo, hi)
    elo, ehi = oracle.channel_ranges(oracle.quantize(X.cpu().numpy(), 0.05))
    assert np.array_equal(lo.cpu().numpy(), elo) and np.array_equal(hi.cpu().numpy(), ehi)


@pytest.mark.parametrize("M,K,dt", [(700, 96, torch.float32), (3000, 768, torch.float16), (129, 1040, torch.int8)])
def test_histogram_and_coverage_ranges(dev, M, K, dt):
    rng = np.random.default_rng(M + K)
    xs = 0.05
    x = (rng.normal(0, 1, (M, K)) * rng.uniform(0.2, 6, (1, K))).astype(np.float32)
    if dt == torch.int8:
        X = torch.from_numpy(oracle.quantize(x, xs)).to(dev)
        q = X.cpu().numpy()
    else:
        X = torch.from_numpy(x).to(dt).to(dev)
        q = oracle.quantize(X.float().cpu().numpy(), xs)
    hist = torch.empty((K, 256), dtype=torch.int32, device=dev)
    half = M // 2
    fx.flexiq_calib_channel_histogram(X[:half], fx._dtype_code(X), half, K, xs, False, hist)
    fx.flexiq_calib_channel_histogram(X[half:], fx._dtype_code(X), M - half, K, xs, True, hist)
    eh = oracle.channel_histogram(q)
    assert np.array_equal(hist.cpu().numpy().view(np.uint32), eh)
    lo = torch.empty(K, dtype=torch.int32, device=dev)
    hi = torch.empty(K, dtype=torch.int32, device=dev)
    for tail in (0, int(M * 0.01 / 2), M):
        fx.flexiq_calib_ranges_from_histogram(hist, K, tail, lo, hi)
        elo, ehi = oracle.ranges_from_histogram(eh, tail)
        assert np.array_equal(lo.cpu().numpy(), elo) and np.array_equal(hi.cpu().numpy(), ehi)


def test_absmax_ema(dev):
    rng = np.random.default_rng(5)
    x = (rng.normal(0, 1, (7, 4096)) * rng.uniform(0.5, 4, (7, 1))).astype(np.float32)
    for dt in (torch.float32, torch.float16):
        xb = torch.from_numpy(x).to(dt).to(dev)
        state = torch.zeros(4, dtype=torch.float32, device=dev)
        for b in range(7):
            fx.flexiq_calib_absmax_ema(xb[b], fx._dtype_code(xb), xb[b].numel(), 0.99, state)
        s = state.cpu().numpy()
        assert s[1] == 7.0
        assert s[0] == np.float32(oracle.absmax_ema(xb.float().cpu().numpy(), 0.99))


def test_argument_errors(dev):
    z = torch.zeros(64, dtype=torch.int32, device=dev)
    x = torch.zeros((4, 64), dtype=torch.float32, device=dev)
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_calib_channel_ranges(x, fx.DTYPE_F32, 4, 60, 0.1, False, z, z)       # K not a multiple of 16
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_calib_channel_ranges(x, fx.DTYPE_F32, 4, 64, 0.0, False, z, z)       # scale must be positive
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_calib_prepare(z, z, z, 64, 24, z, z, z, z)                           # group size
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_calib_absmax_ema(x, fx.DTYPE_I8, 256, 0.99, x)                       # integer input has no range to track


def test_front_end_with_coverage(dev):
    case = inputs.vit_linear("v", 64, 768, 768, 16, seed=17)
    Xc = torch.from_numpy(case.Xcal).to(dev)
    perm, xs, info = calib.static_preparation_device(Xc, case.x_scale, torch.from_numpy(case.Wq).to(dev), case.G, batches=3, coverage=0.99)
    q = oracle.quantize(case.Xcal, case.x_scale)
    lo, hi = oracle.ranges_from_histogram(oracle.channel_histogram(q), int(q.shape[0] * (1.0 - 0.99) / 2.0))
    assert np.array_equal(info["lo"].cpu().numpy(), lo) and np.array_equal(info["hi"].cpu().numpy(), hi)
    assert np.array_equal(xs, oracle.static_positions(lo, hi, case.G))
    perm_e, _ = oracle.greedy_order(lo, hi, oracle.weight_absmax_linear(case.Wq), case.G)
    assert np.array_equal(perm, perm_e)
