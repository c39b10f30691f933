"""GPU parity of the fused layer boundary: a mixed GEMM / convolution whose epilogue writes the
next layer's masked slab, against the oracle's chain  epilogue -> (ReLU) -> lowering by the next
layer's layout and positions.  All results are integers: bit-exact."""
import numpy as np
import pytest
import torch

import helpers
import oracle
from paper_2510_02822_b200 import binding as fx
from paper_2510_02822_b200 import calib, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    return torch.device("cuda:0")


def _mk(case, dev, perm, sxg, conv=False):
    return fx.Layer(torch.from_numpy(case.Wq).to(dev), torch.from_numpy(case.w_scale).to(dev),
                    torch.from_numpy(case.bias).to(dev), perm, sxg, case.G,
                    conv=(case.stride, case.pad) if conv else None)


def _expected_slab(q1, nxt_case, perm, sxs, nl, K):
    e4, e8 = oracle.make_slabs(q1.reshape(-1, K), nxt_case.G, perm, sxs, nl)
    lo = helpers.masked_slab(e4, nxt_case.G, sxs, nl) if nl else np.empty((e8.shape[0], 0), np.int8)
    return np.concatenate([lo, e8], axis=1)


def _chain_linear(dev, M, K, N1, N2, G1, G2, ratios, relu, seed):
    a = inputs.ranged_linear("a", M, K, N1, G1, seed=seed, group_structured=True)
    b = inputs.ranged_linear("b", 64, N1, N2, G2, seed=seed + 1, group_structured=True)
    rng = np.random.default_rng(seed)
    shifts_b = rng.integers(0, 5, N1 // G2).astype(np.uint8)  # arbitrary positions: some values saturate
    pa, sga, sxa, swa = helpers.prepare_linear(a)
    pb, sgb, sxb, swb = helpers.prepare_linear(b, shifts_b)
    A, B = _mk(a, dev, pa, sga), _mk(b, dev, pb, sgb)
    # the same layer with its output channels permuted offline into the next layer's slab order
    Wp, wsp, bp = calib.permute_outputs_for_next(torch.from_numpy(a.Wq), torch.from_numpy(a.w_scale), torch.from_numpy(a.bias), pb, G2)
    Ap = fx.Layer(Wp.to(dev), wsp.to(dev), bp.to(dev), pa, sga, G1)
    X = torch.from_numpy(a.X).to(dev)
    qa = oracle.quantize(a.X, a.x_scale)
    xs_b = a.y_scale  # the next layer's activation scale is this layer's output scale
    for ra, rb in ratios:
        A.set_lowbit_ratio(ra)
        B.set_lowbit_ratio(rb)
        nla, nlb = oracle.n_low(ra, K // G1), oracle.n_low(rb, N1 // G2)
        x4, x8, _ = A.quantize_lower(X, a.x_scale)
        slab, guard_ok = helpers.with_guard(torch, (M, N1), torch.uint8, dev)
        A.mixed_gemm_to_slab(x4, x8, M, a.x_scale, B, xs_b, relu=relu, slab=slab)
        torch.cuda.synchronize()
        fx.flexiq_check_status()
        guard_ok()
        acc = oracle.mixed_gemm_acc(qa, a.Wq, G1, pa, sxa, swa, nla)
        q1 = oracle.epilogue_i8(acc, a.x_scale, a.w_scale, a.bias, xs_b)
        if relu:
            q1 = np.maximum(q1, 0)
        exp = _expected_slab(q1, b, pb, sxb, nlb, N1)
        assert np.array_equal(slab.cpu().numpy().view(np.int8), exp)
        Ap.set_lowbit_ratio(ra)
        slab_p, guard_p = helpers.with_guard(torch, (M, N1), torch.uint8, dev)
        Ap.mixed_gemm_to_slab(x4, x8, M, a.x_scale, B, xs_b, relu=relu, slab=slab_p, out_order=fx.ORDER_NEXT_SLAB)
        torch.cuda.synchronize()
        guard_p()
        assert np.array_equal(slab_p.cpu().numpy().view(np.int8), exp)
        # the two-call sequence gives the same slab, and the next layer consumes the fused one
        two = B.quantize_lower(torch.from_numpy(q1).to(dev), xs_b)[0][:M * N1].view(M, N1)
        assert torch.equal(two, slab)
        Y = B.mixed_gemm(slab, None, M, xs_b, b.y_scale, fx.OUT_ACC_I32)
        torch.cuda.synchronize()
        assert np.array_equal(Y.cpu().numpy(), oracle.mixed_gemm_acc(q1, b.Wq, G2, pb, sxb, swb, nlb))
    A.close()
    B.close()
    Ap.close()


@pytest.mark.parametrize("M,K,N1,N2,G1,G2,relu", [(300, 256, 272, 48, 16, 16, False), (129, 128, 64, 32, 16, 32, True),
                                                  (1000, 384, 1024, 80, 16, 64, False), (1, 64, 16, 16, 16, 16, True),
                                                  (515, 192, 400, 64, 32, 16, True),
                                                  (260, 1280, 112, 48, 16, 16, False)])   # one long-K tile per CTA
def test_linear_chain(dev, M, K, N1, N2, G1, G2, relu):
    _chain_linear(dev, M, K, N1, N2, G1, G2, [(0.0, 0.0), (0.5, 0.5), (1.0, 0.25), (0.25, 1.0)], relu, seed=M + N1)


@pytest.mark.parametrize("cg,bn", [(1, 64), (1, 128), (1, 192), (1, 256), (2, 128), (2, 192), (2, 256)])
def test_every_tile_shape(dev, cg, bn):
    fx.flexiq_force_tile(cg, bn)
    try:
        _chain_linear(dev, 700, 256, 720, 32, 16, 16, [(0.5, 0.5), (1.0, 1.0)], True, seed=cg * 1000 + bn)
    finally:
        fx.flexiq_force_tile(0, 0)


@pytest.mark.parametrize("Nb,H,C,Cmid,R,stride", [(2, 14, 128, 64, 3, 1), (3, 28, 64, 128, 3, 2), (2, 14, 128, 256, 1, 1)])
def test_conv_chain(dev, Nb, H, C, Cmid, R, stride):
    a = inputs.resnet_conv("a", Nb, H, C, Cmid, R, seed=H + C, stride=stride)
    P = (H + 2 * a.pad - R) // stride + 1
    b = inputs.resnet_conv("b", Nb, P, Cmid, 64, 3, seed=H + C + 1)
    rng = np.random.default_rng(H * C)
    pa, sga, sxa, swa = helpers.prepare_conv(a)
    pb, sgb, sxb, swb = helpers.prepare_conv(b, rng.integers(0, 5, Cmid // b.G).astype(np.uint8))
    A, B = _mk(a, dev, pa, sga, conv=True), _mk(b, dev, pb, sgb, conv=True)
    Wp, wsp, bp = calib.permute_outputs_for_next(torch.from_numpy(a.Wq), torch.from_numpy(a.w_scale), torch.from_numpy(a.bias), pb, b.G, conv=True)
    Ap = fx.Layer(Wp.to(dev), wsp.to(dev), bp.to(dev), pa, sga, a.G, conv=(a.stride, a.pad))
    X = torch.from_numpy(a.X).to(dev)
    qa = oracle.quantize(a.X, a.x_scale)
    xs_b = a.y_scale
    for ra, rb in [(0.0, 0.5), (0.5, 1.0), (1.0, 0.0)]:
        A.set_lowbit_ratio(ra)
        B.set_lowbit_ratio(rb)
        nla, nlb = oracle.n_low(ra, C // a.G), oracle.n_low(rb, Cmid // b.G)
        x4, x8, _ = A.quantize_lower(X, a.x_scale)
        slab, guard_ok = helpers.with_guard(torch, (Nb * P * P, Cmid), torch.uint8, dev)
        A.mixed_conv_to_slab(x4, x8, Nb, H, H, a.x_scale, B, xs_b, relu=True, slab=slab)
        torch.cuda.synchronize()
        fx.flexiq_check_status()
        guard_ok()
        acc = oracle.mixed_conv_acc(qa, a.Wq, a.stride, a.pad, a.G, pa, sxa, swa, nla)
        q1 = np.maximum(oracle.epilogue_i8(acc, a.x_scale, a.w_scale, a.bias, xs_b), 0)
        exp = _expected_slab(q1, b, pb, sxb, nlb, Cmid)
        assert np.array_equal(slab.cpu().numpy().view(np.int8), exp)
        Ap.set_lowbit_ratio(ra)
        slab_p = Ap.mixed_conv_to_slab(x4, x8, Nb, H, H, a.x_scale, B, xs_b, relu=True, out_order=fx.ORDER_NEXT_SLAB)
        torch.cuda.synchronize()
        assert np.array_equal(slab_p[:exp.size].cpu().numpy().view(np.int8).reshape(exp.shape), exp)
        Y = B.mixed_conv(slab, None, Nb, P, P, xs_b, b.y_scale, fx.OUT_ACC_I32)
        torch.cuda.synchronize()
        assert np.array_equal(Y.cpu().numpy(), oracle.mixed_conv_acc(q1.reshape(Nb, P, P, Cmid), b.Wq, b.stride, b.pad, b.G, pb, sxb, swb, nlb))
    for L in (A, B, Ap):
        L.close()


def test_argument_errors(dev):
    a = inputs.ranged_linear("a", 32, 64, 64, 16, seed=5)
    b = inputs.ranged_linear("b", 32, 128, 16, 16, seed=6)
    pa, sga, _, _ = helpers.prepare_linear(a)
    pb, sgb, _, _ = helpers.prepare_linear(b)
    A, B = _mk(a, dev, pa, sga), _mk(b, dev, pb, sgb)
    x4, x8, _ = A.quantize_lower(torch.from_numpy(a.X).to(dev), a.x_scale)
    slab = torch.empty(32 * 128, dtype=torch.uint8, device=dev)
    with pytest.raises(fx.FlexiqError) as e:  # 64 output channels into a layer of 128 input channels
        A.mixed_gemm_to_slab(x4, x8, 32, a.x_scale, B, 0.1, slab=slab)
    assert e.value.code == fx.ERR_INVALID_ARG
    A2 = _mk(a, dev, pa, sga)
    with pytest.raises(fx.FlexiqError) as e:
        A.mixed_gemm_to_slab(x4, x8, 32, a.x_scale, A2, 0.0, slab=slab)  # scale must be positive
    assert e.value.code == fx.ERR_INVALID_ARG
    with pytest.raises(fx.FlexiqError) as e:
        A.mixed_gemm_to_slab(x4, x8, 32, a.x_scale, A2, 0.1, slab=slab, out_order=7)
    assert e.value.code == fx.ERR_INVALID_ARG
    A2.set_lowbit_path(fx.LOWBIT_PACKED_U4)
    with pytest.raises(fx.FlexiqError) as e:
        A.mixed_gemm_to_slab(x4, x8, 32, a.x_scale, A2, 0.1, slab=slab)
    assert e.value.code == fx.ERR_UNSUPPORTED
    for L in (A, B, A2):
        L.close()


@pytest.mark.parametrize("M,K,G,dt", [(300, 256, 16, torch.int8), (129, 192, 32, torch.float16), (1000, 768, 16, torch.float32),
                                      (1, 64, 64, torch.int8), (12608, 768, 16, torch.int8)])
def test_residual_reorder(dev, M, K, G, dt):
    rng = np.random.default_rng(M + K)
    perm = rng.permutation(K // G).astype(np.int32)
    Wq = torch.zeros((K, 16), dtype=torch.int8, device=dev)
    L = fx.Layer(Wq, torch.ones(16, device=dev), torch.zeros(16, device=dev), perm, np.zeros(K // G, np.uint8), G)
    X = torch.from_numpy(rng.integers(-120, 120, (M, K)).astype(np.int32)).to(dt).to(dev)
    xn = X.cpu().numpy()
    Y, guard_ok = helpers.with_guard(torch, (M, K), dt, dev)
    L.reorder_channels(X, fx.REORDER_TO_SLAB, Y=Y)
    torch.cuda.synchronize()
    guard_ok()
    assert np.array_equal(Y.cpu().numpy(), oracle.reorder_channels(xn, G, perm, True))
    Z = L.reorder_channels(X, fx.REORDER_FROM_SLAB)
    assert np.array_equal(Z.cpu().numpy(), oracle.reorder_channels(xn, G, perm, False))
    assert torch.equal(L.reorder_channels(Y, fx.REORDER_FROM_SLAB), X)
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_reorder_channels(L.h, X, X.element_size(), M, fx.REORDER_TO_SLAB, X)  # in place
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_reorder_channels(L.h, X, 3, M, fx.REORDER_TO_SLAB, Y)
    L.close()
