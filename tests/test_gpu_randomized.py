"""Seeded random runs of the CUDA path against the CPU oracle, bit-exact: shapes, group sizes, ratios,
extraction positions, low-bit paths, input and output types are drawn from a generator with a fixed
seed, so every run checks the same cases.  The hand-picked cases of the other files cover the edges
one knows about; these cover combinations nobody listed (a convolution whose padded row does not
fit its tile pitch was found this way)."""
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


def _ratio(rng, n_g):
    return float(rng.choice([0.0, 1.0 / n_g, 1.0, float(rng.random()), float(rng.random())]))


def _expected(acc, case, mode, y_scale):
    if mode == fx.OUT_ACC_I32:
        return acc
    if mode == fx.OUT_REQUANT_I8:
        return oracle.epilogue_i8(acc, case.x_scale, case.w_scale, case.bias, y_scale)
    if mode == fx.OUT_DEQUANT_F16:
        return oracle.epilogue_f16(acc, case.x_scale, case.w_scale, case.bias).view(np.uint16)
    return oracle.epilogue_bf16_bits(acc, case.x_scale, case.w_scale, case.bias)


def _bits(Y, mode):
    if mode in (fx.OUT_DEQUANT_F16, fx.OUT_DEQUANT_BF16):
        return Y.view(torch.int16).cpu().numpy().view(np.uint16)
    return Y.cpu().numpy()


MODES = [fx.OUT_ACC_I32, fx.OUT_REQUANT_I8, fx.OUT_DEQUANT_F16, fx.OUT_DEQUANT_BF16]


@pytest.mark.parametrize("seed", [11, 12])
def test_random_convolutions(dev, seed):
    """Square inputs of 3 to 69 pixels, 16 to 384 input channels, 1x1 / 3x3 / 5x5 taps, stride 1 or 2:
    all three launch kinds (plain, im2col, halo patch) and their ragged tiles."""
    for i in range(40):
        rng = np.random.default_rng(seed * 100000 + i)
        C = 16 * int(rng.choice([1, 2, 3, 4, 6, 8, 12, 16, 24]))
        Cout = 16 * int(rng.integers(1, 20))
        R = int(rng.choice([1, 3, 3, 3, 5]))
        stride = int(rng.choice([1, 1, 1, 2])) if R > 1 else 1
        H = int(rng.integers(3, 70))
        Nb = int(rng.integers(1, 5)) if H < 40 else 1
        G = int(rng.choice([16, 16, 32])) if C % 32 == 0 else 16
        case = inputs.resnet_conv("rc", Nb, H, C, Cout, R, G=G, seed=i, stride=stride)
        perm, sxg, sxs, sw = helpers.prepare_conv(case, rng.integers(0, 5, C // G).astype(np.uint8))
        q = oracle.quantize(case.X, case.x_scale)
        X = torch.from_numpy(case.X).to(dev)
        L = _mk(case, dev, perm, sxg, conv=True)
        for _ in range(2):
            r = _ratio(rng, C // G)
            L.set_lowbit_ratio(r)
            nl = oracle.n_low(r, C // G)
            x4, x8, _ = L.quantize_lower(X, case.x_scale)
            acc = oracle.mixed_conv_acc(q, case.Wq, case.stride, case.pad, G, perm, sxs, sw, nl)
            for mode in (fx.OUT_ACC_I32, int(rng.choice(MODES[1:]))):
                Y = L.mixed_conv(x4, x8, Nb, H, H, case.x_scale, case.y_scale, mode)
                torch.cuda.synchronize()
                assert np.array_equal(_bits(Y, mode), _expected(acc, case, mode, case.y_scale)), \
                    f"conv {(Nb, H, C, Cout, R, stride, G)} ratio {r} mode {mode}"
        fx.flexiq_check_status()
        L.close()


@pytest.mark.parametrize("seed", [21, 22])
def test_random_layers_paths_types_positions(dev, seed):
    """One layer per case: masked or packed 4-bit slabs, fp32 / fp16 / bf16 input, static or dynamic
    extraction positions, any output type."""
    for i in range(40):
        rng = np.random.default_rng(seed * 100000 + i)
        G = int(rng.choice([16, 32, 64]))
        conv = bool(rng.integers(0, 3) == 0)
        path = fx.LOWBIT_PACKED_U4 if rng.integers(0, 2) else fx.LOWBIT_MASKED_I8
        if conv:
            G = 16
            C = 16 * int(rng.choice([1, 2, 4, 6, 8, 16, 20]))
            N = 16 * int(rng.integers(1, 14))
            R = int(rng.choice([1, 3, 5]))
            H = int(rng.integers(5, 36))
            Nb = int(rng.integers(1, 4))
            case = inputs.resnet_conv("rl", Nb, H, C, N, R, seed=i, stride=int(rng.choice([1, 1, 2])))
            perm, sxg, sxs, sw = helpers.prepare_conv(case, rng.integers(0, 5, C // G).astype(np.uint8))
            K, M = C, Nb * H * H
            if C % 32:
                path = fx.LOWBIT_MASKED_I8  # the packed convolution needs whole 16-byte weight taps
        else:
            K = G * int(rng.integers(1, 48))
            N = 16 * int(rng.integers(1, 40))
            M = int(rng.integers(1, 2000))
            case = inputs.ranged_linear("rl", M, K, N, G, seed=i, group_structured=True)
            perm, sxg, sxs, sw = helpers.prepare_linear(case, rng.integers(0, 5, K // G).astype(np.uint8))
        n_g = K // G
        L = _mk(case, dev, perm, sxg, conv=conv)
        L.set_lowbit_path(path)
        dt = int(rng.integers(0, 3))
        Xt, code = torch.from_numpy(case.X), fx.DTYPE_F32
        if dt == 1:
            Xt, code = Xt.to(torch.float16), fx.DTYPE_F16
        elif dt == 2:
            Xt, code = Xt.to(torch.bfloat16), fx.DTYPE_BF16
        q = oracle.quantize(Xt.to(torch.float32).numpy(), case.x_scale)  # the 16-bit values are exact in fp32
        Xd = Xt.to(dev)
        for _ in range(3):
            r = _ratio(rng, n_g)
            dyn = bool(rng.integers(0, 3) == 0)
            L.set_lowbit_ratio(r)
            nl = oracle.n_low(r, n_g)
            x4, x8 = L.alloc_slabs(M)
            shifts = torch.zeros(n_g, dtype=torch.uint8, device=dev) if dyn else None
            scratch = torch.full((n_g,), -1, dtype=torch.int32, device=dev) if dyn else None
            fx.flexiq_quantize_lower(L.h, Xd, code, M, case.x_scale, 1 if dyn else 0, x4, x8, shifts, scratch)
            sx_use = oracle.dynamic_positions(q.reshape(M, K), G, perm) if dyn else sxs
            mode = int(rng.choice(MODES))
            if conv:
                Y = L.mixed_conv(x4, x8, case.Nb, H, H, case.x_scale, case.y_scale, mode, x_shift=shifts)
                acc = oracle.mixed_conv_acc(q, case.Wq, case.stride, case.pad, G, perm, sx_use, sw, nl)
            else:
                Y = L.mixed_gemm(x4, x8, M, case.x_scale, case.y_scale, mode, x_shift=shifts)
                acc = oracle.mixed_gemm_acc(q, case.Wq, G, perm, sx_use, sw, nl)
            torch.cuda.synchronize()
            what = f"{'conv' if conv else 'linear'} {(M, K, N, G)} path {path} input {dt} dynamic {dyn} mode {mode} ratio {r}"
            if dyn:
                assert np.array_equal(shifts.cpu().numpy(), sx_use), what
            assert np.array_equal(_bits(Y, mode), _expected(acc, case, mode, case.y_scale)), what
        fx.flexiq_check_status()
        L.close()


def _expected_slab(q1, G, perm, sxs, nl, K):
    e4, e8 = oracle.make_slabs(q1.reshape(-1, K), G, perm, sxs, nl)
    lo = helpers.masked_slab(e4, G, sxs, nl) if nl else np.empty((e8.shape[0], 0), np.int8)
    return np.concatenate([lo, e8], axis=1)


def test_random_fused_boundaries(dev):
    """Two-layer chains whose first epilogue writes the second layer's slab (original and slab output order,
    with and without ReLU), then the second layer on that slab."""
    for i in range(24):
        rng = np.random.default_rng(3100000 + i)
        conv = bool(i % 2)
        if conv:
            C = 16 * int(rng.choice([1, 2, 4, 8, 16]))
            Cmid = 16 * int(rng.integers(1, 12))
            R = int(rng.choice([1, 3]))
            H = int(rng.integers(4, 40))
            Nb = int(rng.integers(1, 4))
            a = inputs.resnet_conv("fa", Nb, H, C, Cmid, R, seed=i, stride=int(rng.choice([1, 1, 2])))
            P = (H + 2 * a.pad - R) // a.stride + 1
            b = inputs.resnet_conv("fb", Nb, P, Cmid, 16 * int(rng.integers(1, 6)), int(rng.choice([1, 3])), seed=i + 1)
            pa, sga, sxa, swa = helpers.prepare_conv(a)
            pb, sgb, sxb, swb = helpers.prepare_conv(b, rng.integers(0, 5, Cmid // b.G).astype(np.uint8))
            M, K, N1 = Nb * P * P, C, Cmid
        else:
            G1, G2 = int(rng.choice([16, 32, 64])), int(rng.choice([16, 32, 64]))
            K, N1 = G1 * int(rng.integers(1, 30)), G2 * int(rng.integers(1, 20))
            M = int(rng.integers(1, 1500))
            a = inputs.ranged_linear("fa", M, K, N1, G1, seed=i, group_structured=True)
            b = inputs.ranged_linear("fb", 64, N1, 16 * int(rng.integers(1, 8)), G2, seed=i + 1, group_structured=True)
            pa, sga, sxa, swa = helpers.prepare_linear(a)
            pb, sgb, sxb, swb = helpers.prepare_linear(b, rng.integers(0, 5, N1 // G2).astype(np.uint8))
        A, B = _mk(a, dev, pa, sga, conv), _mk(b, dev, pb, sgb, conv)
        Wp, wsp, bp = calib.permute_outputs_for_next(torch.from_numpy(a.Wq), torch.from_numpy(a.w_scale),
                                                     torch.from_numpy(a.bias), pb, b.G, conv=conv)
        Ap = fx.Layer(Wp.to(dev), wsp.to(dev), bp.to(dev), pa, sga, a.G, conv=(a.stride, a.pad) if conv else None)
        X = torch.from_numpy(a.X).to(dev)
        qa = oracle.quantize(a.X, a.x_scale)
        for _ in range(2):
            ra, rb = _ratio(rng, K // a.G), _ratio(rng, N1 // b.G)
            relu = bool(rng.integers(0, 2))
            for L, r in ((A, ra), (Ap, ra), (B, rb)):
                L.set_lowbit_ratio(r)
            nla, nlb = oracle.n_low(ra, K // a.G), oracle.n_low(rb, N1 // b.G)
            x4, x8, _ = A.quantize_lower(X, a.x_scale)
            slab, g1 = helpers.with_guard(torch, (M, N1), torch.uint8, dev)
            slab_p, g2 = helpers.with_guard(torch, (M, N1), torch.uint8, dev)
            if conv:
                A.mixed_conv_to_slab(x4, x8, Nb, H, H, a.x_scale, B, a.y_scale, relu=relu, slab=slab)
                Ap.mixed_conv_to_slab(x4, x8, Nb, H, H, a.x_scale, B, a.y_scale, relu=relu, slab=slab_p, out_order=fx.ORDER_NEXT_SLAB)
                Y = B.mixed_conv(slab, None, Nb, P, P, a.y_scale, b.y_scale, fx.OUT_REQUANT_I8)
                acc = oracle.mixed_conv_acc(qa, a.Wq, a.stride, a.pad, a.G, pa, sxa, swa, nla)
            else:
                A.mixed_gemm_to_slab(x4, x8, M, a.x_scale, B, a.y_scale, relu=relu, slab=slab)
                Ap.mixed_gemm_to_slab(x4, x8, M, a.x_scale, B, a.y_scale, relu=relu, slab=slab_p, out_order=fx.ORDER_NEXT_SLAB)
                Y = B.mixed_gemm(slab, None, M, a.y_scale, b.y_scale, fx.OUT_REQUANT_I8)
                acc = oracle.mixed_gemm_acc(qa, a.Wq, a.G, pa, sxa, swa, nla)
            torch.cuda.synchronize()
            fx.flexiq_check_status()
            g1()
            g2()
            q1 = oracle.epilogue_i8(acc, a.x_scale, a.w_scale, a.bias, a.y_scale)
            if relu:
                q1 = np.maximum(q1, 0)
            exp = _expected_slab(q1, b.G, pb, sxb, nlb, N1)
            what = f"chain {i} ratios {ra} {rb} relu {relu}"
            assert np.array_equal(slab.cpu().numpy().view(np.int8), exp), what
            assert np.array_equal(slab_p.cpu().numpy().view(np.int8), exp), what + " (slab output order)"
            if conv:
                acc2 = oracle.mixed_conv_acc(q1.reshape(Nb, P, P, N1), b.Wq, b.stride, b.pad, b.G, pb, sxb, swb, nlb)
            else:
                acc2 = oracle.mixed_gemm_acc(q1, b.Wq, b.G, pb, sxb, swb, nlb)
            assert np.array_equal(Y.cpu().numpy(), oracle.epilogue_i8(acc2, a.y_scale, b.w_scale, b.bias, b.y_scale)), what
        for L in (A, B, Ap):
            L.close()


def test_random_call_sequences_on_one_handle(dev):
    """Sec. 7, run-time ratio adjustment, as a state machine: on one handle a random sequence of ratio
    switches, eager prologue + GEMM calls, GEMM-only calls on a slab prepared earlier at the current
    ratio, CUDA-graph captures (with or without the prologue) and replays of any earlier graph at
    whatever ratio the handle has by then.  Every result is the oracle's at the ratio its slab was
    written at, with the output scale of its own call."""
    side = torch.cuda.Stream()
    for li in range(16):
        rng = np.random.default_rng(4100000 + li)
        conv = bool(li % 2)
        G = 16
        if conv:
            K = 16 * int(rng.choice([2, 4, 8, 12, 16]))
            N = 16 * int(rng.integers(1, 12))
            H = int(rng.integers(5, 20))
            Nb = int(rng.integers(1, 4))
            case = inputs.resnet_conv("sq", Nb, H, K, N, int(rng.choice([1, 3])), G=G, seed=li)
            perm, sxg, sxs, sw = helpers.prepare_conv(case, rng.integers(0, 5, K // G).astype(np.uint8))
            M = Nb * H * H
        else:
            K = G * int(rng.integers(2, 40))
            N = 16 * int(rng.integers(1, 24))
            M = int(rng.integers(1, 700))
            case = inputs.ranged_linear("sq", M, K, N, G, seed=li, group_structured=True)
            perm, sxg, sxs, sw = helpers.prepare_linear(case, rng.integers(0, 5, K // G).astype(np.uint8))
        n_g = K // G
        q = oracle.quantize(case.X, case.x_scale)
        X = torch.from_numpy(case.X).to(dev)
        L = _mk(case, dev, perm, sxg, conv)
        ratios = [0.0, 1.0 / n_g, 0.3, 0.5, 0.7, 1.0]
        y_scales = [case.y_scale * f for f in (1.0, 1.5, 0.6, 2.2, 0.9, 3.0)]  # more than the handle's factor tables
        accs = {}

        def want(r, ys, mode):
            if r not in accs:
                nl = oracle.n_low(r, n_g)
                accs[r] = (oracle.mixed_conv_acc(q, case.Wq, case.stride, case.pad, G, perm, sxs, sw, nl) if conv
                           else oracle.mixed_gemm_acc(q, case.Wq, G, perm, sxs, sw, nl))
            return _expected(accs[r], case, mode, ys)

        def out_buf(mode):
            shape = (case.Nb, H, H, N) if conv else (M, N)
            return torch.zeros(shape, dtype=torch.int8 if mode == fx.OUT_REQUANT_I8 else torch.float16, device=dev)

        def prologue(slab):
            fx.flexiq_quantize_lower(L.h, X, fx.DTYPE_F32, M, case.x_scale, 0, slab, None)

        def gemm(slab, ys, mode, Y):
            if conv:
                fx.flexiq_mixed_conv(L.h, slab, None, None, case.Nb, H, H, case.x_scale, ys, mode, Y)
            else:
                fx.flexiq_mixed_gemm(L.h, slab, None, None, M, case.x_scale, ys, mode, Y)

        def verify(Y, r, ys, mode, what):
            torch.cuda.synchronize()
            assert np.array_equal(_bits(Y, mode), want(r, ys, mode)), f"layer {li} step {step}: {what} at ratio {r}"

        graphs, prepared, cur = [], {}, 0.0
        L.set_lowbit_ratio(cur)
        for step in range(30):
            op = int(rng.integers(0, 6))
            mode = fx.OUT_REQUANT_I8 if rng.integers(0, 3) else fx.OUT_DEQUANT_F16
            ys = float(y_scales[int(rng.integers(0, len(y_scales)))])
            if op == 0:
                cur = float(ratios[int(rng.integers(0, len(ratios)))])
                L.set_lowbit_ratio(cur)
            elif op == 1:
                slab = torch.empty(M * K + 16, dtype=torch.uint8, device=dev)
                Y = out_buf(mode)
                prologue(slab)
                gemm(slab, ys, mode, Y)
                prepared[cur] = slab
                verify(Y, cur, ys, mode, "eager prologue + GEMM")
            elif op == 2 and cur in prepared:
                Y = out_buf(mode)
                gemm(prepared[cur], ys, mode, Y)
                verify(Y, cur, ys, mode, "eager GEMM")
            elif op == 3 and len(graphs) < 6:
                slab = torch.empty(M * K + 16, dtype=torch.uint8, device=dev)
                Y = out_buf(mode)
                gemm_only = bool(rng.integers(0, 2)) and cur in prepared
                torch.cuda.synchronize()
                side.wait_stream(torch.cuda.current_stream())
                g = torch.cuda.CUDAGraph()
                with torch.cuda.stream(side):
                    with torch.cuda.graph(g, stream=side):
                        if gemm_only:
                            gemm(prepared[cur], ys, mode, Y)
                        else:
                            prologue(slab)
                            gemm(slab, ys, mode, Y)
                torch.cuda.synchronize()
                graphs.append((g, Y, cur, ys, mode, prepared[cur] if gemm_only else slab))
            elif op >= 4 and graphs:
                g, Y, r, g_ys, g_mode, _ = graphs[int(rng.integers(0, len(graphs)))]
                Y.zero_()
                g.replay()
                verify(Y, r, g_ys, g_mode, "graph replay")
        torch.cuda.synchronize()
        fx.flexiq_check_status()
        del graphs
        L.close()


def test_random_auxiliary_kernels(dev):
    """The kernels around the layer path on drawn shapes: calibration ranges (one or several batches), histogram
    and coverage ranges, static preparation (positions, scores, greedy order), the residual reorder operator in
    both directions and three element sizes, and the squared distance of the selection search."""
    for i in range(30):
        rng = np.random.default_rng(5100000 + i)
        G = int(rng.choice([16, 32, 64]))
        K = G * int(rng.integers(1, 70))
        N = 16 * int(rng.integers(1, 20))
        M = int(rng.integers(1, 900))
        dt = [torch.float32, torch.float16, torch.bfloat16][int(rng.integers(0, 3))]
        xs = float(rng.uniform(0.01, 0.2))
        x = (rng.normal(0, 1, (M, K)) * rng.uniform(0.05, 8, (1, K))).astype(np.float32)
        X = torch.from_numpy(x).to(dt).to(dev)
        q = oracle.quantize(X.float().cpu().numpy(), xs)
        # ranges, accumulated over two uneven parts
        lo = torch.empty(K, dtype=torch.int32, device=dev)
        hi = torch.empty(K, dtype=torch.int32, device=dev)
        cut = int(rng.integers(0, M + 1))
        code = fx._dtype_code(X)
        if cut:
            fx.flexiq_calib_channel_ranges(X[:cut], code, cut, K, xs, False, lo, hi)
        if M - cut:
            fx.flexiq_calib_channel_ranges(X[cut:], code, M - cut, K, xs, bool(cut), lo, hi)
        elo, ehi = oracle.channel_ranges(q)
        assert np.array_equal(lo.cpu().numpy(), elo) and np.array_equal(hi.cpu().numpy(), ehi), f"ranges {(M, K, dt)}"
        # histogram and coverage ranges
        hist = torch.empty((K, 256), dtype=torch.int32, device=dev)
        fx.flexiq_calib_channel_histogram(X, code, M, K, xs, False, hist)
        eh = oracle.channel_histogram(q)
        assert np.array_equal(hist.cpu().numpy().view(np.uint32), eh), f"histogram {(M, K, dt)}"
        tail = int(rng.integers(0, max(1, M // 8) + 1))
        clo, chi = torch.empty_like(lo), torch.empty_like(hi)
        fx.flexiq_calib_ranges_from_histogram(hist, K, tail, clo, chi)
        e_clo, e_chi = oracle.ranges_from_histogram(eh, tail)
        assert np.array_equal(clo.cpu().numpy(), e_clo) and np.array_equal(chi.cpu().numpy(), e_chi), f"coverage {(M, K, tail)}"
        # weight ranges, positions, scores, greedy order
        Wq = rng.integers(-127, 128, (K, N)).astype(np.int8)
        Wq[rng.integers(0, K, K // 3)] //= 16   # some narrow input channels
        perm, sx, info = calib.static_preparation_device(X, xs, torch.from_numpy(Wq).to(dev), G)
        wmax = oracle.weight_absmax_linear(Wq)
        perm_e, score_e = oracle.greedy_order(elo, ehi, wmax, G)
        assert np.array_equal(info["wmax"].cpu().numpy(), wmax)
        assert np.array_equal(sx, oracle.static_positions(elo, ehi, G))
        assert np.array_equal(info["score"].cpu().numpy(), score_e) and np.array_equal(perm, perm_e), f"order {(K, N, G)}"
        # residual reorder in the order just found
        L = fx.Layer(torch.from_numpy(Wq).to(dev), torch.ones(N, device=dev), torch.zeros(N, device=dev), perm, sx, G)
        rdt = [torch.int8, torch.float16, torch.float32][int(rng.integers(0, 3))]
        R = torch.from_numpy(rng.integers(-120, 120, (M, K)).astype(np.int32)).to(rdt).to(dev)
        Y, guard_ok = helpers.with_guard(torch, (M, K), rdt, dev)
        L.reorder_channels(R, fx.REORDER_TO_SLAB, Y=Y)
        torch.cuda.synchronize()
        guard_ok()
        assert np.array_equal(Y.cpu().numpy(), oracle.reorder_channels(R.cpu().numpy(), G, perm, True)), f"reorder {(M, K, G, rdt)}"
        assert torch.equal(L.reorder_channels(Y, fx.REORDER_FROM_SLAB), R)
        L.close()
        # squared distance of two int8 tensors
        n = int(rng.integers(0, 300000))
        a = rng.integers(-128, 128, n).astype(np.int8)
        b = rng.integers(-128, 128, n).astype(np.int8)
        out = torch.full((1,), -5, dtype=torch.int64, device=dev)
        fx.flexiq_sq_distance_i8(torch.from_numpy(a).to(dev), torch.from_numpy(b).to(dev), out)
        assert int(out.item()) == int(((a.astype(np.int64) - b.astype(np.int64)) ** 2).sum())
    fx.flexiq_check_status()


def test_random_large_linears_on_sampled_rows(dev):
    """Linears of 2,000 to 30,000 rows, up to 4096 input and output channels: several waves of tiles per CTA, CTA pairs,
    ragged last tiles in both directions.  The oracle computes 150 random rows, the first rows and the last 40;
    a second launch must give the same bytes as the first everywhere."""
    for i in range(10):
        rng = np.random.default_rng(6100000 + i)
        G = int(rng.choice([16, 32, 64]))
        K = G * int(rng.integers(4, 4096 // G + 1))
        N = 16 * int(rng.integers(8, 257))
        M = int(rng.integers(2000, 30000))
        case = inputs.vit_linear("rb", M, K, N, G, seed=i)
        perm, sxg, sxs, sw = helpers.prepare_linear(case, rng.integers(0, 5, K // G).astype(np.uint8))
        L = _mk(case, dev, perm, sxg)
        X = torch.from_numpy(case.X).to(dev)
        rows = np.unique(np.concatenate([rng.integers(0, M, 150), np.arange(M - 40, M), np.arange(0, 8)])).astype(np.int64)
        ridx = torch.from_numpy(rows).to(dev)
        q_rows = oracle.quantize(case.X[rows], case.x_scale)
        for r in (float(rng.random()), float(rng.choice([0.0, 0.5, 1.0]))):
            L.set_lowbit_ratio(r)
            nl = oracle.n_low(r, K // G)
            x4, x8, _ = L.quantize_lower(X, case.x_scale)
            mode = int(rng.choice([fx.OUT_REQUANT_I8, fx.OUT_DEQUANT_F16, fx.OUT_ACC_I32]))
            Y = L.mixed_gemm(x4, x8, M, case.x_scale, case.y_scale, mode)
            Y2 = L.mixed_gemm(x4, x8, M, case.x_scale, case.y_scale, mode)
            torch.cuda.synchronize()
            fx.flexiq_check_status()
            acc = oracle.mixed_gemm_acc(q_rows, case.Wq, G, perm, sxs, sw, nl)
            what = f"linear {(M, K, N, G)} ratio {r} mode {mode}"
            assert np.array_equal(_bits(Y[ridx], mode), _expected(acc, case, mode, case.y_scale)), what
            assert torch.equal(Y.view(torch.uint8), Y2.view(torch.uint8)), what
        L.close()
