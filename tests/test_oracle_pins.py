"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test compares the oracle with something other than itself: a value printed in the
paper (tests/golden/paper_worked_examples.txt), a closed form, an invariant, a library
routine on a special case, or a brute-force computation on tiny inputs.
"""
import itertools
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_worked_examples.txt")


def golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


# ------------------------------------------------------------------ Eq. 1 (Sec. 2.1)
def test_quantize_worked_examples():
    g = golden()
    S = np.float32(g["derived_scale"])
    q = oracle.quantize(np.array([g["ex1_fp"], g["ex2_fp"]], np.float32), S)
    assert q.tolist() == [int(g["ex1_q8"]), int(g["ex2_q8"])]


def test_quantize_clip_and_ties():
    S = 0.25  # power of two: x / S is exact, so ties are real ties
    x = np.array([0.5 * S, 1.5 * S, 2.5 * S, -0.5 * S, -1.5 * S, -2.5 * S, 1e9, -1e9, 127.4 * S, 127.5 * S,
                  -128.5 * S, -129 * S, 0.0], np.float32)
    q = oracle.quantize(x, S)
    assert q.tolist() == [0, 2, 2, 0, -2, -2, 127, -128, 127, 127, -128, -128, 0]


def test_quantize_monotone_and_step():
    # invariants of Eq. 1: monotone in x, |x/S - q| <= 1/2 inside the clip range
    rng = np.random.default_rng(1)
    S = np.float32(0.0173)
    x = np.sort(rng.uniform(-2.0, 2.0, 5000).astype(np.float32))
    q = oracle.quantize(x, S).astype(np.int64)
    assert np.all(np.diff(q) >= 0)
    t = x.astype(np.float64) / np.float64(S)
    inside = np.abs(t) < 127
    assert np.all(np.abs(t[inside] - q[inside]) <= 0.5 + 1e-4)


# ------------------------------------------------------------------ positions (Sec. 4.1)
def test_position_worked_examples():
    g = golden()
    # "maximum is less than 32" -> two unused bits -> keep bits 3..6 -> shift right by 2
    assert oracle.position_from_range(0, int(g["ex1_channel_max_below"]) - 1) == 4 - int(g["ex1_unused_bits"])
    # "minimum larger than -16" -> three unused bits -> shift right by 1
    assert oracle.position_from_range(int(g["ex2_channel_min_above"]) + 1, 0) == 4 - int(g["ex2_unused_bits"])
    # naive conversion = highest four bits = position 4 = a full-range channel
    assert oracle.position_from_range(-128, 127) == 4
    assert oracle.position_from_range(0, 0) == 0
    assert oracle.position_from_range(-8, 7) == 0  # 4 or more unused bits: lossless at position 0


def test_position_is_smallest_non_saturating_shift():
    # independent definition: the smallest shift s for which no value of [lo, hi] leaves [-8, 7]
    for lo in range(-128, 1):
        for hi in range(0, 128):
            s_def = next(s for s in range(0, 5) if (lo >> s) >= -8 and (hi >> s) <= 7)
            assert oracle.position_from_range(lo, hi) == s_def, (lo, hi)


def test_bitlen():
    for v in range(0, 300):
        assert oracle.bitlen(v) == v.bit_length()


# ------------------------------------------------------------------ lowering (Sec. 4.1, Fig. 3)
def test_lower_worked_examples():
    g = golden()
    q1, q2 = int(g["ex1_q8"]), int(g["ex2_q8"])
    s1 = oracle.position_from_range(0, 31)
    s2 = oracle.position_from_range(-15, 0)
    assert oracle.lower(q1, s1) == int(g["derived_ex1_q4"])
    assert oracle.lower(q2, s2) == int(g["derived_ex2_q4"])
    # reconstruction error of example 1 is below 4 %; six effective bits = position 2 + 4 bits
    rec = oracle.lower(q1, s1) << s1
    assert abs(rec - q1) / q1 < g["ex1_flexiq_error_below"]
    # the naive top-four-bits conversion of the same value has about 10 % error
    naive = round(q1 / 16) * 16
    assert abs(abs(naive - q1) / q1 - g["ex1_naive_error_about"]) < 0.01
    # bit patterns quoted in the text
    assert (q1 & 0xFF) == 0b00011101 and (oracle.lower(q1, s1) & 15) == 0b0111
    assert (q2 & 0xFF) == 0b11110111 and (oracle.lower(q2, s2) & 15) == 0b1011


def test_lower_exhaustive_bit_subset():
    # Sec. 2.3: the low-bit value is a bit-subset of the 8-bit one.  For every int8 value
    # and position: unsaturated values keep exactly bits s..s+3; the dropped part is the
    # s low bits; saturated values clamp to the nearest end of [-8, 7].
    for q in range(-128, 128):
        for s in range(0, 5):
            v = oracle.lower(q, s)
            assert -8 <= v <= 7
            if -8 <= (q >> s) <= 7:
                assert (v & 15) == ((q & 0xFF) >> s) & 15
                assert 0 <= q - (v << s) < (1 << s)
            else:
                assert v == (7 if q > 0 else -8)
    for q in range(-8, 8):
        assert oracle.lower(q, 0) == q


# ------------------------------------------------------------------ dynamic positions
def test_dynamic_positions_equal_exact_range_rule():
    rng = np.random.default_rng(3)
    G, K, M = 16, 128, 37
    scale = rng.choice([1, 3, 9, 20, 60, 127], size=K)
    q = (rng.standard_normal((M, K)) * scale / 3).clip(-128, 127).astype(np.int8)
    perm = rng.permutation(K // G).astype(np.int32)
    sx = oracle.dynamic_positions(q, G, perm)
    for j, g in enumerate(perm):
        blk = q[:, g * G:(g + 1) * G].astype(int)
        assert sx[j] == oracle.position_from_range(min(0, blk.min()), max(0, blk.max()))
        low = np.array([[oracle.lower(int(v), int(sx[j])) for v in row] for row in blk])
        assert np.array_equal(low, blk >> int(sx[j]))  # never saturates


def test_static_positions_group_max_and_ranges():
    rng = np.random.default_rng(4)
    G, K = 16, 64
    qcal = (rng.standard_normal((50, K)) * rng.choice([2, 10, 40, 120], size=K) / 3).clip(-128, 127).astype(np.int8)
    lo, hi = oracle.channel_ranges(qcal)
    assert np.array_equal(lo, np.minimum(qcal.min(0), 0)) and np.array_equal(hi, np.maximum(qcal.max(0), 0))
    sx = oracle.static_positions(lo, hi, G)
    for g in range(K // G):
        assert sx[g] == max(oracle.position_from_range(int(lo[c]), int(hi[c])) for c in range(g * G, (g + 1) * G))


# ------------------------------------------------------------------ selection order (Sec. 4.2)
def test_greedy_order_nested_and_sorted():
    rng = np.random.default_rng(5)
    G, K, N = 16, 256, 48
    lo = -rng.integers(0, 128, K).astype(np.int32)
    hi = rng.integers(0, 128, K).astype(np.int32)
    Wq = rng.integers(-127, 128, (K, N)).astype(np.int8)
    wmax = oracle.weight_absmax_linear(Wq)
    assert np.array_equal(wmax, np.abs(Wq.astype(int)).max(1))
    perm, score = oracle.greedy_order(lo, hi, wmax, G)
    assert sorted(perm.tolist()) == list(range(K // G))
    ch = np.maximum(hi, -lo).astype(np.int64) * wmax
    assert np.array_equal(score, ch.reshape(-1, G).max(1))
    assert np.all(np.diff(score[perm]) >= 0)
    # nestedness: the low set at a smaller ratio is a subset (prefix) of the one at a larger ratio
    sets = [set(perm[:oracle.n_low(r, K // G)].tolist()) for r in (0.0, 0.25, 0.5, 0.75, 1.0)]
    for a, b in zip(sets, sets[1:]):
        assert a <= b
    assert len(sets[0]) == 0 and len(sets[-1]) == K // G


def test_n_low_rounds_up_to_meet_target():
    for ng in (4, 8, 16, 24, 32, 48, 64, 96, 192, 256):
        for r in (0.0, 0.25, 0.5, 0.75, 1.0):
            assert oracle.n_low(r, ng) == round(r * ng)
    assert oracle.n_low(0.3, 10) == 3 and oracle.n_low(0.31, 10) == 4 and oracle.n_low(0.01, 10) == 1


# ------------------------------------------------------------------ mixed accumulate (Sec. 7)
def _random_problem(rng, M, K, N, G):
    scale = rng.choice([2, 5, 12, 30, 70, 127], size=K)
    Xq = (rng.standard_normal((M, K)) * scale / 2.5).clip(-128, 127).astype(np.int8)
    Wq = (rng.standard_normal((K, N)) * rng.choice([3, 10, 40, 127], size=(K, 1)) / 2.5).clip(-127, 127).astype(np.int8)
    perm = rng.permutation(K // G).astype(np.int32)
    # static positions from a different (smaller-range) draw so some values saturate
    sx = rng.integers(0, 5, K // G).astype(np.uint8)
    sw = oracle.weight_positions_linear(Wq, G, perm)
    return Xq, Wq, perm, sx, sw


def _masked_operands(Xq, Wq, G, perm, sx, sw, n_low):
    """X' and W' of the closed form: 4-bit value shifted back to its position, in slab order."""
    K = Xq.shape[1]
    cols = np.concatenate([np.arange(g * G, (g + 1) * G) for g in perm])
    Xs = Xq[:, cols].astype(np.int64)
    Ws = Wq[cols, :].astype(np.int64)
    for j in range(n_low):
        sl = slice(j * G, (j + 1) * G)
        s = int(sx[j])
        Xs[:, sl] = np.clip(Xs[:, sl] >> s, -8, 7) << s
        sh = sw[j].astype(np.int64)[None, :]
        Ws[sl, :] = (Ws[sl, :] >> sh) << sh
    return Xs, Ws


@pytest.mark.parametrize("M,K,N,G", [(5, 64, 16, 16), (33, 128, 48, 32), (17, 192, 32, 64), (7, 96, 16, 16)])
def test_mixed_gemm_closed_form_all_prefixes(M, K, N, G):
    rng = np.random.default_rng(M * 1000 + K)
    Xq, Wq, perm, sx, sw = _random_problem(rng, M, K, N, G)
    for n_low in range(0, K // G + 1):
        acc = oracle.mixed_gemm_acc(Xq, Wq, G, perm, sx, sw, n_low)
        Xs, Ws = _masked_operands(Xq, Wq, G, perm, sx, sw, n_low)
        assert np.array_equal(acc.astype(np.int64), Xs @ Ws), n_low


def test_ratio_zero_is_the_int8_gemm():
    rng = np.random.default_rng(11)
    Xq, Wq, perm, sx, sw = _random_problem(rng, 29, 160, 32, 16)
    acc = oracle.mixed_gemm_acc(Xq, Wq, 16, perm, sx, sw, 0)
    assert np.array_equal(acc.astype(np.int64), Xq.astype(np.int64) @ Wq.astype(np.int64))


def test_ratio_one_is_the_pure_4bit_computation():
    rng = np.random.default_rng(12)
    G = 16
    Xq, Wq, perm, sx, sw = _random_problem(rng, 13, 96, 16, G)
    ng = 96 // G
    acc = oracle.mixed_gemm_acc(Xq, Wq, G, perm, sx, sw, ng)
    ref = np.zeros((13, 16), np.int64)
    for j, g in enumerate(perm):
        x4 = np.clip(Xq[:, g * G:(g + 1) * G].astype(np.int64) >> int(sx[j]), -8, 7)
        w4 = Wq[g * G:(g + 1) * G, :].astype(np.int64) >> sw[j].astype(np.int64)[None, :]
        assert w4.min() >= -8 and w4.max() <= 7  # weights never saturate
        ref += (x4 @ w4) << (int(sx[j]) + sw[j].astype(np.int64))[None, :]
    assert np.array_equal(acc.astype(np.int64), ref)


def test_brute_force_dot_products_tiny():
    rng = np.random.default_rng(13)
    G = 16
    for (M, K, N) in [(1, 16, 16), (3, 32, 16), (4, 64, 16)]:
        Xq, Wq, perm, sx, sw = _random_problem(rng, M, K, N, G)
        for n_low in range(K // G + 1):
            acc = oracle.mixed_gemm_acc(Xq, Wq, G, perm, sx, sw, n_low)
            for m in range(M):
                for n in range(0, N, 5):
                    total = 0
                    for j, g in enumerate(perm):
                        for i in range(G):
                            x = int(Xq[m, g * G + i])
                            w = int(Wq[g * G + i, n])
                            if j < n_low:
                                s, t = int(sx[j]), int(sw[j, n])
                                x4 = max(-8, min(7, x >> s))
                                w4 = w >> t
                                total += (x4 * w4) << (s + t)
                            else:
                                total += x * w
                    assert int(acc[m, n]) == total


def test_lossless_low_groups_contribute_their_int8_value():
    rng = np.random.default_rng(14)
    G, K, N, M = 16, 64, 16, 9
    Xq = rng.integers(-8, 8, (M, K)).astype(np.int8)
    Wq = rng.integers(-8, 8, (K, N)).astype(np.int8)
    perm = rng.permutation(K // G).astype(np.int32)
    sx = np.zeros(K // G, np.uint8)
    sw = oracle.weight_positions_linear(Wq, G, perm)
    assert not sw.any()
    acc = oracle.mixed_gemm_acc(Xq, Wq, G, perm, sx, sw, K // G)
    assert np.array_equal(acc.astype(np.int64), Xq.astype(np.int64) @ Wq.astype(np.int64))


def test_row_sampled_accumulators_match_full():
    rng = np.random.default_rng(15)
    Xq, Wq, perm, sx, sw = _random_problem(rng, 40, 128, 32, 16)
    full = oracle.mixed_gemm_acc(Xq, Wq, 16, perm, sx, sw, 3)
    rows = np.array([0, 7, 39, 12], np.int64)
    assert np.array_equal(oracle.mixed_gemm_acc(Xq, Wq, 16, perm, sx, sw, 3, rows=rows), full[rows])


def test_slab_format():
    G, K = 16, 32
    q = np.arange(-16, 16, dtype=np.int8)[None, :].repeat(2, 0)
    q[1] = q[1][::-1]
    perm = np.array([1, 0], np.int32)
    sx = np.array([1, 0], np.uint8)
    X4, X8 = oracle.make_slabs(q, G, perm, sx, 1)
    assert X4.shape == (2, 16) and X8.shape == (2, 16)
    # slab group 0 = original group 1 = values 0..15 >> 1 = 0,0,1,1,...,7,7 ; byte t = ch 2t | ch 2t+1 << 4
    assert X4[0, :8].tolist() == [((2 * t) >> 1) | (((2 * t + 1) >> 1) << 4) for t in range(8)]
    assert X8[0].tolist() == list(range(-16, 0))
    assert oracle.x4_pitch(16) == 16 and oracle.x4_pitch(96) == 48 and oracle.x4_pitch(48) == 32


def test_unused_bit_histogram_and_ema():
    # Sec. 4.1's two worked ranges: max < 32 leaves two magnitude bits unused, min > -16 three
    lo = np.array([0, -15, -128, 0, -1, 0, -64, 0], np.int32)
    hi = np.array([31, 0, 127, 0, 0, 7, 63, 64], np.int32)
    #  used bits:   5    4    7   0   0   3    6   7   ->  unused 2, 3, 0, 7, 7, 4, 1, 0  (>= 4 counted together)
    assert oracle.unused_bits_histogram(lo, hi).tolist() == [2, 1, 1, 1, 3]
    # consistency with the extraction position: position = max(0, 4 - unused) for every int8 range
    for l in range(-128, 1, 7):
        for h in range(0, 128, 5):
            u = int(np.argmax(oracle.unused_bits_histogram([l], [h])))
            assert oracle.position_from_range(l, h) == max(0, 4 - u) or u == 4
    # EMA: constant batches are a fixed point; momentum 0 follows the last batch; momentum 0.5 by hand
    x = np.array([[1.0, -3.0], [2.0, 0.5], [-8.0, 1.0]], np.float32)
    assert oracle.absmax_ema(np.tile(np.float32([[1.5, -2.5]]), (5, 1)), 0.99) == np.float32(2.5)
    assert oracle.absmax_ema(x, 0.0) == 8.0
    assert oracle.absmax_ema(x, 0.5) == 0.5 * (0.5 * 3.0 + 0.5 * 2.0) + 0.5 * 8.0
    assert oracle.absmax_ema(x[:1], 0.99) == 3.0


def test_coverage_ranges_from_histogram():
    rng = np.random.default_rng(11)
    q = np.clip(np.rint(rng.normal(0, 20, (1000, 8)) * np.array([0.1, 0.5, 1, 2, 4, 0.2, 1, 3])), -128, 127).astype(np.int8)
    q[:, 5] = np.abs(q[:, 5])          # a one-sided channel: its lower end stays at zero
    hist = oracle.channel_histogram(q)
    assert hist.sum(1).tolist() == [1000] * 8
    assert np.array_equal(hist[2], np.bincount(q[:, 2].astype(np.int64) + 128, minlength=256))
    # no tail dropped: the exact ranges
    lo0, hi0 = oracle.ranges_from_histogram(hist, 0)
    elo, ehi = oracle.channel_ranges(q)
    assert np.array_equal(lo0, elo) and np.array_equal(hi0, ehi)
    # 99 % coverage = 5 samples per tail: the 6th smallest / largest value (order statistics), never past zero
    lo, hi = oracle.ranges_from_histogram(hist, 5)
    for c in range(8):
        srt = np.sort(q[:, c].astype(np.int64))
        # dropping whole bins only: the bound is the value v with at most 5 samples strictly beyond it
        assert lo[c] == min(0, max(v for v in range(-128, 1) if (srt < v).sum() <= 5))
        assert hi[c] == max(0, min(v for v in range(0, 128) if (srt > v).sum() <= 5))
        assert ((srt < lo[c]).sum() <= 5) and ((srt > hi[c]).sum() <= 5) and lo[c] <= 0 <= hi[c]
    assert lo[5] == 0
    # hand case: values -3 (x1), 0 (x7), 5 (x2); one sample per tail may go
    h = np.zeros((1, 256), np.uint32)
    h[0, 125], h[0, 128], h[0, 133] = 1, 7, 2
    assert [x.tolist() for x in oracle.ranges_from_histogram(h, 1)] == [[0], [5]]
    assert [x.tolist() for x in oracle.ranges_from_histogram(h, 2)] == [[0], [0]]


def test_residual_reorder_moves_whole_groups():
    # hand case (Sec. 5 step 3): three groups of 2 channels, slab group j holds original group perm[j]
    x = np.array([[10, 11, 20, 21, 30, 31]], np.int8)
    perm = np.array([2, 0, 1], np.int32)
    assert oracle.reorder_channels(x, 2, perm, True).tolist() == [[30, 31, 10, 11, 20, 21]]
    assert oracle.reorder_channels(x, 2, perm, False).tolist() == [[20, 21, 30, 31, 10, 11]]
    rng = np.random.default_rng(7)
    for dt in (np.int8, np.float16, np.float32):
        G, n_g, M = 16, 12, 9
        X = rng.integers(-100, 100, (M, G * n_g)).astype(dt)
        perm = rng.permutation(n_g).astype(np.int32)
        cols = np.concatenate([np.arange(g * G, (g + 1) * G) for g in perm])
        Y = oracle.reorder_channels(X, G, perm, True)
        assert np.array_equal(Y, X[:, cols])                                     # a column gather
        assert np.array_equal(oracle.reorder_channels(Y, G, perm, False), X)     # and its inverse
    # the 8-bit slab of the prologue at ratio 0 is the same gather
    q = rng.integers(-128, 128, (5, 64)).astype(np.int8)
    perm = rng.permutation(4).astype(np.int32)
    assert np.array_equal(oracle.make_slabs(q, 16, perm, np.zeros(4, np.uint8), 0)[1], oracle.reorder_channels(q, 16, perm, True))


# ------------------------------------------------------------------ epilogue
def test_epilogue_identity_scale_is_a_clip():
    acc = np.array([[-300, -128, -1, 0, 1, 127, 128, 100000] * 2], np.int32)
    out = oracle.epilogue_i8(acc, 1.0, np.ones(16, np.float32), None, 1.0)
    assert np.array_equal(out, np.clip(acc, -128, 127).astype(np.int8))
    f = oracle.epilogue_f32(acc, 1.0, np.ones(16, np.float32), None)
    assert np.array_equal(f, acc.astype(np.float32))


def test_epilogue_ties_and_bias():
    acc = np.array([[1, 3, 5, -1, -3, 7, 2, 2] * 2], np.int32)
    ws = np.full(16, 0.5, np.float32)
    out = oracle.epilogue_i8(acc, 1.0, ws, None, 1.0)  # 0.5 1.5 2.5 -0.5 -1.5 3.5 1 1
    assert out[0, :8].tolist() == [0, 2, 2, 0, -2, 4, 1, 1]
    bias = np.full(16, 0.25, np.float32)
    out = oracle.epilogue_i8(acc, 1.0, ws, bias, 0.5)  # alpha = 1, beta = 0.5 -> acc + 0.5 -> ties to even
    assert out[0, :8].tolist() == [2, 4, 6, 0, -2, 8, 2, 2]
    f = oracle.epilogue_f32(acc, 2.0, ws, bias)
    assert np.array_equal(f[0, :8], acc[0, :8].astype(np.float32) + 0.25)


# ------------------------------------------------------------------ convolution (Fig. 4)
def _conv_problem(rng, Nb, H, W, C, Cout, R, S, G):
    Xq = (np.abs(rng.standard_normal((Nb, H, W, C))) * rng.choice([3, 10, 40, 100], size=C)).clip(0, 127).astype(np.int8)
    Xq[::2] = -Xq[::2]  # exercise negative values too
    Wq = (rng.standard_normal((Cout, R, S, C)) * rng.choice([3, 12, 50], size=C) ).clip(-127, 127).astype(np.int8)
    perm = rng.permutation(C // G).astype(np.int32)
    sx = rng.integers(0, 5, C // G).astype(np.uint8)
    sw = oracle.weight_positions_conv(Wq, G, perm)
    return Xq, Wq, perm, sx, sw


def _im2col(Xq, R, S, stride, pad):
    Nb, H, W, C = Xq.shape
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    Xp = np.zeros((Nb, H + 2 * pad, W + 2 * pad, C), np.int8)
    Xp[:, pad:pad + H, pad:pad + W] = Xq
    cols = np.zeros((Nb, P, Q, R, S, C), np.int8)
    for r in range(R):
        for s in range(S):
            cols[:, :, :, r, s] = Xp[:, r:r + stride * P:stride, s:s + stride * Q:stride]
    return cols.reshape(Nb * P * Q, R * S * C), P, Q


@pytest.mark.parametrize("R,S,stride,pad", [(3, 3, 1, 1), (1, 1, 1, 0), (3, 3, 2, 1)])
def test_conv_equals_gemm_on_explicit_im2col(R, S, stride, pad):
    rng = np.random.default_rng(20 + R + stride)
    G, C, Cout = 16, 48, 16
    Xq, Wq, perm, sx, sw = _conv_problem(rng, 2, 7, 6, C, Cout, R, S, G)
    A, P, Q = _im2col(Xq, R, S, stride, pad)
    ng, T = C // G, R * S
    Wmat = Wq.reshape(Cout, T * C).T.copy()  # [(r,s,c), Cout]
    for n_low in (0, 1, ng):
        acc = oracle.mixed_conv_acc(Xq, Wq, stride, pad, G, perm, sx, sw, n_low)
        # the same problem as a GEMM whose groups are (tap, channel group): low ones first
        order = [(t, j) for j in range(n_low) for t in range(T)] + [(t, j) for j in range(n_low, ng) for t in range(T)]
        perm2 = np.array([t * ng + perm[j] for t, j in order], np.int32)
        sx2 = np.array([sx[j] for t, j in order], np.uint8)
        sw2 = np.stack([sw[j] for t, j in order])
        ref = oracle.mixed_gemm_acc(A, Wmat, G, perm2, sx2, sw2, n_low * T)
        assert np.array_equal(acc.reshape(-1, Cout), ref)


def test_conv_ratio_zero_equals_float64_conv2d():
    import torch
    rng = np.random.default_rng(31)
    Xq, Wq, perm, sx, sw = _conv_problem(rng, 2, 9, 8, 32, 16, 3, 3, 16)
    acc = oracle.mixed_conv_acc(Xq, Wq, 1, 1, 16, perm, sx, sw, 0)
    x = torch.from_numpy(Xq.astype(np.float64)).permute(0, 3, 1, 2)
    w = torch.from_numpy(Wq.astype(np.float64)).permute(0, 3, 1, 2)
    ref = torch.nn.functional.conv2d(x, w, stride=1, padding=1).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(acc.astype(np.float64), ref)


def test_weight_positions_never_saturate():
    rng = np.random.default_rng(40)
    Wq = (rng.standard_normal((64, 32)) * rng.choice([2, 9, 30, 127], size=(64, 1))).clip(-128, 127).astype(np.int8)
    perm = rng.permutation(4).astype(np.int32)
    sw = oracle.weight_positions_linear(Wq, 16, perm)
    for j, g in enumerate(perm):
        blk = Wq[g * 16:(g + 1) * 16].astype(int)
        w4 = blk >> sw[j].astype(int)[None, :]
        assert w4.min() >= -8 and w4.max() <= 7
        # and the position is tight: one less would saturate (unless already 0)
        for n in range(32):
            if sw[j, n] > 0:
                t = blk[:, n] >> (int(sw[j, n]) - 1)
                assert t.min() < -8 or t.max() > 7


def test_epilogue_half_precision_roundings():
    """fp16 / bf16 outputs = the fp32 value rounded to nearest even: hand-picked ties, and a library
    conversion (torch on the CPU) as an independent reference for both formats."""
    import torch
    ws = np.ones(16, np.float32)
    # acc * 2^-12: 4097 -> 1 + 2^-12 (rounds down to 1 in fp16: spacing 2^-10), 4098 -> 1 + 2^-11 is the tie -> even (1.0),
    # 4102 -> 1 + 3 * 2^-11 is the tie above 1 + 2^-10 -> even (1 + 2^-9)
    acc = np.array([[4096, 4097, 4098, 4099, 4102, -4098, 4128, 4160, 0, 1, -1, 70000, 123456, -99999, 33, 65]], np.int32)
    s = float(2.0 ** -12)
    f32 = oracle.epilogue_f32(acc, s, ws, None)
    f16 = oracle.epilogue_f16(acc, s, ws, None)
    assert f16.dtype == np.float16
    assert f16[0, :6].tolist() == [1.0, 1.0, 1.0, 1.0 + 2.0 ** -10, 1.0 + 2.0 ** -9, -1.0]
    assert np.array_equal(f16, torch.from_numpy(f32).to(torch.float16).numpy())
    # bf16 keeps 8 significant bits: spacing 2^-7 at 1.0; 1 + 2^-8 (acc 4112) is a tie -> 1.0; 1 + 3 * 2^-8 (4144) -> 1 + 2^-6
    acc_b = np.array([[4096, 4112, 4113, 4144, 4128, -4112, 12345678, -7654321, 0, 5, 4111, 4145, 1 << 30, -(1 << 30), 77, 99]], np.int32)
    f32b = oracle.epilogue_f32(acc_b, s, ws, None)
    bits = oracle.epilogue_bf16_bits(acc_b, s, ws, None)
    as_f32 = (bits.astype(np.uint32) << 16).view(np.float32)
    assert as_f32[0, :6].tolist() == [1.0, 1.0, 1.0 + 2.0 ** -7, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7, -1.0]
    want = torch.from_numpy(f32b).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, want)
    rng = np.random.default_rng(0)
    acc_r = rng.integers(-2 ** 24, 2 ** 24, (64, 16)).astype(np.int32)
    wsr = rng.uniform(0.5, 2.0, 16).astype(np.float32)
    br = rng.normal(0, 1, 16).astype(np.float32)
    f = oracle.epilogue_f32(acc_r, 3.1e-4, wsr, br)
    assert np.array_equal(oracle.epilogue_f16(acc_r, 3.1e-4, wsr, br), torch.from_numpy(f).to(torch.float16).numpy())
    assert np.array_equal(oracle.epilogue_bf16_bits(acc_r, 3.1e-4, wsr, br),
                          torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))


# ------------------------------------------------------------------ convolution weight tables (Fig. 4, Sec. 4.1, 4.2)
def _conv_weights(rng, Cout, R, S, Cin):
    """Weights whose range differs by tap, by input channel and by output channel, so that a table taken over
    one tap only, over the wrong axis, or per group instead of per (group, output channel) is wrong."""
    tap = rng.choice([0.1, 0.3, 1.0], size=(1, R, S, 1))
    tap.flat[rng.integers(tap.size)] = 1.0
    cin = rng.choice([0.5, 1.0], size=(1, 1, 1, Cin))
    cell = np.repeat(rng.choice([1, 3, 8, 20, 50], size=(Cout, 1, 1, Cin // 16)), 16, axis=3)  # per (output, group)
    W = rng.standard_normal((Cout, R, S, Cin)) * tap * cin * cell
    return W.clip(-128, 127).astype(np.int8)


@pytest.mark.parametrize("R,S", [(3, 3), (1, 1), (1, 3)])
def test_conv_weight_positions_cover_all_taps_and_are_tight(R, S):
    """Fig. 4 / Sec. 4.1: one extraction position per (channel group, output channel); for a convolution the group's
    weights are those of ALL taps.  The position is the smallest shift for which no weight of the group leaves
    [-8, 7] (weights never saturate), checked by brute force over the taps."""
    rng = np.random.default_rng(60 + R * S)
    G, Cin, Cout = 16, 64, 12
    Wq = _conv_weights(rng, Cout, R, S, Cin)
    perm = rng.permutation(Cin // G).astype(np.int32)
    sw = oracle.weight_positions_conv(Wq, G, perm)
    assert sw.shape == (Cin // G, Cout) and sw.max() <= 4
    seen = set()
    for j, g in enumerate(perm):
        for n in range(Cout):
            blk = Wq[n, :, :, g * G:(g + 1) * G].astype(int)  # every tap, the group's G channels
            s = int(sw[j, n])
            assert (blk >> s).min() >= -8 and (blk >> s).max() <= 7, "a weight would saturate"
            if s > 0:
                t = blk >> (s - 1)
                assert t.min() < -8 or t.max() > 7, "position is not the smallest that fits"
            seen.add(s)
    assert len(seen) >= 3  # the draw exercises several positions
    if R * S > 1:
        # the widest tap decides: positions from the centre tap alone are somewhere smaller
        one_tap = oracle.weight_positions_conv(Wq[:, :1, :1].copy(), G, perm)
        assert np.all(one_tap <= sw) and np.any(one_tap < sw)


def test_conv_1x1_weight_tables_equal_the_linear_ones():
    """A 1x1 convolution is the linear layer with the transposed weight matrix: both tables must agree."""
    rng = np.random.default_rng(71)
    G, Cin, Cout = 16, 80, 24
    Wq = _conv_weights(rng, Cout, 1, 1, Cin)
    perm = rng.permutation(Cin // G).astype(np.int32)
    Wlin = Wq.reshape(Cout, Cin).T.copy()
    assert np.array_equal(oracle.weight_positions_conv(Wq, G, perm), oracle.weight_positions_linear(Wlin, G, perm))
    assert np.array_equal(oracle.weight_absmax_conv(Wq), oracle.weight_absmax_linear(Wlin))


def test_conv_weight_absmax_over_outputs_and_taps():
    """Sec. 4.2: a feature channel's maximum weight range, here over every output channel and every tap."""
    rng = np.random.default_rng(72)
    Wq = _conv_weights(rng, 10, 3, 3, 48)
    Wq[3, 2, 0, 5] = -128  # |-128| = 128 does not fit int8: the table is int32
    got = oracle.weight_absmax_conv(Wq)
    assert got.dtype == np.int32 and got[5] == 128
    assert np.array_equal(got, np.abs(Wq.astype(np.int32)).max(axis=(0, 1, 2)))
    # one tap or one output channel alone gives something smaller somewhere
    assert np.any(np.abs(Wq[:, 1, 1].astype(np.int32)).max(axis=0) < got)
    assert np.any(np.abs(Wq[0].astype(np.int32)).max(axis=(0, 1)) < got)


# ------------------------------------------------------------------ epilogue: ONE rounding at general scales
def _round_to_f32(v):
    """Exact rational -> nearest float32, ties to even, decided with exact comparisons."""
    from fractions import Fraction
    c = np.float32(float(v))
    cands = [c, np.nextafter(c, np.float32(np.inf)), np.nextafter(c, np.float32(-np.inf))]
    best = None
    for x in cands:
        d = abs(Fraction(float(x)) - v)
        even = (int(np.float32(x).view(np.uint32)) & 1) == 0
        if best is None or d < best[0] or (d == best[0] and even and not best[2]):
            best = (d, x, even)
    return np.float32(best[1])


def test_epilogue_is_one_fused_rounding_at_general_scales():
    """y = acc * alpha + beta rounded ONCE to fp32 (a fused multiply-add), then, for int8, to the nearest integer
    (ties to even) and clipped.  The expectation is exact rational arithmetic on the fp32 factors; a product
    rounded before the addition, a factor associated differently, or float(acc) rounded twice fails it."""
    from fractions import Fraction
    rng = np.random.default_rng(80)
    N = 16
    acc = np.concatenate([
        rng.integers(-2 ** 24, 2 ** 24, (40, N)),
        rng.integers(-2 ** 31, 2 ** 31, (40, N)),       # beyond 2^24: float(acc) itself rounds
        rng.integers(-3000, 3000, (40, N)),
    ]).astype(np.int32)
    x_scale, y_scale = np.float32(0.0137), np.float32(0.0911)
    w_scale = rng.uniform(1e-3, 3e-2, N).astype(np.float32)
    bias = rng.normal(0, 0.7, N).astype(np.float32)
    # the factors, each operation rounded to fp32 (the oracle's stated association)
    sxw = (x_scale * w_scale).astype(np.float32)
    alpha = (sxw / y_scale).astype(np.float32)
    beta = (bias / y_scale).astype(np.float32)
    got8 = oracle.epilogue_i8(acc, float(x_scale), w_scale, bias, float(y_scale))
    got32 = oracle.epilogue_f32(acc, float(x_scale), w_scale, bias)
    n_double_rounding_differs = 0
    for m in range(acc.shape[0]):
        for n in range(N):
            a = Fraction(float(np.float32(acc[m, n])))  # int -> fp32, nearest even (numpy's conversion)
            y32 = _round_to_f32(a * Fraction(float(sxw[n])) + Fraction(float(bias[n])))
            assert got32[m, n] == y32, (m, n)
            y = _round_to_f32(a * Fraction(float(alpha[n])) + Fraction(float(beta[n])))
            want = min(127, max(-128, round(Fraction(float(y)))))  # round(): half to even on exact rationals
            assert int(got8[m, n]) == want, (m, n)
            two = np.float32(np.float32(np.float32(acc[m, n]) * sxw[n]) + bias[n])
            n_double_rounding_differs += int(two != y32)
    assert n_double_rounding_differs > 20  # the case set tells one rounding from two


def test_epilogue_int8_decisions_next_to_ties():
    """The int8 output at accumulators chosen (by a scan in float64) so that y lies within a few fp32 ulps of a
    half-integer: there a product rounded before the addition, or alpha built as x_scale * (w_scale / y_scale),
    decides differently from the single fused rounding of the stated factors.  Expectations in exact rationals."""
    from fractions import Fraction
    rng = np.random.default_rng(81)
    N = 512
    x_scale, y_scale = np.float32(0.0137), np.float32(0.0911)
    w_scale = rng.uniform(1e-3, 3e-2, N).astype(np.float32)
    bias = rng.normal(0, 0.7, N).astype(np.float32)
    alpha = ((x_scale * w_scale).astype(np.float32) / y_scale).astype(np.float32)
    alpha_alt = (x_scale * (w_scale / y_scale).astype(np.float32)).astype(np.float32)
    beta = (bias / y_scale).astype(np.float32)
    cases = []  # (n, acc)
    n_two, n_alt = 0, 0
    for n in range(N):
        lim = int(120.0 / float(alpha[n]))
        a = np.arange(-lim, lim + 1, dtype=np.int64)
        a32 = a.astype(np.float32)
        fused = (a32.astype(np.float64) * np.float64(alpha[n]) + np.float64(beta[n])).astype(np.float32)
        two = ((a32 * alpha[n]).astype(np.float32) + beta[n]).astype(np.float32)
        alt = (a32.astype(np.float64) * np.float64(alpha_alt[n]) + np.float64(beta[n])).astype(np.float32)
        pick_two = np.nonzero(np.rint(fused) != np.rint(two))[0]
        pick_alt = np.nonzero(np.rint(fused) != np.rint(alt))[0]
        n_two += pick_two.size
        n_alt += pick_alt.size
        for i in np.concatenate([pick_two[:2], pick_alt[:2]]):
            cases.append((n, int(a[i])))
    assert n_two >= 8 and n_alt >= 4, (n_two, n_alt)  # the scan found cases that tell the readings apart
    acc = np.zeros((len(cases), N), np.int32)
    for r, (n, v) in enumerate(cases):
        acc[r, n] = v
    got = oracle.epilogue_i8(acc, float(x_scale), w_scale, bias, float(y_scale))
    for r, (n, v) in enumerate(cases):
        y = _round_to_f32(Fraction(v) * Fraction(float(alpha[n])) + Fraction(float(beta[n])))
        assert int(got[r, n]) == min(127, max(-128, round(Fraction(float(y))))), (n, v)
