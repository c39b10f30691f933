"""FlexiQ CPU oracle (numpy front end of ``flexiq_oracle.c``).

TEST INFRASTRUCTURE, NOT A PRODUCT PATH: only the tests, the smoke check and the
CPU-baseline leg of the benchmark import this package.  It shares nothing with the
CUDA library and never imports it.

Every function here only marshals numpy arrays into the C routine of the same name;
the arithmetic, and the citation of the passage of the paper it follows, live in the
C file.  ``build()`` compiles the C file with gcc (building the checker is not using it).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "flexiq_oracle.c")
_LIB = os.path.join(_DIR, "libflexiq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc; strict IEEE flags so fp32 steps round once."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fno-fast-math", "-ffp-contract=off",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.fqo_quantize_one.restype = C.c_int8
        _lib.fqo_quantize_one.argtypes = [C.c_float, C.c_float]
        _lib.fqo_n_low.argtypes = [C.c_double, C.c_int]
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def max_threads() -> int:
    return int(lib().fqo_max_threads())


def quantize(x, S: float) -> np.ndarray:
    x = _c(x, np.float32)
    q = np.empty(x.shape, np.int8)
    lib().fqo_quantize_f32(_p(x), C.c_int64(x.size), C.c_float(S), _p(q))
    return q


def bitlen(v: int) -> int:
    return int(lib().fqo_bitlen(C.c_int(v)))


def position_from_range(lo: int, hi: int) -> int:
    return int(lib().fqo_position_from_range(C.c_int(lo), C.c_int(hi)))


def lower(q: int, s: int) -> int:
    return int(lib().fqo_lower(C.c_int(q), C.c_int(s)))


def n_low(ratio: float, n_groups: int) -> int:
    return int(lib().fqo_n_low(float(np.float32(ratio)), n_groups))


def channel_ranges(qcal):
    qcal = _c(qcal, np.int8)
    Mc, K = qcal.shape
    lo = np.empty(K, np.int32)
    hi = np.empty(K, np.int32)
    lib().fqo_channel_ranges(_p(qcal), C.c_int64(Mc), K, _p(lo), _p(hi))
    return lo, hi


def static_positions(lo, hi, G: int) -> np.ndarray:
    lo = _c(lo, np.int32)
    hi = _c(hi, np.int32)
    K = lo.size
    sx = np.empty(K // G, np.uint8)
    lib().fqo_static_positions(_p(lo), _p(hi), K, G, _p(sx))
    return sx


def weight_absmax_linear(Wq) -> np.ndarray:
    Wq = _c(Wq, np.int8)
    K, N = Wq.shape
    out = np.empty(K, np.int32)
    lib().fqo_weight_absmax_linear(_p(Wq), K, N, _p(out))
    return out


def weight_absmax_conv(Wq) -> np.ndarray:
    Wq = _c(Wq, np.int8)
    Cout, R, S, Cin = Wq.shape
    out = np.empty(Cin, np.int32)
    lib().fqo_weight_absmax_conv(_p(Wq), Cout, R, S, Cin, _p(out))
    return out


def greedy_order(lo, hi, wabs_max, G: int):
    lo = _c(lo, np.int32)
    hi = _c(hi, np.int32)
    wabs_max = _c(wabs_max, np.int32)
    K = lo.size
    score = np.empty(K // G, np.int64)
    perm = np.empty(K // G, np.int32)
    lib().fqo_greedy_order(_p(lo), _p(hi), _p(wabs_max), K, G, _p(score), _p(perm))
    return perm, score


def weight_positions_linear(Wq, G: int, perm) -> np.ndarray:
    Wq = _c(Wq, np.int8)
    perm = _c(perm, np.int32)
    K, N = Wq.shape
    sw = np.empty((K // G, N), np.uint8)
    lib().fqo_weight_positions_linear(_p(Wq), K, N, G, _p(perm), _p(sw))
    return sw


def weight_positions_conv(Wq, G: int, perm) -> np.ndarray:
    Wq = _c(Wq, np.int8)
    perm = _c(perm, np.int32)
    Cout, R, S, Cin = Wq.shape
    sw = np.empty((Cin // G, Cout), np.uint8)
    lib().fqo_weight_positions_conv(_p(Wq), Cout, R, S, Cin, G, _p(perm), _p(sw))
    return sw


def dynamic_positions(q, G: int, perm) -> np.ndarray:
    q = _c(q, np.int8)
    q2 = q.reshape(-1, q.shape[-1])
    perm = _c(perm, np.int32)
    M, K = q2.shape
    sx = np.empty(K // G, np.uint8)
    lib().fqo_dynamic_positions(_p(q2), C.c_int64(M), K, G, _p(perm), _p(sx))
    return sx


def x4_pitch(K_lo: int) -> int:
    """Row pitch in bytes of the packed low-bit slab: K_lo/2 rounded up to 16."""
    return ((K_lo // 2 + 15) // 16) * 16


def make_slabs(q, G: int, perm, sx_slab, n_low_groups: int):
    q = _c(q, np.int8)
    q2 = q.reshape(-1, q.shape[-1])
    perm = _c(perm, np.int32)
    sx_slab = _c(sx_slab, np.uint8)
    M, K = q2.shape
    K_lo = n_low_groups * G
    pitch = x4_pitch(K_lo)
    X4 = np.zeros((M, pitch), np.uint8)
    X8 = np.empty((M, K - K_lo), np.int8)
    lib().fqo_make_slabs(_p(q2), C.c_int64(M), K, G, _p(perm), _p(sx_slab), n_low_groups,
                         _p(X4), C.c_int64(pitch), _p(X8))
    return X4, X8


def mixed_gemm_acc(Xq, Wq, G: int, perm, sx_slab, sw, n_low_groups: int, rows=None) -> np.ndarray:
    Xq = _c(Xq, np.int8)
    Wq = _c(Wq, np.int8)
    perm = _c(perm, np.int32)
    sx_slab = _c(sx_slab, np.uint8)
    sw = _c(sw, np.uint8)
    M, K = Xq.shape
    K2, N = Wq.shape
    assert K == K2 and sw.shape == (K // G, N)
    if rows is None:
        acc = np.empty((M, N), np.int32)
        st = lib().fqo_mixed_gemm_acc(_p(Xq), _p(Wq), C.c_int64(M), K, N, G, _p(perm), _p(sx_slab),
                                      _p(sw), n_low_groups, _p(acc))
    else:
        rows = _c(rows, np.int64)
        acc = np.empty((rows.size, N), np.int32)
        st = lib().fqo_mixed_gemm_acc_rows(_p(Xq), _p(Wq), _p(rows), C.c_int64(rows.size), K, N, G,
                                           _p(perm), _p(sx_slab), _p(sw), n_low_groups, _p(acc))
    if st != 0:
        raise OverflowError(f"oracle status {st}")
    return acc


def mixed_conv_acc(Xq, Wq, stride: int, pad: int, G: int, perm, sx_slab, sw,
                   n_low_groups: int) -> np.ndarray:
    Xq = _c(Xq, np.int8)
    Wq = _c(Wq, np.int8)
    perm = _c(perm, np.int32)
    sx_slab = _c(sx_slab, np.uint8)
    sw = _c(sw, np.uint8)
    Nb, H, W, Cin = Xq.shape
    Cout, R, S, Cin2 = Wq.shape
    assert Cin == Cin2
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    acc = np.empty((Nb, P, Q, Cout), np.int32)
    st = lib().fqo_mixed_conv_acc(_p(Xq), _p(Wq), Nb, H, W, Cin, Cout, R, S, stride, pad, G,
                                  _p(perm), _p(sx_slab), _p(sw), n_low_groups, _p(acc))
    if st != 0:
        raise OverflowError(f"oracle status {st}")
    return acc


def epilogue_i8(acc, x_scale, w_scale, bias, y_scale) -> np.ndarray:
    acc = _c(acc, np.int32)
    N = acc.shape[-1]
    a2 = acc.reshape(-1, N)
    w_scale = _c(w_scale, np.float32)
    b = None if bias is None else _c(bias, np.float32)
    out = np.empty(a2.shape, np.int8)
    lib().fqo_epilogue_i8(_p(a2), C.c_int64(a2.shape[0]), N, C.c_float(x_scale), _p(w_scale),
                          _p(b) if b is not None else None, C.c_float(y_scale), _p(out))
    return out.reshape(acc.shape)


def epilogue_f32(acc, x_scale, w_scale, bias) -> np.ndarray:
    acc = _c(acc, np.int32)
    N = acc.shape[-1]
    a2 = acc.reshape(-1, N)
    w_scale = _c(w_scale, np.float32)
    b = None if bias is None else _c(bias, np.float32)
    out = np.empty(a2.shape, np.float32)
    lib().fqo_epilogue_f32(_p(a2), C.c_int64(a2.shape[0]), N, C.c_float(x_scale), _p(w_scale),
                           _p(b) if b is not None else None, _p(out))
    return out.reshape(acc.shape)


def epilogue_f16(acc, x_scale, w_scale, bias) -> np.ndarray:
    """16-bit floating-point output (the operators between the quantized layers run in fp16): the fp32
    epilogue value rounded once more to fp16, to nearest even (numpy's float32 -> float16 conversion)."""
    return epilogue_f32(acc, x_scale, w_scale, bias).astype(np.float16)


def epilogue_bf16_bits(acc, x_scale, w_scale, bias) -> np.ndarray:
    """The same for bfloat16, returned as the 16-bit patterns (numpy has no bfloat16): the upper half of
    the fp32 pattern after adding half an ulp of the kept part, ties to the even pattern (finite values)."""
    u = epilogue_f32(acc, x_scale, w_scale, bias).view(np.uint32).astype(np.uint64)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def reorder_channels(x, G: int, perm, to_slab: bool = True) -> np.ndarray:
    x = np.ascontiguousarray(x)
    K = x.shape[-1]
    perm = _c(perm, np.int32)
    y = np.empty_like(x)
    lib().fqo_reorder_channels(_p(x), C.c_int64(x.size // K), K, G, x.itemsize, _p(perm), int(bool(to_slab)), _p(y))
    return y


def unused_bits_histogram(lo, hi) -> np.ndarray:
    lo = _c(lo, np.int32)
    hi = _c(hi, np.int32)
    hist = np.zeros(5, np.int32)
    lib().fqo_unused_bits_histogram(_p(lo), _p(hi), lo.size, _p(hist))
    return hist


def absmax_ema(x_batches, momentum: float) -> float:
    x = _c(x_batches, np.float32)
    b = x.shape[0]
    f = lib().fqo_absmax_ema
    f.restype = C.c_float
    return float(f(_p(x), C.c_int64(b), C.c_int64(x.size // b), C.c_float(momentum)))


def channel_histogram(q) -> np.ndarray:
    q = _c(q, np.int8)
    M, K = q.shape
    hist = np.empty((K, 256), np.uint32)
    lib().fqo_channel_histogram(_p(q), C.c_int64(M), K, _p(hist))
    return hist


def ranges_from_histogram(hist, tail: int):
    hist = _c(hist, np.uint32)
    K = hist.shape[0]
    lo = np.empty(K, np.int32)
    hi = np.empty(K, np.int32)
    lib().fqo_ranges_from_histogram(_p(hist), K, C.c_int64(tail), _p(lo), _p(hi))
    return lo, hi
