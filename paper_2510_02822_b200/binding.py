"""ctypes binding of libflexiq.so: argument marshalling only.

Every function named ``flexiq_*`` here forwards to the C entry point of the same name
(see ``include/flexiq.h``); ``Layer`` is a small convenience wrapper that owns a handle
and allocates the slabs with torch.  Nothing here computes: every step of the path runs
in the CUDA kernels of the library.
"""
from __future__ import annotations

import ctypes as C
import os

_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_DIR, "libflexiq.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT = 0, -1, -2, -3, -4
DTYPE_F32, DTYPE_F16, DTYPE_BF16, DTYPE_I8 = 0, 1, 2, 3
OUT_ACC_I32, OUT_REQUANT_I8, OUT_DEQUANT_F32 = 0, 1, 2
OUT_DEQUANT_F16, OUT_DEQUANT_BF16 = 4, 5
LOWBIT_MASKED_I8, LOWBIT_PACKED_U4 = 0, 1
ORDER_ORIGINAL, ORDER_NEXT_SLAB = 0, 1
REORDER_TO_SLAB, REORDER_FROM_SLAB = 0, 1

EXPORTS = [
    "flexiq_layer_create_linear", "flexiq_layer_create_conv", "flexiq_layer_destroy",
    "flexiq_layer_set_group_perm", "flexiq_layer_set_lowbit_path", "flexiq_layer_sync_ratio", "flexiq_layer_set_slab_check", "flexiq_set_lowbit_ratio", "flexiq_get_max_4bit_ch",
    "flexiq_x4_pitch", "flexiq_quantize_lower", "flexiq_quantize_lower_dynamic_noalloc", "flexiq_mixed_gemm", "flexiq_mixed_conv",
    "flexiq_mixed_gemm_to_slab", "flexiq_mixed_conv_to_slab", "flexiq_reorder_channels",
    "flexiq_calib_channel_ranges", "flexiq_calib_channel_histogram", "flexiq_calib_ranges_from_histogram",
    "flexiq_calib_weight_absmax", "flexiq_calib_prepare", "flexiq_calib_absmax_ema",
    "flexiq_controller_create", "flexiq_controller_destroy", "flexiq_controller_level", "flexiq_controller_update",
    "flexiq_serving_simulate", "flexiq_evo_init", "flexiq_evo_next_generation", "flexiq_sq_distance_i8",
    "flexiq_layer_export", "flexiq_selftest_wait_expiry", "flexiq_force_tile", "flexiq_choose_tile", "flexiq_check_status", "flexiq_last_error",
]

_lib = None


class FlexiqError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"flexiq error {code}: {msg}")
        self.code = code


def lib():
    """Loads the CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with __graft_entry__.build() "
                "(python -m paper_2510_02822_b200.build); there is no CPU fallback")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, f32 = C.c_void_p, C.c_int, C.c_int64, C.c_float
        L.flexiq_last_error.restype = C.c_char_p
        L.flexiq_layer_create_linear.argtypes = [C.POINTER(vp), i32, i32, i32, vp, vp, vp, vp, vp, vp]
        L.flexiq_layer_create_conv.argtypes = [C.POINTER(vp), i32, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        L.flexiq_layer_destroy.argtypes = [vp]
        L.flexiq_layer_set_lowbit_path.argtypes = [vp, i32]
        L.flexiq_layer_sync_ratio.argtypes = [vp, vp]
        L.flexiq_layer_set_slab_check.argtypes = [vp, i32]
        L.flexiq_layer_set_group_perm.argtypes = [vp, vp, vp, vp, vp]
        L.flexiq_set_lowbit_ratio.argtypes = [vp, f32]
        L.flexiq_get_max_4bit_ch.argtypes = [vp, C.POINTER(i32)]
        L.flexiq_x4_pitch.argtypes = [vp, i32, C.POINTER(i64)]
        L.flexiq_quantize_lower.argtypes = [vp, vp, i32, i64, f32, i32, vp, vp, vp, vp, vp]
        L.flexiq_quantize_lower_dynamic_noalloc.argtypes = [vp, vp, i32, i64, f32, vp, vp, vp, vp]
        L.flexiq_mixed_gemm.argtypes = [vp, vp, vp, vp, i64, f32, f32, i32, vp, vp]
        L.flexiq_mixed_conv.argtypes = [vp, vp, vp, vp, i32, i32, i32, f32, f32, i32, vp, vp]
        L.flexiq_mixed_gemm_to_slab.argtypes = [vp, vp, vp, vp, i64, f32, vp, f32, i32, i32, vp, vp]
        L.flexiq_mixed_conv_to_slab.argtypes = [vp, vp, vp, vp, i32, i32, i32, f32, vp, f32, i32, i32, vp, vp]
        L.flexiq_reorder_channels.argtypes = [vp, vp, i32, i64, i32, vp, vp]
        L.flexiq_calib_channel_ranges.argtypes = [vp, i32, i64, i32, f32, i32, vp, vp, vp]
        L.flexiq_calib_channel_histogram.argtypes = [vp, i32, i64, i32, f32, i32, vp, vp]
        L.flexiq_calib_ranges_from_histogram.argtypes = [vp, i32, i64, vp, vp, vp]
        L.flexiq_calib_weight_absmax.argtypes = [vp, i32, i32, i32, i32, vp, vp]
        L.flexiq_calib_prepare.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, vp, vp]
        L.flexiq_calib_absmax_ema.argtypes = [vp, i32, i64, f32, vp, vp]
        L.flexiq_layer_export.argtypes = [vp, vp, vp, vp]
        L.flexiq_check_status.argtypes = [vp]
        L.flexiq_selftest_wait_expiry.argtypes = [vp, vp]
        f64 = C.c_double
        L.flexiq_controller_create.argtypes = [C.POINTER(vp), i32, i32, vp, vp, f64, f64, i32]
        L.flexiq_controller_destroy.argtypes = [vp]
        L.flexiq_controller_level.argtypes = [vp, C.POINTER(i32)]
        L.flexiq_controller_update.argtypes = [vp, f64, C.POINTER(i32)]
        L.flexiq_serving_simulate.argtypes = [vp, i32, i64, vp, i32, i32, vp, vp, vp]
        u64 = C.c_uint64
        L.flexiq_evo_init.argtypes = [i32, vp, vp, vp, vp, i32, u64, vp, C.POINTER(i64)]
        L.flexiq_evo_next_generation.argtypes = [i32, vp, vp, vp, i64, i32, i32, i32, i32, u64, i32, vp, vp, vp]
        L.flexiq_sq_distance_i8.argtypes = [vp, vp, i64, vp, vp]
        _lib = L
    return _lib


def last_error() -> str:
    return lib().flexiq_last_error().decode()


def _check(rc: int):
    if rc != OK:
        raise FlexiqError(rc, last_error())


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


_raw_stream = None


def _stream():
    """The current CUDA stream of the current device as a void*.  torch's raw-stream accessor is
    an order of magnitude cheaper than building a Stream object per call; fall back if absent."""
    global _raw_stream
    import torch
    if _raw_stream is None:
        _raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", False)
    if _raw_stream:
        return C.c_void_p(_raw_stream(torch.cuda.current_device()))
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


# ---- one function per C entry point ------------------------------------------------
def flexiq_layer_create_linear(K, N, G, Wq_dev, w_scale_dev, bias_dev, perm_host, x_shift_host):
    h = C.c_void_p()
    _check(lib().flexiq_layer_create_linear(C.byref(h), K, N, G, _ptr(Wq_dev), _ptr(w_scale_dev), _ptr(bias_dev),
                                            perm_host.ctypes.data_as(C.c_void_p),
                                            None if x_shift_host is None else x_shift_host.ctypes.data_as(C.c_void_p),
                                            _stream()))
    return h


def flexiq_layer_create_conv(Cin, Cout, R, S, stride, pad, G, Wq_dev, w_scale_dev, bias_dev, perm_host, x_shift_host):
    h = C.c_void_p()
    _check(lib().flexiq_layer_create_conv(C.byref(h), Cin, Cout, R, S, stride, pad, G, _ptr(Wq_dev), _ptr(w_scale_dev),
                                          _ptr(bias_dev), perm_host.ctypes.data_as(C.c_void_p),
                                          None if x_shift_host is None else x_shift_host.ctypes.data_as(C.c_void_p),
                                          _stream()))
    return h


def flexiq_layer_destroy(h):
    _check(lib().flexiq_layer_destroy(h))


def flexiq_layer_set_lowbit_path(h, path):
    _check(lib().flexiq_layer_set_lowbit_path(h, path))


def flexiq_layer_set_slab_check(h, enabled):
    _check(lib().flexiq_layer_set_slab_check(h, int(bool(enabled))))


def flexiq_set_lowbit_ratio(h, ratio):
    _check(lib().flexiq_set_lowbit_ratio(h, ratio))


def flexiq_get_max_4bit_ch(h) -> int:
    v = C.c_int()
    _check(lib().flexiq_get_max_4bit_ch(h, C.byref(v)))
    return v.value


def flexiq_x4_pitch(h, K_lo) -> int:
    v = C.c_int64()
    _check(lib().flexiq_x4_pitch(h, K_lo, C.byref(v)))
    return v.value


def flexiq_quantize_lower(h, X_dev, x_dtype, M, x_scale, dynamic_pos, X4_dev, X8_dev, x_shift_out_dev=None,
                          scratch_dev=None):
    _check(lib().flexiq_quantize_lower(h, _ptr(X_dev), x_dtype, M, x_scale, int(dynamic_pos), _ptr(X4_dev), _ptr(X8_dev),
                                       _ptr(x_shift_out_dev), _ptr(scratch_dev), _stream()))


def flexiq_quantize_lower_dynamic_noalloc(h, X_dev, x_dtype, M, x_scale, X4_dev, X8_dev, x_shift_out_dev):
    """Dynamic-position prologue that allocates nothing: its scratch is a fixed array inside the
    library (at most 4096 channel groups; calls on one device must not overlap)."""
    _check(lib().flexiq_quantize_lower_dynamic_noalloc(h, _ptr(X_dev), x_dtype, M, x_scale, _ptr(X4_dev), _ptr(X8_dev),
                                                       _ptr(x_shift_out_dev), _stream()))


def flexiq_mixed_gemm(h, X4_dev, X8_dev, x_shift_dev, M, x_scale, y_scale, out_mode, Y_dev):
    _check(lib().flexiq_mixed_gemm(h, _ptr(X4_dev), _ptr(X8_dev), _ptr(x_shift_dev), M, x_scale, y_scale, out_mode,
                                   _ptr(Y_dev), _stream()))


def flexiq_mixed_conv(h, X4_dev, X8_dev, x_shift_dev, Nb, H, W, x_scale, y_scale, out_mode, Y_dev):
    _check(lib().flexiq_mixed_conv(h, _ptr(X4_dev), _ptr(X8_dev), _ptr(x_shift_dev), Nb, H, W, x_scale, y_scale,
                                   out_mode, _ptr(Y_dev), _stream()))


def flexiq_mixed_gemm_to_slab(h, X4_dev, X8_dev, x_shift_dev, M, x_scale, next_h, next_x_scale, relu, out_order, next_X4_dev):
    _check(lib().flexiq_mixed_gemm_to_slab(h, _ptr(X4_dev), _ptr(X8_dev), _ptr(x_shift_dev), M, x_scale, next_h,
                                           next_x_scale, int(relu), out_order, _ptr(next_X4_dev), _stream()))


def flexiq_mixed_conv_to_slab(h, X4_dev, X8_dev, x_shift_dev, Nb, H, W, x_scale, next_h, next_x_scale, relu, out_order, next_X4_dev):
    _check(lib().flexiq_mixed_conv_to_slab(h, _ptr(X4_dev), _ptr(X8_dev), _ptr(x_shift_dev), Nb, H, W, x_scale, next_h,
                                           next_x_scale, int(relu), out_order, _ptr(next_X4_dev), _stream()))


def flexiq_reorder_channels(h, X_dev, elem_bytes, M, direction, Y_dev):
    _check(lib().flexiq_reorder_channels(h, _ptr(X_dev), elem_bytes, M, direction, _ptr(Y_dev), _stream()))


def flexiq_calib_channel_ranges(X_dev, x_dtype, M, K, x_scale, accumulate, lo_dev, hi_dev):
    _check(lib().flexiq_calib_channel_ranges(_ptr(X_dev), x_dtype, M, K, x_scale, int(accumulate), _ptr(lo_dev), _ptr(hi_dev), _stream()))


def flexiq_calib_channel_histogram(X_dev, x_dtype, M, K, x_scale, accumulate, hist_dev):
    _check(lib().flexiq_calib_channel_histogram(_ptr(X_dev), x_dtype, M, K, x_scale, int(accumulate), _ptr(hist_dev), _stream()))


def flexiq_calib_ranges_from_histogram(hist_dev, K, tail, lo_dev, hi_dev):
    _check(lib().flexiq_calib_ranges_from_histogram(_ptr(hist_dev), K, int(tail), _ptr(lo_dev), _ptr(hi_dev), _stream()))


def flexiq_calib_weight_absmax(Wq_dev, is_conv, K, N, taps, wmax_dev):
    _check(lib().flexiq_calib_weight_absmax(_ptr(Wq_dev), int(is_conv), K, N, taps, _ptr(wmax_dev), _stream()))


def flexiq_calib_prepare(lo_dev, hi_dev, wmax_dev, K, G, perm_dev, x_shift_dev, score_dev, hist_dev):
    _check(lib().flexiq_calib_prepare(_ptr(lo_dev), _ptr(hi_dev), _ptr(wmax_dev), K, G, _ptr(perm_dev), _ptr(x_shift_dev),
                                      _ptr(score_dev), _ptr(hist_dev), _stream()))


def flexiq_calib_absmax_ema(X_dev, x_dtype, count, momentum, state_dev):
    _check(lib().flexiq_calib_absmax_ema(_ptr(X_dev), x_dtype, count, momentum, _ptr(state_dev), _stream()))


def flexiq_layer_export(h, sw_host=None, w8_host=None, w4_host=None):
    def hp(a):
        return None if a is None else a.ctypes.data_as(C.c_void_p)
    _check(lib().flexiq_layer_export(h, hp(sw_host), hp(w8_host), hp(w4_host)))


def flexiq_force_tile(cta_group, tile_n):
    _check(lib().flexiq_force_tile(cta_group, tile_n))


def flexiq_choose_tile(M, N, k_blocks, block_k=128, sm_count=148):
    """(CTAs per tile, tile width) of the automatic choice; host-only."""
    cg, bn = C.c_int(0), C.c_int(0)
    _check(lib().flexiq_choose_tile(C.c_int64(M), N, k_blocks, block_k, sm_count, C.byref(cg), C.byref(bn)))
    return cg.value, bn.value


def flexiq_selftest_wait_expiry(result_dev):
    _check(lib().flexiq_selftest_wait_expiry(_ptr(result_dev), _stream()))


def flexiq_check_status():
    _check(lib().flexiq_check_status(_stream()))


# ---- convenience wrapper ------------------------------------------------------------
_TORCH_DTYPE = {}


def _dtype_code(t):
    import torch
    if not _TORCH_DTYPE:
        _TORCH_DTYPE.update({torch.float32: DTYPE_F32, torch.float16: DTYPE_F16, torch.bfloat16: DTYPE_BF16,
                             torch.int8: DTYPE_I8})
    return _TORCH_DTYPE[t.dtype]


class Layer:
    """Owns one flexiq layer handle plus reusable slab buffers (torch device memory)."""

    def __init__(self, Wq, w_scale, bias, perm, x_shift, G=16, conv=None):
        import numpy as np
        self.G = G
        self.conv = conv  # None or (stride, pad)
        perm = np.ascontiguousarray(perm, np.int32)
        x_shift = None if x_shift is None else np.ascontiguousarray(x_shift, np.uint8)
        if conv is None:
            self.K, self.N = Wq.shape
            self.h = flexiq_layer_create_linear(self.K, self.N, G, Wq, w_scale, bias, perm, x_shift)
        else:
            self.N, self.R, self.S, self.K = Wq.shape
            self.h = flexiq_layer_create_conv(self.K, self.N, self.R, self.S, conv[0], conv[1], G, Wq, w_scale, bias,
                                              perm, x_shift)
        self.device = Wq.device
        self._slabs = {}

    def close(self):
        if self.h is not None:
            flexiq_layer_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_lowbit_path(self, path):
        flexiq_layer_set_lowbit_path(self.h, path)

    def set_lowbit_ratio(self, ratio):
        flexiq_set_lowbit_ratio(self.h, ratio)

    def set_group_perm(self, Wq, group_perm, x_shift=None):
        """Layout post-processing again for another group order (no allocation, stream-ordered)."""
        import numpy as np
        perm = np.ascontiguousarray(group_perm, dtype=np.int32)
        xs = None if x_shift is None else np.ascontiguousarray(x_shift, dtype=np.uint8)
        _check(lib().flexiq_layer_set_group_perm(self.h, _ptr(Wq), _np_ptr(perm), None if xs is None else _np_ptr(xs), _stream()))

    def sync_ratio(self):
        """Writes the ratio-dependent weight K block for the ratio in force on the current stream, if it is not there yet."""
        _check(lib().flexiq_layer_sync_ratio(self.h, _stream()))

    @property
    def K_lo(self):
        return flexiq_get_max_4bit_ch(self.h)

    def alloc_slabs(self, M):
        """Slab buffers sized for any ratio (allocated once per M, reused)."""
        import torch
        if M not in self._slabs:
            x4 = torch.empty(max(M, 1) * self.K + 16, dtype=torch.uint8, device=self.device)
            x8 = torch.empty(max(M, 1) * self.K + 16, dtype=torch.int8, device=self.device)
            self._slabs[M] = (x4, x8)
        return self._slabs[M]

    def quantize_lower(self, X, x_scale, dynamic=False, slabs=None):
        import torch
        M = X.numel() // self.K
        x4, x8 = slabs if slabs is not None else self.alloc_slabs(M)
        shifts = scratch = None
        if dynamic:
            shifts = torch.empty(self.K // self.G, dtype=torch.uint8, device=self.device)
            scratch = torch.empty(self.K // self.G, dtype=torch.int32, device=self.device)
        flexiq_quantize_lower(self.h, X, _dtype_code(X), M, x_scale, dynamic, x4, x8, shifts, scratch)
        return x4, x8, shifts

    def mixed_gemm(self, x4, x8, M, x_scale, y_scale, out_mode, Y=None, x_shift=None):
        import torch
        if Y is None:
            dt = {OUT_ACC_I32: torch.int32, OUT_REQUANT_I8: torch.int8, OUT_DEQUANT_F32: torch.float32,
                  OUT_DEQUANT_F16: torch.float16, OUT_DEQUANT_BF16: torch.bfloat16}[out_mode]
            Y = torch.empty((M, self.N), dtype=dt, device=self.device)
        flexiq_mixed_gemm(self.h, x4, x8, x_shift, M, x_scale, y_scale, out_mode, Y)
        return Y

    def reorder_channels(self, X, direction=REORDER_TO_SLAB, Y=None):
        """Residual-branch reorder of a [..., K] tensor between original and slab channel order."""
        import torch
        if Y is None:
            Y = torch.empty_like(X)
        flexiq_reorder_channels(self.h, X, X.element_size(), X.numel() // self.K, direction, Y)
        return Y

    def mixed_gemm_to_slab(self, x4, x8, M, x_scale, nxt, next_x_scale, relu=False, slab=None, x_shift=None, out_order=ORDER_ORIGINAL):
        """Mixed GEMM whose epilogue writes the masked slab of the layer `nxt` (fused layer boundary)."""
        if slab is None:
            slab = nxt.alloc_slabs(M)[0]
        flexiq_mixed_gemm_to_slab(self.h, x4, x8, x_shift, M, x_scale, nxt.h, next_x_scale, relu, out_order, slab)
        return slab

    def mixed_conv_to_slab(self, x4, x8, Nb, H, W, x_scale, nxt, next_x_scale, relu=False, slab=None, x_shift=None, out_order=ORDER_ORIGINAL):
        stride, pad = self.conv
        P = (H + 2 * pad - self.R) // stride + 1
        Q = (W + 2 * pad - self.S) // stride + 1
        if slab is None:
            slab = nxt.alloc_slabs(Nb * P * Q)[0]
        flexiq_mixed_conv_to_slab(self.h, x4, x8, x_shift, Nb, H, W, x_scale, nxt.h, next_x_scale, relu, out_order, slab)
        return slab

    def mixed_conv(self, x4, x8, Nb, H, W, x_scale, y_scale, out_mode, Y=None, x_shift=None):
        import torch
        stride, pad = self.conv
        P = (H + 2 * pad - self.R) // stride + 1
        Q = (W + 2 * pad - self.S) // stride + 1
        if Y is None:
            dt = {OUT_ACC_I32: torch.int32, OUT_REQUANT_I8: torch.int8, OUT_DEQUANT_F32: torch.float32,
                  OUT_DEQUANT_F16: torch.float16, OUT_DEQUANT_BF16: torch.bfloat16}[out_mode]
            Y = torch.empty((Nb, P, Q, self.N), dtype=dt, device=self.device)
        flexiq_mixed_conv(self.h, x4, x8, x_shift, Nb, H, W, x_scale, y_scale, out_mode, Y)
        return Y


# ------------------------------------------------------------------ ratio controller and request queue (host only)
def _np_ptr(a):
    return C.c_void_p(a.ctypes.data)


class Controller:
    """Run-time ratio controller (flexiq_controller_*): levels are the ratios l / (n_levels - 1)."""

    def __init__(self, rate_grid, latency, threshold, window_s, initial_level=0):
        import numpy as np
        self.rate_grid = np.ascontiguousarray(rate_grid, dtype=np.float64)
        self.latency = np.ascontiguousarray(latency, dtype=np.float64)
        if self.latency.ndim != 2 or self.latency.shape[1] != self.rate_grid.size:
            raise ValueError("latency must be [n_levels][n_rates]")
        self.n_levels = self.latency.shape[0]
        h = C.c_void_p()
        _check(lib().flexiq_controller_create(C.byref(h), self.n_levels, self.rate_grid.size, _np_ptr(self.rate_grid),
                                              _np_ptr(self.latency), float(threshold), float(window_s), int(initial_level)))
        self.h = h

    @property
    def level(self) -> int:
        v = C.c_int()
        _check(lib().flexiq_controller_level(self.h, C.byref(v)))
        return v.value

    def update(self, rate: float) -> int:
        v = C.c_int()
        _check(lib().flexiq_controller_update(self.h, float(rate), C.byref(v)))
        return v.value

    def ratio(self) -> float:
        return self.level / max(1, self.n_levels - 1)

    def close(self):
        if self.h is not None and self.h.value:
            _check(lib().flexiq_controller_destroy(self.h))
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def flexiq_serving_simulate(ctrl, fixed_level, arrival, service, max_batch):
    """Request queue in virtual time; returns (response seconds [n], level [n])."""
    import numpy as np
    arrival = np.ascontiguousarray(arrival, dtype=np.float64)
    service = np.ascontiguousarray(service, dtype=np.float64)
    if service.ndim != 2 or service.shape[1] != max_batch:
        raise ValueError("service must be [n_levels][max_batch]")
    response = np.zeros(arrival.size, dtype=np.float64)
    level = np.zeros(arrival.size, dtype=np.int32)
    _check(lib().flexiq_serving_simulate(ctrl.h if ctrl is not None else None, int(fixed_level), arrival.size, _np_ptr(arrival),
                                         service.shape[0], int(max_batch), _np_ptr(service), _np_ptr(response), _np_ptr(level)))
    return response, level


# ------------------------------------------------------------------ evolutionary selection (Sec. 4.2, Algorithm 1)
def _evo_args(groups, score, locked):
    import numpy as np
    groups = np.ascontiguousarray(groups, dtype=np.int32)
    score = np.ascontiguousarray(score, dtype=np.int64)
    if score.size != int(groups.sum()):
        raise ValueError("score must hold one value per group of every layer")
    if locked is not None:
        locked = np.ascontiguousarray(locked, dtype=np.uint8)
        if locked.size != score.size:
            raise ValueError("locked must hold one flag per group")
    return groups, score, locked


def flexiq_evo_init(groups, score, per_layer_target, N, seed, locked=None):
    """Seed population [N][total] uint8 and the number of set flags every chromosome holds."""
    import numpy as np
    groups, score, locked = _evo_args(groups, score, locked)
    tgt = np.ascontiguousarray(per_layer_target, dtype=np.int32)
    if tgt.size != groups.size:
        raise ValueError("per_layer_target must hold one value per layer")
    pop = np.zeros((int(N), score.size), dtype=np.uint8)
    target = C.c_int64()
    _check(lib().flexiq_evo_init(groups.size, _np_ptr(groups), _np_ptr(score), None if locked is None else _np_ptr(locked),
                                 _np_ptr(tgt), int(N), int(seed), _np_ptr(pop), C.byref(target)))
    return pop, target.value


def flexiq_evo_next_generation(pop, distance, groups, score, target, k, r, mutation_bp, seed, generation, locked=None):
    import numpy as np
    groups, score, locked = _evo_args(groups, score, locked)
    pop = np.ascontiguousarray(pop, dtype=np.uint8)
    distance = np.ascontiguousarray(distance, dtype=np.int64)
    if pop.ndim != 2 or pop.shape[1] != score.size or distance.size != pop.shape[0]:
        raise ValueError("pop must be [N][total] and distance [N]")
    nxt = np.zeros_like(pop)
    _check(lib().flexiq_evo_next_generation(groups.size, _np_ptr(groups), _np_ptr(score), None if locked is None else _np_ptr(locked),
                                            int(target), pop.shape[0], int(k), int(r), int(mutation_bp), int(seed), int(generation),
                                            _np_ptr(distance), _np_ptr(pop), _np_ptr(nxt)))
    return nxt


def flexiq_sq_distance_i8(A, B, out):
    """out (int64 device tensor, one element) = sum (A - B)^2 over two int8 device tensors."""
    if A.numel() != B.numel():
        raise ValueError("A and B differ in size")
    _check(lib().flexiq_sq_distance_i8(_ptr(A), _ptr(B), A.numel(), _ptr(out), _stream()))
