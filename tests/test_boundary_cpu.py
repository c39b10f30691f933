"""CPU-only checks of the boundary and the host logic: the C-ABI library loads, exports
every symbol the header declares, and rejects bad arguments before touching a device."""
import ctypes as C
import os
import re

import numpy as np
import pytest
import torch

import oracle
from paper_2510_02822_b200 import binding as fx
from paper_2510_02822_b200 import build as fxbuild
from paper_2510_02822_b200 import calib, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    fxbuild.build_library()
    return fx.lib()


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "flexiq.h")).read()
    declared = set(re.findall(r"\b(flexiq_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(fx.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_create_rejects_bad_arguments_without_a_device(lib):
    h = C.c_void_p()
    perm = np.arange(8, dtype=np.int32)
    dummy = C.c_void_p(16)  # never dereferenced: validation fails first
    pp = perm.ctypes.data_as(C.c_void_p)
    cases = [
        (dict(K=100, N=16, G=16), "multiple of group_size"),
        (dict(K=128, N=16, G=8), "group_size"),
        (dict(K=128, N=20, G=16), "multiple of 16"),
        (dict(K=0, N=16, G=16), "positive"),
    ]
    for kw, msg in cases:
        rc = lib.flexiq_layer_create_linear(C.byref(h), kw["K"], kw["N"], kw["G"], dummy, dummy, None, pp, None, None)
        assert rc == fx.ERR_INVALID_ARG and msg in fx.last_error(), (kw, fx.last_error())
    rc = lib.flexiq_layer_create_linear(C.byref(h), 128, 16, 16, None, dummy, None, pp, None, None)
    assert rc == fx.ERR_INVALID_ARG
    bad = np.array([0, 1, 2, 3, 4, 5, 6, 6], np.int32)
    rc = lib.flexiq_layer_create_linear(C.byref(h), 128, 16, 16, dummy, dummy, None, bad.ctypes.data_as(C.c_void_p), None, None)
    assert rc == fx.ERR_INVALID_ARG and "permutation" in fx.last_error()
    shifts = np.array([0, 1, 2, 3, 4, 5, 0, 0], np.uint8)
    rc = lib.flexiq_layer_create_linear(C.byref(h), 128, 16, 16, dummy, dummy, None, pp, shifts.ctypes.data_as(C.c_void_p), None)
    assert rc == fx.ERR_INVALID_ARG and "exceeds 4" in fx.last_error()
    assert lib.flexiq_layer_create_linear(None, 128, 16, 16, dummy, dummy, None, pp, None, None) == fx.ERR_INVALID_ARG


def test_calls_reject_dead_handles(lib):
    assert lib.flexiq_set_lowbit_ratio(None, 0.5) == fx.ERR_INVALID_ARG
    assert lib.flexiq_layer_destroy(None) == fx.ERR_INVALID_ARG
    assert lib.flexiq_mixed_gemm(None, None, None, None, 1, 1.0, 1.0, 0, None, None) == fx.ERR_INVALID_ARG
    assert lib.flexiq_mixed_conv(None, None, None, None, 1, 1, 1, 1.0, 1.0, 0, None, None) == fx.ERR_INVALID_ARG
    assert lib.flexiq_quantize_lower(None, None, 0, 1, 1.0, 0, None, None, None, None, None) == fx.ERR_INVALID_ARG
    assert "handle" in fx.last_error()


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(fx, "_lib", None)
    monkeypatch.setattr(fx, "LIB_PATH", "/nonexistent/libflexiq.so")
    with pytest.raises(FileNotFoundError, match="no CPU fallback"):
        fx.lib()


def test_host_calibration_matches_oracle():
    for case in (inputs.config1(), inputs.ranged_linear("g", 64, 256, 32, 32, seed=9, group_structured=True)):
        qcal = oracle.quantize(case.Xcal, case.x_scale)
        q2 = calib.quantize_reference(torch.from_numpy(case.Xcal), case.x_scale).numpy()
        assert np.array_equal(qcal, q2)
        lo, hi = oracle.channel_ranges(qcal)
        sx = oracle.static_positions(lo, hi, case.G)
        perm, _ = oracle.greedy_order(lo, hi, oracle.weight_absmax_linear(case.Wq), case.G)
        p2, s2 = calib.static_preparation(torch.from_numpy(q2), torch.from_numpy(case.Wq), case.G)
        assert np.array_equal(perm, p2) and np.array_equal(sx, s2)
    c = inputs.resnet_conv("c", 2, 6, 64, 16, 3, seed=3)
    qcal = oracle.quantize(c.Xcal, c.x_scale).reshape(-1, c.C)
    lo, hi = oracle.channel_ranges(qcal)
    perm, _ = oracle.greedy_order(lo, hi, oracle.weight_absmax_conv(c.Wq), c.G)
    p2, s2 = calib.static_preparation(torch.from_numpy(qcal), torch.from_numpy(c.Wq), c.G, conv=True)
    assert np.array_equal(perm, p2) and np.array_equal(oracle.static_positions(lo, hi, c.G), s2)


def test_inputs_are_seeded_and_shaped():
    a, b = inputs.config1(), inputs.config1()
    assert np.array_equal(a.X, b.X) and np.array_equal(a.Wq, b.Wq) and a.y_scale == b.y_scale
    assert a.X.shape == (256, 384) and a.Wq.shape == (384, 384) and a.Wq.dtype == np.int8
    u = inputs.uniform(1, 2, 1000)
    assert 0 <= u.min() and u.max() < 1 and abs(u.mean() - 0.5) < 0.05
    z = inputs.normal(1, 2, 20000)
    assert abs(z.mean()) < 0.05 and abs(z.std() - 1) < 0.05
    v = inputs.vit_linear("v", 32, 768, 64, seed=5)
    assert 20 <= v.meta["outlier_channels"] <= 60  # about 5 % of 768


def test_tile_choice_host_logic(lib):
    """The automatic tile shape (host-only hook): what the benchmark's four ViT-B layers get on 148 SMs, and
    properties that hold for every shape."""
    M = 64 * 197
    assert fx.flexiq_choose_tile(M, 2304, 6) == (2, 256)      # QKV: CTA pairs, 256 x 256
    assert fx.flexiq_choose_tile(M, 3072, 6) == (2, 256)      # fc1
    assert fx.flexiq_choose_tile(M, 768, 24) == (2, 192)      # fc2: 200 pair tiles fill three waves better than 150
    assert fx.flexiq_choose_tile(M, 768, 6) == (1, 192)       # proj
    rng = np.random.default_rng(5)
    for _ in range(300):
        m, n = int(rng.integers(1, 40000)), 16 * int(rng.integers(1, 300))
        kb, bk, sms = int(rng.integers(1, 40)), int(rng.choice([64, 128])), int(rng.choice([74, 132, 148]))
        cg, bn = fx.flexiq_choose_tile(m, n, kb, bk, sms)
        assert cg in (1, 2) and bn in (64, 128, 192, 256)
        assert not (cg == 2 and bn < 128)
        assert (cg, bn) == fx.flexiq_choose_tile(m, n, kb, bk, sms)      # a pure function of its arguments
    for bad in [(0, 64, 1, 128, 148), (5, 0, 1, 128, 148), (5, 64, 0, 128, 148), (5, 64, 1, 96, 148), (5, 64, 1, 128, 0)]:
        with pytest.raises(fx.FlexiqError):
            fx.flexiq_choose_tile(*bad)
