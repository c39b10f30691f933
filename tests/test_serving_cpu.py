"""Serving experiment (Sec. 8): the library's host-side ratio controller and request queue against
the oracle.  No GPU: these entry points do no device work."""
import math

import numpy as np
import pytest

from oracle import serving as osv
from paper_2510_02822_b200 import binding as fx
from paper_2510_02822_b200 import inputs


# ------------------------------------------------------------------ library against the oracle
def _table(n_levels, max_batch, base=0.5e-3):
    return np.array([[base * (1.0 - 0.1 * l) * (1.0 + 0.15 * (b - 1)) for b in range(1, max_batch + 1)] for l in range(n_levels)])


@pytest.mark.parametrize("max_batch", [1, 4, 16])
@pytest.mark.parametrize("rate", [300.0, 1500.0, 2600.0])
def test_library_queue_fixed_level(max_batch, rate):
    arr = inputs.poisson_arrivals(21, rate, 3000)
    service = _table(5, max_batch)
    for level in (0, 3):
        want_r, want_l = osv.simulate(arr, service, max_batch, fixed_level=level)
        got_r, got_l = fx.flexiq_serving_simulate(None, level, arr, service, max_batch)
        assert np.array_equal(got_l, want_l)
        assert np.array_equal(got_r, want_r)     # same float64 operations in the same order


@pytest.mark.parametrize("max_batch", [1, 8])
def test_library_queue_with_controller(max_batch):
    arr = inputs.fluctuating_arrivals(31, 500.0, 1500.0, 4.0, 8.0)
    service = _table(5, max_batch, base=0.7e-3)
    grid = np.array([250.0, 500.0, 1000.0, 1500.0, 2000.0])
    lat = np.array([[1e-3 * (1.0 - 0.12 * l) * math.exp(r / 600.0) for r in grid] for l in range(5)])
    thr = 5e-3
    want_r, want_l = osv.simulate(arr, service, max_batch,
                                  controller=dict(rate_grid=grid, latency=lat, threshold=thr, window=0.2, level=1))
    ctrl = fx.Controller(grid, lat, thr, 0.2, initial_level=1)
    got_r, got_l = fx.flexiq_serving_simulate(ctrl, 0, arr, service, max_batch)
    assert len(set(want_l.tolist())) >= 3        # the trace does move the ratio
    assert np.array_equal(got_l, want_l)
    assert np.array_equal(got_r, want_r)
    assert ctrl.level == int(want_l[-1])         # the level after the run is the last decision's
    ctrl.close()


def test_library_controller_update_matches_oracle():
    grid = np.array([100.0, 400.0, 900.0, 3000.0])
    rng_lat = np.array([[2e-3 * (1 + i) / (1 + 0.5 * l) for i in range(4)] for l in range(5)])
    ctrl = fx.Controller(grid, rng_lat, 3e-3, 1.0)
    level = 0
    rates = inputs.uniform(41, 0, 400) * 3500.0
    for r in rates:
        level = osv.controller_update(level, float(r), grid, rng_lat, 3e-3)
        assert ctrl.update(float(r)) == level
    assert ctrl.level == level
    ctrl.close()


def test_library_serving_argument_errors():
    grid, lat = np.array([1.0, 2.0]), np.ones((3, 2))
    with pytest.raises(fx.FlexiqError):
        fx.Controller(np.array([2.0, 1.0]), lat, 1.0, 1.0)          # grid not ascending
    with pytest.raises(fx.FlexiqError):
        fx.Controller(grid, lat, 1.0, 0.0)                           # empty window
    with pytest.raises(fx.FlexiqError):
        fx.Controller(grid, lat, 1.0, 1.0, initial_level=3)
    service = np.ones((3, 2))
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_serving_simulate(None, 3, np.array([0.0, 1.0]), service, 2)      # level out of range
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_serving_simulate(None, 0, np.array([1.0, 0.0]), service, 2)      # arrivals not ascending
    ctrl = fx.Controller(grid, lat, 1.0, 1.0)
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_serving_simulate(ctrl, 0, np.array([0.0]), np.ones((4, 2)), 2)   # level count mismatch
    r, l = fx.flexiq_serving_simulate(ctrl, 0, np.zeros(0), service, 2)            # empty trace
    assert r.size == 0 and l.size == 0
    ctrl.close()
