"""Serving experiment (Sec. 8): pins of the queue / rate-monitor / ratio-controller oracle against
hand-worked cases, Lindley's recursion and the M/D/1 mean delay."""
import numpy as np
import pytest

from oracle import serving as osv
from paper_2510_02822_b200 import inputs


# ------------------------------------------------------------------ oracle pins
def test_queue_hand_worked():
    # one server, 0.2 s per request: the second and third requests queue behind the first
    resp, lvl = osv.simulate([0.0, 0.1, 0.15, 1.0], [[0.2]], max_batch=1)
    assert np.allclose(resp, [0.2, 0.3, 0.45, 0.2], rtol=0, atol=1e-15)
    assert lvl.tolist() == [0, 0, 0, 0]


def test_queue_equals_lindley_recursion():
    # single-server FIFO queue: wait_{i+1} = max(0, wait_i + S - gap_i)  (Lindley's recursion)
    arr = inputs.poisson_arrivals(3, 800.0, 5000)
    S = 1.0e-3
    resp, _ = osv.simulate(arr, [[S]], max_batch=1)
    wait = 0.0
    for i in range(arr.size):
        assert abs(resp[i] - (wait + S)) < 1e-12
        if i + 1 < arr.size:
            wait = max(0.0, wait + S - (arr[i + 1] - arr[i]))


def test_queue_mean_wait_matches_pollaczek_khinchine():
    # M/D/1: mean queueing delay = rho * S / (2 (1 - rho))
    lam, S = 1000.0, 0.6e-3
    arr = inputs.poisson_arrivals(5, lam, 200000)
    resp, _ = osv.simulate(arr, [[S]], max_batch=1)
    rho = lam * S
    expect = rho * S / (2.0 * (1.0 - rho))
    got = float(np.mean(resp) - S)
    assert abs(got - expect) / expect < 0.03


def test_queue_batches_take_everything_waiting_up_to_the_limit():
    # ten requests at t = 0, at most four per batch: batches of 4, 4 and 2, each batch completes together
    service = [[1.0, 1.5, 2.0, 2.5]]
    resp, _ = osv.simulate([0.0] * 10, service, max_batch=4)
    assert np.allclose(resp, [2.5] * 4 + [5.0] * 4 + [6.5] * 2)
    # a request that arrives while a batch runs waits for the next one
    resp, _ = osv.simulate([0.0, 0.5, 0.6], service, max_batch=4)
    assert np.allclose(resp, [1.0, 1.0 + 1.5 - 0.5, 1.0 + 1.5 - 0.6])


def test_queue_invariants_with_batching():
    arr = inputs.poisson_arrivals(7, 2000.0, 4000)
    service = [[0.4e-3 + 0.05e-3 * b for b in range(1, 9)]]
    resp, _ = osv.simulate(arr, service, max_batch=8)
    done = arr + resp
    assert np.all(np.diff(done) >= -1e-15)                      # first come, first served
    assert np.all(resp >= service[0][0] - 1e-15)                 # nobody is served faster than a batch of one
    assert done[-1] >= arr[-1] + service[0][0] - 1e-15


def test_profiled_latency_interpolates_and_clamps():
    grid, row = [100.0, 200.0, 400.0], [1.0, 2.0, 6.0]
    assert osv.profiled_latency(grid, row, 50.0) == 1.0
    assert osv.profiled_latency(grid, row, 100.0) == 1.0
    assert osv.profiled_latency(grid, row, 150.0) == pytest.approx(1.5)
    assert osv.profiled_latency(grid, row, 300.0) == pytest.approx(4.0)
    assert osv.profiled_latency(grid, row, 1000.0) == 6.0


def test_controller_steps_by_one_level():
    grid = [100.0, 1000.0]
    lat = [[1.0, 10.0], [0.8, 6.0], [0.5, 3.0]]   # higher ratio, lower latency
    thr = 4.0
    # at rate 1000 level 0 profiles 10 > 4: one step (25 % in the paper) up, not two
    assert osv.controller_update(0, 1000.0, grid, lat, thr) == 1
    assert osv.controller_update(1, 1000.0, grid, lat, thr) == 2
    assert osv.controller_update(2, 1000.0, grid, lat, thr) == 2      # top level holds
    # at rate 100 every level is within the threshold: step down one at a time
    assert osv.controller_update(2, 100.0, grid, lat, thr) == 1
    assert osv.controller_update(0, 100.0, grid, lat, thr) == 0
    # level 1 is fine at rate 500 (3.69) but level 0 would not be (5.0): stay
    assert osv.controller_update(1, 500.0, grid, lat, thr) == 1
    # the threshold itself is not exceeded
    assert osv.controller_update(0, 1000.0, grid, [[1.0, 4.0], [1.0, 1.0]], 4.0) == 0


def test_controller_in_the_queue_follows_a_rate_step():
    # 2 s at 200 requests/s, then 2 s at 2000 requests/s, then 2 s at 200 again
    a = inputs.poisson_arrivals(11, 200.0, 400)
    a = a[a < 2.0]
    b = 2.0 + inputs.poisson_arrivals(12, 2000.0, 4800)
    b = b[b < 4.0]
    c = 4.0 + inputs.poisson_arrivals(13, 200.0, 400)
    c = c[c < 6.0]
    arr = np.concatenate([a, b, c])
    service = [[0.45e-3], [0.40e-3], [0.35e-3]]
    ctrl = dict(rate_grid=[200.0, 2000.0], latency=[[0.5e-3, 5e-3], [0.45e-3, 2e-3], [0.4e-3, 0.8e-3]],
                threshold=1e-3, window=0.25, level=0)
    resp, lvl = osv.simulate(arr, service, max_batch=1, controller=ctrl)
    assert lvl[0] == 0
    assert lvl[(arr > 1.0) & (arr < 2.0)].max() == 0          # low rate: stays at the lowest ratio
    assert lvl[(arr > 3.0) & (arr < 4.0)].min() == 2          # high rate: climbed to the top, one step per window
    assert lvl[(arr > 5.2) & (arr < 6.0)].max() == 0          # and back down
    change = np.flatnonzero(np.diff(lvl) != 0)
    assert np.all(np.abs(np.diff(lvl)[change]) == 1)
    starts = (arr + resp - np.array([service[l][0] for l in lvl]))[change + 1]
    assert np.all(np.diff(starts) >= 0.25 - 1e-12)             # decisions are a window apart


