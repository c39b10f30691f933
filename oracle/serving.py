"""CPU oracle of the serving experiment: request queue, rate monitor and ratio controller.

TEST INFRASTRUCTURE, NOT A PRODUCT PATH: only the tests, the smoke check and the
CPU-baseline leg of the benchmark import this module.  It shares nothing with the CUDA
library and never imports it.  Plain Python loops over float64 values, one request at a time.

What it follows (Sec. 8, "end-to-end request response times" and "Adapting to Workload
Fluctuation"): requests arrive at given times (a Poisson process in the experiment; the
arrival times are an input here), wait in one first-come-first-served queue in front of one
accelerator, and a response time is completion minus arrival, queueing delay included.  At
run time the request rate is monitored, and whenever the latency that was profiled for the
current rate at the current low-bit ratio is above a threshold, the ratio goes up by one
step of 25 %.

Readings where the text is silent (each is also listed in the design notes):
  * batching: when the accelerator becomes free it takes every request that has arrived by
    then, oldest first, up to ``max_batch``; ``max_batch = 1`` is the plain single-server queue;
  * service time: a table ``service[level][batch - 1]`` in seconds (measured per ratio and batch);
  * request rate: arrivals inside the last ``window`` seconds before a dispatch, divided by
    ``window``; the controller decides at a dispatch when at least ``window`` seconds have
    passed since its previous decision (the first decision is due at time ``window``);
  * profiled latency at a rate between two profiled rates: linear interpolation, clamped to
    the first and last profiled rate outside the grid;
  * stepping down (the text only states the step up, its figure needs both directions): one
    step down when the profiled latency of the next lower ratio at the current rate is
    within the threshold; a decision moves one step at most.
"""
from __future__ import annotations

import numpy as np


def profiled_latency(rate_grid, latency_row, rate: float) -> float:
    """Latency profiled for one ratio, read at ``rate`` (linear between grid points, clamped outside)."""
    g = [float(v) for v in rate_grid]
    y = [float(v) for v in latency_row]
    if rate <= g[0]:
        return y[0]
    if rate >= g[-1]:
        return y[-1]
    for i in range(1, len(g)):
        if rate <= g[i]:
            t = (rate - g[i - 1]) / (g[i] - g[i - 1])
            return y[i - 1] + t * (y[i] - y[i - 1])
    return y[-1]


def controller_update(level: int, rate: float, rate_grid, latency, threshold: float) -> int:
    """One decision (Sec. 8): step the ratio up when the profiled latency of the current ratio at the
    observed rate exceeds the threshold; otherwise step down when the next lower ratio would do."""
    n_levels = len(latency)
    if profiled_latency(rate_grid, latency[level], rate) > threshold:
        return level + 1 if level + 1 < n_levels else level
    if level > 0 and profiled_latency(rate_grid, latency[level - 1], rate) <= threshold:
        return level - 1
    return level


def simulate(arrival, service, max_batch: int, fixed_level: int = 0, controller: dict | None = None):
    """Run the queue over ``arrival`` (ascending seconds).  ``service[level][b - 1]`` = seconds for a
    batch of ``b``.  ``controller`` = dict(rate_grid, latency, threshold, window, level) or None for a
    fixed ratio.  Returns (response seconds per request, level that served each request)."""
    arrival = [float(t) for t in arrival]
    n = len(arrival)
    response = np.zeros(n, dtype=np.float64)
    served_level = np.zeros(n, dtype=np.int32)
    level = int(controller["level"]) if controller else int(fixed_level)
    last_decision = 0.0
    free_at = 0.0
    i = 0
    while i < n:
        start = free_at if free_at > arrival[i] else arrival[i]
        b = 1
        while i + b < n and b < max_batch and arrival[i + b] <= start:
            b += 1
        if controller and start - last_decision >= controller["window"]:
            w = float(controller["window"])
            count = 0
            for t in arrival:
                if start - w < t <= start:
                    count += 1
            level = controller_update(level, count / w, controller["rate_grid"], controller["latency"], controller["threshold"])
            last_decision = start
        done = start + float(service[level][b - 1])
        for r in range(i, i + b):
            response[r] = done - arrival[r]
            served_level[r] = level
        free_at = done
        i += b
    return response, served_level
