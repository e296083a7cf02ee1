"""Runs the CPU oracle on every host core at once -- TEST / BASELINE INFRASTRUCTURE, not a product path.

The oracle's arithmetic is untouched: every worker process calls dvm_oracle.evaluate on its own window of the
inputs, again and again for a fixed time; the windows are independent row blocks, so no result is combined.  What
is reported is the total work of all workers over the slowest worker's time."""
from __future__ import annotations

import multiprocessing
import os
import time

_JOB = None  # (nodes, list of input lists (float64 numpy arrays), params, seconds): set before the workers fork


def _work(i):
    from oracle import dvm_oracle as orc
    nodes, cases, params, seconds = _JOB
    ins = cases[i % len(cases)]
    t0 = time.perf_counter()
    k = 0
    while time.perf_counter() - t0 < seconds or k == 0:
        orc.evaluate(nodes, ins, params)
        k += 1
    return k, time.perf_counter() - t0


def evaluate_on_all_cores(nodes, cases, params=(), seconds=10.0, workers=None):
    """cases: one list of float64 input arrays per window (workers take them round-robin).  Returns
    (evaluations done in total, seconds of the slowest worker, number of worker processes)."""
    global _JOB
    n = workers or os.cpu_count() or 1
    _JOB = (nodes, cases, tuple(params), float(seconds))
    ctx = multiprocessing.get_context("fork")   # the windows are inherited, not pickled; workers only use numpy
    with ctx.Pool(n) as pool:
        res = pool.map(_work, range(n), chunksize=1)
    _JOB = None
    return sum(k for k, _ in res), max(t for _, t in res), n


def _once(i):
    from oracle import dvm_oracle as orc
    nodes, cases, params, _ = _JOB
    orc.evaluate(nodes, cases[i % len(cases)], params)
    return 1


class StepPool:
    """A pool of worker processes, one per host core, that evaluates the same sample once per worker and step
    (the reference arm's "step"): step() returns when every worker is done."""

    def __init__(self, nodes, cases, params=(), workers=None):
        global _JOB
        self.n = workers or os.cpu_count() or 1
        _JOB = (nodes, cases, tuple(params), 0.0)
        self.pool = multiprocessing.get_context("fork").Pool(self.n)

    def step(self):
        return sum(self.pool.map(_once, range(self.n), chunksize=1))

    def close(self):
        self.pool.close()
        self.pool.join()
