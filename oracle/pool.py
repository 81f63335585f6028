"""Runs the fp64 oracle on several host cores at once (test and benchmark infrastructure, like the rest of `oracle/`).

The oracle itself is untouched: every worker process calls `gdn_oracle.chunk_prepare` on its own share of the
chunks, in the same small batches a single-core run uses. The inputs are handed to each worker once, when the
pool starts; a task names a range of chunks only. This module imports numpy and the oracle, nothing else, so a
worker starts in a fraction of a second.
"""
from __future__ import annotations

import multiprocessing
import os
import time

import numpy as np

from . import gdn_oracle as orc

_DATA = None


def _init(K, V, beta, g):
    global _DATA
    _DATA = (K, V, beta, g)
    orc.chunk_prepare(K[:2], V[:2], beta[:2], g[:2])  # first-call costs stay out of the timed part


def _run(lo: int, hi: int, batch: int) -> int:
    K, V, beta, g = _DATA
    n = K.shape[0]
    done = 0
    i = lo
    while i < hi:
        j = i % n
        m = min(batch, hi - i, n - j)
        orc.chunk_prepare(K[j:j + m], V[j:j + m], beta[j:j + m], g[j:j + m])
        done += m
        i += m
    return done


def _worker(K, V, beta, g, lo, hi, batch, ready, go, results):
    _init(K, V, beta, g)
    ready.put(os.getpid())
    go.wait()
    t0 = time.time()
    done = _run(lo, hi, batch)
    results.put((done, t0, time.time()))


def usable_cores() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def timed_chunk_prepare(K, V, beta, g, n_chunks: int, workers: int | None = None, batch: int = 32):
    """Processes `n_chunks` chunk evaluations (cycling through the given stack of chunks), split evenly over
    `workers` processes that all start together. Returns (chunks done, wall seconds from the first start to the
    last finish, workers used)."""
    workers = usable_cores() if workers is None else max(1, workers)
    K = np.ascontiguousarray(K, dtype=np.float64)
    V = np.ascontiguousarray(V, dtype=np.float64)
    beta = np.ascontiguousarray(beta, dtype=np.float64)
    g = np.ascontiguousarray(g, dtype=np.float64)
    if workers == 1:
        _init(K, V, beta, g)
        t0 = time.perf_counter()
        done = _run(0, n_chunks, batch)
        return done, time.perf_counter() - t0, 1
    ctx = multiprocessing.get_context("spawn")
    ready, results, go = ctx.Queue(), ctx.Queue(), ctx.Event()
    share = -(-n_chunks // workers)
    procs = []
    for w in range(workers):
        lo, hi = w * share, min((w + 1) * share, n_chunks)
        procs.append(ctx.Process(target=_worker, args=(K, V, beta, g, lo, hi, batch, ready, go, results), daemon=True))
        procs[-1].start()
    try:
        for _ in procs:
            ready.get(timeout=300)  # every worker has started and warmed up before the clock starts
        go.set()
        out = [results.get(timeout=3600) for _ in procs]
    finally:
        for p in procs:
            p.join(timeout=5)
            if p.is_alive():
                p.terminate()
    done = sum(o[0] for o in out)
    wall = max(o[2] for o in out) - min(o[1] for o in out)
    return done, wall, workers
