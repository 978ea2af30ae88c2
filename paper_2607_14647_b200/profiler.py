"""Start-up cost profiling (Appendix C, "Cost-table profiling protocol"): host logic around the library's calls.

The paper's system fills C(B, rho) before serving by running dummy speculative steps, at every captured batch size and
ratio bucket, through the same pipeline and CUDA-graph configuration as serving, and keeps the median step latency of a
few repetitions.  `profile_cost_grid` does that for a `binding.CostGrid`; `profile_dense` does the same along the packed
length T for the dense table that `dcut_set_cost_dense` takes, and `isotonic_non_decreasing` turns its noisy points into
a table that never charges a longer batch less.  The steps themselves are the caller's (they run the library's kernels);
nothing here computes any part of the method.
"""
from __future__ import annotations

from typing import Callable, Dict, List, Optional, Sequence

import numpy as np
import torch


def time_replays(run: Callable[[], None], reps: int, warmup: int = 2, inner: int = 1) -> List[float]:
    """`reps` samples of the milliseconds one call of `run` takes, each sample `inner` consecutive calls between its own
    pair of CUDA events on the current stream, divided by `inner`.  CUDA event stamps step by one to two microseconds
    on this GPU: with `inner` = 1 a 0.3 ms step is read to within half a percent, and a cost curve whose whole slope
    is 50 us over 1000 packed tokens comes out in stairs."""
    for _ in range(warmup):
        run()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
    ev[0].record()
    for k in range(reps):
        for _ in range(inner):
            run()
        ev[k + 1].record()
    ev[-1].synchronize()
    return [ev[k].elapsed_time(ev[k + 1]) / inner for k in range(reps)]


def profile_cost_grid(grid, make_step: Callable[[int, int], Callable[[], None]], reps: int = 7, warmup: int = 3,
                      inner: int = 1) -> np.ndarray:
    """Fills every cell of `grid` (a binding.CostGrid).  `make_step(B, K)` returns a callable that runs one whole step
    of a dummy batch of B requests whose selector is forced to the budget K (a one-bucket table), the way serving
    would run it (a captured CUDA graph's replay, if serving replays graphs).  Returns the table of medians [n_B, n_rho]."""
    for b, B in enumerate(grid.batch_sizes):
        for r in range(len(grid.ratios)):
            run = make_step(B, grid.budget(B, r))
            grid.record(b, r, time_replays(run, reps, warmup, inner))
    return grid.table()


def isotonic_non_decreasing(y: Sequence[float], w: Optional[Sequence[float]] = None) -> np.ndarray:
    """Least-squares non-decreasing fit (pool adjacent violators).  A longer packed batch never costs less, so a
    profiled point that lies below its shorter neighbour is measurement noise: the fit replaces each run of violating
    points by their weighted mean and leaves points that already ascend untouched."""
    y = np.asarray(y, np.float64)
    w = np.ones_like(y) if w is None else np.asarray(w, np.float64)
    vals: List[float] = []
    wts: List[float] = []
    cnt: List[int] = []
    for yi, wi in zip(y, w):
        vals.append(float(yi))
        wts.append(float(wi))
        cnt.append(1)
        while len(vals) > 1 and vals[-2] > vals[-1]:
            tot = wts[-2] + wts[-1]
            vals[-2] = (vals[-2] * wts[-2] + vals[-1] * wts[-1]) / tot
            wts[-2] = tot
            cnt[-2] += cnt[-1]
            vals.pop()
            wts.pop()
            cnt.pop()
    return np.concatenate([np.full(c, v) for v, c in zip(vals, cnt)])


def dense_table(points_T: Sequence[int], points_ms: Sequence[float], n: int) -> np.ndarray:
    """cost[T] for T = 0 .. n-1 from profiled (T, ms) points: isotonic fit of the points, then linear interpolation
    (flat outside the profiled range).  The result is non-decreasing and strictly positive wherever the points are."""
    t = np.asarray(points_T, np.float64)
    order = np.argsort(t)
    fit = isotonic_non_decreasing(np.asarray(points_ms, np.float64)[order])
    return np.interp(np.arange(n), t[order], fit).astype(np.float32)


def profile_dense(points_T: Sequence[int], make_step: Callable[[int], Callable[[], None]], reps: int = 21,
                  warmup: int = 3) -> Dict[str, list]:
    """Median step latency at each packed length of `points_T`; `make_step(T)` returns the callable that runs one
    step whose selector is forced to the packed length T."""
    med, p25 = [], []
    for T in points_T:
        ts = time_replays(make_step(int(T)), reps, warmup)
        med.append(float(np.median(ts)))
        p25.append(float(np.percentile(ts, 25)))
    return {"T": [int(t) for t in points_T], "median_ms": med, "p25_ms": p25}
