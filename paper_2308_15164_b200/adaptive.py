"""Adaptive batch size driver (Algorithm 1, Step 2 of arXiv 2308.15164): workers keep computing
reference batches for as long as the synchronisation of the delayed gradients (Step 1) is running,
so the per-iteration micro-batch counts b_i are not preset -- they come out of the timing.

The W workers are logical (gradient buffers of one GPU), so their relative speed is simulated the
way the paper simulates heterogeneous clusters (Section 6.1), in virtual time whose unit is the
reference-batch time of an undisturbed worker:

  static heterogeneity   every reference batch of worker i is prolonged by a fixed fraction
                         static[i] (the paper: 0 %, 100 %, 200 %, 300 % for its 4 workers);
  dynamic heterogeneity  every reference batch is prolonged by a random fraction drawn uniformly
                         from [0, dynamic] (the paper: 0 % .. 50 %), on top of the static one;
  both                   the two combined, the random part relative to the statically prolonged time.

One polling round advances virtual time by one unit; a worker hands over a gradient in the round in
which its reference batch completes.  After every round the driver asks abs_step1_finished; every
worker contributes at least `min_batches` per iteration (Assumption 5: the batch of an iteration
is at least N * M_r)."""

from __future__ import annotations

from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np


def heterogeneity(kind: str, W: int) -> Tuple[List[float], float]:
    """(static[i], dynamic) of the paper's three simulated clusters (Sections 6.2 - 6.4); for W other
    than 4 the static pattern 0, 1, 2, 3 repeats."""
    pattern = [float(i % 4) for i in range(W)]
    if kind == "static":
        return pattern, 0.0
    if kind == "dynamic":
        return [0.0] * W, 0.5
    if kind == "both":
        return pattern, 0.5
    raise ValueError("kind must be 'static', 'dynamic' or 'both'")


def run_adaptive(eng, next_gradient: Callable[[int, int, int], object], iterations: int,
                 period: Optional[Sequence[int]] = None, min_batches: int = 1, max_batches: int = 64,
                 static: Optional[Sequence[float]] = None, dynamic: float = 0.0, seed: int = 0,
                 trace: Optional[list] = None) -> List[List[int]]:
    """Drive `eng` (a pipelined binding.AbsSgd) for `iterations` iterations.

    next_gradient(t, worker, k) returns the device gradient (tensor or address) of worker's k-th
    micro-batch of iteration t.  Worker speeds: either `period` (worker i needs period[i] rounds per
    reference batch; the same as static[i] = period[i] - 1) or `static` / `dynamic` as described in
    the module docstring (random draws from numpy's default_rng(seed), on the host).
    Returns the realised schedule b[t][i], decided here on the host from abs_step1_finished polls --
    nothing read back from the device enters it.  If `trace` is a list, (t, worker, k) of every
    gradient is appended to it in arrival order."""
    W = eng.W
    if period is not None:
        if static is not None:
            raise ValueError("give either period or static, not both")
        static = [float(p) - 1.0 for p in period]
    if static is None:
        static = [0.0] * W
    if len(static) != W or min(static) < 0.0 or dynamic < 0.0:
        raise ValueError("static needs one non-negative entry per worker, dynamic must be >= 0")
    rng = np.random.default_rng(seed)

    def duration(i: int) -> float:
        d = 1.0 + static[i]
        return d * (1.0 + rng.uniform(0.0, dynamic)) if dynamic > 0.0 else d

    schedule = []
    for t in range(iterations):
        counts = [0] * W
        due = [duration(i) for i in range(W)]       # virtual completion time of each worker's current batch
        now = 0.0
        while True:
            now += 1.0
            for i in range(W):
                while due[i] <= now + 1e-9 and counts[i] < max_batches:
                    eng.accumulate(i, next_gradient(t, i, counts[i]))
                    if trace is not None:
                        trace.append((t, i, counts[i]))
                    counts[i] += 1
                    due[i] += duration(i)
            enough = all(c >= min_batches for c in counts)
            capped = all(c >= max_batches for c in counts)
            if enough and (eng.step1_finished() or capped):
                break
        eng.sync_step()            # ends the iteration; launches Step 1 for what was just accumulated
        schedule.append(counts)
    return schedule
