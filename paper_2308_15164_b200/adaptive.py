"""Adaptive batch size driver (Algorithm 1, Step 2 of arXiv 2308.15164): workers keep computing
reference batches for as long as the synchronisation of the delayed gradients (Step 1) is running,
so the per-iteration micro-batch counts b_i are not preset -- they come out of the timing.

The W workers are logical (gradient buffers of one GPU), so their relative speed is simulated the
way the paper simulates heterogeneity (Section 6.1): worker i needs `period[i]` polling rounds per
reference batch (period 1 = fastest).  Every worker contributes at least `min_batches` per
iteration (Assumption 5: the batch of an iteration is at least N * M_r)."""

from __future__ import annotations

from typing import Callable, List, Sequence


def run_adaptive(eng, next_gradient: Callable[[int, int, int], object], iterations: int, period: Sequence[int],
                 min_batches: int = 1, max_batches: int = 64) -> List[List[int]]:
    """Drive `eng` (a pipelined binding.AbsSgd) for `iterations` iterations.

    next_gradient(t, worker, k) returns the device gradient (tensor or address) of worker's k-th
    micro-batch of iteration t.  Returns the realised schedule b[t][i], decided here on the host from
    abs_step1_finished polls -- nothing read back from the device enters it."""
    W = eng.W
    schedule = []
    for t in range(iterations):
        counts = [0] * W
        rounds = 0
        while True:
            rounds += 1
            for i in range(W):
                if rounds % period[i] == 0 and counts[i] < max_batches:
                    eng.accumulate(i, next_gradient(t, i, counts[i]))
                    counts[i] += 1
            enough = all(c >= min_batches for c in counts)
            capped = all(c >= max_batches for c in counts)
            if enough and (eng.step1_finished() or capped):
                break
        eng.sync_step()            # ends the iteration; launches Step 1 for what was just accumulated
        schedule.append(counts)
    return schedule
