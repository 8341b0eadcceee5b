"""Numerical study (CPU, test infrastructure like the rest of oracle/): what would bf16 gradient
accumulators cost in accuracy?  Halving the accumulator width would take the accumulate kernel from
12 to 8 bytes per parameter and micro-batch and the fused step from 8 W + 16 to 4 W + 16, so the
question is whether Algorithm 1's G_t^i survives being rounded to bf16 after every addition.

    python -m oracle.study_bf16_accumulators          # prints the table below for workload 2 (small)

The variant differs from AbsSgdOracle in one line: the accumulator is rounded to bf16 (nearest even)
after every `G += g`.  Everything else (fp64 update, weighted average) is unchanged."""

from __future__ import annotations

import numpy as np

from oracle.abs_oracle import AbsSgdOracle, bf16_round


class Bf16AccumulatorOracle(AbsSgdOracle):
    def accumulate(self, i, g):
        super().accumulate(i, g)
        self.acc[self.cur, i] = bf16_round(self.acc[self.cur, i]).astype(np.float32)


def deviation(x0, W, lr, momentum, weight_decay, calls_per_iteration):
    """calls_per_iteration: list over iterations of lists of (worker, gradient).  Returns
    (max |x_bf16acc - x_fp32acc| / max |x_fp32acc|, same for the parameter change since x0)."""
    a = AbsSgdOracle(x0, W, lr, momentum, weight_decay)
    b = Bf16AccumulatorOracle(x0, W, lr, momentum, weight_decay)
    for calls in calls_per_iteration:
        for (i, g) in calls:
            a.accumulate(i, g)
            b.accumulate(i, g)
        a.sync_step()
        b.sync_step()
    xa, xb = a.x, b.x
    err = np.abs(xa - xb).max()
    return err / np.abs(xa).max(), err / max(np.abs(xa - np.asarray(x0, dtype=np.float64)).max(), 1e-300)


def main():
    from paper_2308_15164_b200 import workloads as wlm   # seeded input generators only

    for T in (10, 30, 100):
        wl = wlm.config(2, small=True, T=T)
        x0, pool = wlm.params0(wl), wlm.grad_pool(wl)
        calls = [[(i, pool[c % wl.pool_size]) for (i, k, c) in it] for it in wlm.iter_calls(wl)]
        rel_x, rel_dx = deviation(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay, calls)
        print(f"workload 2 (small), T = {T:3d}: max|dx| / max|x| = {rel_x:.2e}   relative to the distance moved: {rel_dx:.2e}")


if __name__ == "__main__":
    main()
