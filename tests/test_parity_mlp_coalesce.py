"""ABS_FLAG_MLP_COALESCE: single abs_accumulate_mlp calls of a worker are gathered (up to four) and run as one
batch.  Checked: (1) bit-identical to explicit abs_accumulate_mlp_batch calls over the same groups, eager and
pipelined; (2) against the CPU oracle (2e-3 bars) with workers interleaved, more workers than groups may wait,
idle workers, other kinds of accumulate calls in between, and reads of the accumulator in mid-iteration;
(3) counters bit-exact after every call."""

import dataclasses

import numpy as np
import pytest

from oracle.abs_oracle import AbsSgdOracle, mlp_loss_and_grad
from paper_2308_15164_b200 import workloads as wlm

pytestmark = pytest.mark.gpu

TOL = 2e-3


def _engine(wl, x0, pipelined, coalesce, overwrite_first=False):
    import torch

    from paper_2308_15164_b200 import binding as B

    d = wl.mlp
    return B.AbsSgd(torch.from_numpy(x0).cuda(), wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=pipelined,
                    mlp=(d.d_in, d.d_hidden, d.d_out, d.mb), overwrite_first=overwrite_first, mlp_coalesce=coalesce)


@pytest.mark.parametrize("overwrite_first", [False, True], ids=["clear-in-sync", "overwrite-first"])
@pytest.mark.parametrize("small", [True, False], ids=["384x512", "3072x4096"])
def test_gathered_single_calls_equal_explicit_batch_calls_bit_for_bit(small, overwrite_first):
    import torch

    T = 6 if small else 3
    wl = wlm.config(4, small=small, T=T)
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    torch.cuda.synchronize()
    sched = wlm.schedule(wl)
    outs = {}
    for mode in ("batch-eager", "single-eager", "single-pipelined"):
        eng = _engine(wl, x0, pipelined=mode.endswith("pipelined"), coalesce=mode.startswith("single"),
                      overwrite_first=overwrite_first)
        for t, b_row in enumerate(sched):
            for i, b in enumerate(b_row):            # worker by worker: groups are runs of up to four
                lo = (5 * t + 11 * i) % (wl.mlp_pool - 8)
                if mode.startswith("single"):
                    for k in range(int(b)):
                        eng.accumulate_mlp(i, xs_d[lo + k], ys_d[lo + k])
                        assert eng.counters()[0][eng.counters()[1]][i] == k + 1       # counted at once
                else:
                    for k in range(0, int(b), 4):
                        n = min(4, int(b) - k)
                        eng.accumulate_mlp_batch(i, n, xs_d[lo + k:lo + k + n], ys_d[lo + k:lo + k + n])
            eng.sync_step()
        eng.check()
        outs[mode] = (eng.params_host(), [eng.consumed(s) for s in range(T)])
        eng.destroy()
    assert np.abs(outs["batch-eager"][0] - x0).max() > 1e-5
    for mode in ("single-eager", "single-pipelined"):
        assert np.array_equal(outs[mode][0], outs["batch-eager"][0]), mode
        for a, b in zip(outs[mode][1], outs["batch-eager"][1]):
            assert np.array_equal(a, b)


# per iteration: (worker, kind, count); kinds: "one" single MLP calls, "batch" one batch call, "vec" a plain gradient
_PLAN = [
    [(0, "one", 1), (1, "one", 1), (2, "one", 1), (3, "one", 1), (4, "one", 1), (5, "one", 1), (0, "one", 2), (3, "one", 3)],
    [(2, "one", 5), (1, "one", 2), (1, "batch", 3), (1, "one", 1), (4, "vec", 1), (4, "one", 2)],
    [(5, "one", 3), (5, "vec", 1), (5, "one", 1), (0, "batch", 2), (0, "one", 6)],
    [(3, "one", 1)],
    [],
    [(i, "one", 2) for i in range(6)] + [(i, "one", 1) for i in range(6)],
]


@pytest.mark.parametrize("pipelined", [False, True], ids=["eager", "pipelined"])
def test_interleaved_workers_mixed_calls_against_the_oracle(pipelined):
    import torch

    wl = dataclasses.replace(wlm.config(4, small=True, T=len(_PLAN)), W=6)
    d = wl.mlp
    dims = (d.d_in, d.d_hidden, d.d_out)
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    vec = np.random.default_rng(5).standard_normal((2, wl.P)).astype(np.float32) * 1e-3
    o = AbsSgdOracle(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    eng = _engine(wl, x0, pipelined, True)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    vec_d = [torch.from_numpy(vec[j]).cuda() for j in range(2)]
    torch.cuda.synchronize()
    c = 0
    for t, calls in enumerate(_PLAN):
        p = o.params()
        for (i, kind, n) in calls:
            lo = c % (wl.mlp_pool - 8)
            for j in range(n):
                if kind == "vec":
                    o.accumulate(i, vec[c % 2])
                else:
                    o.accumulate(i, mlp_loss_and_grad(p, xs[lo + j], ys[lo + j], *dims, mode="bf16")[1].astype(np.float32))
            if kind == "one":
                for j in range(n):
                    eng.accumulate_mlp(i, xs_d[lo + j], ys_d[lo + j])
            elif kind == "batch":
                eng.accumulate_mlp_batch(i, n, xs_d[lo:lo + n], ys_d[lo:lo + n])
            else:
                eng.accumulate(i, vec_d[c % 2])
            c += n
            cg, curg, tg = eng.counters()
            cr, curr, tr = o.counters()
            assert np.array_equal(cg, cr) and (curg, tg) == (curr, tr)
        if t == 2:        # reading an accumulator in mid-iteration starts the waiting groups first
            got = eng.accumulator(eng.counters()[1], 0).clone()
            eng.stream_acc.synchronize()
            want = o.acc[o.cur][0].astype(np.float64)
            # norm-wise: single hidden units whose ReLU gate is numerically undecided may differ (see test_parity_mlp)
            assert np.linalg.norm(got.cpu().numpy() - want) <= 1e-2 * np.linalg.norm(want)
        o.sync_step()
        eng.sync_step()
    eng.check()
    got = eng.params_host()
    consumed = [eng.consumed(s) for s in range(len(_PLAN))]
    eng.destroy()
    ref = o.params()
    assert np.abs(ref - x0).max() > 1e-5
    assert np.abs(got.astype(np.float64) - ref).max() <= TOL * np.abs(ref).max()
    for a, b in zip(consumed, o.consumed):
        assert np.array_equal(a, b)


def test_flag_needs_the_mlp_flag():
    from paper_2308_15164_b200 import binding as B

    cfg = B.make_config(P=4096, W=2, lr=0.1, flags=B.FLAG_MLP_COALESCE, stream_acc=1)
    assert B.abs_workspace_bytes(cfg) == 0
