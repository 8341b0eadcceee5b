"""GPU parity of ABS_FLAG_MLP_DEFER: the layer-1 weight gradient of a worker is contracted once per iteration,
over all its micro-batches (every gradient of an iteration is evaluated at the same x_t: Algorithm 1, Step 2),
instead of once per call.  Checked against the CPU oracle, through the C ABI, at the bars of the per-call path
(2e-3 of the tensor maximum element-wise and 2e-3 in Frobenius norm; counters bit-exact):

  * a worker's accumulator row after several single and batch calls (read through abs_accumulator, which makes
    the library contract what is waiting) against the oracle's sum of gradients;
  * reading the row in the middle of an iteration and going on (the second contraction adds to the first);
  * more micro-batches in one iteration than the operand pool holds (early contraction);
  * whole training runs -- eager, pipelined, with gathered calls, in overwrite-first mode -- against the oracle run,
    eager and pipelined bit-identical;
  * gradient vectors (abs_accumulate) and MLP calls mixed within an iteration, idle workers;
  * export / import in the middle of an iteration;
  * the two forms of the deferred step -- W1 slice updated straight from the pooled operands (one contraction over
    all micro-batches inside the update kernel) or from the rows (per-worker contractions first) -- against each
    other after the same iterations, with and without Eq. 6."""

import numpy as np
import pytest

from oracle.abs_oracle import AbsSgdOracle, mlp_loss_and_grad
from paper_2308_15164_b200 import workloads as wlm

pytestmark = pytest.mark.gpu

TOL = 2e-3


def _engine(wl, x0, W=None, pipelined=False, coalesce=False, overwrite_first=False, defer=True):
    import torch

    from paper_2308_15164_b200 import binding as B

    d = wl.mlp
    return B.AbsSgd(torch.from_numpy(x0).cuda(), W or wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=pipelined,
                    mlp=(d.d_in, d.d_hidden, d.d_out, d.mb), overwrite_first=overwrite_first, mlp_coalesce=coalesce,
                    mlp_defer=defer)


def _grad(p, xs, ys, c, wl):
    d = wl.mlp
    return mlp_loss_and_grad(p, xs[c % wl.mlp_pool], ys[c % wl.mlp_pool], d.d_in, d.d_hidden, d.d_out, mode="bf16")[1].astype(np.float32)


def _close_row(got, ref, wl, what):
    """Tensor by tensor (W1, b1, W2, b2 slices of the flat row)."""
    d = wl.mlp
    o = [0, d.d_in * d.d_hidden, d.d_in * d.d_hidden + d.d_hidden, d.d_in * d.d_hidden + d.d_hidden + d.d_hidden * d.d_out, wl.P]
    for name, lo, hi in zip(("dW1", "db1", "dW2", "db2"), o[:-1], o[1:]):
        g, r = got[lo:hi].astype(np.float64), ref[lo:hi].astype(np.float64)
        assert np.abs(g - r).max() <= TOL * np.abs(r).max(), f"{what}: {name} max err {np.abs(g - r).max():.3e} vs {TOL}*{np.abs(r).max():.3e}"
        assert np.linalg.norm(g - r) <= TOL * np.linalg.norm(r), f"{what}: {name} Frobenius"


@pytest.mark.parametrize("small", [True, False], ids=["384x512", "3072x4096"])
def test_row_after_several_calls_and_a_read_in_the_middle(small):
    import torch

    wl = wlm.config(4, small=small, T=1)
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    eng = _engine(wl, x0)
    # worker 2: 1 + 3 + 1 micro-batches; worker 0: 2; workers 1, 3 idle
    plan = [(2, 1), (0, 2), (2, 3), (2, 1)]
    ref = {0: np.zeros(wl.P, np.float32), 2: np.zeros(wl.P, np.float32)}
    c = 0
    for (i, n) in plan:
        eng.accumulate_mlp_batch(i, n, xs_d[c:c + n], ys_d[c:c + n]) if n > 1 else eng.accumulate_mlp(i, xs_d[c], ys_d[c])
        for j in range(n):
            ref[i] = ref[i] + _grad(x0, xs, ys, c + j, wl)
        c += n
    cur = eng.counters()[1]
    for i in (0, 2):
        _close_row(eng.accumulator(cur, i).cpu().numpy(), ref[i], wl, f"worker {i}")
    for i in (1, 3):
        assert not eng.accumulator(cur, i).any()
    # the iteration goes on: what comes now is added to what the read made the library contract
    for (i, n) in [(2, 2), (1, 1)]:
        eng.accumulate_mlp_batch(i, n, xs_d[c:c + n], ys_d[c:c + n]) if n > 1 else eng.accumulate_mlp(i, xs_d[c], ys_d[c])
        for j in range(n):
            ref[i] = ref.get(i, np.zeros(wl.P, np.float32)) + _grad(x0, xs, ys, c + j, wl)
        c += n
    for i in (0, 1, 2):
        _close_row(eng.accumulator(cur, i).cpu().numpy(), ref[i], wl, f"worker {i}, second read")
    assert eng.counters()[0][cur].tolist() == [2, 1, 7, 0]
    eng.check()
    eng.destroy()


@pytest.mark.parametrize("calls", ["single", "batches-of-3"])
def test_more_microbatches_than_the_pool_holds(calls):
    """W = 2: the pool holds 32 micro-batches; 45 arrive in one iteration (worker 0: 30, worker 1: 15)."""
    import torch

    wl = wlm.config(4, small=True, T=1)
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    o = AbsSgdOracle(x0, 2, wl.lr, wl.momentum, wl.weight_decay)
    eng = _engine(wl, x0, W=2, pipelined=True)
    step = 1 if calls == "single" else 3
    c = 0
    for rnd in range(15 // step):
        for i, n in ((0, 2 * step), (1, step)):
            for lo in range(0, n, step):
                at = c % (wl.mlp_pool - step)
                if step == 1:
                    eng.accumulate_mlp(i, xs_d[at], ys_d[at])
                else:
                    eng.accumulate_mlp_batch(i, step, xs_d[at:at + step], ys_d[at:at + step])
                for j in range(step):
                    o.accumulate(i, _grad(x0, xs, ys, at + j, wl))
                c += step
    cur = eng.counters()[1]
    assert eng.counters()[0][cur].tolist() == [30, 15]
    for _ in range(3):
        eng.sync_step(); o.sync_step()
    eng.check()
    got = eng.params_host()
    ref = o.params()
    assert np.abs(ref - x0).max() > 1e-4
    assert np.abs(got.astype(np.float64) - ref).max() <= TOL * np.abs(ref).max()
    assert np.array_equal(eng.consumed(1), np.array([30, 15]))
    eng.destroy()


def _run(wl, x0, xs_d, ys_d, rows_only=False, **kw):
    from paper_2308_15164_b200 import binding as B

    eng = _engine(wl, x0, **kw)
    if rows_only:                                    # the fused step never works from the pooled operands
        eng.set_launch(B.K_MLP_BWD, 1)
    states = []
    for t, calls in enumerate(wlm.iter_calls(wl)):
        for (i, k, c) in calls:
            eng.accumulate_mlp(i, xs_d[c % wl.mlp_pool], ys_d[c % wl.mlp_pool])
        eng.sync_step()
        states.append(eng.counters())
    eng.check()
    out = eng.params_host()
    consumed = [eng.consumed(s) for s in range(len(states))]
    eng.destroy()
    return out, states, consumed


@pytest.mark.parametrize("small,T", [(True, 12), (False, 5)], ids=["384x512-T12", "3072x4096-T5"])
def test_training_run_matches_oracle(small, T):
    import torch

    wl = wlm.config(4, small=small, T=T)
    d = wl.mlp
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    o = AbsSgdOracle(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    ref_states = []
    for calls in wlm.iter_calls(wl):
        p = o.params()
        for (i, k, c) in calls:
            o.accumulate(i, _grad(p, xs, ys, c, wl))
        o.sync_step()
        ref_states.append(o.counters())
    ref = o.params()
    assert np.abs(ref - x0).max() > 1e-4
    outs = {}
    for name, kw in (("eager", dict()), ("pipelined", dict(pipelined=True)), ("gathered", dict(pipelined=True, coalesce=True)),
                     ("overwrite-first", dict(pipelined=True, overwrite_first=True)), ("per-call", dict(pipelined=True, defer=False)),
                     ("rows-only", dict(pipelined=True, rows_only=True)), ("rows-only-eager", dict(rows_only=True))):
        got, states, consumed = _run(wl, x0, xs_d, ys_d, **kw)
        err = np.abs(got.astype(np.float64) - ref).max()
        assert err <= TOL * np.abs(ref).max(), f"{name}: {err:.3e}"
        for (c1, cur1, t1), (c2, cur2, t2) in zip(states, ref_states):
            assert np.array_equal(c1, c2) and (cur1, t1) == (cur2, t2)
        for a, b in zip(consumed, o.consumed):
            assert np.array_equal(a, b)
        outs[name] = got
    assert np.array_equal(outs["eager"], outs["pipelined"]), "eager and pipelined runs must be bit-identical"
    assert np.array_equal(outs["overwrite-first"], outs["pipelined"]), "overwrite-first mode must give the same parameters"
    assert np.array_equal(outs["rows-only"], outs["rows-only-eager"])
    # against the per-call path, and between the two forms of the deferred step, only the order of the fp32 additions
    # differs (and 1 / B is multiplied by instead of divided by)
    assert np.abs(outs["pipelined"] - outs["per-call"]).max() <= 1e-4 * np.abs(ref).max()
    assert np.abs(outs["rows-only"] - outs["per-call"]).max() <= 1e-4 * np.abs(ref).max()


@pytest.mark.parametrize("lambda_dc", [0.0, 0.3], ids=["plain", "eq6"])
@pytest.mark.parametrize("small", [True, False], ids=["384x512", "3072x4096"])
def test_one_step_from_the_pooled_operands_against_the_step_from_the_rows(small, lambda_dc):
    """The same three iterations with the W1 slice updated straight from the pooled operands (one contraction over all
    micro-batches, inside the update kernel) and from the rows (per-worker contractions, then the row-based fused
    step): parameters, momentum and the next iteration's gradients (which read the bf16 copy of the new weights)
    agree to fp32 rounding, element by element."""
    import torch

    from paper_2308_15164_b200 import binding as B

    wl = wlm.config(4, small=small, T=3)
    d = wl.mlp
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    res = []
    for knob in (0, 1, 2):                           # pooled step (128 x 256 tiles), rows first, pooled step with 128 x 128 tiles
        eng = B.AbsSgd(torch.from_numpy(x0).cuda(), wl.W, wl.lr, wl.momentum, 1e-3, lambda_dc, pipelined=True,
                       mlp=(d.d_in, d.d_hidden, d.d_out, d.mb), mlp_defer=True)
        if knob:
            eng.set_launch(B.K_MLP_BWD, knob)
        for t, calls in enumerate(wlm.iter_calls(wl)):
            for (i, k, c) in calls:
                eng.accumulate_mlp(i, xs_d[c % wl.mlp_pool], ys_d[c % wl.mlp_pool])
            eng.sync_step()
        eng.sync_step()
        eng.wait(); eng.synchronize(); eng.check()
        x, v = eng.params_host().copy(), eng.momentum().cpu().numpy().copy()
        eng.accumulate_mlp(1, xs_d[5], ys_d[5])      # a gradient at the new parameters: reads their bf16 copy
        g = eng.accumulator(eng.counters()[1], 1).cpu().numpy().copy()
        res.append((x, v, g))
        eng.destroy()
    (xa, va, ga), (xb, vb, gb), (xc, vc, gc) = res
    assert np.abs(xa - x0).max() > 1e-4
    assert np.abs(xa - xb).max() <= 2e-6 * np.abs(xb).max()
    assert np.abs(va - vb).max() <= 2e-5 * np.abs(vb).max()
    assert np.abs(ga - gb).max() <= TOL * np.abs(gb).max()
    # the two tile widths contract the same operands in the same order: the same bits
    assert np.array_equal(xa, xc) and np.array_equal(va, vc) and np.array_equal(ga, gc)


_MIXED = [
    [(0, "mlp", 1), (1, "vec", 1), (0, "mlp", 2), (3, "mlp", 4)],
    [(2, "vec", 2), (2, "mlp", 3), (0, "mlp", 1), (2, "vec", 1), (2, "mlp", 1)],
    [],
    [(1, "mlp", 2), (1, "mlp", 2), (3, "vec", 1)],
    [(0, "mlp", 4), (1, "mlp", 4), (2, "mlp", 4), (3, "mlp", 4)],
]


@pytest.mark.parametrize("overwrite_first", [False, True], ids=["clear-in-sync", "overwrite-first"])
@pytest.mark.parametrize("pipelined", [False, True], ids=["eager", "pipelined"])
def test_gradient_vectors_and_mlp_calls_mixed(pipelined, overwrite_first):
    import torch

    wl = wlm.config(4, small=True, T=len(_MIXED))
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    vec = np.random.default_rng(11).standard_normal((3, wl.P)).astype(np.float32) * 1e-3
    o = AbsSgdOracle(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    eng = _engine(wl, x0, pipelined=pipelined, overwrite_first=overwrite_first)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    vec_d = [torch.from_numpy(vec[j]).cuda() for j in range(3)]
    c = 0
    for t, calls in enumerate(_MIXED + [[], []]):
        p = o.params()
        for (i, kind, n) in calls:
            lo = c % (wl.mlp_pool - 4)
            if kind == "mlp":
                eng.accumulate_mlp_batch(i, n, xs_d[lo:lo + n], ys_d[lo:lo + n])
                for j in range(n):
                    o.accumulate(i, _grad(p, xs, ys, lo + j, wl))
            else:
                for j in range(n):
                    eng.accumulate(i, vec_d[(c + j) % 3])
                    o.accumulate(i, vec[(c + j) % 3])
            c += n
        eng.sync_step(); o.sync_step()
        cnt, cur, tt = eng.counters()
        assert np.array_equal(cnt, o.counters()[0]) and (cur, tt) == o.counters()[1:]
    eng.check()
    got = eng.params_host()
    ref = o.params()
    assert np.abs(ref - x0).max() > 1e-5
    assert np.abs(got.astype(np.float64) - ref).max() <= TOL * np.abs(ref).max()
    for s, b in enumerate(o.consumed):
        assert np.array_equal(eng.consumed(s), b)
    eng.destroy()


def test_export_in_the_middle_of_an_iteration_and_resume_in_a_fresh_context():
    import torch

    wl = wlm.config(4, small=True, T=4)
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    its = list(wlm.iter_calls(wl))

    def feed(eng, calls):
        for (i, k, c) in calls:
            eng.accumulate_mlp(i, xs_d[c % wl.mlp_pool], ys_d[c % wl.mlp_pool])

    a = _engine(wl, x0, pipelined=True)
    for calls in its[:2]:
        feed(a, calls); a.sync_step()
    half = len(its[2]) // 2
    feed(a, its[2][:half])
    blob = a.state_export()                      # the operands waiting in the pool are contracted into the rows first
    b = _engine(wl, (x0 * 0.5).astype(np.float32), pipelined=True)
    b.state_import(blob)
    for eng in (a, b):
        feed(eng, its[2][half:]); eng.sync_step()
        feed(eng, its[3]); eng.sync_step(); eng.sync_step()
        eng.check()
    assert np.array_equal(a.params_host(), b.params_host())
    assert np.array_equal(a.momentum().cpu().numpy(), b.momentum().cpu().numpy())
    assert np.array_equal(a.counters()[0], b.counters()[0])
    # and the run as a whole still follows the oracle
    o = AbsSgdOracle(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    for calls in its:
        p = o.params()
        for (i, k, c) in calls:
            o.accumulate(i, _grad(p, xs, ys, c, wl))
        o.sync_step()
    o.sync_step()
    assert np.abs(a.params_host().astype(np.float64) - o.params()).max() <= TOL * np.abs(o.params()).max()
    a.destroy(); b.destroy()


def test_eager_mode_reading_a_closed_set_that_still_waits_in_pooled_form():
    """Eager mode applies a set one call after its iteration ended; until then its W1 gradients wait in pooled form.
    Reading the closed set's rows (abs_accumulator) or exporting the state makes the library complete the rows
    first; the step that follows then runs row-based and the run still follows the oracle."""
    import torch

    wl = wlm.config(4, small=True, T=3)
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    its = list(wlm.iter_calls(wl))
    o = AbsSgdOracle(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    eng = _engine(wl, x0, pipelined=False)
    for t, calls in enumerate(its):
        p = o.params()
        sums = {}
        for (i, k, c) in calls:
            g = _grad(p, xs, ys, c, wl)
            o.accumulate(i, g)
            sums[i] = sums.get(i, 0) + g
            eng.accumulate_mlp(i, xs_d[c % wl.mlp_pool], ys_d[c % wl.mlp_pool])
        closed = eng.counters()[1]
        eng.sync_step(); o.sync_step()               # the set just filled is now closed and waits for the next call
        if t == 0:
            for i, s in sums.items():
                _close_row(eng.accumulator(closed, i).cpu().numpy(), s, wl, f"closed set, worker {i}")
        elif t == 1:
            blob = eng.state_export()
            assert blob.nbytes > 0
    eng.sync_step(); o.sync_step()
    eng.check()
    ref = o.params()
    assert np.abs(ref - x0).max() > 1e-4
    assert np.abs(eng.params_host().astype(np.float64) - ref).max() <= TOL * np.abs(ref).max()
    for s in range(len(its) + 1):
        assert np.array_equal(eng.consumed(s), o.consumed[s])
    eng.destroy()


def test_gathered_single_calls_of_several_workers_share_a_group():
    """ABS_FLAG_MLP_COALESCE with ABS_FLAG_MLP_DEFER gathers consecutive single calls four at a time whoever their
    workers are: every worker's b_i and row must still be its own."""
    import torch

    wl = wlm.config(4, small=True, T=1)
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    eng = _engine(wl, x0, pipelined=True, coalesce=True)
    order = [2, 0, 2, 3, 3, 0, 2, 2, 0, 3, 2]        # 11 calls: two full groups and one of three; worker 1 idle
    ref = {}
    for c, i in enumerate(order):
        eng.accumulate_mlp(i, xs_d[c], ys_d[c])
        ref[i] = ref.get(i, 0) + _grad(x0, xs, ys, c, wl)
    cur = eng.counters()[1]
    assert eng.counters()[0][cur].tolist() == [3, 0, 5, 3]
    for i, want in ref.items():
        _close_row(eng.accumulator(cur, i).cpu().numpy(), want, wl, f"worker {i}")
    assert not eng.accumulator(cur, 1).any()
    o = AbsSgdOracle(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    for c, i in enumerate(order):
        o.accumulate(i, _grad(x0, xs, ys, c, wl))
    for _ in range(2):
        eng.sync_step(); o.sync_step()
    eng.check()
    assert np.array_equal(eng.consumed(1), np.array([3, 0, 5, 3]))
    assert np.abs(eng.params_host().astype(np.float64) - o.params()).max() <= TOL * np.abs(o.params()).max()
    eng.destroy()


@pytest.mark.parametrize("defer", [False, True], ids=["per-call-dw1", "deferred-dw1"])
@pytest.mark.parametrize("shape", [(128, 128, 10), (256, 128, 3), (128, 384, 16)])
def test_smallest_layer_sizes(shape, defer):
    """One tile in one or both directions, one and sixteen outputs: three iterations against the oracle."""
    import dataclasses

    import torch

    from paper_2308_15164_b200 import binding as B

    d_in, d_h, d_out = shape
    dims = wlm.MlpDims(d_in, d_h, d_out, 64)
    wl = dataclasses.replace(wlm.config(4, small=True, T=3), mlp=dims, P=dims.P)
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    o = AbsSgdOracle(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    eng = B.AbsSgd(torch.from_numpy(x0).cuda(), wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=True,
                   mlp=(d_in, d_h, d_out, 64), mlp_defer=defer)
    for t, calls in enumerate(wlm.iter_calls(wl)):
        p = o.params()
        for (i, k, c) in calls:
            g = mlp_loss_and_grad(p, xs[c % wl.mlp_pool], ys[c % wl.mlp_pool], d_in, d_h, d_out, mode="bf16")[1].astype(np.float32)
            o.accumulate(i, g)
            eng.accumulate_mlp(i, xs_d[c % wl.mlp_pool], ys_d[c % wl.mlp_pool])
        eng.sync_step(); o.sync_step()
    eng.sync_step(); o.sync_step()
    eng.check()
    ref = o.params()
    assert np.abs(ref - x0).max() > 1e-4
    assert np.abs(eng.params_host().astype(np.float64) - ref).max() <= TOL * np.abs(ref).max()
    for s in range(4):
        assert np.array_equal(eng.consumed(s), o.consumed[s])
    eng.destroy()


@pytest.mark.parametrize("mode", ["deferred", "deferred-gathered", "deferred-rows", "per-call"])
def test_twelve_workers(mode):
    """W = 12 (more workers than internal streams; the row-based step in its chunked form), two of them idle."""
    import dataclasses

    import torch

    from paper_2308_15164_b200 import binding as B

    W = 12
    wl = dataclasses.replace(wlm.config(4, small=True, T=3), W=W)
    d = wl.mlp
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    rng = np.random.default_rng(5)
    sched = rng.integers(0, 4, size=(3, W))
    sched[:, 3] = 0; sched[:, 7] = 0
    o = AbsSgdOracle(x0, W, wl.lr, wl.momentum, wl.weight_decay)
    eng = B.AbsSgd(torch.from_numpy(x0).cuda(), W, wl.lr, wl.momentum, wl.weight_decay, pipelined=True,
                   mlp=(d.d_in, d.d_hidden, d.d_out, d.mb), mlp_defer=mode != "per-call", mlp_coalesce=mode == "deferred-gathered")
    if mode == "deferred-rows":
        eng.set_launch(B.K_MLP_BWD, 1)
    c = 0
    for t in range(3):
        p = o.params()
        for k in range(int(sched[t].max())):          # round-robin over the workers, as they would arrive
            for i in range(W):
                if k < sched[t, i]:
                    o.accumulate(i, _grad(p, xs, ys, c, wl))
                    eng.accumulate_mlp(i, xs_d[c % wl.mlp_pool], ys_d[c % wl.mlp_pool])
                    c += 1
        eng.sync_step(); o.sync_step()
        cnt, cur, tt = eng.counters()
        assert np.array_equal(cnt, o.counters()[0])
    eng.sync_step(); o.sync_step()
    eng.check()
    ref = o.params()
    assert np.abs(ref - x0).max() > 1e-4
    assert np.abs(eng.params_host().astype(np.float64) - ref).max() <= TOL * np.abs(ref).max()
    for s in range(4):
        assert np.array_equal(eng.consumed(s), o.consumed[s])
    eng.destroy()


def test_learning_rate_schedule_eq6_and_weight_decay_in_the_pooled_step():
    """gamma_t changing every iteration, Eq. 6 and weight decay through the step that works from the pooled operands
    (the rate travels with the gradients: the set of iteration t is applied with the rate in effect when it ended),
    eager and pipelined, against the oracle."""
    import torch

    from paper_2308_15164_b200 import binding as B

    T = 6
    wl = wlm.config(4, small=True, T=T)
    d = wl.mlp
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    lrs = [0.05, 0.02, 0.08, 0.01, 0.04, 0.03, 0.03]
    lam, wd = 0.3, 1e-3
    o = AbsSgdOracle(x0, wl.W, lrs[0], wl.momentum, wd, lam)
    its = list(wlm.iter_calls(wl))
    for t, calls in enumerate(its):
        o.lr = lrs[t]
        p = o.params()
        for (i, k, c) in calls:
            o.accumulate(i, _grad(p, xs, ys, c, wl))
        o.sync_step()
    o.lr = lrs[T]
    o.sync_step()
    ref = o.params()
    assert np.abs(ref - x0).max() > 1e-4
    outs = []
    for pipelined in (False, True):
        eng = B.AbsSgd(torch.from_numpy(x0).cuda(), wl.W, lrs[0], wl.momentum, wd, lam, pipelined=pipelined,
                       mlp=(d.d_in, d.d_hidden, d.d_out, d.mb), mlp_defer=True)
        for t, calls in enumerate(its):
            eng.set_lr(lrs[t + 1])                   # gamma_{t+1}: supplied one iteration ahead
            for (i, k, c) in calls:
                eng.accumulate_mlp(i, xs_d[c % wl.mlp_pool], ys_d[c % wl.mlp_pool])
            eng.sync_step()
        eng.sync_step()
        eng.check()
        got = eng.params_host()
        assert np.abs(got.astype(np.float64) - ref).max() <= TOL * np.abs(ref).max(), f"pipelined={pipelined}"
        outs.append(got)
        eng.destroy()
    assert np.array_equal(outs[0], outs[1])


@pytest.mark.parametrize("pipelined", [False, True], ids=["eager", "pipelined"])
def test_one_worker(pipelined):
    """W = 1 (every kernel chained, deep pipelines): single and batch calls over three iterations against the oracle."""
    import dataclasses

    import torch

    from paper_2308_15164_b200 import binding as B

    wl = dataclasses.replace(wlm.config(4, small=True, T=3), W=1)
    d = wl.mlp
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    o = AbsSgdOracle(x0, 1, wl.lr, wl.momentum, wl.weight_decay)
    eng = B.AbsSgd(torch.from_numpy(x0).cuda(), 1, wl.lr, wl.momentum, wl.weight_decay, pipelined=pipelined,
                   mlp=(d.d_in, d.d_hidden, d.d_out, d.mb), mlp_defer=True)
    c = 0
    for t, plan in enumerate([(1, 3, 1), (8,), (2, 1, 1, 5)]):
        p = o.params()
        for n in plan:
            if n == 1:
                eng.accumulate_mlp(0, xs_d[c], ys_d[c])
            else:
                eng.accumulate_mlp_batch(0, n, xs_d[c:c + n], ys_d[c:c + n])
            for j in range(n):
                o.accumulate(0, _grad(p, xs, ys, c + j, wl))
            c += n
        eng.sync_step(); o.sync_step()
    eng.sync_step(); o.sync_step()
    eng.check()
    ref = o.params()
    assert np.abs(ref - x0).max() > 1e-4
    assert np.abs(eng.params_host().astype(np.float64) - ref).max() <= TOL * np.abs(ref).max()
    assert [int(eng.consumed(s)[0]) for s in range(4)] == [0, 5, 8, 9]
    eng.destroy()


@pytest.mark.parametrize("defer", [False, True], ids=["per-call-dw1", "deferred-dw1"])
def test_list_call_equals_the_batch_call_bit_for_bit(defer):
    """abs_accumulate_mlp_list over n separate buffers = abs_accumulate_mlp_batch over the same micro-batches laid
    out contiguously: same kernels behind one cast launch, same bits (rows, counters, parameters after the steps)."""
    import torch

    from paper_2308_15164_b200 import binding as B

    wl = wlm.config(4, small=True, T=2)
    d = wl.mlp
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    plan = [(0, [3, 9, 1]), (2, [5]), (0, [7, 2, 11, 4, 6, 8, 10, 12]), (3, [13, 14])]   # worker, pool indices (scattered)
    outs = []
    for form in ("list", "batch"):
        eng = B.AbsSgd(torch.from_numpy(x0).cuda(), wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=True,
                       mlp=(d.d_in, d.d_hidden, d.d_out, d.mb), mlp_defer=defer)
        for t in range(2):
            for (i, idx) in plan:
                if form == "list":
                    eng.accumulate_mlp_list(i, [xs_d[j] for j in idx], [ys_d[j] for j in idx])
                else:
                    xc = torch.stack([xs_d[j] for j in idx]).contiguous()
                    yc = torch.stack([ys_d[j] for j in idx]).contiguous()
                    torch.cuda.synchronize()
                    eng.accumulate_mlp_batch(i, len(idx), xc, yc)
                    eng.synchronize()                # xc / yc go out of scope: their reads must have happened
            if t == 1:
                cur = eng.counters()[1]
                rows = [eng.accumulator(cur, i).cpu().numpy().copy() for i in range(wl.W)]
            eng.sync_step()
        eng.sync_step()
        eng.check()
        outs.append((rows, eng.params_host().copy(), [eng.consumed(s).copy() for s in range(3)]))
        eng.destroy()
    (ra, xa, ca), (rb, xb, cb) = outs
    assert np.abs(xa - x0).max() > 1e-5
    assert np.array_equal(xa, xb)
    for a, b in zip(ra, rb):
        assert np.array_equal(a, b)
    for a, b in zip(ca, cb):
        assert np.array_equal(a, b)
    assert ca[1].tolist() == [11, 0, 1, 2]


def test_list_call_argument_checks():
    import ctypes

    import torch

    from paper_2308_15164_b200 import binding as B

    wl = wlm.config(4, small=True)
    d = wl.mlp
    x = torch.zeros((2, d.mb, d.d_in), device="cuda")
    y = torch.zeros((2, d.mb), dtype=torch.int32, device="cuda")
    eng = B.AbsSgd(torch.from_numpy(wlm.params0(wl)).cuda(), wl.W, wl.lr, mlp=(d.d_in, d.d_hidden, d.d_out, d.mb))
    n0 = eng.launch_count()
    xa = (ctypes.c_void_p * 2)(x[0].data_ptr(), x[1].data_ptr())
    ya = (ctypes.c_void_p * 2)(y[0].data_ptr(), y[1].data_ptr())
    bad = (ctypes.c_void_p * 2)(x[0].data_ptr(), None)
    mis = (ctypes.c_void_p * 2)(x[0].data_ptr(), x[1].data_ptr() + 4)
    f = B.lib.abs_accumulate_mlp_list
    assert f(eng._h, 0, 0, xa, ya) == B.EINVAL
    assert f(eng._h, 0, 9, xa, ya) == B.EINVAL
    assert f(eng._h, wl.W, 2, xa, ya) == B.EINVAL
    assert f(eng._h, 0, 2, None, ya) == B.EINVAL
    assert f(eng._h, 0, 2, bad, ya) == B.EINVAL
    assert f(eng._h, 0, 2, mis, ya) == B.EINVAL
    assert f(eng._h, 0, 2, xa, bad) == B.EINVAL
    assert eng.launch_count() == n0 and not eng.counters()[0].any()
    assert f(eng._h, 0, 2, xa, ya) == B.OK
    eng.check()
    eng.destroy()


def test_bf16_inputs_in_deferred_mode():
    """ABS_FLAG_MLP_X_BF16 with ABS_FLAG_MLP_DEFER: X handed over as bf16 values gives the same bits as the same
    values handed over as fp32 (the cast copies them as they are), single, batch and list calls."""
    import torch

    from paper_2308_15164_b200 import binding as B

    wl = wlm.config(4, small=True, T=2)
    d = wl.mlp
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xb = torch.from_numpy(xs).cuda().to(torch.bfloat16)          # the values both runs see
    xf = xb.to(torch.float32)
    ys_d = torch.from_numpy(ys).cuda()
    outs = []
    for x_bf16, xd in ((True, xb), (False, xf)):
        eng = B.AbsSgd(torch.from_numpy(x0).cuda(), wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=True,
                       mlp=(d.d_in, d.d_hidden, d.d_out, d.mb), mlp_defer=True, mlp_x_bf16=x_bf16)
        for t in range(2):
            eng.accumulate_mlp(0, xd[3], ys_d[3])
            eng.accumulate_mlp_batch(1, 3, xd[4:7], ys_d[4:7])
            eng.accumulate_mlp_list(2, [xd[9], xd[1]], [ys_d[9], ys_d[1]])
            eng.sync_step()
        eng.sync_step()
        eng.check()
        outs.append(eng.params_host().copy())
        eng.destroy()
    assert np.abs(outs[0] - x0).max() > 1e-5
    assert np.array_equal(outs[0], outs[1])


def test_gradient_norm_flag_in_deferred_mode():
    """ABS_FLAG_GRAD_NORM with ABS_FLAG_MLP_DEFER: the norm is formed by the row-based step, so every iteration's rows
    are completed first; |Gbar|^2 and the parameters follow the oracle."""
    import torch

    from paper_2308_15164_b200 import binding as B

    wl = wlm.config(4, small=True, T=3)
    d = wl.mlp
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    o = AbsSgdOracle(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    eng = B.AbsSgd(torch.from_numpy(x0).cuda(), wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=True,
                   mlp=(d.d_in, d.d_hidden, d.d_out, d.mb), mlp_defer=True, grad_norm=True)
    for t, calls in enumerate(wlm.iter_calls(wl)):
        p = o.params()
        for (i, k, c) in calls:
            o.accumulate(i, _grad(p, xs, ys, c, wl))
            eng.accumulate_mlp(i, xs_d[c % wl.mlp_pool], ys_d[c % wl.mlp_pool])
        eng.sync_step(); o.sync_step()
    eng.sync_step(); o.sync_step()
    eng.check()
    assert np.abs(eng.params_host().astype(np.float64) - o.params()).max() <= TOL * np.abs(o.params()).max()
    for s in range(1, 4):
        want = o.gnorm2[s]
        assert want > 0
        assert abs(eng.grad_norm2(s) - want) <= 2 * TOL * want, (s, eng.grad_norm2(s), want)
    eng.destroy()
