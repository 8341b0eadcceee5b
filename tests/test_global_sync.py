"""Step 1 across GPUs (abs_global_*): G ranks, each a context with W_local workers, driven in one process on one
GPU (dist.LocalRanks: plain pointers instead of peer mappings, events instead of collectives; no kernel waits
for another rank's).  Checked against
  * the CPU oracle with G * W_local workers (the paper's definition: the average runs over ALL workers), within
    1e-5 * max|param|, counters bit-exact;
  * a one-GPU context with G * W_local workers fed the same gradients: parameters bit for bit, the rank's slice
    of the momentum bit for bit.
"""

import ctypes

import numpy as np
import pytest

from paper_2308_15164_b200 import workloads as wlm
from tests import harness as H

pytestmark = pytest.mark.gpu


def _pool_on_device(pool, dev):
    import torch

    src = torch.from_numpy(pool.view(np.int16) if pool.dtype == np.uint16 else pool)
    pool_d = torch.zeros((pool.shape[0], (pool.shape[1] + 7) // 8 * 8), dtype=src.dtype, device=dev)
    pool_d[:, :pool.shape[1]] = src.to(dev)
    return pool_d


def _run(wl, sched, G, lambda_dc=0.0, overwrite_first=False, lr_schedule=None):
    """Runs the schedule `sched` [T][W] three ways on the same gradients and returns
    (oracle xs, one-context xs, ranks xs [T][G], extras)."""
    import torch

    from oracle.abs_oracle import AbsSgdOracle
    from paper_2308_15164_b200 import binding as B
    from paper_2308_15164_b200 import dist as D

    dev = torch.device("cuda:0")
    W = wl.W
    assert W % G == 0
    Wl = W // G
    x0 = wlm.params0(wl)
    pool = wlm.grad_pool(wl)
    pool_d = _pool_on_device(pool, dev)
    gd = B.GRAD_BF16 if wl.grad_dtype == "bf16" else B.GRAD_F32
    x0_d = torch.from_numpy(x0).to(dev)
    torch.cuda.synchronize()

    ref = AbsSgdOracle(x0, W, wl.lr, wl.momentum, wl.weight_decay, lambda_dc)
    one = B.AbsSgd(x0_d, W, wl.lr, wl.momentum, wl.weight_decay, lambda_dc, grad_dtype=gd, pipelined=True,
                   overwrite_first=overwrite_first)
    ranks = [B.AbsSgd(x0_d, Wl, wl.lr, wl.momentum, wl.weight_decay, lambda_dc, grad_dtype=gd, pipelined=True,
                      overwrite_first=overwrite_first) for _ in range(G)]
    grp = D.LocalRanks(ranks)

    def read(eng):
        with torch.cuda.stream(eng.stream_acc):
            p = eng.params().clone()
        eng.stream_acc.synchronize()
        return p.cpu().numpy()

    xs_ref, xs_one, xs_rk, states = [], [], [], []
    c = 0
    for t, b_row in enumerate(sched):
        if lr_schedule is not None and t + 1 < len(lr_schedule):
            for e in [one] + ranks:
                e.set_lr(float(lr_schedule[t + 1]))
        if lr_schedule is not None:
            ref.lr = lr_schedule[t]
        for (i, k) in wlm.call_order(b_row):
            g = pool[c % wl.pool_size]
            ref.accumulate(i, g)
            one.accumulate(i, pool_d[c % wl.pool_size])
            ranks[i // Wl].accumulate(i % Wl, pool_d[c % wl.pool_size])     # global worker i = rank * W_local + local
            c += 1
        ref.sync_step()
        one.sync_step()
        grp.sync_step()
        xs_ref.append(ref.params().copy())
        xs_one.append(read(one))
        xs_rk.append([read(e) for e in ranks])
        states.append((ref.counters(), [e.counters() for e in ranks]))
    T = len(sched)
    extras = dict(consumed_ref=[np.asarray(b) for b in ref.consumed],
                  consumed_rk=[[e.global_consumed(s) for s in range(max(0, T - 60), T)] for e in ranks],
                  consumed_from=max(0, T - 60), slices=[e.global_slice() for e in ranks], states=states)
    # momentum: the in-flight kernels are one step ahead of the published parameters on every path alike
    one.wait()
    for e in ranks:
        e.wait()
    torch.cuda.synchronize()
    extras["v_one"] = one.momentum().clone().cpu().numpy()
    extras["v_rk"] = [e.momentum().clone().cpu().numpy() for e in ranks]
    for e in [one] + ranks:
        e.check()
        e.destroy()
    return xs_ref, xs_one, xs_rk, extras


def _assert_all(wl, sched, G, xs_ref, xs_one, xs_rk, ex):
    Wl = wl.W // G
    for t in range(len(sched)):
        for r in range(G):
            assert np.array_equal(xs_rk[t][r], xs_one[t]), f"x_{t + 1} on rank {r} differs from the one-GPU context"
        H.assert_params_close(xs_rk[t][0], xs_ref[t], what=f"x_{t + 1}")
        (cr, curr, tr), per_rank = ex["states"][t]
        for r, (cg, curg, tg) in enumerate(per_rank):
            assert np.array_equal(cg, cr[:, r * Wl:(r + 1) * Wl]) and (curg, tg) == (curr, tr)
    f = ex["consumed_from"]
    for r in range(G):
        for s, b in enumerate(ex["consumed_rk"][r]):
            assert np.array_equal(b, ex["consumed_ref"][f + s]), (r, f + s, b, ex["consumed_ref"][f + s])
    at = 0
    for r, (first, count) in enumerate(ex["slices"]):
        assert first == at or count == 0
        at = first + count
        assert np.array_equal(ex["v_rk"][r][first:first + count], ex["v_one"][first:first + count]), f"momentum slice of rank {r}"
    assert at == wl.P


@pytest.mark.parametrize("G", [2, 4])
def test_workload2_small_ranks_equal_one_context_and_oracle(G):
    wl = wlm.config(2, small=True, T=12)
    sched = wlm.schedule(wl)
    out = _run(wl, sched, G)
    _assert_all(wl, sched, G, *out)
    assert np.array_equal(out[2][0][0], wlm.params0(wl))       # x_1 = x_0


@pytest.mark.parametrize("G", [2, 8])
def test_workload3_small_idle_workers_and_an_idle_iteration(G):
    wl = wlm.config(3, small=True, T=24)
    sched = wlm.schedule(wl).copy()
    assert (sched == 0).any()
    sched[5, :] = 0                  # nobody computed anything: x_7 = x_6 on every rank, v untouched
    sched[11, :wl.W // 2] = 0        # the first half of the ranks idle (whole ranks when G = 2)
    out = _run(wl, sched, G)
    _assert_all(wl, sched, G, *out)
    assert np.array_equal(out[2][6][0], out[2][5][0])


def test_workload5_small_bf16_gradients_sixteen_workers_on_four_ranks():
    wl = wlm.config(5, small=True, T=6)
    sched = wlm.schedule(wl)
    out = _run(wl, sched, 4)
    _assert_all(wl, sched, 4, *out)


def test_overwrite_first_mode_and_learning_rate_schedule():
    wl = wlm.config(3, small=True, T=12)
    sched = wlm.schedule(wl)
    lrs = [wl.lr * (0.5 ** (t // 4)) for t in range(wl.T)]
    out = _run(wl, sched, 4, overwrite_first=True, lr_schedule=lrs)
    _assert_all(wl, sched, 4, *out)


@pytest.mark.parametrize("lam", [0.5, 2.0])
def test_compensation_eq6_across_ranks_with_a_no_op_step_in_between(lam):
    import dataclasses

    wl = dataclasses.replace(wlm.config(3, small=True, T=10), grad_std=1.0, lr=0.02)
    sched = wlm.schedule(wl).copy()
    sched[4, :] = 0                  # the step after it must use x_t - x_{t-1} = 0 (decided on the device)
    out = _run(wl, sched, 2, lambda_dc=lam)
    _assert_all(wl, sched, 2, *out)
    plain = _run(wl, sched, 2, lambda_dc=0.0)
    assert np.abs(plain[0][-1] - out[0][-1]).max() > 1e-4 * np.abs(out[0][-1]).max()     # the term is visible


def test_small_vector_leaves_trailing_ranks_without_a_slice():
    import dataclasses

    wl = dataclasses.replace(wlm.config(3, small=True, T=6), P=2500, W=8)
    sched = wlm.schedule(wl)
    out = _run(wl, sched, 4)
    _assert_all(wl, sched, 4, *out)
    assert [s[1] for s in out[3]["slices"]] == [1024, 1024, 452, 0]


def test_call_order_and_mode_errors():
    import torch

    from paper_2308_15164_b200 import binding as B

    dev = torch.device("cuda:0")
    x0 = torch.zeros(4096, device=dev)
    eager = B.AbsSgd(x0, 2, 0.1)
    with pytest.raises(B.AbsError):
        eager.global_attach(0, [eager.workspace.data_ptr()])          # needs two parameter buffers
    eager.destroy()
    a = B.AbsSgd(x0, 2, 0.1, pipelined=True)
    b = B.AbsSgd(x0, 2, 0.1, pipelined=True)
    with pytest.raises(B.AbsError):
        a.global_begin()                                              # not attached
    spaces = [a.workspace.data_ptr(), b.workspace.data_ptr()]
    with pytest.raises(B.AbsError):
        a.global_attach(1, spaces)                                    # own workspace is not at [rank]
    with pytest.raises(B.AbsError):
        a.global_attach(0, spaces + [0])                              # NULL peer
    a.global_attach(0, spaces)
    b.global_attach(1, spaces)
    with pytest.raises(B.AbsError):
        a.global_attach(0, spaces)                                    # twice
    with pytest.raises(B.AbsError):
        a.sync_step()                                                 # one-GPU step on a multi-GPU context
    for call in (a.global_step, a.global_end):
        with pytest.raises(B.AbsError):
            call()                                                    # before abs_global_begin
    a.global_begin()
    with pytest.raises(B.AbsError):
        a.global_begin()
    with pytest.raises(B.AbsError):
        a.global_end()
    b.global_begin()
    torch.cuda.synchronize()
    a.global_step(); b.global_step()
    with pytest.raises(B.AbsError):
        a.global_step()
    torch.cuda.synchronize()
    a.global_end(); b.global_end()
    big = [B.AbsSgd(x0, 33, 0.1, pipelined=True) for _ in range(2)]
    with pytest.raises(B.AbsError):
        big[0].global_attach(0, [e.workspace.data_ptr() for e in big])    # 2 * 33 workers > 64
    for e in [a, b] + big:
        e.check()
        e.destroy()


@pytest.mark.parametrize("defer", [False, True], ids=["per-call-dw1", "deferred-dw1"])
def test_mlp_gradients_computed_on_two_ranks_match_one_context_and_oracle(defer):
    """Workload 4 (small layer sizes): every rank computes its workers' MLP gradients at x_t (single and batch
    calls) -- the fused kernel must also refresh every rank's bf16 copy of the weights, which the next forward
    pass reads.  With ABS_FLAG_MLP_DEFER the ranks complete their rows when the iteration ends (one contraction per
    worker); the one-GPU context they are compared with bit for bit does the same (its step from the pooled
    operands would sum in another order)."""
    import torch

    from oracle.abs_oracle import AbsSgdOracle, mlp_loss_and_grad
    from paper_2308_15164_b200 import binding as B
    from paper_2308_15164_b200 import dist as D

    G, T = 2, 8
    wl = wlm.config(4, small=True, T=T)
    d = wl.mlp
    Wl = wl.W // G
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    sched = wlm.schedule(wl).copy()
    sched[2, 1] = 0                                   # an idle worker
    dev = torch.device("cuda:0")
    xs_d, ys_d = torch.from_numpy(xs).to(dev), torch.from_numpy(ys).to(dev)
    x0_d = torch.from_numpy(x0).to(dev)
    torch.cuda.synchronize()
    mlp = (d.d_in, d.d_hidden, d.d_out, d.mb)
    one = B.AbsSgd(x0_d, wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=True, mlp=mlp, mlp_defer=defer)
    if defer:
        one.set_launch(B.K_MLP_BWD, 1)
    ranks = [B.AbsSgd(x0_d, Wl, wl.lr, wl.momentum, wl.weight_decay, pipelined=True, mlp=mlp, mlp_defer=defer) for _ in range(G)]
    grp = D.LocalRanks(ranks)
    ref = AbsSgdOracle(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    for t, b_row in enumerate(sched):
        p = ref.params()
        for i, b in enumerate(b_row):                 # worker by worker: up to 2 reference batches per call
            lo = (7 * t + 3 * i) % (wl.mlp_pool - 8)
            k = 0
            while k < int(b):
                n = min(2, int(b) - k)
                for j in range(n):
                    _, g, _ = mlp_loss_and_grad(p, xs[lo + k + j], ys[lo + k + j], d.d_in, d.d_hidden, d.d_out, mode="bf16")
                    ref.accumulate(i, g.astype(np.float32))
                for eng, w in ((one, i), (ranks[i // Wl], i % Wl)):
                    if n == 1:
                        eng.accumulate_mlp(w, xs_d[lo + k], ys_d[lo + k])
                    else:
                        eng.accumulate_mlp_batch(w, n, xs_d[lo + k:lo + k + n], ys_d[lo + k:lo + k + n])
                k += n
        ref.sync_step()
        one.sync_step()
        grp.sync_step()
        got_one = one.params_host()
        for r, e in enumerate(ranks):
            assert np.array_equal(e.params_host(), got_one), f"x_{t + 1} on rank {r}"
    want = ref.params()
    assert np.abs(want - x0).max() > 1e-4
    assert np.abs(got_one.astype(np.float64) - want).max() <= H.TOL_BF16 * np.abs(want).max()
    for r, e in enumerate(ranks):
        for s in range(T):
            assert np.array_equal(e.global_consumed(s), np.asarray(ref.consumed[s]))
    for e in [one] + ranks:
        e.check()
        e.destroy()
