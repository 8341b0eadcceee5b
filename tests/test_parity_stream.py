"""GPU parity of the streaming path (accumulate + fused sync step, eager and pipelined) against
the CPU oracle on identical seeded inputs, through the C ABI.

Bars: parameters within 1e-5 * max|param| (fp32 arithmetic; the only differences from the
oracle are fp32-vs-fp64 evaluation of the update and of the W-way sum); b_i counters, set
index and iteration counter bit-exact."""

import dataclasses

import numpy as np
import pytest

from paper_2308_15164_b200 import workloads as wlm
from tests import harness as H

pytestmark = pytest.mark.gpu


def _check(wl, pipelined, columns=None, every_iteration=True, lambda_dc=0.0, lr_schedule=None, host_input=False):
    x0 = wlm.params0(wl)
    pool = wlm.grad_pool(wl) if wl.pool_size else None
    ref = H.oracle_run(wl, x0, pool, columns=columns, lambda_dc=lambda_dc, lr_schedule=lr_schedule)
    got = H.gpu_run(wl, x0, pool, pipelined, columns=columns, lambda_dc=lambda_dc,
                    every_iteration=every_iteration, lr_schedule=lr_schedule, host_input=host_input)
    H.assert_states_equal(got, ref)
    if every_iteration:
        assert len(got["xs"]) == wl.T
        for s, (a, b) in enumerate(zip(got["xs"], ref["xs"])):
            H.assert_params_close(a, b, what=f"{wl.name} x_{s + 1}")
        # x_1 = x_0 exactly (nothing to apply at t = 0)
        x0c = x0 if columns is None else x0[columns]
        assert np.array_equal(got["xs"][0], x0c)
    else:
        H.assert_params_close(got["xs"][-1], ref["xs"][-1], what=f"{wl.name} x_T")
    if not pipelined:       # (pipelined: the in-flight kernel is already one step ahead on v)
        scale_v = np.abs(ref["v"]).max()
        assert np.abs(got["v"] - ref["v"]).max() <= 1e-5 * max(scale_v, 1e-30)
    calls = int(wlm.schedule(wl).sum())
    assert got["launches"] >= calls          # every accumulate is a kernel launch of this library
    return got, ref


@pytest.mark.parametrize("pipelined", [False, True], ids=["eager", "pipelined"])
def test_cfg1_tiny(pipelined):
    _check(wlm.config(1), pipelined)


@pytest.mark.parametrize("pipelined", [False, True], ids=["eager", "pipelined"])
def test_cfg2_resnet18_small_every_element(pipelined):
    _check(wlm.config(2, small=True, T=30), pipelined)


@pytest.mark.parametrize("pipelined", [False, True], ids=["eager", "pipelined"])
def test_cfg3_dynamic_small_every_element(pipelined):
    wl = wlm.config(3, small=True, T=40)
    assert (wlm.schedule(wl) == 0).any()       # idle workers occur
    _check(wl, pipelined)


@pytest.mark.parametrize("pipelined", [False, True], ids=["eager", "pipelined"])
def test_cfg5_bf16_small_every_element(pipelined):
    _check(wlm.config(5, small=True, T=10), pipelined)


def test_host_input_path_matches():
    _check(wlm.config(2, small=True, T=6), True, host_input=True)
    _check(wlm.config(5, small=True, T=4), False, host_input=True)


@pytest.mark.parametrize("lam", [0.5, 2.0])
@pytest.mark.parametrize("pipelined", [False, True], ids=["eager", "pipelined"])
def test_compensation_eq6(pipelined, lam):
    # gradients of size ~1 so that the lambda * Gbar^2 * (x_t - x_{t-1}) term is visible
    wl = dataclasses.replace(wlm.config(1), T=8)
    got, ref = _check(wl, pipelined, lambda_dc=lam)
    plain = H.oracle_run(wl, wlm.params0(wl), None, lambda_dc=0.0)
    assert np.abs(plain["xs"][-1] - ref["xs"][-1]).max() > 1e-3 * np.abs(ref["xs"][-1]).max()


def test_learning_rate_schedule():
    wl = wlm.config(3, small=True, T=12)
    lrs = [0.05 * (0.8 ** t) for t in range(wl.T)]
    _check(wl, False, lr_schedule=lrs)
    _check(wl, True, lr_schedule=lrs)


# ------------------------------------------------------------------ full sizes, sampled outputs
@pytest.mark.parametrize("cfg,T", [(2, 100), (3, 200), (5, 20)])
def test_full_size_sampled_columns(cfg, T):
    """The bench's launch configuration (pipelined) at full size; the oracle follows a sample of
    ~100k parameter positions (windows at both ends and the quarter points plus random picks)."""
    wl = wlm.config(cfg, T=T)
    cols = wlm.sample_columns(wl.P)
    _check(wl, True, columns=cols, every_iteration=False)


@pytest.mark.slow
@pytest.mark.parametrize("cfg,T", [(2, 100), (3, 200), (5, 20)])
def test_full_size_every_element(cfg, T):
    """Workloads 2, 3 and 5 at their full size and length in the bench's launch configuration (pipelined), EVERY
    parameter compared with the oracle -- its C form, which the CPU suite holds to the NumPy oracle within 1e-7
    and which runs the full vectors in tens of seconds on the host cores."""
    from oracle.c_oracle import AbsSgdOracleC

    wl = wlm.config(cfg, T=T)
    x0 = wlm.params0(wl)
    pool = wlm.grad_pool(wl)
    ref = H.oracle_run(wl, x0, pool, oracle_cls=AbsSgdOracleC, every_iteration=False)
    got = H.gpu_run(wl, x0, pool, True, every_iteration=False)
    H.assert_states_equal(got, ref)
    assert got["xs"][-1].shape == (wl.P,)
    rel = H.assert_params_close(got["xs"][-1], ref["xs"][-1], what=f"{wl.name} x_T, all {wl.P} parameters")
    assert np.abs(ref["xs"][-1] - x0).max() > 1e-3 * np.abs(x0).max()      # the run moved the parameters
    print(f"workload {cfg}: max |x_gpu - x_oracle| / max|x| = {rel:.2e} over {wl.P} parameters")


# ------------------------------------------------------------------ edge cases
@pytest.mark.parametrize("P", [1, 3, 4, 5, 255, 256, 257, 1023, 4097, 65537])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_ragged_sizes(P, dtype):
    wl = dataclasses.replace(wlm.config(3, small=True, T=5), P=P, W=3, grad_dtype=dtype, pool_size=4)
    _check(wl, False)
    _check(wl, True)


@pytest.mark.parametrize("W", [1, 2, 7, 16, 17, 33, 64])
def test_worker_counts(W):
    wl = dataclasses.replace(wlm.config(3, small=True, T=6), P=70_001, W=W, pool_size=5)
    _check(wl, False)
    _check(wl, True)


def test_all_idle_iterations_and_double_sync():
    """sum_i b_i = 0: the step is a no-op on x and v, counters and set index still advance."""
    import torch

    from oracle.abs_oracle import AbsSgdOracle
    from paper_2308_15164_b200 import binding as B

    rng = np.random.default_rng(0)
    P, W = 5003, 3
    x0 = rng.standard_normal(P).astype(np.float32)
    grads = [rng.standard_normal(P).astype(np.float32) for _ in range(6)]
    plan = [[(0, 0), (2, 1)], [], [], [(1, 2), (1, 3), (0, 4)], [], [(2, 5)], [], []]
    for pipelined in (False, True):
        o = AbsSgdOracle(x0, W, 0.1, 0.9, 1e-2)
        e = B.AbsSgd(torch.from_numpy(x0).cuda(), W, 0.1, 0.9, 1e-2, pipelined=pipelined)
        gd = [torch.from_numpy(g).cuda() for g in grads]
        torch.cuda.synchronize()
        for step in plan:
            for (i, gi) in step:
                o.accumulate(i, grads[gi]); e.accumulate(i, gd[gi])
            o.sync_step(); e.sync_step()
            c1, cur1, t1 = e.counters(); c2, cur2, t2 = o.counters()
            assert np.array_equal(c1, c2) and (cur1, t1) == (cur2, t2)
            H.assert_params_close(e.params_host(), o.params(), what="x")
        for s in range(len(plan)):
            assert np.array_equal(e.consumed(s), o.consumed[s])
        e.destroy()


def test_eager_and_pipelined_are_bit_identical():
    """Overlapping Step 1 with the next iteration's Step 2 must not change any result."""
    wl = wlm.config(3, small=True, T=25)
    x0 = wlm.params0(wl); pool = wlm.grad_pool(wl)
    a = H.gpu_run(wl, x0, pool, pipelined=False)
    b = H.gpu_run(wl, x0, pool, pipelined=True)
    for s, (xa, xb) in enumerate(zip(a["xs"], b["xs"])):
        assert np.array_equal(xa, xb), f"x_{s + 1} differs between eager and pipelined mode"
    for (c1, cur1, t1), (c2, cur2, t2) in zip(a["states"], b["states"]):
        assert np.array_equal(c1, c2) and (cur1, t1) == (cur2, t2)
    for b1, b2 in zip(a["consumed"], b["consumed"]):
        assert np.array_equal(b1, b2)


@pytest.mark.parametrize("cfg,T", [(2, 12), (3, 40), (5, 6)])
@pytest.mark.parametrize("pipelined", [False, True], ids=["eager", "pipelined"])
def test_overwrite_first_mode_gives_the_same_results(cfg, T, pipelined):
    """Byte-saving variant (no zero writes in the fused step, first micro-batch of a worker stores instead of
    adds): same parameters bit for bit as the default mode, idle workers included, and oracle parity."""
    wl = wlm.config(cfg, small=True, T=T)
    x0 = wlm.params0(wl); pool = wlm.grad_pool(wl)
    a = H.gpu_run(wl, x0, pool, pipelined=pipelined)
    b = H.gpu_run(wl, x0, pool, pipelined=pipelined, overwrite_first=True)
    for s, (xa, xb) in enumerate(zip(a["xs"], b["xs"])):
        assert np.array_equal(xa, xb), f"x_{s + 1} differs in overwrite-first mode"
    ref = H.oracle_run(wl, x0, pool)
    H.assert_states_equal(b, ref)
    H.assert_params_close(b["xs"][-1], ref["xs"][-1], what="overwrite-first x_T")


@pytest.mark.parametrize("batch", [2, 3, 8])
@pytest.mark.parametrize("overwrite_first", [False, True], ids=["clear-in-sync", "overwrite-first"])
@pytest.mark.parametrize("cfg,T", [(2, 12), (3, 30), (5, 6)])
def test_accumulate_batch_equals_single_calls(cfg, T, overwrite_first, batch):
    """abs_accumulate_batch adds a worker's gradients one after the other in list order, in one pass over its
    row: bit-identical parameters to single abs_accumulate calls (fp32 and bf16 gradients, ragged P, idle
    workers), same counters, oracle parity."""
    wl = wlm.config(cfg, small=True, T=T)
    x0 = wlm.params0(wl); pool = wlm.grad_pool(wl)
    a = H.gpu_run(wl, x0, pool, pipelined=True, overwrite_first=overwrite_first)
    b = H.gpu_run(wl, x0, pool, pipelined=True, overwrite_first=overwrite_first, batch=batch)
    assert b["launches"] < a["launches"]
    for s, (xa, xb) in enumerate(zip(a["xs"], b["xs"])):
        assert np.array_equal(xa, xb), f"x_{s + 1} differs with batched accumulation"
    ref = H.oracle_run(wl, x0, pool)
    H.assert_states_equal(b, ref)
    H.assert_params_close(b["xs"][-1], ref["xs"][-1], what="batched accumulate x_T")


@pytest.mark.parametrize("P", [5, 257, 4099])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_accumulate_batch_ragged_and_argument_errors(P, dtype):
    import torch

    from paper_2308_15164_b200 import binding as B

    rng = np.random.default_rng(P)
    n = 5
    g = rng.standard_normal((n, P)).astype(np.float32)
    if dtype == "bf16":
        bits = wlm.f32_to_bf16_bits(g)
        g = (bits.astype(np.uint32) << 16).view(np.float32)
        g_d = [torch.from_numpy(bits[k].view(np.int16)).cuda() for k in range(n)]
    else:
        g_d = [torch.from_numpy(g[k]).cuda() for k in range(n)]
    eng = B.AbsSgd(torch.zeros(P, device="cuda"), 2, 0.1, grad_dtype=B.GRAD_BF16 if dtype == "bf16" else B.GRAD_F32)
    eng.accumulate_batch(1, g_d[:2])
    eng.accumulate_batch(1, g_d[2:])
    want = np.zeros(P, dtype=np.float32)
    for k in range(n):
        want = want + g[k]                       # fp32 adds, same order
    got = eng.accumulator(0, 1)[:P].cpu().numpy()
    assert np.array_equal(got, want)
    assert eng.counters()[0][0].tolist() == [0, n]
    import ctypes
    arr = (ctypes.c_void_p * 9)(*[g_d[0].data_ptr()] * 9)
    assert B.lib.abs_accumulate_batch(eng._h, 0, 9, arr) == B.EINVAL           # more than 8
    assert B.lib.abs_accumulate_batch(eng._h, 0, 0, arr) == B.EINVAL
    assert B.lib.abs_accumulate_batch(eng._h, 2, 1, arr) == B.EINVAL           # worker out of range
    arr[1] = None
    assert B.lib.abs_accumulate_batch(eng._h, 0, 2, arr) == B.EINVAL           # NULL entry
    assert eng.counters()[0][0].tolist() == [0, n]                              # nothing was enqueued
    eng.destroy()


def test_accumulator_matches_oracle_bitwise():
    """fp32 adds of the same operands in the same order: the accumulators agree bit for bit."""
    import torch

    from oracle.abs_oracle import AbsSgdOracle
    from paper_2308_15164_b200 import binding as B

    wl = wlm.config(2, small=True, T=1)
    x0 = wlm.params0(wl); pool = wlm.grad_pool(wl)
    o = AbsSgdOracle(x0, wl.W, wl.lr)
    e = B.AbsSgd(torch.from_numpy(x0).cuda(), wl.W, wl.lr)
    pool_d = torch.from_numpy(pool).cuda()
    torch.cuda.synchronize()
    for (i, k, c) in next(iter(wlm.iter_calls(wl))):
        o.accumulate(i, pool[c % wl.pool_size]); e.accumulate(i, pool_d[c % wl.pool_size])
    e.synchronize()
    for i in range(wl.W):
        assert np.array_equal(e.accumulator(0, i).cpu().numpy(), o.acc[0, i])
    e.destroy()


def test_cuda_graph_replay_of_the_tiny_workload():
    """Workload 1 is launch-bound (5 launches of a few microseconds per iteration).  In eager mode every call
    enqueues on stream_acc only, so two iterations (the accumulator sets alternate with period 2) can be captured
    into a CUDA graph and replayed; the parameters after R replays match the oracle after 2 + 2 R iterations."""
    import torch

    from oracle.abs_oracle import AbsSgdOracle
    from paper_2308_15164_b200 import binding as B

    wl = wlm.config(1)
    order = wlm.call_order(wlm.schedule(wl)[0])                 # b = (3, 1): 4 calls per iteration
    rng = np.random.default_rng(21)
    x0 = wlm.params0(wl)
    pool = (rng.standard_normal((8, wl.P)) * 0.5).astype(np.float32)
    pool_d = [torch.from_numpy(pool[j]).cuda() for j in range(8)]
    eng = B.AbsSgd(torch.from_numpy(x0).cuda(), wl.W, wl.lr, wl.momentum, wl.weight_decay)   # eager
    c = [0]

    def two_iterations():
        for _ in range(2):
            for (i, k) in order:
                eng.accumulate(i, pool_d[c[0] % 8]); c[0] += 1
            eng.sync_step()

    with torch.cuda.stream(eng.stream_acc):
        two_iterations()                                        # iterations 0, 1 (the first step applies nothing)
    eng.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=eng.stream_acc):
        two_iterations()                                        # recorded, not run
    R = 25
    for _ in range(R):
        g.replay()
    torch.cuda.synchronize()
    got = eng.params_host()
    eng.destroy()

    o = AbsSgdOracle(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    cc = 0
    for _ in range(2 + 2 * R):
        for (i, k) in order:
            o.accumulate(i, pool[cc % 8]); cc += 1
        o.sync_step()
    want = o.params()
    assert np.abs(want - x0).max() > 1e-3
    assert np.abs(got - want).max() <= H.TOL_F32 * np.abs(want).max()
