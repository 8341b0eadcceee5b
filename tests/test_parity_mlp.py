"""GPU parity of the MLP micro-batch gradient (forward, loss, backward, tcgen05 dW1 GEMM with the
accumulate epilogue) and of full MLP training runs against the CPU oracle, through the C ABI.

Bars: every gradient tensor within 2e-3 * max|ref| element-wise and 2e-3 in Frobenius norm of the
bf16-emulating oracle evaluated at the same parameters; end-of-run parameters within
2e-3 * max|param|; counters bit-exact.

The ReLU gate [Z > 0] is a discrete decision taken on a floating-point number.  The GPU
accumulates Z in fp32, the oracle in fp64, so for the handful of pre-activations with
|Z| < 1e-4 (fp32 accumulation error is ~1e-6 here) either gate value is a valid outcome.  Those
hidden units are compared against every valid outcome; all others are compared strictly."""

import itertools

import numpy as np
import pytest

from oracle.abs_oracle import AbsSgdOracle, bf16_round, mlp_loss_and_grad, mlp_split
from paper_2308_15164_b200 import workloads as wlm

pytestmark = pytest.mark.gpu

TOL = 2e-3
TAU = 1e-4


def _engine(wl, x0, pipelined=False, epilogue=0, overwrite_first=False):
    import torch

    from paper_2308_15164_b200 import binding as B

    d = wl.mlp
    eng = B.AbsSgd(torch.from_numpy(x0).cuda(), wl.W, wl.lr, wl.momentum, wl.weight_decay,
                   pipelined=pipelined, mlp=(d.d_in, d.d_hidden, d.d_out, d.mb), overwrite_first=overwrite_first)
    eng.set_launch(B.K_MLP_DW1, epilogue)
    return eng


def _close(got, ref, what):
    scale = np.abs(ref).max()
    assert np.abs(got - ref).max() <= TOL * scale, f"{what}: max err {np.abs(got - ref).max():.3e} vs {TOL}*{scale:.3e}"
    assert np.linalg.norm(got - ref) <= TOL * np.linalg.norm(ref), f"{what}: Frobenius"


def _check_gradient(got_flat, params, X, y, dims):
    d_in, d_h, d_out = dims
    _, ref, aux = mlp_loss_and_grad(params, X, y, d_in, d_h, d_out, mode="bf16")
    dW1, db1, dW2, db2 = mlp_split(ref, d_in, d_h, d_out)
    gW1, gb1, gW2, gb2 = mlp_split(got_flat.astype(np.float64), d_in, d_h, d_out)
    Z = aux["Z"]
    amb = np.argwhere(np.abs(Z) < TAU)
    amb_cols = sorted(set(int(h) for _, h in amb))
    assert len(amb) < 1e-3 * Z.size
    clear = np.setdiff1d(np.arange(d_h), amb_cols)
    _close(gW2, dW2, "dW2")
    _close(gb2, db2, "db2")
    _close(gW1[:, clear], dW1[:, clear], "dW1")
    _close(gb1[clear], db1[clear], "db1")
    # undecided gates: the column must equal the reference with some subset of them inverted
    sW1, sb1 = TOL * np.abs(dW1).max(), TOL * np.abs(db1).max()
    for h in amb_cols:
        rows = [int(r) for r, hh in amb if hh == h]
        assert len(rows) <= 4
        ok = False
        for k in range(len(rows) + 1):
            for sub in itertools.combinations(rows, k):
                col, b = dW1[:, h].copy(), db1[h]
                for r in sub:
                    sign = -1.0 if Z[r, h] > 0 else 1.0          # gate on -> remove, gate off -> add
                    col += sign * aux["X"][r] * bf16_round(aux["dH"][r, h])
                    b += sign * aux["dH"][r, h]
                if np.abs(gW1[:, h] - col).max() <= sW1 and abs(gb1[h] - b) <= sb1:
                    ok = True
        assert ok, f"hidden unit {h}: no valid gate assignment reproduces the GPU column"
    return len(amb)


@pytest.mark.parametrize("epilogue", [0, 16, 1, 2, 64, 4, 8],
                         ids=["auto", "tma-load-add-store", "tma-reduce", "cuda-core-forward", "cluster-fused-forward",
                              "persistent-ring-dw1", "register-prefetch-dw1"])
@pytest.mark.parametrize("small", [True, False], ids=["384x512", "3072x4096"])
def test_single_microbatch_gradient(small, epilogue):
    wl = wlm.config(4, small=small)
    d = wl.mlp
    dims = (d.d_in, d.d_hidden, d.d_out)
    x0 = wlm.params0(wl)
    # non-zero biases so that b1 / b2 handling is exercised
    rng = np.random.default_rng(7)
    o_w1, o_b1, o_w2, o_b2 = d.offsets
    x0[o_b1:o_w2] = rng.standard_normal(d.d_hidden).astype(np.float32) * 0.1
    x0[o_b2:] = rng.standard_normal(d.d_out).astype(np.float32) * 0.1
    xs, ys = wlm.mlp_batches(wl)
    import torch

    eng = _engine(wl, x0, epilogue=epilogue)
    for b in (0, 5):
        xd, yd = torch.from_numpy(xs[b]).cuda(), torch.from_numpy(ys[b]).cuda()
        torch.cuda.synchronize()
        eng.accumulate_mlp(b % wl.W, xd, yd)
        eng.check()
        got = eng.accumulator(0, b % wl.W).cpu().numpy()
        _check_gradient(got, x0, xs[b], ys[b], dims)
    cnt, cur, t = eng.counters()
    assert cnt[0].tolist() == [1, 1, 0, 0] and cur == 0 and t == 0
    # A worker's first gradient of an iteration is stored, later ones are added: the second call on worker 0
    # takes the read-modify-write path; what it added must be the gradient of its micro-batch.
    before = eng.accumulator(0, 0).cpu().numpy().astype(np.float64)
    xd, yd = torch.from_numpy(xs[3]).cuda(), torch.from_numpy(ys[3]).cuda()
    torch.cuda.synchronize()
    eng.accumulate_mlp(0, xd, yd)
    eng.check()
    after = eng.accumulator(0, 0).cpu().numpy().astype(np.float64)
    _check_gradient(after - before, x0, xs[3], ys[3], dims)
    assert eng.counters()[0][0].tolist() == [2, 1, 0, 0]
    eng.destroy()


def test_two_microbatches_add_up():
    """The epilogue accumulates: two calls into the same worker give the sum of both gradients."""
    import torch

    wl = wlm.config(4, small=True)
    d = wl.mlp
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    eng = _engine(wl, x0)
    want = np.zeros(wl.P)
    for b in (1, 2, 3):
        xd, yd = torch.from_numpy(xs[b]).cuda(), torch.from_numpy(ys[b]).cuda()
        torch.cuda.synchronize()
        eng.accumulate_mlp(2, xd, yd)
        eng.check()
        want += mlp_loss_and_grad(x0, xs[b], ys[b], d.d_in, d.d_hidden, d.d_out, mode="bf16")[1]
    got = eng.accumulator(0, 2).cpu().numpy().astype(np.float64)
    # norm-wise: a few undecided ReLU gates may differ (see module docstring)
    assert np.linalg.norm(got - want) <= 2e-2 * np.linalg.norm(want)
    dW2g, dW2w = mlp_split(got, d.d_in, d.d_hidden, d.d_out)[2], mlp_split(want, d.d_in, d.d_hidden, d.d_out)[2]
    _close(dW2g, dW2w, "dW2 (3 micro-batches)")
    assert eng.counters()[0][0].tolist() == [0, 0, 3, 0]
    eng.destroy()


def _run_training(wl, pipelined, x0, xs, ys, eng=None, overwrite_first=False):
    import torch

    d = wl.mlp
    own = eng is None
    if own:
        eng = _engine(wl, x0, pipelined=pipelined, overwrite_first=overwrite_first)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    torch.cuda.synchronize()
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


def _oracle_training(wl, x0, xs, ys):
    d = wl.mlp
    o = AbsSgdOracle(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    states = []
    for t, calls in enumerate(wlm.iter_calls(wl)):
        p = o.params()                                # all micro-batches of iteration t see x_t
        for (i, k, c) in calls:
            _, g, _ = mlp_loss_and_grad(p, xs[c % wl.mlp_pool], ys[c % wl.mlp_pool], d.d_in, d.d_hidden, d.d_out, mode="bf16")
            o.accumulate(i, g.astype(np.float32))
        o.sync_step()
        states.append(o.counters())
    return o.params(), states, o.consumed


@pytest.mark.parametrize("small,T", [(True, 12), (False, 5)], ids=["384x512-T12", "3072x4096-T5"])
def test_training_run_matches_oracle(small, T):
    wl = wlm.config(4, small=small, T=T)
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    ref, ref_states, ref_consumed = _oracle_training(wl, x0, xs, ys)
    assert np.abs(ref - x0).max() > 1e-4              # the run moved the parameters
    outs = []
    for pipelined in (False, True):
        got, states, consumed = _run_training(wl, pipelined, x0, xs, ys)
        err = np.abs(got.astype(np.float64) - ref).max()
        assert err <= TOL * np.abs(ref).max(), f"pipelined={pipelined}: {err:.3e}"
        for (c1, cur1, t1), (c2, cur2, t2) in zip(states, ref_states):
            assert np.array_equal(c1, c2) and (cur1, t1) == (cur2, t2)
        for a, b in zip(consumed, ref_consumed):
            assert np.array_equal(a, b)
        outs.append(got)
    assert np.array_equal(outs[0], outs[1]), "eager and pipelined runs must be bit-identical"
    # byte-saving mode (accumulator rows are not cleared; every worker's first gradient overwrites its row)
    got, states, consumed = _run_training(wl, True, x0, xs, ys, overwrite_first=True)
    assert np.array_equal(got, outs[0]), "overwrite-first mode must give the same parameters"
    for a, b in zip(consumed, ref_consumed):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("epilogue", [0, 8, 4, 36], ids=["auto", "tile-per-cta", "persistent-ring-128x128", "persistent-ring-128x64"])
@pytest.mark.parametrize("n", [2, 3, 4])
@pytest.mark.parametrize("small", [True, False], ids=["384x512", "3072x4096"])
def test_batched_microbatches_match_the_sum_of_gradients(small, n, epilogue):
    """abs_accumulate_mlp_batch: n reference batches of one worker contracted by one K = 64 n GEMM give the sum
    of the n micro-batch gradients (b_i += n)."""
    import torch

    wl = wlm.config(4, small=small)
    d = wl.mlp
    dims = (d.d_in, d.d_hidden, d.d_out)
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    eng = _engine(wl, x0, epilogue=epilogue)
    b0 = 8
    xd, yd = torch.from_numpy(xs[b0:b0 + n]).cuda().contiguous(), torch.from_numpy(ys[b0:b0 + n]).cuda().contiguous()
    torch.cuda.synchronize()
    eng.accumulate_mlp_batch(3, n, xd, yd)
    eng.check()
    got = eng.accumulator(0, 3).cpu().numpy().astype(np.float64)
    assert eng.counters()[0][0].tolist() == [0, 0, 0, n]
    want = np.zeros(wl.P)
    undecided = set()
    for j in range(n):
        _, g, aux = mlp_loss_and_grad(x0, xs[b0 + j], ys[b0 + j], *dims, mode="bf16")
        want += g
        undecided |= set(int(h) for _, h in np.argwhere(np.abs(aux["Z"]) < TAU))
    clear = np.setdiff1d(np.arange(d.d_hidden), sorted(undecided))
    gW1, gb1, gW2, gb2 = mlp_split(got, *dims)
    wW1, wb1, wW2, wb2 = mlp_split(want, *dims)
    _close(gW2, wW2, "dW2"); _close(gb2, wb2, "db2")
    _close(gW1[:, clear], wW1[:, clear], "dW1"); _close(gb1[clear], wb1[clear], "db1")
    # hidden units with an undecided ReLU gate: bounded by the contribution of those few gates
    if undecided:
        u = sorted(undecided)
        assert np.abs(gW1[:, u] - wW1[:, u]).max() <= 0.2 * np.abs(wW1).max()
    # and the same data through n single calls agrees to fp32 rounding of the sums
    eng2 = _engine(wl, x0, epilogue=epilogue)
    for j in range(n):
        eng2.accumulate_mlp(3, xd[j], yd[j])
    eng2.check()
    single = eng2.accumulator(0, 3).cpu().numpy().astype(np.float64)
    assert np.abs(got - single).max() <= 1e-5 * np.abs(single).max()
    # a second call on the same worker takes the adding path: the row doubles
    eng.accumulate_mlp_batch(3, n, xd, yd)
    eng.check()
    twice = eng.accumulator(0, 3).cpu().numpy().astype(np.float64)
    assert np.abs(twice - 2.0 * got).max() <= 1e-5 * np.abs(got).max()
    assert eng.counters()[0][0].tolist() == [0, 0, 0, 2 * n]
    eng.destroy(); eng2.destroy()


# Hand-made schedule for the small network: idle workers (rows of zeros stay stale in overwrite-first mode), all
# workers idle, batch calls of every size, and precomputed gradients (abs_accumulate) mixed into the same rows
# before and after a device-computed one -- the first call of a worker in an iteration stores, whatever its kind.
# Entry: (worker, kind, n) with kind "mlp" (n micro-batches in one call) or "vec" (one precomputed gradient).
_MIXED = [
    [(0, "mlp", 1), (2, "mlp", 3), (0, "mlp", 2), (3, "vec", 1), (3, "mlp", 1)],
    [(1, "mlp", 4), (1, "vec", 1), (0, "mlp", 1)],
    [],
    [(3, "mlp", 2), (3, "mlp", 2), (2, "vec", 1), (2, "vec", 1), (2, "mlp", 1)],
    [(0, "vec", 1)],
    [(1, "mlp", 1), (2, "mlp", 4), (3, "mlp", 3), (0, "mlp", 2)],
    [(2, "mlp", 1)],
]


@pytest.mark.parametrize("overwrite_first", [False, True], ids=["clear-in-sync", "overwrite-first"])
@pytest.mark.parametrize("pipelined", [False, True], ids=["eager", "pipelined"])
def test_mixed_calls_idle_workers_and_batches(pipelined, overwrite_first):
    import torch

    wl = wlm.config(4, small=True, T=len(_MIXED))
    d = wl.mlp
    dims = (d.d_in, d.d_hidden, d.d_out)
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    vec = np.random.default_rng(11).standard_normal((3, wl.P)).astype(np.float32) * 1e-3
    # oracle
    o = AbsSgdOracle(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    ref_states, c = [], 0
    for calls in _MIXED:
        p = o.params()
        for (i, kind, n) in calls:
            for _ in range(n):
                if kind == "mlp":
                    g = mlp_loss_and_grad(p, xs[c % wl.mlp_pool], ys[c % wl.mlp_pool], *dims, mode="bf16")[1].astype(np.float32)
                else:
                    g = vec[c % 3]
                o.accumulate(i, g)
                c += 1
        o.sync_step()
        ref_states.append(o.counters())
    ref = o.params()
    assert np.abs(ref - x0).max() > 1e-5
    # library
    eng = _engine(wl, x0, pipelined=pipelined, overwrite_first=overwrite_first)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    vec_d = [torch.from_numpy(vec[j]).cuda() for j in range(3)]   # one allocation each: 16-byte aligned
    torch.cuda.synchronize()
    c = 0
    for t, calls in enumerate(_MIXED):
        for (i, kind, n) in calls:
            if kind == "mlp":
                lo = c % wl.mlp_pool
                assert lo + n <= wl.mlp_pool
                eng.accumulate_mlp_batch(i, n, xs_d[lo:lo + n], ys_d[lo:lo + n])
            else:
                eng.accumulate(i, vec_d[c % 3])
            c += n
        eng.sync_step()
        cnt, cur, tt = eng.counters()
        assert np.array_equal(cnt, ref_states[t][0]) and (cur, tt) == ref_states[t][1:]
    eng.check()
    got = eng.params_host()
    consumed = [eng.consumed(s) for s in range(len(_MIXED))]
    eng.destroy()
    assert np.abs(got.astype(np.float64) - ref).max() <= TOL * np.abs(ref).max()
    for a, b in zip(consumed, o.consumed):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("n", [1, 2, 3, 4])
@pytest.mark.parametrize("small", [True, False], ids=["384x512", "3072x4096"])
def test_cluster_fused_forward_is_bit_identical_to_the_two_kernel_forward(small, n):
    """The cluster kernel adds the K-split partial sums in the same order as k_fwd2 does: same H, same logits,
    hence the same accumulator bits."""
    import torch

    wl = wlm.config(4, small=small)
    x0 = wlm.params0(wl)
    rng = np.random.default_rng(3)
    d = wl.mlp
    o_w1, o_b1, o_w2, o_b2 = d.offsets
    x0[o_b1:o_w2] = rng.standard_normal(d.d_hidden).astype(np.float32) * 0.1
    xs, ys = wlm.mlp_batches(wl)
    xd, yd = torch.from_numpy(xs[20:20 + n]).cuda().contiguous(), torch.from_numpy(ys[20:20 + n]).cuda().contiguous()
    torch.cuda.synchronize()
    outs = []
    for variant in (0, 64):
        eng = _engine(wl, x0, epilogue=variant)
        eng.accumulate_mlp_batch(1, n, xd, yd)
        eng.accumulate_mlp_batch(1, n, xd, yd)
        eng.check()
        outs.append(eng.accumulator(0, 1).cpu().numpy())
        eng.destroy()
    assert np.array_equal(outs[0], outs[1])
