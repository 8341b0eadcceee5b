"""Pins for the CPU oracle: facts fixed by Algorithm 1 (arXiv 2308.15164) and by mathematics.

Each pin is a function taking a *factory* ``make(x0, W, lr, momentum, weight_decay,
lambda_dc) -> oracle`` and raising AssertionError when the oracle breaks the fact.
tests/test_oracle_pins.py runs every pin on the real oracles (all must pass) and on
deliberately broken copies (each must be caught by at least one pin).
"""

from __future__ import annotations

import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split()
            out[k] = float(v)
    return out


def _grads(rng, P, counts, integer=True):
    """{(i,k): g} with small-integer entries, so fp32 accumulation is exact."""
    out = {}
    for i, b in enumerate(counts):
        for k in range(b):
            g = rng.integers(-8, 9, size=P).astype(np.float32) if integer else rng.standard_normal(P).astype(np.float32)
            out[(i, k)] = g
    return out


def _run(o, schedule, grads_per_iter):
    """Feed iterations; return [x after sync call #0, #1, ...] (i.e. x_1, x_2, ...)."""
    xs = []
    for counts, grads in zip(schedule, grads_per_iter):
        for i, b in enumerate(counts):
            for k in range(b):
                o.accumulate(i, grads[(i, k)])
        o.sync_step()
        xs.append(o.params().astype(np.float64))
    return xs


def _gbar(counts, grads):
    tot = sum(grads[(i, k)].astype(np.float64) for i, b in enumerate(counts) for k in range(b))
    return tot / sum(counts)


# P1 ---------------------------------------------------------------------------------------
def pin_single_worker_is_delayed_momentum_sgd(make):
    """W=1: the run is plain momentum SGD on Gbar_t = mean of the worker's micro-batch
    gradients, applied one iteration late."""
    rng = np.random.default_rng(11)
    P, T, lr, mu, wd = 37, 6, 0.05, 0.9, 0.01
    x0 = rng.standard_normal(P).astype(np.float32)
    sched = [(int(rng.integers(1, 5)),) for _ in range(T)]
    gl = [_grads(rng, P, c) for c in sched]
    xs = _run(make(x0, 1, lr, mu, wd, 0.0), sched, gl)
    x = x0.astype(np.float64); v = np.zeros(P)
    assert np.array_equal(xs[0], x0.astype(np.float64))
    for s in range(1, T):
        g = _gbar(sched[s - 1], gl[s - 1]) + wd * x
        v = mu * v + g
        x = x - lr * v
        np.testing.assert_allclose(xs[s], x, rtol=0, atol=2e-6 * np.abs(x).max())


# P2 ---------------------------------------------------------------------------------------
def pin_equal_counts_give_uniform_average(make):
    """All b_i equal: the weighted average equals the plain mean of the per-worker means."""
    rng = np.random.default_rng(12)
    P, W, b = 29, 3, 4
    x0 = np.zeros(P, dtype=np.float32)
    counts = (b,) * W
    g0 = _grads(rng, P, counts)
    o = make(x0, W, 1.0, 0.0, 0.0, 0.0)
    xs = _run(o, [counts, (1,) * W], [g0, _grads(rng, P, (1,) * W)])
    worker_means = [sum(g0[(i, k)].astype(np.float64) for k in range(b)) / b for i in range(W)]
    expect = -np.mean(worker_means, axis=0)            # x_2 = x_1 - 1.0 * Gbar_0
    np.testing.assert_allclose(xs[1], expect, rtol=0, atol=1e-6)


# P3 ---------------------------------------------------------------------------------------
def pin_idle_worker_contributes_nothing(make):
    """A worker with b_i = 0 changes nothing: same result as the run without that worker."""
    rng = np.random.default_rng(13)
    P, T = 23, 5
    x0 = rng.standard_normal(P).astype(np.float32)
    sched3 = [(2, 0, 3), (1, 0, 1), (4, 0, 2), (1, 0, 1), (2, 0, 2)]
    gl3 = [_grads(rng, P, c, integer=False) for c in sched3]
    sched2 = [(c[0], c[2]) for c in sched3]
    gl2 = [{(0 if i == 0 else 1, k): g for (i, k), g in gr.items()} for gr in gl3]
    xa = _run(make(x0, 3, 0.1, 0.9, 1e-3, 0.0), sched3, gl3)
    xb = _run(make(x0, 2, 0.1, 0.9, 1e-3, 0.0), sched2, gl2)
    for a, b in zip(xa, xb):
        assert np.array_equal(a, b)


# P4 ---------------------------------------------------------------------------------------
def pin_first_step_is_noop(make):
    """G_{-1} = 0 (Algorithm 1, Initialization): x_1 = x_0 bit for bit, momentum untouched,
    even with weight decay and momentum switched on; an all-idle iteration behaves the same."""
    rng = np.random.default_rng(14)
    P = 19
    x0 = rng.standard_normal(P).astype(np.float32)
    o = make(x0, 2, 0.1, 0.9, 0.1, 0.0)
    o.accumulate(0, rng.standard_normal(P).astype(np.float32))
    o.sync_step()
    assert np.array_equal(o.params(), x0)
    assert np.all(np.asarray(o.v) == 0.0)
    # two sync steps in a row: the second has an empty delayed set only after the first
    # consumed the pending one.
    o.sync_step()                      # applies iteration 0's gradient
    x2 = o.params().copy(); v2 = np.asarray(o.v).copy()
    o.sync_step()                      # nothing pending (no accumulate in between): no-op
    o.sync_step()
    assert np.array_equal(o.params(), x2)
    assert np.array_equal(np.asarray(o.v), v2)


# P5 ---------------------------------------------------------------------------------------
def pin_delay_is_exactly_one_iteration(make):
    """Changing the gradients of iteration t leaves x_0..x_{t+1} bit-identical and changes x_{t+2}."""
    rng = np.random.default_rng(15)
    P, T, tp = 17, 6, 2
    x0 = rng.standard_normal(P).astype(np.float32)
    sched = [(2, 1)] * T
    gl = [_grads(rng, P, c, integer=False) for c in sched]
    gl2 = [dict(g) for g in gl]
    gl2[tp] = {key: g + 1.0 for key, g in gl[tp].items()}
    xa = _run(make(x0, 2, 0.1, 0.9, 0.0, 0.0), sched, gl)     # xa[s] = x_{s+1}
    xb = _run(make(x0, 2, 0.1, 0.9, 0.0, 0.0), sched, gl2)
    for s in range(0, tp + 1):                                # x_1 .. x_{tp+1}
        assert np.array_equal(xa[s], xb[s]), f"x_{s + 1} saw iteration {tp}'s gradients"
    assert not np.array_equal(xa[tp + 1], xb[tp + 1]), "x_{t+2} must contain iteration t's gradients"


# P6 ---------------------------------------------------------------------------------------
def pin_matches_library_sgd_shifted_by_one(make):
    """With gradients that do not depend on the parameters, x^{ABS}_{t+1} = x^{BSP}_t, where
    BSP is torch.optim.SGD (lr, momentum, weight_decay) fed Gbar_0, Gbar_1, ..."""
    import torch

    rng = np.random.default_rng(16)
    P, W, T, lr, mu, wd = 41, 4, 7, 0.07, 0.8, 5e-3
    x0 = rng.standard_normal(P).astype(np.float32)
    sched = [tuple(int(v) for v in rng.integers(0, 5, size=W)) for _ in range(T)]
    sched = [c if sum(c) > 0 else (1,) + c[1:] for c in sched]
    gl = [_grads(rng, P, c) for c in sched]
    xs = _run(make(x0, W, lr, mu, wd, 0.0), sched, gl)
    p = torch.tensor(x0.astype(np.float64), requires_grad=True)
    opt = torch.optim.SGD([p], lr=lr, momentum=mu, weight_decay=wd)
    np.testing.assert_allclose(xs[0], x0.astype(np.float64), rtol=0, atol=0)
    for s in range(1, T):
        p.grad = torch.tensor(_gbar(sched[s - 1], gl[s - 1]))
        opt.step()
        ref = p.detach().numpy()
        np.testing.assert_allclose(xs[s], ref, rtol=0, atol=2e-6 * np.abs(ref).max())


# P7 ---------------------------------------------------------------------------------------
def pin_plain_sgd_telescopes(make):
    """mu = wd = 0: x_T = x_0 - lr * sum_{t=0}^{T-2} Gbar_t (the last iteration's gradients are
    accumulated but never applied; Algorithm 1 returns x_T)."""
    rng = np.random.default_rng(17)
    P, W, T, lr = 31, 3, 6, 0.25
    x0 = rng.standard_normal(P).astype(np.float32)
    sched = [tuple(int(v) for v in rng.integers(1, 4, size=W)) for _ in range(T)]
    gl = [_grads(rng, P, c) for c in sched]
    xs = _run(make(x0, W, lr, 0.0, 0.0, 0.0), sched, gl)
    expect = x0.astype(np.float64) - lr * sum(_gbar(sched[t], gl[t]) for t in range(T - 1))
    np.testing.assert_allclose(xs[-1], expect, rtol=0, atol=2e-6 * np.abs(expect).max())


# P8 ---------------------------------------------------------------------------------------
def pin_weights_are_batch_counts(make):
    """Constant gradient c_i per worker: Gbar = sum_i b_i c_i / sum_i b_i exactly.  Separates
    the weighted average from a uniform one and from dividing by the worker count."""
    P, lr = 8, 1.0
    x0 = np.zeros(P, dtype=np.float32)
    counts = (3, 1, 4)
    c = (1.0, 10.0, -2.0)
    grads = {(i, k): np.full(P, c[i], dtype=np.float32) for i, b in enumerate(counts) for k in range(b)}
    o = make(x0, 3, lr, 0.0, 0.0, 0.0)
    xs = _run(o, [counts, counts], [grads, grads])
    expect = -(3 * 1.0 + 1 * 10.0 + 4 * -2.0) / 8.0            # = -0.625
    np.testing.assert_allclose(xs[1], np.full(P, expect), rtol=0, atol=1e-12)


# P9 ---------------------------------------------------------------------------------------
def pin_momentum_hand_example(make):
    gold = read_golden("p9_momentum_hand_example.txt")
    o = make(np.array([1.0], dtype=np.float32), 2, 0.1, 0.9, 0.0, 0.0)
    per_iter = [([1.0, 2.0, 3.0], [10.0]), ([1.0] * 3, [1.0]), ([0.0] * 3, [0.0]), ([0.0] * 3, [0.0])]
    xs, vs = [], []
    for w0, w1 in per_iter:
        for g in w0:
            o.accumulate(0, np.array([g], dtype=np.float32))
        for g in w1:
            o.accumulate(1, np.array([g], dtype=np.float32))
        o.sync_step()
        xs.append(float(o.params()[0])); vs.append(float(np.asarray(o.v)[0]))
    for k, x in zip(("x1", "x2", "x3", "x4"), xs):
        assert abs(x - gold[k]) < 1e-6, (k, x, gold[k])
    for k, v in zip(("v_after_step1", "v_after_step2", "v_after_step3"), vs[1:]):
        assert abs(v - gold[k]) < 1e-9, (k, v, gold[k])


def pin_compensation_hand_example(make):
    """Eq. 6 on a one-parameter example worked by hand."""
    gold = read_golden("eq6_compensation_hand_example.txt")
    o = make(np.array([1.0], dtype=np.float32), 2, 0.1, 0.0, 0.0, 0.5)
    per_iter = [([1.0, 2.0, 3.0], [10.0]), ([1.0] * 3, [1.0]), ([2.0] * 3, [2.0]), ([0.0] * 3, [0.0])]
    xs = []
    for w0, w1 in per_iter:
        for g in w0:
            o.accumulate(0, np.array([g], dtype=np.float32))
        for g in w1:
            o.accumulate(1, np.array([g], dtype=np.float32))
        o.sync_step()
        xs.append(float(o.params()[0]))
    for k, x in zip(("x1", "x2", "x3", "x4"), xs):
        assert abs(x - gold[k]) < 1e-6, (k, x, gold[k])


def pin_compensation_uses_parameter_displacement(make):
    """Eq. 6 written out on vectors: with mu = wd = 0,
    x_{t+1} = x_t - lr * (Gbar_{t-1} + lambda * Gbar_{t-1}^2 * (x_t - x_{t-1}))."""
    rng = np.random.default_rng(18)
    P, W, T, lr, lam = 13, 2, 6, 0.1, 0.5
    x0 = rng.standard_normal(P).astype(np.float32)
    sched = [(2, 1)] * T
    gl = [_grads(rng, P, c) for c in sched]
    xs = _run(make(x0, W, lr, 0.0, 0.0, lam), sched, gl)
    x_prev = x0.astype(np.float64); x = x0.astype(np.float64)
    for s in range(1, T):
        G = _gbar(sched[s - 1], gl[s - 1])
        Gt = G + lam * G * G * (x - x_prev)
        x_prev, x = x, x - lr * Gt
        np.testing.assert_allclose(xs[s], x, rtol=0, atol=3e-6 * np.abs(x).max())


# counters ---------------------------------------------------------------------------------
def pin_counters_and_swap(make):
    """b_i counts calls; the set index alternates 0,1,0,...; a sync clears the set it consumed."""
    P = 4
    o = make(np.zeros(P, dtype=np.float32), 3, 0.1, 0.0, 0.0, 0.0)
    g = np.ones(P, dtype=np.float32)
    cnt, cur, t = o.counters()
    assert cur == 0 and t == 0 and not cnt.any()
    for i, b in enumerate((2, 0, 5)):
        for _ in range(b):
            o.accumulate(i, g)
    cnt, cur, t = o.counters()
    assert cnt[0].tolist() == [2, 0, 5] and cnt[1].tolist() == [0, 0, 0]
    assert o.sync_step() == 0                      # delayed set (index 1) is empty
    cnt, cur, t = o.counters()
    assert cur == 1 and t == 1 and cnt[0].tolist() == [2, 0, 5]
    o.accumulate(1, g)
    cnt, _, _ = o.counters()
    assert cnt[1].tolist() == [0, 1, 0]
    assert o.sync_step() == 7                      # consumes set 0
    cnt, cur, t = o.counters()
    assert cur == 0 and t == 2 and cnt[0].tolist() == [0, 0, 0] and cnt[1].tolist() == [0, 1, 0]
    assert [c.tolist() for c in o.consumed] == [[0, 0, 0], [2, 0, 5]]
    # the consumed set was cleared: filling it again starts from zero
    o.accumulate(0, g)
    assert o.sync_step() == 1                      # consumes set 1 (the single call of worker 1)
    o.sync_step()                                  # consumes set 0: exactly one gradient of ones
    np.testing.assert_allclose(o.params(), np.zeros(P) - 0.1 * (7 / 7 + 1 + 1), atol=1e-6)


def pin_bf16_gradients_are_widened_exactly(make):
    """bf16 micro-batch gradients (bit patterns) enter the fp32 accumulator by exact widening."""
    rng = np.random.default_rng(19)
    P = 64
    vals = rng.standard_normal(P).astype(np.float32)
    bits = (vals.view(np.uint32) >> 16).astype(np.uint16)          # truncation: some bf16 values
    widened = (bits.astype(np.uint32) << 16).view(np.float32)
    o1 = make(np.zeros(P, dtype=np.float32), 1, 1.0, 0.0, 0.0, 0.0)
    o2 = make(np.zeros(P, dtype=np.float32), 1, 1.0, 0.0, 0.0, 0.0)
    o1.accumulate(0, bits)                       # uint16 arrays are bf16 bit patterns
    o2.accumulate(0, widened)
    for o in (o1, o2):
        o.sync_step(); o.sync_step()
    assert np.array_equal(o1.params(), o2.params())
    np.testing.assert_allclose(o2.params(), -widened, atol=0)


ALL_PINS = [
    pin_single_worker_is_delayed_momentum_sgd,
    pin_equal_counts_give_uniform_average,
    pin_idle_worker_contributes_nothing,
    pin_first_step_is_noop,
    pin_delay_is_exactly_one_iteration,
    pin_matches_library_sgd_shifted_by_one,
    pin_plain_sgd_telescopes,
    pin_weights_are_batch_counts,
    pin_momentum_hand_example,
    pin_compensation_hand_example,
    pin_compensation_uses_parameter_displacement,
    pin_counters_and_swap,
    pin_bf16_gradients_are_widened_exactly,
]
