"""CPU-only: the seeded synthetic input generators (shapes, determinism, schedule structure)."""

import numpy as np

from paper_2308_15164_b200 import workloads as wl


def test_resnet18_layout_has_62_tensors_and_11689512_params():
    tens = wl.resnet18_tensors()
    assert len(tens) == 62
    assert sum(int(np.prod(s)) for _, s in tens) == 11_689_512
    assert sum(1 for _, s in tens if len(s) == 4) == 20
    cfg = wl.config(2)
    assert cfg.P == 11_689_512 and cfg.W == 4 and cfg.T == 100
    assert wl.schedule(cfg)[17].tolist() == [2, 2, 4, 8]


def test_config_sizes():
    assert wl.config(1).P == 4096 and wl.schedule(wl.config(1))[0].tolist() == [3, 1]
    assert wl.config(3).P == 25_557_032 and wl.config(3).W == 8
    assert wl.config(4).P == 12_627_978 and wl.config(4).mlp.offsets == (0, 12_582_912, 12_587_008, 12_627_968)
    assert wl.config(5).P == 124_439_808 and wl.config(5).grad_dtype == "bf16"


def test_schedules():
    c3 = wl.config(3)
    b = wl.schedule(c3)
    assert b.shape == (200, 8) and b.min() == 0 and b.max() <= 16
    assert all((b[t] == 0).any() for t in range(7, 200, 10))
    assert 3.5 < b.mean() < 6.0
    assert np.array_equal(b, wl.schedule(c3))
    b5 = wl.schedule(wl.config(5))
    assert b5.min() >= 1 and b5.max() <= 12 and set(np.unique(b5)) == set(range(1, 13))
    b4 = wl.schedule(wl.config(4))
    assert b4.min() >= 1 and b4.max() <= 8


def test_call_order_interleaves_by_virtual_time():
    order = wl.call_order((2, 2, 4, 8))
    assert len(order) == 16
    for i, b in enumerate((2, 2, 4, 8)):
        assert [k for (w, k) in order if w == i] == list(range(b))     # per-worker order kept
    assert order[0] == (3, 0) and order[-1] == (3, 7) or order[-1][1] == (2, 2, 4, 8)[order[-1][0]] - 1
    assert wl.call_order((0, 3)) == [(1, 0), (1, 1), (1, 2)]
    calls = list(wl.iter_calls(wl.config(1)))
    assert len(calls) == 5 and [c for it in calls for (_, _, c) in it] == list(range(20))


def test_inputs_are_deterministic_and_scaled():
    c = wl.config(2, small=True)
    x0 = wl.params0(c)
    assert x0.dtype == np.float32 and x0.shape == (c.P,) and np.array_equal(x0, wl.params0(c))
    pool = wl.grad_pool(c)
    assert pool.shape == (16, c.P) and pool.dtype == np.float32
    # stem conv: fan_in 147 -> std 147^-1/2
    assert abs(pool[:, :9408].std() - 147 ** -0.5) < 2e-3
    cols = np.array([0, 5, 9407, 9408, c.P - 1])
    assert np.array_equal(wl.grad_pool(c, columns=cols), pool[:, cols])
    c5 = wl.config(5, small=True)
    p5 = wl.grad_pool(c5)
    assert p5.dtype == np.uint16
    assert abs(wl.bf16_bits_to_f32(p5).std() - 0.02) < 1e-3
    g = wl.fresh_grad(wl.config(1), 2, 1, 0)
    assert np.array_equal(g, wl.fresh_grad(wl.config(1), 2, 1, 0))
    assert not np.array_equal(g, wl.fresh_grad(wl.config(1), 2, 0, 0))


def test_bf16_bits_round_to_nearest_even():
    import torch

    v = (np.random.default_rng(0).standard_normal(4096) * 5).astype(np.float32)
    ref = torch.tensor(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(wl.f32_to_bf16_bits(v), ref)


def test_mlp_batches_and_sample_columns():
    c = wl.config(4, small=True)
    x, y = wl.mlp_batches(c)
    assert x.shape == (64, 64, 384) and y.shape == (64, 64) and y.min() == 0 and y.max() == 9
    idx = wl.sample_columns(25_557_032)
    assert idx[0] == 0 and idx[-1] == 25_557_031 and np.all(np.diff(idx) > 0)


def test_bench_byte_model_of_the_mlp_runs():
    """bench.mlp_run_bytes on a schedule small enough to add up by hand (d_in = d_hidden = 128, 10 outputs)."""
    import importlib.util
    import os

    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(os.path.dirname(os.path.dirname(__file__)), "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    d = wl.MlpDims(128, 128, 10, 64)
    w1, P = 128 * 128, d.P
    ops = 2 * 64 * (128 + 128)                         # bf16 X^T and dZ^T of one micro-batch
    sched = [[3, 0], [1, 2]]                           # two iterations, two workers
    # per-call mode, single calls: worker 0 stores once and adds twice; the second iteration's step applies the first's set
    total, calls, stored, mbs = bench.mlp_run_bytes(sched, d, P, 1, False)
    assert (calls, stored, mbs) == (6, 3, 6)
    assert total == 6 * 2 * w1 + (3 * 4 + 3 * 8) * w1 + 6 * ops + (8 * 1 + 18) * P
    # batch calls of up to 4: one call per active worker and iteration, all of them store
    total4, calls4, stored4, _ = bench.mlp_run_bytes(sched, d, P, 4, False)
    assert (calls4, stored4) == (3, 3)
    assert total4 == 3 * 2 * w1 + 3 * 4 * w1 + 6 * ops + (8 * 1 + 18) * P
    # deferred, rows written: the slice once per active worker and iteration, operands written and read
    rows, _, _, _ = bench.mlp_run_bytes(sched, d, P, 1, False, "rows")
    assert rows == 6 * 2 * w1 + 3 * 4 * w1 + 2 * 6 * ops + (8 * 1 + 18) * P
    # deferred, Step 1 from the pool: no accumulator traffic for W1; 18 bytes per W1 element in the step
    pool, _, _, _ = bench.mlp_run_bytes(sched, d, P, 1, False, "pool")
    assert pool == 6 * 2 * w1 + 2 * 6 * ops + 18 * w1 + (8 * 1 + 18) * (P - w1)
    assert pool < rows < total
