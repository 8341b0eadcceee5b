"""GPU test of abs_sync_step_noalloc, the entry point for callers that cannot allocate device
memory (code living inside another component's memory budget: a framework extension under a
pre-reserved pool, a job with all device memory carved up front, a loop that cannot take the
device-wide synchronisation of cudaMalloc).  Its working memory is a small array built into the
library, shared by every call, so every case makes calls in a row on the same device and checks
each of them: against the CPU oracle's sync step fed the same gradients (the parity bar of the fp32
path) and against the context-based abs_sync_step fed the same accumulators (bit for bit: whichever
form of the fused kernel the context picks, both forms compute the same bits).

Kept in a file of its own that sorts last, so that a run stopping at the first failure has
already gone through every other test."""

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = 1e-5      # max |x - x_oracle| <= TOL * max |x_oracle|, as for every fp32 parity case

# (P, W, micro-batch counts of the consecutive calls).  P % 4 == 0 throughout (the entry point's contract).
CASES = {
    # just under 2^18 vectors, five workers, idle workers in both calls, then a call with every worker idle
    "W5-1M": (1_000_448, 5, [(3, 0, 1, 2, 1), (1, 2, 0, 0, 4), (0, 0, 0, 0, 0), (2, 1, 1, 0, 0)]),
    # more than 2^20 elements with a ragged last tile (P % 1024 = 4): the size at which abs_sync_step would
    # switch to its bulk-copy form for W = 5; this entry point must stay on the load/store form and agree
    "W5-1.3M-ragged": (1_310_724, 5, [(1, 1, 2, 0, 3), (2, 0, 0, 1, 1)]),
    # compile-time worker counts of the kernel
    "W2": (300_004, 2, [(2, 1), (0, 3), (0, 0)]),
    "W1": (65_540, 1, [(2,), (1,)]),
    "W4": (200_000, 4, [(1, 0, 2, 1), (1, 1, 1, 1)]),
    # chunked rows beyond eight workers
    "W12": (120_004, 12, [tuple(int(b) for b in np.arange(12) % 3), tuple([1] * 12)]),
}


@pytest.mark.parametrize("name", list(CASES))
def test_noalloc_matches_oracle_and_context_sync_step_on_consecutive_calls(name):
    import torch

    from oracle.abs_oracle import AbsSgdOracle
    from paper_2308_15164_b200 import binding as B

    P, W, counts_per_call = CASES[name]
    rng = np.random.default_rng(42)
    lr, mu, wd = 0.05, 0.9, 1e-3
    x0 = (rng.standard_normal(P) * 0.05).astype(np.float32)
    dev = torch.device("cuda:0")
    ref = AbsSgdOracle(x0, W, lr, mu, wd)                                   # the oracle
    eng = B.AbsSgd(torch.from_numpy(x0).to(dev), W, lr, mu, wd)            # eager context: the existing entry point
    x = torch.from_numpy(x0).to(dev)                                        # caller-owned state for the new one
    v = torch.zeros(P, dtype=torch.float32, device=dev)
    stride = P + 64
    acc = torch.zeros((W, stride), dtype=torch.float32, device=dev)
    cnt = torch.zeros(W, dtype=torch.int32, device=dev)
    stream = eng.stream_acc
    eng.sync_step(); ref.sync_step()                                        # t = 0: nothing pending
    moved = False
    for call, counts in enumerate(counts_per_call):
        grads = [[rng.standard_normal(P).astype(np.float32) for _ in range(b)] for b in counts]
        grads_d = [[torch.from_numpy(g).to(dev) for g in gs] for gs in grads]
        torch.cuda.synchronize()
        cur = eng.counters()[1]
        for i, gs in enumerate(grads):
            for g, gd in zip(gs, grads_d[i]):
                ref.accumulate(i, g)
                eng.accumulate(i, gd)
        eng.synchronize()
        with torch.cuda.stream(stream):
            for i in range(W):                                              # same accumulator contents for both paths
                acc[i, :P].copy_(eng.accumulator(cur, i))
            cnt.copy_(torch.tensor(counts, dtype=torch.int32))
            acc[:, P:] = 7.0                                                # padding between rows must stay untouched
        stream.synchronize()
        x_before, v_before = x.cpu().numpy(), v.cpu().numpy()
        for o in (eng, ref):
            o.sync_step()                                                   # ends the iteration (the set becomes pending)
            o.sync_step()                                                   # applies it (no accumulate in between)
        rc = B.sync_step_noalloc(x, v, acc, cnt, lr, mu, wd, stream=stream)
        assert rc == B.OK
        stream.synchronize()
        got_x, got_v = x.cpu().numpy(), v.cpu().numpy()
        want_x = ref.params()
        assert np.abs(got_x - want_x).max() <= TOL * np.abs(want_x).max(), f"call {call}: parameters against the oracle"
        assert np.abs(got_v - ref.v).max() <= TOL * max(np.abs(ref.v).max(), 1e-30), f"call {call}: momentum against the oracle"
        assert np.array_equal(got_x, eng.params_host()), f"call {call}: parameters against abs_sync_step"
        assert np.array_equal(got_v, eng.momentum().cpu().numpy()), f"call {call}: momentum against abs_sync_step"
        if sum(counts) == 0:                                                # every worker idle: nothing may change
            assert np.array_equal(got_x, x_before) and np.array_equal(got_v, v_before)
        else:
            moved = moved or not np.array_equal(got_x, x_before)
        a = acc.cpu().numpy()
        assert np.all(a[:, :P] == 0.0), "consumed accumulators are cleared (idle ones were zero already)"
        assert np.all(a[:, P:] == 7.0), "row padding was written"
        assert cnt.cpu().numpy().tolist() == [0] * W
    assert moved
    eng.check()
    eng.destroy()


def test_noalloc_rejects_bad_arguments_without_launching():
    import torch

    from paper_2308_15164_b200 import binding as B

    dev = torch.device("cuda:0")
    x = torch.ones(1024, device=dev); v = torch.zeros(1024, device=dev)
    acc = torch.ones((65, 1024), device=dev); cnt = torch.ones(65, dtype=torch.int32, device=dev)
    assert B.sync_step_noalloc(x, v, acc, cnt, 0.1) == B.ELIMIT             # W = 65 > 64
    assert B.sync_step_noalloc(x[:1022], v[:1022], acc[:4, :1022], cnt[:4], 0.1) == B.EINVAL   # P % 4 != 0
    assert B.sync_step_noalloc(x[1:1021], v[:1020], acc[:4, :1020], cnt[:4], 0.1) == B.EINVAL  # misaligned x
    host = torch.zeros(1024).pin_memory()                                   # not device memory of the current device
    s = torch.cuda.current_stream(dev).cuda_stream
    assert B.lib.abs_sync_step_noalloc(host.data_ptr(), v.data_ptr(), acc.data_ptr(), 1024, 1024, 4, cnt.data_ptr(),
                                       0.1, 0.0, 0.0, s) == B.EINVAL
    torch.cuda.synchronize()
    assert torch.all(x == 1) and torch.all(acc == 1) and torch.all(cnt == 1)
