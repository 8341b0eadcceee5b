"""GPU test of abs_sync_step_noalloc, the entry point for callers that cannot allocate device
memory (code living inside another component's memory budget: a framework extension under a
pre-reserved pool, a job with all device memory carved up front, a loop that cannot take the
device-wide synchronisation of cudaMalloc).  Its working memory is a small array built into the
library, shared by every call, so the test makes two calls in a row and checks both against the
context-based abs_sync_step fed the same accumulators.

Kept in a file of its own that sorts last, so that a run stopping at the first failure has
already gone through every other test."""

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_noalloc_matches_context_sync_step_twice():
    import torch

    from paper_2308_15164_b200 import binding as B

    rng = np.random.default_rng(42)
    P, W, lr, mu, wd = 1_000_448, 5, 0.05, 0.9, 1e-3          # P % 4 == 0, several CTAs, ragged last tile
    x0 = (rng.standard_normal(P) * 0.05).astype(np.float32)
    dev = torch.device("cuda:0")
    eng = B.AbsSgd(torch.from_numpy(x0).to(dev), W, lr, mu, wd)            # eager context: the existing entry point
    x = torch.from_numpy(x0).to(dev)                                        # caller-owned state for the new one
    v = torch.zeros(P, dtype=torch.float32, device=dev)
    stride = P + 64
    acc = torch.zeros((W, stride), dtype=torch.float32, device=dev)
    cnt = torch.zeros(W, dtype=torch.int32, device=dev)
    stream = eng.stream_acc
    counts_per_call = [(3, 0, 1, 2, 1), (1, 2, 0, 0, 4)]                    # idle workers in both calls
    eng.sync_step()                                                         # t = 0: nothing pending
    for call, counts in enumerate(counts_per_call):
        grads = [[torch.from_numpy(rng.standard_normal(P).astype(np.float32)).to(dev) for _ in range(b)] for b in counts]
        torch.cuda.synchronize()
        cur = eng.counters()[1]
        for i, gs in enumerate(grads):
            for g in gs:
                eng.accumulate(i, g)
        eng.synchronize()
        with torch.cuda.stream(stream):
            for i in range(W):                                              # same accumulator contents for both paths
                acc[i, :P].copy_(eng.accumulator(cur, i))
            cnt.copy_(torch.tensor(counts, dtype=torch.int32))
            acc[:, P:] = 7.0                                                # padding between rows must stay untouched
        stream.synchronize()
        eng.sync_step()                                                     # ends the iteration (set `cur` becomes pending)
        eng.sync_step()                                                     # applies it (no accumulate in between)
        rc = B.sync_step_noalloc(x, v, acc, cnt, lr, mu, wd, stream=stream)
        assert rc == B.OK
        stream.synchronize()
        want_x, want_v = eng.params_host(), eng.momentum().cpu().numpy()
        got_x, got_v = x.cpu().numpy(), v.cpu().numpy()
        tol = 1e-5
        assert np.abs(got_x - want_x).max() <= tol * np.abs(want_x).max(), f"call {call}: parameters"
        assert np.abs(got_v - want_v).max() <= tol * np.abs(want_v).max(), f"call {call}: momentum"
        assert not np.array_equal(want_x, x0)
        a = acc.cpu().numpy()
        assert np.all(a[:, :P] == 0.0), "consumed accumulators are cleared (idle ones were zero already)"
        assert np.all(a[:, P:] == 7.0), "row padding was written"
        assert cnt.cpu().numpy().tolist() == [0] * W
    eng.destroy()


def test_noalloc_rejects_bad_sizes_without_launching():
    import torch

    from paper_2308_15164_b200 import binding as B

    dev = torch.device("cuda:0")
    x = torch.ones(1024, device=dev); v = torch.zeros(1024, device=dev)
    acc = torch.ones((65, 1024), device=dev); cnt = torch.ones(65, dtype=torch.int32, device=dev)
    assert B.sync_step_noalloc(x, v, acc, cnt, 0.1) == B.ELIMIT             # W = 65 > 64
    assert B.sync_step_noalloc(x[:1022], v[:1022], acc[:4, :1022], cnt[:4], 0.1) == B.EINVAL   # P % 4 != 0
    assert B.sync_step_noalloc(x[1:1021], v[:1020], acc[:4, :1020], cnt[:4], 0.1) == B.EINVAL  # misaligned x
    torch.cuda.synchronize()
    assert torch.all(x == 1) and torch.all(acc == 1) and torch.all(cnt == 1)
