"""Programmatic dependent launch between consecutive kernels of a stream (the default) against plain stream order
(abs_set_launch(ABS_K_CHAIN, 1)): the chain only changes WHEN a kernel's set-up runs, never what it computes, so
every result must agree bit for bit -- streaming path (eager and pipelined, fp32 and bf16 gradients, batch calls,
both forms of the fused step) and MLP path (single, gathered and batch calls, every worker's calls on its own
streams or all on one).  Also the timeline of the timed launches (abs_profile(ctx, 2), abs_profile_timeline)."""

import numpy as np
import pytest

from paper_2308_15164_b200 import workloads as wlm

pytestmark = pytest.mark.gpu


def _stream_run(cfg, T, pipelined, chain, batch=0, sync_shape=0):
    import torch

    from paper_2308_15164_b200 import binding as B

    wl = wlm.config(cfg, small=True, T=T)
    x0 = wlm.params0(wl)
    pool = wlm.grad_pool(wl)
    dev = torch.device("cuda:0")
    src = torch.from_numpy(pool.view(np.int16) if pool.dtype == np.uint16 else pool)
    pool_d = torch.zeros((pool.shape[0], (pool.shape[1] + 7) // 8 * 8), dtype=src.dtype, device=dev)
    pool_d[:, :pool.shape[1]] = src.to(dev)
    eng = B.AbsSgd(torch.from_numpy(x0).to(dev), wl.W, wl.lr, wl.momentum, wl.weight_decay,
                   grad_dtype=B.GRAD_BF16 if wl.grad_dtype == "bf16" else B.GRAD_F32, pipelined=pipelined)
    eng.set_launch(B.K_CHAIN, chain)
    eng.set_launch(B.K_SYNC, sync_shape)
    torch.cuda.synchronize()
    for calls in wlm.iter_calls(wl):
        if batch:
            per = {}
            for (i, k, c) in calls:
                per.setdefault(i, []).append(pool_d[c % wl.pool_size])
            for i, gs in per.items():
                for lo in range(0, len(gs), batch):
                    eng.accumulate_batch(i, gs[lo:lo + batch])
        else:
            for (i, k, c) in calls:
                eng.accumulate(i, pool_d[c % wl.pool_size])
        eng.sync_step()
    eng.check()
    x = eng.params_host()
    eng.wait(); eng.synchronize()
    v = eng.momentum().cpu().numpy()
    eng.destroy()
    return x, v


@pytest.mark.parametrize("cfg,T,batch,sync_shape", [(2, 8, 0, 0), (3, 14, 0, 0), (3, 14, 0, -2), (5, 5, 0, 0), (2, 6, 3, 0)],
                         ids=["resnet18", "dynamic-idle-workers", "dynamic-bulk-copy-step", "bf16-gradients", "batch-calls"])
@pytest.mark.parametrize("pipelined", [False, True], ids=["eager", "pipelined"])
def test_chained_and_plain_launches_give_the_same_bits_streaming(cfg, T, batch, sync_shape, pipelined):
    a = _stream_run(cfg, T, pipelined, 0, batch, sync_shape)
    b = _stream_run(cfg, T, pipelined, 1, batch, sync_shape)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert not np.array_equal(a[0], wlm.params0(wlm.config(cfg, small=True, T=T)))


def _mlp_run(chain, mode, serial, pipelined, defer=False):
    import torch

    from paper_2308_15164_b200 import binding as B

    wl = wlm.config(4, small=True, T=6)
    d = wl.mlp
    xs, ys = wlm.mlp_batches(wl)
    dev = torch.device("cuda:0")
    xs_d, ys_d = torch.from_numpy(xs).to(dev), torch.from_numpy(ys).to(dev)
    eng = B.AbsSgd(torch.from_numpy(wlm.params0(wl)).to(dev), wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=pipelined,
                   mlp=(d.d_in, d.d_hidden, d.d_out, d.mb), mlp_coalesce=(mode == "gathered"), mlp_defer=defer)
    eng.set_launch(B.K_CHAIN, chain)
    eng.set_launch(B.K_MLP_FWD, serial)
    torch.cuda.synchronize()
    n = 0
    for t, b_row in enumerate(wlm.schedule(wl)):
        if mode == "batch":
            for i, b in enumerate(b_row):
                left = int(b)
                while left > 0:
                    k = min(4, left)
                    lo = (n * 7) % (wl.mlp_pool - 4)
                    eng.accumulate_mlp_batch(i, k, xs_d[lo:lo + k], ys_d[lo:lo + k]); left -= k; n += k
        else:
            for (i, k) in wlm.call_order(b_row):
                eng.accumulate_mlp(i, xs_d[n % wl.mlp_pool], ys_d[n % wl.mlp_pool]); n += 1
        eng.sync_step()
    eng.check()
    x = eng.params_host()
    eng.destroy()
    return x


@pytest.mark.parametrize("defer", [False, True], ids=["per-call-dw1", "deferred-dw1"])
@pytest.mark.parametrize("mode", ["single", "gathered", "batch"])
@pytest.mark.parametrize("serial", [0, 1], ids=["worker-streams", "one-stream"])
def test_chained_and_plain_launches_give_the_same_bits_mlp(mode, serial, defer):
    if mode == "gathered" and serial:
        pytest.skip("serial mode runs every call at once: nothing to gather")
    for pipelined in (False, True):
        a = _mlp_run(0, mode, serial, pipelined, defer)
        b = _mlp_run(1, mode, serial, pipelined, defer)
        assert np.array_equal(a, b), f"pipelined={pipelined}"


def test_set_launch_rejects_unknown_values():
    import torch

    from paper_2308_15164_b200 import binding as B

    eng = B.AbsSgd(torch.zeros(1024, device="cuda"), 2, 0.1)
    for cls, val in ((B.K_CHAIN, 2), (B.K_CHAIN, -1), (B.K_MLP_DW1, 1), (B.K_MLP_DW1, 64), (B.K_MLP_DW1, 256),
                     (B.K_MLP_FWD, 2), (B.K_MLP_BWD, 3), (B.K_SYNC, -3), (6, 0), (-1, 0)):
        assert B.lib.abs_set_launch(eng._h, cls, val) == B.EINVAL, (cls, val)
    for cls, val in ((B.K_CHAIN, 1), (B.K_CHAIN, 0), (B.K_MLP_DW1, 4 | 32 | 128), (B.K_MLP_DW1, 8), (B.K_SYNC, -2), (B.K_ACCUMULATE, 4), (B.K_MLP_BWD, 1), (B.K_MLP_BWD, 2)):
        assert B.lib.abs_set_launch(eng._h, cls, val) == B.OK, (cls, val)
    eng.destroy()


def test_timeline_of_the_timed_launches():
    import torch

    from paper_2308_15164_b200 import binding as B

    wl = wlm.config(4, small=True, T=3)
    d = wl.mlp
    xs, ys = wlm.mlp_batches(wl)
    dev = torch.device("cuda:0")
    xs_d, ys_d = torch.from_numpy(xs).to(dev), torch.from_numpy(ys).to(dev)
    eng = B.AbsSgd(torch.from_numpy(wlm.params0(wl)).to(dev), wl.W, wl.lr, wl.momentum, pipelined=True,
                   mlp=(d.d_in, d.d_hidden, d.d_out, d.mb))
    torch.cuda.synchronize()
    eng.profile(2)
    n = 0
    for b_row in wlm.schedule(wl):
        for (i, k) in wlm.call_order(b_row):
            eng.accumulate_mlp(i, xs_d[n % wl.mlp_pool], ys_d[n % wl.mlp_pool]); n += 1
        eng.sync_step()
    spans = eng.profile_timeline()
    eng.profile(False)
    # five timed kernels per call (cast, forward GEMM, bias/ReLU/logits, backward, dW1) and one fused step per
    # iteration (pipelined mode launches Step 1 for the set just filled at the end of every iteration)
    assert len(spans) == 5 * n + 3
    by = {}
    for (cls, part, stream, t0, t1) in spans:
        assert t1 > t0 >= 0.0
        by.setdefault((cls, part), []).append(stream)
    assert sorted(by) == [("mlp_bwd", 0), ("mlp_dw1", 0), ("mlp_fwd", 0), ("mlp_fwd", 1), ("mlp_fwd", 2), ("sync", 0)]
    assert set(by[("mlp_fwd", 0)]) == {0}                       # the cast reads the caller's buffers: stream_acc
    assert set(by[("sync", 0)]) == {1}                          # Step 1 on stream_sync
    assert set(by[("mlp_fwd", 1)]) <= {2, 3, 4, 5}              # the workers' own streams
    assert set(by[("mlp_dw1", 0)]) <= {10, 11, 12, 13}          # dW1: the workers' second streams
    n_st, ms = eng.kernel_stats(B.K_MLP_DW1)
    assert n_st == n and ms > 0
    eng.check()
    eng.destroy()
