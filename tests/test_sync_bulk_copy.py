"""The bulk-copy form of the fused step (abs_set_launch(ABS_K_SYNC, -2): cp.async.bulk loads into shared-memory
stages, update in shared memory, cp.async.bulk stores) gives the same bits as the default kernel: parameters
after every iteration, momentum, consumed counts -- eager and pipelined, idle workers, bf16 gradients, Eq. 6,
ragged sizes, worker counts up to the limit (and beyond it, where the default kernel takes over), the MLP's bf16
copy of the weights, overwrite-first mode."""

import dataclasses

import numpy as np
import pytest

from paper_2308_15164_b200 import workloads as wlm
from tests import harness as H

pytestmark = pytest.mark.gpu


def _run(wl, pipelined, variant, lambda_dc=0.0, overwrite_first=False, sched=None):
    import torch

    from paper_2308_15164_b200 import binding as B

    dev = torch.device("cuda:0")
    x0 = wlm.params0(wl)
    pool = wlm.grad_pool(wl)
    src = torch.from_numpy(pool.view(np.int16) if pool.dtype == np.uint16 else pool)
    pool_d = torch.zeros((pool.shape[0], (pool.shape[1] + 7) // 8 * 8), dtype=src.dtype, device=dev)
    pool_d[:, :pool.shape[1]] = src.to(dev)
    gd = B.GRAD_BF16 if wl.grad_dtype == "bf16" else B.GRAD_F32
    eng = B.AbsSgd(torch.from_numpy(x0).to(dev), wl.W, wl.lr, wl.momentum, wl.weight_decay, lambda_dc, grad_dtype=gd,
                   pipelined=pipelined, overwrite_first=overwrite_first)
    eng.set_launch(B.K_SYNC, variant)
    sched = wlm.schedule(wl) if sched is None else sched
    xs, c = [], 0
    for b_row in sched:
        for (i, k) in wlm.call_order(b_row):
            eng.accumulate(i, pool_d[c % wl.pool_size]); c += 1
        eng.sync_step()
        xs.append(eng.params_host())
    eng.wait()
    eng.synchronize()
    v = eng.momentum().clone().cpu().numpy()
    consumed = [eng.consumed(s) for s in range(len(sched))]
    eng.check()
    eng.destroy()
    return xs, v, consumed


def _same(a, b):
    for t, (x1, x2) in enumerate(zip(a[0], b[0])):
        assert np.array_equal(x1, x2), f"x_{t + 1}"
    assert np.array_equal(a[1], b[1])
    for c1, c2 in zip(a[2], b[2]):
        assert np.array_equal(c1, c2)


@pytest.mark.parametrize("cfg,lam,ow", [(2, 0.0, False), (3, 0.5, False), (5, 0.0, False), (3, 0.0, True)])
@pytest.mark.parametrize("pipelined", [False, True], ids=["eager", "pipelined"])
def test_same_bits_as_the_default_kernel(cfg, lam, ow, pipelined):
    wl = wlm.config(cfg, small=True, T=8)
    sched = wlm.schedule(wl).copy()
    sched[3, :] = 0
    if cfg == 3:
        sched[5, ::2] = 0                              # every other worker idle
    ref = _run(wl, pipelined, -1, lam, ow, sched)      # -1: the load/store kernel, one tile per CTA
    got = _run(wl, pipelined, -2, lam, ow, sched)
    _same(got, ref)
    assert np.abs(ref[0][-1] - wlm.params0(wl)).max() > 0


@pytest.mark.parametrize("P", [1, 5, 255, 1023, 1025, 4097, 65537])
@pytest.mark.parametrize("W", [1, 3, 8, 24, 25])
def test_ragged_sizes_and_worker_counts(P, W):
    wl = dataclasses.replace(wlm.config(3, small=True, T=4), P=P, W=W)
    ref = _run(wl, True, -1)
    got = _run(wl, True, -2)
    _same(got, ref)


def test_mlp_weight_copy_is_refreshed_by_the_bulk_copy_kernel():
    import torch

    from paper_2308_15164_b200 import binding as B

    wl = wlm.config(4, small=True, T=5)
    d = wl.mlp
    x0 = wlm.params0(wl)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()
    torch.cuda.synchronize()
    outs = []
    for variant in (-1, -2):
        eng = B.AbsSgd(torch.from_numpy(x0).cuda(), wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=True,
                       mlp=(d.d_in, d.d_hidden, d.d_out, d.mb))
        eng.set_launch(B.K_SYNC, variant)
        for calls in wlm.iter_calls(wl):
            for (i, k, c) in calls:
                eng.accumulate_mlp(i, xs_d[c % wl.mlp_pool], ys_d[c % wl.mlp_pool])
            eng.sync_step()
        eng.check()
        outs.append(eng.params_host())
        eng.destroy()
    assert np.array_equal(outs[0], outs[1])
    assert np.abs(outs[0] - x0).max() > 1e-5
