"""abs_state_export / abs_state_import: a run that is exported after k iterations and imported into a FRESH
context (created from other initial parameters) continues bit for bit like the uninterrupted run -- parameters,
momentum, counters, consumed-count log -- in eager and pipelined mode, with bf16 gradients, with Eq. 6 and a
learning-rate schedule, for the MLP path, and for ranks in multi-GPU mode."""

import ctypes

import numpy as np
import pytest

from paper_2308_15164_b200 import workloads as wlm

pytestmark = pytest.mark.gpu


def _mk(wl, x0_d, pipelined, lambda_dc=0.0, overwrite_first=False, W=None):
    from paper_2308_15164_b200 import binding as B

    gd = B.GRAD_BF16 if wl.grad_dtype == "bf16" else B.GRAD_F32
    return B.AbsSgd(x0_d, W or wl.W, wl.lr, wl.momentum, wl.weight_decay, lambda_dc, grad_dtype=gd, pipelined=pipelined,
                    overwrite_first=overwrite_first)


def _pool_d(pool, dev):
    import torch

    src = torch.from_numpy(pool.view(np.int16) if pool.dtype == np.uint16 else pool)
    out = torch.zeros((pool.shape[0], (pool.shape[1] + 7) // 8 * 8), dtype=src.dtype, device=dev)
    out[:, :pool.shape[1]] = src.to(dev)
    return out


def _snapshot(eng):
    import torch

    eng.wait()
    eng.synchronize()
    x = eng.params().clone().cpu().numpy()
    v = eng.momentum().clone().cpu().numpy()
    torch.cuda.synchronize()
    return x, v, eng.counters()


@pytest.mark.parametrize("cfg,pipelined,lam,ow", [(2, False, 0.0, False), (2, True, 0.5, False), (3, True, 0.0, True), (5, True, 0.0, False),
                                                 (5, False, 2.0, False)])
def test_resume_is_bit_exact_streaming(cfg, pipelined, lam, ow):
    import torch

    dev = torch.device("cuda:0")
    k = 5
    wl = wlm.config(cfg, small=True, T=2 * k)
    x0_d = torch.from_numpy(wlm.params0(wl)).to(dev)
    pool = _pool_d(wlm.grad_pool(wl), dev)
    lrs = [wl.lr * (0.7 ** t) for t in range(wl.T + 1)]
    calls = list(wlm.iter_calls(wl))

    def run(eng, t0, t1):
        for t in range(t0, t1):
            eng.set_lr(lrs[t + 1])
            for (i, kk, c) in calls[t]:
                eng.accumulate(i, pool[c % wl.pool_size])
            eng.sync_step()

    a = _mk(wl, x0_d, pipelined, lam, ow)
    run(a, 0, 2 * k)
    want = _snapshot(a)
    want_consumed = [a.consumed(s) for s in range(2 * k)]
    a.destroy()

    b = _mk(wl, x0_d, pipelined, lam, ow)
    run(b, 0, k)
    blob = b.state_export()
    b.destroy()
    c = _mk(wl, torch.full_like(x0_d, 7.0), pipelined, lam, ow)          # other parameters: everything must come from the blob
    run(c, 0, 2)                                                         # ... and other history
    c.state_import(blob)
    assert c.counters()[2] == k
    run(c, k, 2 * k)
    got = _snapshot(c)
    assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1])
    assert np.array_equal(got[2][0], want[2][0]) and got[2][1:] == want[2][1:]
    for s in range(2 * k):
        assert np.array_equal(c.consumed(s), want_consumed[s])
    c.destroy()


def test_resume_is_bit_exact_mlp_with_gathered_calls():
    import torch

    from paper_2308_15164_b200 import binding as B

    dev = torch.device("cuda:0")
    k = 3
    wl = wlm.config(4, small=True, T=2 * k)
    d = wl.mlp
    x0_d = torch.from_numpy(wlm.params0(wl)).to(dev)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).to(dev), torch.from_numpy(ys).to(dev)
    torch.cuda.synchronize()
    calls = list(wlm.iter_calls(wl))

    def mk(p0):
        return B.AbsSgd(p0, wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=True, mlp=(d.d_in, d.d_hidden, d.d_out, d.mb),
                        mlp_coalesce=True)

    def run(eng, t0, t1, stop_mid=False):
        for t in range(t0, t1):
            for (i, kk, c) in calls[t]:
                eng.accumulate_mlp(i, xs_d[c % wl.mlp_pool], ys_d[c % wl.mlp_pool])
            eng.sync_step()

    a = mk(x0_d)
    run(a, 0, 2 * k)
    want = _snapshot(a)
    a.destroy()
    b = mk(x0_d)
    run(b, 0, k)
    blob = b.state_export()
    b.destroy()
    c = mk(torch.zeros_like(x0_d))
    c.state_import(blob)
    run(c, k, 2 * k)
    got = _snapshot(c)
    assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1])
    assert np.abs(want[0] - wlm.params0(wl)).max() > 1e-5
    c.check()
    c.destroy()


def test_export_in_mid_iteration_keeps_the_partial_accumulators():
    import torch

    dev = torch.device("cuda:0")
    wl = wlm.config(2, small=True, T=4)
    x0_d = torch.from_numpy(wlm.params0(wl)).to(dev)
    pool = _pool_d(wlm.grad_pool(wl), dev)
    calls = list(wlm.iter_calls(wl))
    flat = [(t, i, c) for t in range(wl.T) for (i, kk, c) in calls[t]]
    ends = {t: max(n for n, (tt, _, _) in enumerate(flat) if tt == t) for t in range(wl.T)}

    def run(eng, n0, n1):
        for n in range(n0, n1):
            t, i, c = flat[n]
            eng.accumulate(i, pool[c % wl.pool_size])
            if n == ends[t]:
                eng.sync_step()

    a = _mk(wl, x0_d, True)
    run(a, 0, len(flat))
    want = _snapshot(a)
    a.destroy()
    cut = ends[1] + 6                                  # six micro-batches into iteration 2
    b = _mk(wl, x0_d, True)
    run(b, 0, cut)
    blob = b.state_export()
    b.destroy()
    c = _mk(wl, torch.zeros_like(x0_d), True)
    c.state_import(blob)
    run(c, cut, len(flat))
    got = _snapshot(c)
    assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1]) and np.array_equal(got[2][0], want[2][0])
    c.destroy()


def test_multi_gpu_ranks_resume():
    import torch

    from paper_2308_15164_b200 import dist as D

    dev = torch.device("cuda:0")
    G, k = 2, 4
    wl = wlm.config(3, small=True, T=2 * k)
    Wl = wl.W // G
    x0_d = torch.from_numpy(wlm.params0(wl)).to(dev)
    pool = _pool_d(wlm.grad_pool(wl), dev)
    calls = list(wlm.iter_calls(wl))

    def mk(p0):
        ranks = [_mk(wl, p0, True, W=Wl) for _ in range(G)]
        return ranks, D.LocalRanks(ranks)

    def run(ranks, grp, t0, t1):
        for t in range(t0, t1):
            for (i, kk, c) in calls[t]:
                ranks[i // Wl].accumulate(i % Wl, pool[c % wl.pool_size])
            grp.sync_step()

    ra, ga = mk(x0_d)
    run(ra, ga, 0, 2 * k)
    want = [_snapshot(e) for e in ra]
    rb, gb = mk(x0_d)
    run(rb, gb, 0, k)
    blobs = [e.state_export() for e in rb]
    rc, gc = mk(torch.zeros_like(x0_d))
    for e, blob in zip(rc, blobs):
        e.state_import(blob)
    run(rc, gc, k, 2 * k)
    got = [_snapshot(e) for e in rc]
    for r in range(G):
        first, count = rc[r].global_slice()
        assert np.array_equal(got[r][0], want[r][0])
        assert np.array_equal(got[r][1][first:first + count], want[r][1][first:first + count])
    with pytest.raises(Exception):
        rc[0].state_import(blobs[1])                   # another rank's state
    for e in ra + rb + rc:
        e.destroy()


def test_import_rejects_foreign_and_truncated_states():
    import torch

    from paper_2308_15164_b200 import binding as B

    dev = torch.device("cuda:0")
    x0 = torch.zeros(4096, device=dev)
    a = B.AbsSgd(x0, 2, 0.1, 0.9)
    blob = a.state_export()
    assert blob.nbytes == int(B.lib.abs_state_bytes(a._h))
    other = B.AbsSgd(x0, 3, 0.1, 0.9)
    with pytest.raises(B.AbsError):
        other.state_import(blob)                       # other worker count
    with pytest.raises(B.AbsError):
        a.state_import(blob[:-1])                      # truncated
    bad = blob.copy(); bad[0] ^= 0xFF
    with pytest.raises(B.AbsError):
        a.state_import(bad)                            # not a state
    assert B.lib.abs_state_export(a._h, None, blob.nbytes) == B.EINVAL
    small = np.empty(16, dtype=np.uint8)
    assert B.lib.abs_state_export(a._h, small.ctypes.data, small.nbytes) == B.EINVAL
    a.state_import(blob)                               # its own state is fine
    a.destroy(); other.destroy()
    assert B.lib.abs_state_bytes(None) == 0
