"""Drives the CUDA path (through the C ABI binding) and the CPU oracle over the same seeded
workload, for the parity tests.  Inputs flow from the workload generators to both sides;
nothing computed by one side is fed to the other."""

from __future__ import annotations

import numpy as np

from paper_2308_15164_b200 import workloads as wlm

TOL_F32 = 1e-5          # max |x_gpu - x_oracle| <= TOL_F32 * max |x_oracle|   (fp32 path)
TOL_BF16 = 2e-3         # same bound for runs whose gradients come from bf16-operand GEMMs


def oracle_run(wl, x0, pool, columns=None, lambda_dc=0.0, oracle_cls=None, lr_schedule=None, every_iteration=True):
    """Run the oracle over the workload (optionally restricted to `columns` of the parameter
    vector -- the path is element-wise, so a column subset evolves independently).
    Returns dict(xs=[x_1, x_2, ...], consumed=[...], states=[(cnt, cur, t) after each sync])."""
    if oracle_cls is None:
        from oracle.abs_oracle import AbsSgdOracle as oracle_cls
    if columns is not None:
        x0 = x0[columns]
        if pool is not None:
            pool = pool[:, columns]
    o = oracle_cls(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay, lambda_dc)
    xs, states = [], []
    for t, calls in enumerate(wlm.iter_calls(wl)):
        if lr_schedule is not None:
            o.lr = lr_schedule[t]
        for (i, k, c) in calls:
            if wl.pool_size:
                g = pool[c % wl.pool_size]
            else:
                g = wlm.fresh_grad(wl, t, i, k)
                if columns is not None:
                    g = g[columns]
            o.accumulate(i, g)
        o.sync_step()
        if every_iteration or t == wl.T - 1:           # (full-size runs keep the final parameters only)
            xs.append(o.params().copy())
        states.append(o.counters())
    return dict(xs=xs, consumed=[np.asarray(c) for c in o.consumed], states=states, v=np.asarray(o.v).copy())


def gpu_run(wl, x0, pool, pipelined, columns=None, lambda_dc=0.0, every_iteration=True, lr_schedule=None,
            host_input=False, overwrite_first=False, batch=0):
    """Run the CUDA path over the workload.  Returns the same dict as oracle_run (xs restricted to
    `columns` when given).  With every_iteration=False only the final parameters are read back.
    batch > 0 (pool workloads): each worker's gradients of an iteration go through abs_accumulate_batch in
    chunks of up to `batch`, in the worker's own arrival order (rows of different workers are independent)."""
    import torch

    from paper_2308_15164_b200 import binding as B

    dev = torch.device("cuda:0")
    x0_d = torch.from_numpy(x0).to(dev)
    gd = B.GRAD_BF16 if wl.grad_dtype == "bf16" else B.GRAD_F32
    eng = B.AbsSgd(x0_d, wl.W, wl.lr, wl.momentum, wl.weight_decay, lambda_dc, grad_dtype=gd,
                   pipelined=pipelined, host_input=host_input, overwrite_first=overwrite_first)
    pool_d = None
    pool_h = None
    if wl.pool_size:
        if host_input:
            pool_h = torch.from_numpy(pool.view(np.int16) if pool.dtype == np.uint16 else pool).pin_memory()
        else:
            # rows padded to a multiple of 8 elements so that every row starts 16-byte aligned
            src = torch.from_numpy(pool.view(np.int16) if pool.dtype == np.uint16 else pool)
            pool_d = torch.zeros((pool.shape[0], (pool.shape[1] + 7) // 8 * 8), dtype=src.dtype, device=dev)
            pool_d[:, :pool.shape[1]] = src.to(dev)
    torch.cuda.synchronize()
    cols_d = torch.from_numpy(columns).to(dev) if columns is not None else None
    xs, states, keep = [], [], []
    n_iter = 0
    for t, calls in enumerate(wlm.iter_calls(wl)):
        if lr_schedule is not None and t + 1 < len(lr_schedule):
            eng.set_lr(float(lr_schedule[t + 1]))     # gamma_{t+1}: supplied one iteration ahead
        if batch and wl.pool_size and not host_input:
            per_worker = {}
            for (i, k, c) in calls:
                per_worker.setdefault(i, []).append(pool_d[c % wl.pool_size])
            for i, gs in per_worker.items():
                for lo in range(0, len(gs), batch):
                    eng.accumulate_batch(i, gs[lo:lo + batch])
            calls = []
        for (i, k, c) in calls:
            if wl.pool_size:
                if host_input:
                    eng.accumulate_host(i, pool_h[c % wl.pool_size])
                else:
                    eng.accumulate(i, pool_d[c % wl.pool_size])
            else:
                g = torch.from_numpy(wlm.fresh_grad(wl, t, i, k)).to(dev)
                torch.cuda.current_stream().synchronize()
                keep.append(g)
                eng.accumulate(i, g)
        eng.sync_step()
        n_iter += 1
        states.append(eng.counters())
        if every_iteration or n_iter == wl.T:
            with torch.cuda.stream(eng.stream_acc):
                p = eng.params()
                p = p[cols_d] if cols_d is not None else p.clone()
            eng.stream_acc.synchronize()
            xs.append(p.cpu().numpy())
    eng.synchronize()
    T = len(states)
    consumed = [eng.consumed(s) for s in range(max(0, T - 60), T)]
    eng.wait()
    v = eng.momentum()
    with torch.cuda.stream(eng.stream_acc):
        v = (v[cols_d] if cols_d is not None else v.clone())
    eng.synchronize()
    out = dict(xs=xs, consumed=consumed, consumed_from=max(0, T - 60), states=states, v=v.cpu().numpy(),
               launches=eng.launch_count())
    eng.destroy()
    return out


def assert_params_close(x_gpu, x_ref, tol=TOL_F32, what=""):
    scale = float(np.abs(x_ref).max())
    err = float(np.abs(x_gpu.astype(np.float64) - x_ref.astype(np.float64)).max())
    assert err <= tol * scale, f"{what}: max abs err {err:.3e} > {tol:g} * max|param| ({scale:.3e})"
    return err / max(scale, 1e-300)


def assert_states_equal(gpu, ref):
    """b_i counters, set index and iteration counter: bit-exact after every sync step."""
    assert len(gpu["states"]) == len(ref["states"])
    for s, ((c1, cur1, t1), (c2, cur2, t2)) in enumerate(zip(gpu["states"], ref["states"])):
        assert np.array_equal(c1, c2), f"counters differ after sync step {s}: {c1} vs {c2}"
        assert (cur1, t1) == (cur2, t2), f"(cur, t) differ after sync step {s}"
    f = gpu["consumed_from"]
    for s, b in enumerate(gpu["consumed"]):
        assert np.array_equal(b, ref["consumed"][f + s]), f"device-side b_i of sync step {f + s}: {b} vs {ref['consumed'][f + s]}"
