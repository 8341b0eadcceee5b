"""Step 1 across GPUs with the count exchanges on NCCL (dist.GlobalStep as the benchmark's multi-GPU section
drives it).  One GPU is at hand, so the process group has ONE rank: the NCCL branch of the exchange -- an in-place
int32 all-reduce ordered on stream_sync, no host block -- and the whole begin / exchange / kernel / exchange / end
sequence run for real, against the CPU oracle; what one GPU cannot show is the traffic between peers (covered, as
far as one GPU goes, by the emulated-rank and two-process tests).  Runs in a child process so that the process
group does not outlive the test."""

import os
import socket
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

pytestmark = pytest.mark.gpu

T = 12


def _child(port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK="0", LOCAL_RANK="0", WORLD_SIZE="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
                      NCCL_NVLS_ENABLE="0")
    try:
        import torch
        import torch.distributed as dist

        from paper_2308_15164_b200 import binding as B
        from paper_2308_15164_b200 import dist as D
        from paper_2308_15164_b200 import workloads as wlm

        dev = torch.device("cuda:0")
        torch.cuda.set_device(dev)
        dist.init_process_group(backend="nccl", rank=0, world_size=1, device_id=dev)
        wl = wlm.config(3, small=True, T=T)
        sched = wlm.schedule(wl).copy()
        sched[5, :] = 0                                   # one iteration in which nobody computed anything
        pool = wlm.grad_pool(wl)
        pool_d = torch.zeros((pool.shape[0], (pool.shape[1] + 7) // 8 * 8), dtype=torch.float32, device=dev)
        pool_d[:, :pool.shape[1]] = torch.from_numpy(pool).to(dev)
        x0_d = torch.from_numpy(wlm.params0(wl)).to(dev)
        torch.cuda.synchronize()
        eng = B.AbsSgd(x0_d, wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=True)
        step = D.GlobalStep(eng)
        assert dist.get_backend() == "nccl"
        xs, c = [], 0
        for b_row in sched:
            for (i, k) in wlm.call_order(b_row):
                eng.accumulate(i, pool_d[c % wl.pool_size]); c += 1
            ev = step.sync_step(timed=True)
            xs.append(eng.params_host())
        eng.check()
        assert ev[0].elapsed_time(ev[1]) > 0.0
        consumed = [eng.global_consumed(s) for s in range(T)]
        step.close()
        eng.destroy()

        # the benchmark's multi-GPU section on the same one-rank group (small vector, a few iterations)
        import bench

        wl2 = wlm.config(2, small=True)
        rows = [pool_d[r].data_ptr() for r in range(pool_d.shape[0])]     # rows of P(workload 3) >= P(workload 2, small) floats
        sec = bench.run_global_step(B, D, wlm, wl2, dev, 0, 1, rows, 5, bench.measured_peaks())
        dist.destroy_process_group()
        out.put(("ok", xs, consumed, sec))
    except Exception as exc:                              # the parent turns this into a test failure
        import traceback

        out.put(("error", traceback.format_exc(), None, None))


def test_global_step_over_a_one_rank_nccl_group_matches_the_oracle():
    from oracle.abs_oracle import AbsSgdOracle
    from paper_2308_15164_b200 import workloads as wlm

    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    p = ctx.Process(target=_child, args=(port, q))
    p.start()
    status, xs, consumed, sec = q.get(timeout=600)
    p.join(timeout=120)
    assert status == "ok", xs
    assert p.exitcode == 0

    wl = wlm.config(3, small=True, T=T)
    sched = wlm.schedule(wl).copy()
    sched[5, :] = 0
    pool = wlm.grad_pool(wl)
    o = AbsSgdOracle(wlm.params0(wl), wl.W, wl.lr, wl.momentum, wl.weight_decay)
    c = 0
    for t, b_row in enumerate(sched):
        for (i, k) in wlm.call_order(b_row):
            o.accumulate(i, pool[c % wl.pool_size]); c += 1
        o.sync_step()
        want = o.params()
        assert np.abs(xs[t] - want).max() <= 1e-5 * np.abs(want).max(), f"x_{t + 1}"
        assert np.array_equal(consumed[t], o.consumed[t])
    assert np.abs(xs[-1] - xs[0]).max() > 0
    # the benchmark section ran and reports finite figures (no peers: nothing crosses NVLink)
    assert sec["ranks"] == 1 and sec["nvlink_bytes_in_per_rank"] == 0 and sec["nvlink_bytes_out_per_rank"] == 0
    assert sec["us_per_iteration_max_over_ranks"] > 0 and sec["us_fused_kernel_max_over_ranks"] > 0
    assert np.isfinite(sec["whole_job_gbs"]) and sec["whole_job_gbs"] > 0
