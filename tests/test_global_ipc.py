"""Step 1 across GPUs with the ranks as separate PROCESSES (dist.GlobalStep): each rank exports its workspace
with abs_ipc_export, maps the other's with abs_ipc_open, and the fused kernel of one process reads and writes
the other process's memory.  Two processes share the one GPU at hand (the mapping mechanism is the same as
between two GPUs of a node; the count exchange runs over gloo on the host, so no kernel ever waits for the
other process).  Checked against the CPU oracle with all workers, and rank against rank bit for bit."""

import os
import socket
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

pytestmark = pytest.mark.gpu

G, T, STRIDE = 2, 8, 97


def _rank_main(rank, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK="0", WORLD_SIZE=str(G), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    try:
        import torch

        from paper_2308_15164_b200 import binding as B
        from paper_2308_15164_b200 import dist as D
        from paper_2308_15164_b200 import workloads as wlm

        D.init("gloo", timeout_s=120)
        dev = torch.device("cuda:0")
        torch.cuda.set_device(dev)
        wl = wlm.config(3, small=True, T=T)
        Wl = wl.W // G
        sched = wlm.schedule(wl).copy()
        sched[3, :] = 0                                   # one iteration in which nobody computed anything
        pool = wlm.grad_pool(wl)
        pool_d = torch.zeros((pool.shape[0], (pool.shape[1] + 7) // 8 * 8), dtype=torch.float32, device=dev)
        pool_d[:, :pool.shape[1]] = torch.from_numpy(pool).to(dev)
        x0_d = torch.from_numpy(wlm.params0(wl)).to(dev)
        torch.cuda.synchronize()
        eng = B.AbsSgd(x0_d, Wl, wl.lr, wl.momentum, wl.weight_decay, pipelined=True)
        step = D.GlobalStep(eng)
        samples, c = [], 0
        for b_row in sched:
            for (i, k) in wlm.call_order(b_row):
                if i // Wl == rank:                       # this rank's workers only
                    eng.accumulate(i % Wl, pool_d[c % wl.pool_size])
                c += 1
            step.sync_step()
            with torch.cuda.stream(eng.stream_acc):
                p = eng.params().clone()
            eng.stream_acc.synchronize()
            samples.append(p[::STRIDE].cpu().numpy())
        final = p.cpu().numpy()
        consumed = [eng.global_consumed(s) for s in range(T)]
        eng.check()
        step.close()
        eng.destroy()
        out.put((rank, "ok", samples, final, consumed))
        D.barrier()
        D.shutdown()
    except Exception as e:  # noqa: BLE001  (reported to the parent, which fails the test)
        import traceback

        out.put((rank, "error", traceback.format_exc(), repr(e), None))


def test_two_processes_share_their_workspaces_over_cuda_ipc():
    from oracle.abs_oracle import AbsSgdOracle
    from paper_2308_15164_b200 import workloads as wlm

    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, port, q)) for r in range(G)]
    for p in procs:
        p.start()
    res = {}
    try:
        for _ in procs:
            r = q.get(timeout=300)
            res[r[0]] = r
    finally:
        for p in procs:
            p.join(timeout=60)
            if p.is_alive():
                p.kill()
    for r in range(G):
        assert res[r][1] == "ok", res[r][2]

    wl = wlm.config(3, small=True, T=T)
    sched = wlm.schedule(wl).copy()
    sched[3, :] = 0
    pool = wlm.grad_pool(wl)
    ref = AbsSgdOracle(wlm.params0(wl), wl.W, wl.lr, wl.momentum, wl.weight_decay)
    c = 0
    for t, b_row in enumerate(sched):
        for (i, k) in wlm.call_order(b_row):
            ref.accumulate(i, pool[c % wl.pool_size]); c += 1
        ref.sync_step()
        want = ref.params()
        assert np.array_equal(res[0][2][t], res[1][2][t]), f"ranks disagree on x_{t + 1}"
        err = np.abs(res[0][2][t].astype(np.float64) - want[::STRIDE]).max()
        assert err <= 1e-5 * np.abs(want).max(), (t, err)
    assert np.array_equal(res[0][3], res[1][3])
    assert np.abs(res[0][3].astype(np.float64) - ref.params()).max() <= 1e-5 * np.abs(ref.params()).max()
    assert np.abs(res[0][3] - wlm.params0(wl)).max() > 0                      # the run did move the parameters
    for r in range(G):
        for s in range(T):
            assert np.array_equal(res[r][4][s], np.asarray(ref.consumed[s])), (r, s)
