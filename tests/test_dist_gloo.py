"""CPU-only: the replica plumbing (barrier, max-over-ranks timing, summed work) on a
world_size-2 gloo group."""

import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2308_15164_b200 import dist as D

    r, lr, w = D.init("gloo")
    assert (r, lr, w) == (rank, rank, world)
    D.barrier()
    secs = 1.0 + rank          # rank 1 is the slow replica
    units = 10.0 * (rank + 1)
    thr, worst = D.aggregate_throughput(units, secs)
    out.put((rank, thr, worst, D.reduce_max(float(rank)), D.reduce_sum(1.0)))
    D.barrier()
    D.shutdown()


def test_two_rank_aggregation():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, thr, worst, mx, sm in res:
        assert worst == 2.0                   # max over ranks
        assert abs(thr - 30.0 / 2.0) < 1e-12  # all units / slowest replica
        assert mx == 1.0 and sm == 2.0


def test_single_process_defaults():
    sys.path.insert(0, ROOT)
    from paper_2308_15164_b200 import dist as D

    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert D.rank_info() == (0, 0, 1)
    assert D.aggregate_throughput(8.0, 2.0) == (4.0, 2.0)


def _exchange_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch

    from paper_2308_15164_b200 import dist as D

    D.init("gloo")
    W = 3                                               # local workers per rank
    # what abs_global_begin leaves in the exchange vector: own b_i in own slots, zeros elsewhere
    own = torch.tensor([[2, 0, 5], [1, 7, 0]], dtype=torch.int32)[rank]
    counts = torch.zeros(world * W, dtype=torch.int32)
    counts[rank * W:(rank + 1) * W] = own
    D.exchange_counts(counts)                           # exchange A
    token = torch.zeros(1, dtype=torch.int32)
    D.exchange_counts(token)                            # exchange B (a barrier)
    infos = D.gather_handles((bytes([rank]) * 64, 4096 * rank, "host", 1000 + rank))
    out.put((rank, counts.tolist(), int(token.item()), infos))
    D.barrier()
    D.shutdown()


def test_two_rank_count_exchange_and_handle_gather():
    """Host side of Step 1 across GPUs on a world_size-2 gloo group: the summed exchange vector holds every
    rank's b_i in global worker order on every rank; the handle gather returns rank order."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_exchange_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, counts, token, infos in res:
        assert counts == [2, 0, 5, 1, 7, 0]
        assert token == 0
        assert [i[0] for i in infos] == [bytes([0]) * 64, bytes([1]) * 64]
        assert [i[1] for i in infos] == [0, 4096] and [i[3] for i in infos] == [1000, 1001]
