"""Process-group plumbing, one process per GPU.

Two uses.  (1) Independent replicas of the one-GPU step (the benchmark's --gpus N): no exchange between
replicas, only a barrier around the timed region and max/sum reductions of the measurements.
(2) Step 1 across GPUs (`GlobalStep`): the paper's workers on different GPUs.  The gradients are moved by the
library's own kernel through peer mappings of the ranks' workspaces; this module only exchanges the workspace
handles once and, per iteration, sums the W * n_ranks micro-batch counts and runs a closing barrier -- both
ordered on the context's stream_sync.  `LocalRanks` drives several ranks of the same protocol inside one
process on one GPU (their kernels never wait for one another; events order them), which is how the multi-rank
arithmetic is checked where only one GPU is at hand."""

from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def rank_info() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str, timeout_s: float = 0.0) -> Tuple[int, int, int]:
    """Joins the process group named by the torchrun environment.  timeout_s > 0 bounds every collective of a
    host-side backend (a rank that never arrives then ends the others with an error instead of a hang)."""
    rank, local_rank, world = rank_info()
    if world > 1 and not dist.is_initialized():
        import datetime

        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        # the collectives of this package carry a few integers: in-switch reduction buys nothing, and a rank that
        # leaves while its memory is bound to an NVLink-switch reduction group is worse than one that simply leaves
        os.environ.setdefault("NCCL_NVLS_ENABLE", "0")
        kw = dict(timeout=datetime.timedelta(seconds=timeout_s)) if timeout_s > 0 else {}
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kw)
    return rank, local_rank, world


def barrier(device=None):
    if dist.is_available() and dist.is_initialized():
        if device is not None and device.type == "cuda":
            dist.barrier(device_ids=[device.index])
        else:
            dist.barrier()


def reduce_max(value: float, device=None) -> float:
    """Max over ranks of a per-rank scalar (e.g. the device-timed duration of the timed region)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def reduce_sum(value: float, device=None) -> float:
    """Sum over ranks (e.g. units of work processed)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def aggregate_throughput(units_this_rank: float, seconds_this_rank: float, device=None) -> Tuple[float, float]:
    """Whole-job throughput of independent replicas: (sum of units) / (max of durations).
    Returns (throughput, max_seconds)."""
    total = reduce_sum(units_this_rank, device)
    worst = reduce_max(seconds_this_rank, device)
    return total / worst, worst


def shutdown():
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------------
# Step 1 across GPUs
# --------------------------------------------------------------------------------------------------
def exchange_counts(counts: torch.Tensor, stream=None, group=None) -> None:
    """Sum the int32 exchange vector over all ranks, in place.  Device tensors on an NCCL group: the collective
    is ordered behind `stream` and `stream` waits for it (no host block).  Otherwise (gloo): the host waits for
    `stream`, sums on the CPU and writes the result back on `stream`."""
    if counts.is_cuda and dist.get_backend(group) == "nccl":
        with torch.cuda.stream(stream):
            dist.all_reduce(counts, op=dist.ReduceOp.SUM, group=group)
        return
    if counts.is_cuda:
        stream.synchronize()
        host = counts.cpu()
        dist.all_reduce(host, op=dist.ReduceOp.SUM, group=group)
        with torch.cuda.stream(stream):
            counts.copy_(host.to(counts.device))
        stream.synchronize()           # the pageable copy above must not outlive `host`
    else:
        dist.all_reduce(counts, op=dist.ReduceOp.SUM, group=group)


def gather_handles(own, group=None) -> list:
    """Every rank's (handle bytes, offset, host name, process id) in rank order."""
    world = dist.get_world_size(group)
    out = [None] * world
    dist.all_gather_object(out, own, group=group)
    return out


class GlobalStep:
    """Ends the iterations of a multi-GPU run.  `eng` is this rank's binding.AbsSgd (pipelined, same
    configuration on every rank); the default process group (or `group`) spans the ranks."""

    def __init__(self, eng, group=None):
        import socket

        from . import binding as B

        self.eng, self.group, self.B = eng, group, B
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        eng.synchronize()                                     # abs_init has finished on this rank ...
        handle, off = B.ipc_export(eng.workspace.data_ptr())
        infos = gather_handles((handle, off, socket.gethostname(), os.getpid()), group)   # ... and on every rank
        self._opened = []
        spaces = []
        with torch.cuda.device(eng.device):
            for q, (h, o, host, pid) in enumerate(infos):
                if q == self.rank:
                    spaces.append(eng.workspace.data_ptr())
                    continue
                if host != infos[self.rank][2]:
                    raise RuntimeError("peer mappings need all ranks on one NVLink node")
                p = B.ipc_open(h, o)
                self._opened.append((p, o))
                spaces.append(p)
        eng.global_attach(self.rank, spaces)
        self._token = torch.zeros(1, dtype=torch.int32, device=eng.device)
        dist.barrier(group=group)

    def sync_step(self, timed: bool = False):
        """One end of iteration.  timed=True returns a CUDA event pair on stream_sync around this rank's fused
        kernel (between the two exchanges)."""
        eng = self.eng
        counts = eng.global_begin()
        exchange_counts(counts, eng.stream_sync, self.group)          # exchange A: all b_i, everywhere
        ev = None
        if timed:
            ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
            ev[0].record(eng.stream_sync)
        eng.global_step()
        if timed:
            ev[1].record(eng.stream_sync)
        exchange_counts(self._token, eng.stream_sync, self.group)     # exchange B: every rank's kernel is done
        eng.global_end()
        return ev

    def close(self):
        self.eng.synchronize()
        dist.barrier(group=self.group)                                # nobody still reads a peer's memory
        for p, o in self._opened:
            self.B.ipc_close(p, o)
        self._opened = []


class LocalRanks:
    """G ranks of the multi-GPU protocol inside one process, all on one device: every rank has its own
    context, workspace and streams, peer pointers are plain pointers, and the two exchanges are done with
    events and a small torch sum on a control stream.  No kernel waits for another rank's kernel."""

    def __init__(self, engines):
        self.engines = list(engines)
        dev = self.engines[0].device
        self.ctrl = torch.cuda.Stream(device=dev)
        for e in self.engines:
            e.synchronize()
        spaces = [e.workspace.data_ptr() for e in self.engines]
        for r, e in enumerate(self.engines):
            e.global_attach(r, spaces)

    def _join(self):
        """Control stream waits for every rank's stream_sync."""
        for e in self.engines:
            self.ctrl.wait_stream(e.stream_sync)

    def _fork(self):
        for e in self.engines:
            e.stream_sync.wait_stream(self.ctrl)

    def sync_step(self, timed: bool = False):
        """One end of iteration on all ranks.  timed=True returns a CUDA event pair on the control stream that
        brackets the G fused kernels (which run side by side on this one GPU)."""
        counts = [e.global_begin() for e in self.engines]
        self._join()
        with torch.cuda.stream(self.ctrl):                    # exchange A
            total = torch.stack(counts).sum(dim=0, dtype=torch.int32)
            for c in counts:
                c.copy_(total)
        ev = None
        if timed:
            ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
            ev[0].record(self.ctrl)
        self._fork()
        for e in self.engines:
            e.global_step()
        self._join()                                          # exchange B
        if timed:
            ev[1].record(self.ctrl)
        self._fork()
        for e in self.engines:
            e.global_end()
        return ev
