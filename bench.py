#!/usr/bin/env python
"""Benchmark of the delayed synchronous step (ABS-SGD, arXiv 2308.15164, Algorithm 1) on B200.

A "step" is one iteration of Algorithm 1 on the ResNet18-sized workload (P = 11,689,512 fp32
parameters, W = 4 workers with b = (2,2,4,8) micro-batches): 16 accumulate launches (Step 2)
plus one fused weighted-reduce/update launch (Step 1), run in pipelined mode so that Step 1 of
iteration t overlaps Step 2 of iteration t+1.  The metric is algorithmic HBM bytes per second:

    bytes per step = 16 * 12 * P  (accumulate: read g, read acc, write acc)
                   + (8 * 4 + 16) * P  (fused step: read 4 acc + x + v, write x + v + 4 zeros)

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (launched by torchrun) every rank runs an independent replica on its own GPU (the
step has no exchange between replicas); rank 0 prints ONE JSON line with the whole-job value.
"""

from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "delayed-sync iteration HBM throughput (16 accumulate + 1 fused sync step, algorithmic bytes)"
UNIT = "GB/s"
HBM_NOMINAL_GBS = 8000.0
HBM_FALLBACK_GBS = 6650.0
NVLINK_MEASURED_GBS = 770.0        # peer copy, per direction and GPU, measured on this machine
# the same string in both arms: the workload the headline metric is quoted on
WORKLOAD = ("cfg2 resnet18-sized static heterogeneity: P=11689512 fp32 (62 tensors), W=4, b=(2,2,4,8), lr=0.1 mu=0.9 "
            "wd=5e-4; one step = one iteration = 16 accumulate + 1 fused sync step")
MIN_TIMED_SECONDS = 1.0            # the --steps-long region is repeated until this much time has been measured
DEFAULT_SECTIONS = "e2e,cpu,mlp,tiny,schedules,batch_curve,sync_curve,global"
GLOBAL_STEP_DEADLINE_S = 180       # multi-GPU section: see run_ours


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=HBM_FALLBACK_GBS, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, local_rank: int):
        # nvidia-smi takes an index or a UUID: with CUDA_VISIBLE_DEVICES set, the local rank's entry as it stands
        self.gpu = str(local_rank)
        try:
            vis = [t.strip() for t in os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",") if t.strip()]
            if vis:
                self.gpu = vis[local_rank]
        except Exception:
            pass
        self.proc = None
        self.path = None
        self.skip = 0

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
            # nvidia-smi takes a few hundred ms to start: wait for its first (idle) sample so that the
            # samples that follow fall inside the timed region
            t0 = time.time()
            while time.time() - t0 < 5.0 and os.path.getsize(self.path) == 0:
                time.sleep(0.02)
            self.skip = sum(1 for _ in open(self.path))
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for n, line in enumerate(open(self.path)):
                if n < self.skip:
                    continue
                f = [s.strip() for s in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


def bytes_per_step(wl, b_row):
    g_bytes = 2 if wl.grad_dtype == "bf16" else 4
    calls = int(sum(b_row))
    w_act = int(sum(1 for b in b_row if b > 0))
    acc = calls * (g_bytes + 8) * wl.P
    sync = (8 * w_act + 16) * wl.P
    return acc, sync


# ------------------------------------------------------------------------------------------
def run_reference(args):
    """The CPU oracle (C twin, OpenMP) timed on the host cores, same workload and metric."""
    from paper_2308_15164_b200 import dist as D
    from paper_2308_15164_b200 import workloads as wlm

    rank, _, world = D.rank_info()
    if rank != 0:
        return
    from oracle.c_oracle import AbsSgdOracleC

    wl = wlm.config(2)
    x0 = wlm.params0(wl)
    pool = wlm.grad_pool(wl)
    b_row = wlm.schedule(wl)[0]
    order = wlm.call_order(b_row)
    acc_b, sync_b = bytes_per_step(wl, b_row)
    o = AbsSgdOracleC(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    c = 0

    def one_step():
        nonlocal c
        for (i, k) in order:
            o.accumulate(i, pool[c % wl.pool_size]); c += 1
        o.sync_step()

    for _ in range(args.warmup):
        one_step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one_step()
    dt = time.perf_counter() - t0
    cores = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
    val = (acc_b + sync_b) * args.steps / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "where": "every step in full on the host cores (C oracle, OpenMP)"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{args.steps} full iterations of the workload (C oracle, OpenMP)"},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------
def run_ours(args):
    import torch

    from paper_2308_15164_b200 import binding as B
    from paper_2308_15164_b200 import dist as D
    from paper_2308_15164_b200 import workloads as wlm

    rank, local_rank, world = D.init("nccl")
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    peaks = measured_peaks()

    wl = wlm.config(2)
    x0 = wlm.params0(wl)
    pool = wlm.grad_pool(wl)                      # 16 x P fp32 = 748 MB (larger than the 126 MB L2)
    b_row = wlm.schedule(wl)[0]
    order = wlm.call_order(b_row)
    n_acc_step = len(order)
    acc_b, sync_b = bytes_per_step(wl, b_row)
    step_bytes = acc_b + sync_b
    per_acc = acc_b // n_acc_step
    pool_d = torch.from_numpy(pool).to(dev)
    x0_d = torch.from_numpy(x0).to(dev)
    torch.cuda.synchronize()

    def make(pipelined, host_input=False, overwrite_first=False):
        return B.AbsSgd(x0_d, wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=pipelined, host_input=host_input,
                        overwrite_first=overwrite_first)

    call_idx = [0]
    rows = [pool_d[r].data_ptr() for r in range(wl.pool_size)]      # raw device addresses of the pool rows

    def accumulates(eng):
        c = call_idx[0]
        for (i, k) in order:
            eng.accumulate(i, rows[c % wl.pool_size]); c += 1
        call_idx[0] = c

    def one_step(eng):
        accumulates(eng)
        eng.sync_step()

    def one_step_batched(eng):
        # every worker hands over its b_i gradients of the iteration in one call (one pass over its row)
        c = call_idx[0]
        per_worker = {}
        for (i, k) in order:
            per_worker.setdefault(i, []).append(rows[c % wl.pool_size]); c += 1
        call_idx[0] = c
        for i, gs in per_worker.items():
            eng.accumulate_batch(i, gs)
        eng.sync_step()

    def timed(eng, steps, warmup, one_step=one_step):
        """`steps` steps between a barrier + synchronize on both sides, timed by CUDA events on stream_acc (the
        stream every accumulate kernel is launched on).  Returns (seconds of the region, seconds from its start
        to the end of the LAST ACCUMULATE kernel, launches)."""
        for _ in range(warmup):
            one_step(eng)
        eng.wait(); eng.synchronize()
        D.barrier(dev)
        torch.cuda.synchronize()
        n0 = eng.launch_count()
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        with torch.cuda.stream(eng.stream_acc):
            e0.record()
            for _ in range(steps):
                one_step(eng)
            e1.record()                     # behind the last accumulate kernel; the last fused step may still run
            eng.wait()                      # stream_acc waits for the last fused kernel on stream_sync
            e2.record()
        torch.cuda.synchronize()
        D.barrier(dev)
        return e0.elapsed_time(e2) / 1e3, e0.elapsed_time(e1) / 1e3, eng.launch_count() - n0

    # ---- pass 1: the timed region (pipelined, nothing instrumented), repeated until >= MIN_TIMED_SECONDS ----
    eng = make(pipelined=True)
    sampler = ClockSampler(local_rank)
    secs_w, _, _ = timed(eng, max(args.steps // 10, 2), args.warmup)      # warm-up (outside the clock samples)
    est = secs_w / max(args.steps // 10, 2)
    repeats = int(min(max(1, np.ceil(args.min_seconds / max(est * args.steps, 1e-9))), 200))
    repeats = int(D.reduce_max(float(repeats), dev))                      # the same count on every rank
    sampler.start()
    regions = [timed(eng, args.steps, 0) for _ in range(repeats)]
    clocks = sampler.stop()
    secs_all = sorted(r[0] for r in regions)
    secs = float(np.median(secs_all))
    acc_chain_secs = float(np.median([r[1] for r in regions]))
    launches = regions[0][2]
    value, worst = D.aggregate_throughput(step_bytes * args.steps / 1e9, secs, dev)

    # ---- pass 2: same region with an event pair around every launch -> per-kernel durations (the events keep
    # consecutive kernels from being chained, so this pass is slower than pass 1) --
    eng.profile(True)
    secs_p2, _, _ = timed(eng, args.steps, 1)
    n_acc, ms_acc = eng.kernel_stats(B.K_ACCUMULATE)
    n_syn, ms_syn = eng.kernel_stats(B.K_SYNC)
    eng.profile(False)
    eng.destroy()

    # ---- pass 3: eager mode (no overlap): each kernel class alone on the GPU ------------------
    eng = make(pipelined=False)
    secs_eager, _, _ = timed(eng, args.steps, args.warmup)
    # the accumulate kernel alone, back to back on its stream (64 launches over the workers' rows, pool cycled)
    for rep_ in range(2):
        eng.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(eng.stream_acc):
            e0.record()
            for _ in range(4):
                accumulates(eng)
            e1.record()
        torch.cuda.synchronize()
    ms_chain, n_chain = e0.elapsed_time(e1), 4 * n_acc_step
    eng.sync_step()
    eng.profile(True)
    timed(eng, min(args.steps, 100), 2)
    n_acc_e, ms_acc_e = eng.kernel_stats(B.K_ACCUMULATE)
    n_syn_e, ms_syn_e = eng.kernel_stats(B.K_SYNC)
    eng.profile(False)
    eng.destroy()

    # ---- pass 4: byte-saving variant (ABS_FLAG_OVERWRITE_FIRST): fewer bytes per step, same results -----
    eng = make(pipelined=True, overwrite_first=True)
    secs_ow, _, _ = timed(eng, args.steps, args.warmup)
    eng.destroy()
    w_act = int(sum(1 for b in b_row if b > 0))
    ow_bytes = (int(sum(b_row)) - w_act) * 12 * wl.P + w_act * 8 * wl.P + (4 * w_act + 16) * wl.P

    # ---- pass 5: batched accumulation (abs_accumulate_batch): each row read and written once per iteration ----
    batched = {}
    for name, ow in (("default_mode", False), ("overwrite_first", True)):
        eng = make(pipelined=True, overwrite_first=ow)
        secs_b, _, launches_b = timed(eng, args.steps, args.warmup, one_step_batched)
        eng.destroy()
        acc_bytes = sum((4 * int(b) + (4 if ow else 8)) * wl.P for b in b_row if b > 0)
        syn_bytes = ((4 if ow else 8) * w_act + 16) * wl.P
        batched[name] = {"ms_per_step": secs_b / args.steps * 1e3, "bytes_per_step": acc_bytes + syn_bytes,
                         "hbm_gbs_on_its_own_bytes": (acc_bytes + syn_bytes) * args.steps / secs_b / 1e9,
                         "step_time_vs_default": secs_b / secs, "launches_per_step": launches_b / args.steps}

    # DRAM bytes (read + write) of ONE launch of each kernel at this workload's size, from an ncu capture of a lone
    # launch of the current kernels: reads equal the algorithmic reads, the writes partly stay in the 126 MB L2.
    NCU_TRAFFIC = {"k_accumulate_f32": 93_521_664 + 2_307_584, "k_sync<4>": 280_567_296 + 219_856_384}

    def roof(alg_bytes, n, ms, name, note):
        ach = alg_bytes / (ms / n / 1e3) / 1e9 if n and ms > 0 else None
        return {"kernel": name, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": (ach / peaks["hbm_gbs"]) if ach else None, "peak_source": "of " + peaks["source"],
                "frac_of_nominal_8TBs": (ach / HBM_NOMINAL_GBS) if ach else None,
                "avg_us": ms / n * 1e3 if n else None, "launches": n, "algorithmic_bytes": alg_bytes,
                "traffic": NCU_TRAFFIC.get(name) if wl.P == 11_689_512 else None,
                "traffic_note": "dram__bytes_read.sum + dram__bytes_write.sum of one LONE launch under ncu (not steady state)",
                "how": note}

    # The dominant kernel inside the timed region: the 16 * steps accumulate launches are back to back on stream_acc
    # (each waits for the one ahead; the fused step runs beside them on stream_sync), so their average duration is
    # the event-timed span from the start of the region to the end of its last accumulate, divided by their number.
    n_acc_region = n_acc_step * args.steps
    roofline = roof(per_acc, n_acc_region, acc_chain_secs * 1e3, "k_accumulate_f32",
                    "CUDA events on stream_acc around the timed region's accumulate launches (back to back on that stream, "
                    "median over the repetitions); the fused step of the previous iteration runs concurrently on "
                    "stream_sync and takes its share of the HBM bandwidth")
    roofline["concurrent_kernel"] = {"kernel": "k_sync<4>", "algorithmic_bytes_per_step": sync_b,
                                     "frac_of_both_kernels_together": value / world / peaks["hbm_gbs"]}
    # 16 accumulate launches, one after the other, fit into a step of the same pass
    assert n_acc_step * roofline["avg_us"] <= secs / args.steps * 1e6 * (1 + 1e-6), "per-kernel time does not reconcile with the step time"
    in_step_pairs = {
        "what": "the same pipelined region once more with an event pair around EVERY launch: the pairs keep consecutive "
                "kernels from being chained, so this pass is slower than the timed one and is no part of the headline",
        "ms_per_step": secs_p2 / args.steps * 1e3,
        "accumulate": roof(per_acc, n_acc, ms_acc, "k_accumulate_f32", "event pair per launch on stream_acc, fused step concurrent"),
        "sync": roof(sync_b, n_syn, ms_syn, "k_sync<4>", "event pair per launch on stream_sync, accumulate kernels concurrent")}
    isolated = {
        "accumulate": roof(per_acc, n_chain, ms_chain, "k_accumulate_f32",
                           "eager mode, 64 launches back to back with nothing else on the GPU, one event pair around all of them"),
        "accumulate_event_pair_per_launch": roof(per_acc, n_acc_e, ms_acc_e, "k_accumulate_f32",
                                                 "eager mode, kernel alone on the GPU, event pair around each launch"),
        "sync": roof(sync_b, n_syn_e, ms_syn_e, "k_sync<4>", "eager mode, kernel alone on the GPU, event pair around each launch"),
        "eager_ms_per_step": secs_eager / args.steps * 1e3,
        "eager_gbs": step_bytes * args.steps / secs_eager / 1e9}
    sync_alone = isolated["sync"]

    ms_step = worst / args.steps * 1e3
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "mode": "pipelined (two streams)", "l2": "inputs larger than L2: gradient pool "
                   "748 MB cycled, accumulators 374 MB", "parallelism": f"replicas x{world}", "bytes_per_step": step_bytes},
        "timing": {"repeats": repeats, "what": f"the {args.steps}-step region repeated {repeats} times (at least "
                   f"{args.min_seconds} s in all); ms_per_step and value are the median repetition",
                   "ms_per_step_min": secs_all[0] / args.steps * 1e3, "ms_per_step_max": secs_all[-1] / args.steps * 1e3,
                   "us_per_step_x_sm_mhz": (ms_step * 1e3 * clocks["sm_mhz"]) if clocks["sm_mhz"] else None},
        "frac_of_measured_hbm": value / world / peaks["hbm_gbs"],
        "frac_of_nominal_8TBs": value / world / HBM_NOMINAL_GBS,
        "sync_step_gbs": sync_alone["achieved"], "sync_step_us": sync_alone["avg_us"],
        "sync_step_frac_of_measured_hbm": sync_alone["frac"], "sync_step_frac_of_nominal_8TBs": sync_alone["frac_of_nominal_8TBs"],
        "sync_step_how": "the fused step alone on the GPU (eager mode), event pair around each launch, (8*4+16)*P bytes",
        "roofline": roofline, "in_step_event_pairs": in_step_pairs, "isolated": isolated,
        "batched_accumulate_variant": dict(batched, what="abs_accumulate_batch: the b_i gradients of a worker in one "
                                           "pass over its accumulator row, (4 b_i + 8) instead of 12 b_i bytes per "
                                           "parameter; bit-identical results"),
        "gpu_launches": launches, "clocks": clocks,
        "overwrite_first_variant": {
            "what": "ABS_FLAG_OVERWRITE_FIRST: no zero writes in the fused step, a worker's first micro-batch stores "
                    "instead of adds (bit-identical results)",
            "ms_per_step": secs_ow / args.steps * 1e3, "bytes_per_step": ow_bytes,
            "hbm_gbs_on_its_own_bytes": ow_bytes * args.steps / secs_ow / 1e9,
            "step_time_vs_default": secs_ow / secs},
    }

    sections = args.sections.split(",")
    if world > 1 and args.sections == DEFAULT_SECTIONS:
        sections = ["e2e", "cpu"]                      # the other GPUs of the job are held while rank 0 measures alone
    if rank == 0:
        if "e2e" in sections:
            line["e2e"] = run_e2e(B, wlm, wl, x0_d, pool, order, step_bytes, min(args.steps, 10))
        if "cpu" in sections:
            line["cpu_baseline"] = run_cpu_baseline(wlm, wl, x0, pool, order, step_bytes)
    if world > 1 or "global_step" in sections:
        # Step 1 across the GPUs of this job (every rank takes part; rank 0 reports).  Nothing here may cost the
        # line above: an exception is reported inside the object, and if the section has not ended by its deadline
        # (a rank that never arrived at a collective) every rank leaves -- rank 0 after printing the line without it.
        # At that point no kernel of this section can be in flight: the fused kernels are launched behind the
        # collective that every rank has to join.
        finished = threading.Event()

        def watchdog():
            if finished.wait(GLOBAL_STEP_DEADLINE_S):
                return
            if rank == 0:
                line["global_step"] = {"error": f"no result within {GLOBAL_STEP_DEADLINE_S} s; left out"}
                print(json.dumps(line), flush=True)
            os._exit(0)

        threading.Thread(target=watchdog, daemon=True).start()
        try:
            if world == 1:                             # asked for on one GPU: a process group of one rank
                import torch.distributed as tdist

                if not tdist.is_initialized():
                    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
                    os.environ.setdefault("MASTER_PORT", "29512")
                    os.environ.setdefault("NCCL_NVLS_ENABLE", "0")
                    tdist.init_process_group(backend="nccl", rank=0, world_size=1, device_id=dev)
            D.barrier(dev)
            line["global_step"] = run_global_step(B, D, wlm, wl, dev, rank, world, rows, min(args.steps, 50), peaks)
        except Exception as exc:                       # the replica figure above stands on its own
            line["global_step"] = {"error": f"{type(exc).__name__}: {exc}"}
        finished.set()
    if rank == 0:
        del pool_d
        torch.cuda.empty_cache()
        if "mlp" in sections:
            line["mlp"] = run_mlp(B, wlm, dev, peaks)
            # the section's headline rows once more, side by side (us per micro-batch of the whole pipelined run)
            line["mlp_us_per_microbatch"] = {k: round(v["us_per_microbatch"], 2) for k, v in line["mlp"].items()
                                             if isinstance(v, dict) and "us_per_microbatch" in v and not k.startswith("serial_")}
        if "tiny" in sections:
            line["tiny"] = run_tiny(B, wlm, dev)
        if "schedules" in sections:
            line["other_schedules"] = run_schedules(B, wlm, dev, peaks)
        if "workloads35" in sections:                 # opt-in: generating workload 5's gradient pool takes a while
            line["workloads_3_and_5"] = run_other_workloads(B, wlm, dev)
        if "sync_curve" in sections:
            line["sync_curve"] = run_sync_curve(B, dev, peaks)
        if "global" in sections:
            line["global_sync_emulated_ranks"] = run_global_sync(B, dev, peaks)
        if "batch_curve" in sections:
            line["accumulate_batch_curve"] = run_batch_curve(B, dev, peaks)
        print(json.dumps(line), flush=True)
    D.barrier(dev)
    D.shutdown()


def run_global_step(B, D, wlm, wl, dev, rank, world, rows, steps, peaks):
    """Step 1 across the job's GPUs (the paper's own setting: Algorithm 1, Step 1 between workers on different
    GPUs; dist.GlobalStep): the workload's W workers are spread over the G = world ranks (W / G local workers each when G
    divides W, else one worker per rank with the b_i pattern repeated); per iteration a rank accumulates its own
    workers' micro-batches and then takes part in the global step, whose kernel reads the peers' rows and writes the
    peers' parameters through NVLink peer mappings.  Reported per rank: time per iteration (max over ranks), time of
    the fused kernel alone (event pair on stream_sync), and its NVLink bytes in / out over that time against the
    measured 770 GB/s per direction."""
    import torch

    G = world
    Wl = wl.W // G if wl.W % G == 0 else 1
    base = wlm.schedule(wl)[0]
    b_all = [int(base[j % len(base)]) for j in range(G * Wl)]          # b_i of the global workers
    mine = [(i, b_all[rank * Wl + i]) for i in range(Wl)]
    x0_d = torch.from_numpy(wlm.params0(wl)).to(dev)
    eng = B.AbsSgd(x0_d, Wl, wl.lr, wl.momentum, wl.weight_decay, pipelined=True)
    step = D.GlobalStep(eng)
    c = [rank * 5]

    def one():
        for (i, k) in wlm.call_order([b for _, b in mine]):
            eng.accumulate(i, rows[c[0] % len(rows)]); c[0] += 1
        return step.sync_step(timed=True)

    for _ in range(3):
        one()
    eng.wait(); eng.synchronize()
    D.barrier(dev)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    pairs = []
    with torch.cuda.stream(eng.stream_acc):
        e0.record()
        for _ in range(steps):
            pairs.append(one())
        eng.wait()
        e1.record()
    torch.cuda.synchronize()
    D.barrier(dev)
    secs = D.reduce_max(e0.elapsed_time(e1) / 1e3, dev)
    k_us = D.reduce_max(float(np.median([a.elapsed_time(b) for a, b in pairs])) * 1e3, dev)
    eng.check()
    step.close()
    eng.destroy()
    P, R = wl.P, G * Wl
    first, count = B.global_partition(P, G, rank)
    nv_in = (G - 1) * Wl * 4 * count                   # the peers' rows of this rank's slice
    nv_out = (G - 1) * (Wl + 1) * 4 * count            # zeros over them, and x' to every peer
    hbm = (8 * R + 12 + 4 * G) * count                 # this GPU's kernel: local and remote bytes together
    acc_bytes = sum(b for _, b in mine) * 12 * P
    out = {"ranks": G, "workers_per_rank": Wl, "b_of_the_global_workers": b_all, "iterations": steps,
           "us_per_iteration_max_over_ranks": secs / steps * 1e6,
           "us_fused_kernel_max_over_ranks": k_us,
           "nvlink_bytes_in_per_rank": nv_in, "nvlink_bytes_out_per_rank": nv_out,
           "nvlink_gbs_in": nv_in / k_us / 1e3 if k_us > 0 else None, "nvlink_gbs_out": nv_out / k_us / 1e3 if k_us > 0 else None,
           "nvlink_frac_of_770_out": (nv_out / k_us / 1e3 / NVLINK_MEASURED_GBS) if k_us > 0 and G > 1 else None,
           "kernel_bytes_per_rank": hbm, "accumulate_bytes_per_rank_and_iteration": acc_bytes,
           "whole_job_gbs": D.reduce_sum(float(acc_bytes + hbm), dev) * steps / secs / 1e9}
    return out


def run_other_workloads(B, wlm, dev):
    """Whole iterations of workloads 3 (W = 8, idle workers) and 5 (W = 16, bf16 gradients) at full size,
    pipelined, with single and with batched accumulate calls: time per iteration and GB/s on the run's own
    algorithmic bytes ((g + 8) P per single call, (g n + 8) P per batch call, (8 W_act + 16) P per fused step)."""
    import numpy as np
    import torch

    out = {}
    for cfg, T in ((3, 60), (5, 20)):
        wl = wlm.config(cfg, T=T)
        x0 = wlm.params0(wl)
        pool = wlm.grad_pool(wl)
        src = torch.from_numpy(pool.view(np.int16) if pool.dtype == np.uint16 else pool)
        pool_d = torch.zeros((pool.shape[0], (pool.shape[1] + 7) // 8 * 8), dtype=src.dtype, device=dev)
        pool_d[:, :pool.shape[1]] = src.to(dev)
        rows = [pool_d[r].data_ptr() for r in range(wl.pool_size)]
        bf16 = wl.grad_dtype == "bf16"
        gb = 2 if bf16 else 4
        sched = wlm.schedule(wl)
        res = {"P": wl.P, "W": wl.W, "iterations": T, "grad_dtype": wl.grad_dtype}
        for name, batched in (("single_calls", False), ("batch_calls", True)):
            eng = B.AbsSgd(torch.from_numpy(x0).to(dev), wl.W, wl.lr, wl.momentum, wl.weight_decay,
                           grad_dtype=B.GRAD_BF16 if bf16 else B.GRAD_F32, pipelined=True)
            for rep_ in range(2):                      # the first round warms up
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                nbytes, prev_active = 0, 0
                with torch.cuda.stream(eng.stream_acc):
                    e0.record()
                    for t, calls in enumerate(wlm.iter_calls(wl)):
                        if batched:
                            per = {}
                            for (i, k, c) in calls:
                                per.setdefault(i, []).append(rows[c % wl.pool_size])
                            for i, gs in per.items():
                                for lo in range(0, len(gs), 8):
                                    eng.accumulate_batch(i, gs[lo:lo + 8])
                                    nbytes += (gb * len(gs[lo:lo + 8]) + 8) * wl.P
                        else:
                            for (i, k, c) in calls:
                                eng.accumulate(i, rows[c % wl.pool_size])
                                nbytes += (gb + 8) * wl.P
                        eng.sync_step()                # applies the previous iteration's set
                        if prev_active:
                            nbytes += (8 * prev_active + 16) * wl.P
                        prev_active = int((sched[t] > 0).sum())
                    eng.wait()
                    e1.record()
                torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            res[name] = {"us_per_iteration": ms / T * 1e3, "gbs_on_its_own_bytes": nbytes / ms / 1e6}
            eng.check(); eng.destroy()
        out[f"workload_{cfg}"] = res
        del pool_d
        torch.cuda.empty_cache()
    return out


def run_sync_curve(B, dev, peaks, P=25_557_032):
    """The fused step alone on the GPU (eager mode, an event pair around every launch -- the pairs keep the launch
    from being chained to the kernel ahead, so every figure includes the kernel's own ramp and tail) for several
    worker counts W, every worker active: GB/s on its algorithmic bytes (8 W + 16) P, at the size of workload 3's
    vector.  For W = 1 the accumulator written just before partly sits in the 126 MB L2: that point is optimistic."""
    import torch

    out = {"P": P, "unit": "GB/s on (8*W + 16) * P bytes", "peak": peaks["hbm_gbs"]}
    gen = torch.Generator(device=dev).manual_seed(2)
    g = torch.randn(P + 8, device=dev, generator=gen)
    for W in (1, 2, 4, 5, 6, 8, 12, 16, 17, 24, 32, 64):
        eng = B.AbsSgd(torch.zeros(P, device=dev), W, 0.1, 0.9, 5e-4)
        for rep_ in range(2):                          # the first round warms up
            eng.profile(True)
            with torch.cuda.stream(eng.stream_acc):
                for it in range(5):
                    for i in range(W):
                        eng.accumulate(i, g)
                    eng.sync_step()
            n, ms = eng.kernel_stats(B.K_SYNC)
            eng.profile(False)
        gbs = (8 * W + 16) * P / (ms / n) / 1e6
        out[str(W)] = {"us": ms / n * 1e3, "gbs": gbs, "frac_of_measured_hbm": gbs / peaks["hbm_gbs"]}
        eng.check(); eng.destroy()
    return out


def run_global_sync(B, dev, peaks):
    """Step 1 across GPUs (abs_global_*), G ranks emulated in one process on this one GPU (dist.LocalRanks).  The
    G fused kernels of an iteration run side by side (as they would on G GPUs) but here share one HBM, so the
    figure is all ranks' bytes over the time from the first kernel's start to the last one's end (an event pair
    on the control stream).  Bytes per parameter, R = G * W_local rows: read R rows + x + v, write R zero rows +
    v + x into G buffers = 8 R + 12 + 4 G.  Every one of them is local HBM traffic here; between real GPUs
    (G - 1) / G of the row and x traffic crosses NVLink instead, so this is the kernel's streaming rate on one
    GPU, not a multi-GPU measurement."""
    import torch

    from paper_2308_15164_b200 import dist as D

    out = {"unit": "GB/s on (8*R + 12 + 4*G) * P bytes per iteration, all ranks on one GPU", "peak": peaks["hbm_gbs"]}
    gen = torch.Generator(device=dev).manual_seed(3)
    for name, P, G, Wl in (("resnet18_4_ranks_x_1_worker", 11_689_512, 4, 1), ("resnet50_4_ranks_x_2_workers", 25_557_032, 4, 2),
                           ("resnet50_8_ranks_x_1_worker", 25_557_032, 8, 1)):
        g = torch.randn(P + 8, device=dev, generator=gen)
        x0 = torch.zeros(P, device=dev)
        ranks = [B.AbsSgd(x0, Wl, 0.1, 0.9, 5e-4, pipelined=True) for _ in range(G)]
        grp = D.LocalRanks(ranks)
        evs = []
        for it in range(13):
            for e in ranks:
                for i in range(Wl):
                    e.accumulate(i, g)
            ev = grp.sync_step(timed=True)
            if it >= 3:                                 # the first rounds warm up
                evs.append(ev)
        torch.cuda.synchronize()
        ms = sum(a.elapsed_time(b) for a, b in evs) / len(evs)
        R = G * Wl
        nbytes = (8 * R + 12 + 4 * G) * P
        out[name] = {"P": P, "ranks": G, "workers_per_rank": Wl, "us_all_ranks": ms * 1e3,
                     "gbs": nbytes / ms / 1e6, "frac_of_measured_hbm": nbytes / ms / 1e6 / peaks["hbm_gbs"]}
        for e in ranks:
            e.check(); e.destroy()
        del ranks, grp, g, x0
        torch.cuda.empty_cache()
    return out


def run_batch_curve(B, dev, peaks, P=40_000_000):
    """abs_accumulate_batch alone on the GPU (eager mode, an event pair around every launch) for n = 1..8
    gradients per call, fp32 and bf16: GB/s on the call's own algorithmic bytes, (g n + 8) P with g = 4 or 2."""
    import torch

    out = {"P": P, "unit": "GB/s on (g*n + 8) * P bytes", "peak": peaks["hbm_gbs"]}
    for dtype, gd, gb in (("f32", B.GRAD_F32, 4), ("bf16", B.GRAD_BF16, 2)):
        gen = torch.Generator(device=dev).manual_seed(1)
        pool = [torch.randn(P, device=dev, generator=gen).to(torch.float32 if gb == 4 else torch.bfloat16) for _ in range(12)]
        eng = B.AbsSgd(torch.zeros(P, device=dev), 4, 0.1, grad_dtype=gd)
        res = {}
        for n in range(1, 9):
            for rep_ in range(2):                      # the first round warms up
                eng.profile(True)
                with torch.cuda.stream(eng.stream_acc):
                    for it in range(24):
                        gs = [pool[(it * 5 + k) % 12] for k in range(n)]
                        if n == 1:
                            eng.accumulate(it % 4, gs[0])
                        else:
                            eng.accumulate_batch(it % 4, gs)
                cnt, ms = eng.kernel_stats(B.K_ACCUMULATE)
                eng.profile(False)
            res[str(n)] = {"us": ms / cnt * 1e3, "gbs": (gb * n + 8) * P / (ms / cnt) / 1e6}
        out[dtype] = res
        eng.check(); eng.destroy()
        del pool
        torch.cuda.empty_cache()
    return out


def run_tiny(B, wlm, dev, iters=2000):
    """Workload 1 (P = 4096, W = 2, b = (3, 1)) moves 131 KB per iteration: it is bound by launches, not bytes,
    so it is reported as microseconds per iteration (4 accumulate + 1 fused step): plain calls in eager and in
    pipelined mode, two iterations captured into a CUDA graph and replayed (eager mode enqueues on stream_acc
    only; the accumulator sets alternate with period 2), and the C oracle on the host."""
    import time

    import torch

    from oracle.c_oracle import AbsSgdOracleC

    wl = wlm.config(1)
    order = wlm.call_order(wlm.schedule(wl)[0])
    x0 = wlm.params0(wl)
    pool = [wlm.fresh_grad(wl, 0, 0, k) for k in range(8)]
    pool_d = [torch.from_numpy(g).to(dev) for g in pool]
    x0_d = torch.from_numpy(x0).to(dev)
    out = {"workload": "cfg1 tiny: P=4096, W=2, b=(3,1); 5 launches per iteration", "iterations": iters}

    def iterate(eng, n, c0=0, batched=False):
        c = c0
        for _ in range(n):
            if batched:                                   # one abs_accumulate_batch per worker: 3 launches per iteration
                per_worker = {}
                for (i, k) in order:
                    per_worker.setdefault(i, []).append(pool_d[c % 8]); c += 1
                for i, gs in per_worker.items():
                    eng.accumulate_batch(i, gs)
            else:
                for (i, k) in order:
                    eng.accumulate(i, pool_d[c % 8]); c += 1
            eng.sync_step()

    for name, pipelined in (("eager", False), ("pipelined", True)):
        eng = B.AbsSgd(x0_d, wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=pipelined)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(eng.stream_acc):
            iterate(eng, 20)
            eng.wait(); e0.record()
            iterate(eng, iters)
            eng.wait(); e1.record()
        torch.cuda.synchronize()
        out["us_per_iteration_" + name] = e0.elapsed_time(e1) / iters * 1e3
        eng.check(); eng.destroy()

    for name, batched in (("cuda_graph", False), ("cuda_graph_batched_accumulate", True)):
        eng = B.AbsSgd(x0_d, wl.W, wl.lr, wl.momentum, wl.weight_decay)
        with torch.cuda.stream(eng.stream_acc):
            iterate(eng, 2, batched=batched)
        eng.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=eng.stream_acc):
            iterate(eng, 2, batched=batched)              # recorded, not run: two iterations
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(eng.stream_acc):
            for _ in range(10):
                g.replay()
            e0.record()
            for _ in range(iters // 2):
                g.replay()
            e1.record()
        torch.cuda.synchronize()
        out["us_per_iteration_" + name] = e0.elapsed_time(e1) / (iters // 2 * 2) * 1e3
        eng.check(); eng.destroy()

    o = AbsSgdOracleC(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    c = 0
    t0 = time.perf_counter()
    for _ in range(iters):
        for (i, k) in order:
            o.accumulate(i, pool[c % 8]); c += 1
        o.sync_step()
    out["us_per_iteration_cpu_oracle"] = (time.perf_counter() - t0) / iters * 1e6
    return out


def mlp_run_bytes(sched, d, P, max_batch, overwrite_first, defer=None):
    """Algorithmic HBM bytes of an MLP run over the schedule `sched` [T, W] when every worker hands over its b_i
    micro-batches in calls of up to `max_batch`: per call the bf16 weights are streamed once (2 bytes per W1
    element) and the W1 slice of the accumulator is written (4 bytes per element: the worker's first call of the
    iteration stores) or read and written (8: later calls add); per micro-batch the bf16 operands of dW1; per
    iteration the fused step, (8 W_act + 16 + 2) bytes per parameter (the 2: the bf16 copy of the new weights;
    4 W_act + 18 when the step does not write zeros).
    defer = "rows" (ABS_FLAG_MLP_DEFER with the rows written): the slice is written once per active worker and
    iteration (4 bytes per element), never read by a gradient call, and the operands are written by the call and read
    by that one contraction.  defer = "pool" (Step 1 from the pooled operands): no accumulator traffic for W1 at all;
    the step moves 18 bytes per W1 element and the row-based amount on the rest of the vector.
    Returns (bytes, calls, stored calls, micro-batches)."""
    w1 = d.d_in * d.d_hidden
    total = calls = stored = mbs = 0
    prev_active = 0
    for b_row in sched:
        if prev_active:
            row_based = ((4 if overwrite_first else 8) * prev_active + 18)
            total += 18 * w1 + row_based * (P - w1) if defer == "pool" else row_based * P
        for b in b_row:
            left, first = int(b), True
            while left > 0:
                n = min(max_batch, left)
                if defer:
                    total += 2 * w1 + (4 * w1 if first and defer == "rows" else 0) + 2 * n * 2 * d.mb * (d.d_in + d.d_hidden)
                else:
                    total += 2 * w1 + (4 if first else 8) * w1 + n * 2 * d.mb * (d.d_in + d.d_hidden)
                calls += 1; stored += 1 if first else 0; mbs += n
                left -= n; first = False
        prev_active = int(sum(1 for b in b_row if b > 0))
    return total, calls, stored, mbs


def run_mlp(B, wlm, dev, peaks, iters=12):
    """The MLP workload (3072-4096-10, W=4, b_i ~ U{1..8}), pipelined: time per micro-batch of the whole run (all
    workers' gradient calls overlapping on their streams, the fused step included) with single calls, with single
    calls gathered by the library, and with batch calls of up to 4; each against the run's HBM floor (its
    algorithmic bytes, see mlp_run_bytes, over the measured copy bandwidth).  In serial mode (every kernel alone on
    the GPU, an event pair around each kernel group) also the per-kernel durations, with the dW1 = X^T dZ GEMM
    (M=3072, N=4096, K=64 n) as TFLOP/s and as GB/s on the bytes its launches moved (4 bytes per W1 element when
    the tile is stored, 8 when it is added to): at K = 64 n it is bound by that traffic, not by the tensor pipe."""
    import torch

    wl = wlm.config(4, T=iters)
    d = wl.mlp
    x0_d = torch.from_numpy(wlm.params0(wl)).to(dev)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).to(dev), torch.from_numpy(ys).to(dev)
    xp = [xs_d[b].data_ptr() for b in range(wl.mlp_pool)]      # raw device addresses of the micro-batches
    yp = [ys_d[b].data_ptr() for b in range(wl.mlp_pool)]
    torch.cuda.synchronize()
    calls = list(wlm.iter_calls(wl))
    sched = wlm.schedule(wl)
    w1 = d.d_in * d.d_hidden
    flop = 2.0 * w1 * d.mb
    out = {"workload": "cfg4 mlp 3072-4096-10, mb=64, W=4, b_i~U{1..8}, pipelined", "iterations": iters,
           "dw1_flop_per_microbatch": flop}

    def run_case(max_batch, variant=0, coalesce=False, overwrite_first=False, serial=0, defer=None):
        eng = B.AbsSgd(x0_d, wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=True, mlp=(d.d_in, d.d_hidden, d.d_out, d.mb),
                       mlp_coalesce=coalesce, overwrite_first=overwrite_first, mlp_defer=defer is not None)
        eng.set_launch(B.K_MLP_DW1, variant)
        eng.set_launch(B.K_MLP_FWD, serial)
        if defer == "rows":
            eng.set_launch(B.K_MLP_BWD, 1)

        def run(profile):
            eng.profile(profile)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n_mb = 0
            with torch.cuda.stream(eng.stream_acc):
                e0.record()
                if max_batch == 1:
                    for it in calls:                     # the workload's interleaved arrival order
                        for (i, k, c) in it:
                            eng.accumulate_mlp(i, xp[c % wl.mlp_pool], yp[c % wl.mlp_pool]); n_mb += 1
                        eng.sync_step()
                else:
                    for b_row in sched:
                        for i, b in enumerate(b_row):
                            left = int(b)
                            while left > 0:
                                n = min(max_batch, left)
                                p0 = (n_mb * 7) % (wl.mlp_pool - max_batch)
                                eng.accumulate_mlp_batch(i, n, xp[p0], yp[p0]); left -= n; n_mb += n
                        eng.sync_step()
                eng.wait()
                e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1), n_mb

        run(False)                                       # warm-up
        ms = min(run(False)[0] for _ in range(3))
        n_mb = run(False)[1]
        res = {"us_per_microbatch": ms / n_mb * 1e3, "microbatches": n_mb}
        if serial:
            run(True)
            st = {nm: eng.kernel_stats(k) for nm, k in (("fwd", B.K_MLP_FWD), ("bwd", B.K_MLP_BWD), ("dw1", B.K_MLP_DW1),
                                                        ("sync", B.K_SYNC))}
            _, n_calls, n_stored, _ = mlp_run_bytes(sched, d, wl.P, max_batch, overwrite_first)
            us = {nm: v[1] / max(v[0], 1) * 1e3 for nm, v in st.items()}
            us["fwd"] = st["fwd"][1] / n_calls * 1e3      # three timed kernels per call: cast, forward GEMM, bias / ReLU / logits
            dw1_bytes = ((4 * n_stored + 8 * (n_calls - n_stored)) * w1 + n_mb * 2 * d.mb * (d.d_in + d.d_hidden)) / n_calls
            res.update({"us_cast_fwd1_fwd2_per_call": us["fwd"], "us_bwd_per_call": us["bwd"], "us_dw1_per_call": us["dw1"],
                        "us_sync": us["sync"], "calls": n_calls, "calls_that_store": n_stored,
                        "dw1_tflops": flop * n_mb / n_calls / us["dw1"] / 1e6,
                        "dw1_frac_of_bf16_peak_sustained": flop * n_mb / n_calls / us["dw1"] / 1e6 / peaks["bf16_tflops_sustained"],
                        "dw1_bytes_per_call": dw1_bytes, "dw1_hbm_gbs": dw1_bytes / us["dw1"] / 1e3,
                        "dw1_frac_of_hbm": dw1_bytes / us["dw1"] / 1e3 / peaks["hbm_gbs"]})
        else:
            nbytes, n_calls, n_stored, _ = mlp_run_bytes(sched, d, wl.P, 4 if coalesce else max_batch, overwrite_first, defer)
            floor_us = nbytes / peaks["hbm_gbs"] / 1e3 / n_mb
            res.update({"algorithmic_bytes_per_microbatch": nbytes / n_mb, "hbm_floor_us_per_microbatch": floor_us,
                        "frac_of_hbm_floor": floor_us / res["us_per_microbatch"]})
        eng.check()
        eng.destroy()
        return res

    for name, kw in (("single_calls", dict(max_batch=1)),
                     ("single_calls_gathered_by_the_library", dict(max_batch=1, coalesce=True)),
                     ("batch_calls_up_to_4", dict(max_batch=4)),
                     ("batch_calls_up_to_4_overwrite_first", dict(max_batch=4, overwrite_first=True)),
                     ("batch_calls_up_to_4_deep_pipelines", dict(max_batch=4, variant=128)),
                     ("batch_calls_up_to_8", dict(max_batch=8)),
                     # ABS_FLAG_MLP_DEFER: Step 1 of the W1 slice straight from the pooled dW1 operands (one contraction
                     # over all micro-batches of the iteration inside the update kernel) ...
                     ("deferred_single_calls", dict(max_batch=1, defer="pool")),
                     ("deferred_single_calls_gathered_by_the_library", dict(max_batch=1, coalesce=True, defer="pool")),
                     ("deferred_batch_calls_up_to_4", dict(max_batch=4, defer="pool")),
                     ("deferred_batch_calls_up_to_8", dict(max_batch=8, defer="pool")),
                     # ... or one dW1 contraction per worker and iteration into the rows (K = 64 b_i), then the row-based step
                     ("deferred_rows_single_calls", dict(max_batch=1, defer="rows")),
                     ("deferred_rows_batch_calls_up_to_4", dict(max_batch=4, defer="rows"))):
        out[name] = run_case(**kw)
    # The deferred mode's step alone on the GPU (k_sync_small_pooled + k_sync_w1, the library's event pair around
    # them), 18 micro-batches pooled per iteration (the workload's mean): against the bytes it has to move --
    # 18 per W1 element (x, v in; x', v, bf16 x' out), the pooled operands once, the bias / W2 part.
    def pooled_step(n_mb=18, iters=8):
        eng = B.AbsSgd(x0_d, wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=True, mlp=(d.d_in, d.d_hidden, d.d_out, d.mb),
                       mlp_defer=True)

        def run(k):
            n = 0
            with torch.cuda.stream(eng.stream_acc):
                for _ in range(k):
                    for j in range(n_mb):
                        eng.accumulate_mlp(j % wl.W, xp[n % wl.mlp_pool], yp[n % wl.mlp_pool]); n += 1
                    eng.sync_step(); eng.wait()
                    eng.stream_acc.synchronize()
            torch.cuda.synchronize()

        run(2)
        eng.profile(True)
        run(iters)
        ns, ms = eng.kernel_stats(B.K_SYNC)
        eng.profile(False)
        eng.check(); eng.destroy()
        us = ms / ns * 1e3
        nbytes = 18 * w1 + n_mb * 2 * d.mb * (d.d_in + d.d_hidden) + (n_mb + 18) * (wl.P - w1)
        return {"microbatches_pooled": n_mb, "us": us, "algorithmic_bytes": nbytes, "gbs": nbytes / us / 1e3,
                "frac_of_measured_hbm": nbytes / us / 1e3 / peaks["hbm_gbs"],
                "contraction_tflops": 2.0 * w1 * d.mb * n_mb / us / 1e6}

    out["deferred_step_alone"] = pooled_step()
    for name, kw in (("single_calls", dict(max_batch=1)), ("single_calls_ring_dw1", dict(max_batch=1, variant=4)),
                     ("batch_calls_up_to_4", dict(max_batch=4)), ("batch_calls_up_to_4_tile_per_cta_dw1", dict(max_batch=4, variant=8))):
        out["serial_" + name] = run_case(serial=1, **kw)
    return out


def run_schedules(B, wlm, dev, peaks, steps=200):
    """Workload 2's vector with the paper's own static cluster (Section 6.1-6.2: iteration times in the ratio
    1 : 2 : 3 : 4, so the workers finish 12, 6, 4 and 3 reference batches in the same span) beside the benchmark's
    b = (2, 2, 4, 8): whole pipelined iterations, GB/s on each schedule's own algorithmic bytes."""
    import dataclasses

    import torch

    wl0 = wlm.config(2)
    x0_d = torch.from_numpy(wlm.params0(wl0)).to(dev)
    gen = torch.Generator(device=dev).manual_seed(7)
    pool_d = torch.randn((16, wl0.P), device=dev, generator=gen)
    rows = [pool_d[r].data_ptr() for r in range(16)]
    out = {}
    for name, b_row in (("b_2_2_4_8", (2, 2, 4, 8)), ("paper_static_cluster_b_12_6_4_3", (12, 6, 4, 3))):
        wl = dataclasses.replace(wl0, sched_arg=tuple(b_row))
        order = wlm.call_order(b_row)
        acc_b, sync_b = bytes_per_step(wl, b_row)
        eng = B.AbsSgd(x0_d, wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=True)
        c = 0
        for rep_ in range(2):                              # the first round warms up
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(eng.stream_acc):
                e0.record()
                for _ in range(steps):
                    for (i, k) in order:
                        eng.accumulate(i, rows[c % 16]); c += 1
                    eng.sync_step()
                eng.wait()
                e1.record()
            torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        out[name] = {"b": list(b_row), "us_per_iteration": ms * 1e3, "bytes_per_iteration": acc_b + sync_b,
                     "gbs": (acc_b + sync_b) / ms / 1e6, "frac_of_measured_hbm": (acc_b + sync_b) / ms / 1e6 / peaks["hbm_gbs"]}
        eng.check(); eng.destroy()
    return out


def run_e2e(B, wlm, wl, x0_d, pool, order, step_bytes, steps):
    """Same metric through the public API with HOST buffers: every step copies its 16 gradient
    micro-batches from pinned host memory and reads the published parameters back."""
    import torch

    pool_h = torch.from_numpy(pool).pin_memory()
    out_h = torch.empty(wl.P, dtype=torch.float32).pin_memory()
    eng = B.AbsSgd(x0_d, wl.W, wl.lr, wl.momentum, wl.weight_decay, pipelined=True, host_input=True)
    c = 0

    def one():
        nonlocal c
        for (i, k) in order:
            eng.accumulate_host(i, pool_h[c % wl.pool_size]); c += 1
        eng.sync_step()
        eng.params_host(out_h.numpy())

    for _ in range(2):
        one()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    eng.destroy()
    return {"value": step_bytes * steps / dt / 1e9, "unit": UNIT, "ms_per_step": dt / steps * 1e3, "steps": steps,
            "h2d_bytes_per_step": len(order) * wl.P * 4, "d2h_bytes_per_step": wl.P * 4,
            "note": "PCIe-bound: 16 gradient vectors in, parameters out, every step"}


def run_cpu_baseline(wlm, wl, x0, pool, order, step_bytes):
    from oracle.c_oracle import AbsSgdOracleC

    o = AbsSgdOracleC(x0, wl.W, wl.lr, wl.momentum, wl.weight_decay)
    c = 0

    def one():
        nonlocal c
        for (i, k) in order:
            o.accumulate(i, pool[c % wl.pool_size]); c += 1
        o.sync_step()

    one()
    t0 = time.perf_counter()
    n = 0
    while n < 600 and (time.perf_counter() - t0) < 12.0:       # about 12 s of wall time on the host cores
        one(); n += 1
    dt = time.perf_counter() - t0
    o.close()
    return {"value": step_bytes * n / dt / 1e9, "unit": UNIT, "cores": int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1)),
            "kind": "oracle", "ms_per_step": dt / n * 1e3,
            "sample": f"{n} full iterations of the same workload (C oracle, OpenMP, all host cores)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_SECONDS,
                    help="the --steps-long timed region is repeated until this much time has been measured (0: once)")
    ap.add_argument("--sections", default=DEFAULT_SECTIONS,
                    help="extra measurements after the timed region (drop them for a profiler's launch list)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
