"""Small, short runs of one kernel class, sized for a profiler capture.

    python -m paper_2308_15164_b200.profile_case sync       [--P 11689512] [--W 4] [--iters 3]
    python -m paper_2308_15164_b200.profile_case accumulate [--P 11689512] [--W 4] [--iters 3] [--bf16]
    python -m paper_2308_15164_b200.profile_case mlp        [--iters 2] [--batch 4] [--calls 2]
    python -m paper_2308_15164_b200.profile_case global     [--P 25557032] [--ranks 4] [--W 2] [--iters 2]
    python -m paper_2308_15164_b200.profile_case timeline   [--iters 3] [--batch 4] [--defer]   (no profiler: prints the library's
                                                            own timeline of the MLP workload's kernels)

Each case keeps its working set larger than the 126 MB L2 but to a few hundred MB, launches the
kernel of interest a handful of times and exits, so that a multi-pass capture ends by itself.
Every kernel launched here is the library's own (through the C ABI); nothing is timed.
"""

from __future__ import annotations

import argparse
import sys

import numpy as np
import torch


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["sync", "accumulate", "mlp", "global", "timeline"])
    ap.add_argument("--P", type=int, default=11_689_512)
    ap.add_argument("--W", type=int, default=4)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--bf16", action="store_true")
    ap.add_argument("--pipelined", action="store_true")
    ap.add_argument("--epilogue", type=int, default=0)
    ap.add_argument("--batch", type=int, default=1, help="mlp: reference batches per call (1..4)")
    ap.add_argument("--ranks", type=int, default=4, help="global: ranks emulated in this process (W = workers per rank)")
    ap.add_argument("--calls", type=int, default=1, help="mlp: calls per worker and iteration (the first one stores)")
    ap.add_argument("--defer", action="store_true", help="mlp, timeline: ABS_FLAG_MLP_DEFER (one dW1 contraction per worker and iteration)")
    args = ap.parse_args(argv)

    from . import binding as B
    from . import workloads as wlm

    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    if args.case == "timeline":
        return timeline(args, B, wlm, dev)
    if args.case == "global":
        from . import dist as D

        g = torch.Generator(device="cpu").manual_seed(0)
        x0 = (torch.randn(args.P, generator=g) * 0.02).to(dev)
        grad = torch.randn((args.P + 7) // 8 * 8, generator=g).to(dev)
        ranks = [B.AbsSgd(x0, args.W, 0.1, 0.9, 5e-4, pipelined=True) for _ in range(args.ranks)]
        grp = D.LocalRanks(ranks)
        for _ in range(args.iters):
            for e in ranks:
                for i in range(args.W):
                    e.accumulate(i, grad)
            grp.sync_step()
        for e in ranks:
            e.check()
            e.destroy()
    elif args.case in ("sync", "accumulate"):
        g = torch.Generator(device="cpu").manual_seed(0)
        x0 = (torch.randn(args.P, generator=g) * 0.02).to(dev)
        pool = torch.randn((4, (args.P + 7) // 8 * 8), generator=g)
        pool = (pool.to(torch.bfloat16) if args.bf16 else pool).to(dev)
        eng = B.AbsSgd(x0, args.W, 0.1, 0.9, 5e-4, grad_dtype=B.GRAD_BF16 if args.bf16 else B.GRAD_F32,
                       pipelined=args.pipelined)
        torch.cuda.synchronize()
        c = 0
        for _ in range(args.iters + 1):          # the first sync step has nothing to apply
            for i in range(args.W):
                eng.accumulate(i, pool[c % 4]); c += 1
            eng.sync_step()
        eng.check()
        eng.destroy()
    else:
        wl = wlm.config(4)
        d = wl.mlp
        x0 = torch.from_numpy(wlm.params0(wl)).to(dev)
        xs, ys = wlm.mlp_batches(wl)
        xs_d, ys_d = torch.from_numpy(xs[:8]).to(dev), torch.from_numpy(ys[:8]).to(dev)
        eng = B.AbsSgd(x0, wl.W, wl.lr, wl.momentum, pipelined=args.pipelined, mlp=(d.d_in, d.d_hidden, d.d_out, d.mb),
                       mlp_defer=args.defer)
        eng.set_launch(B.K_MLP_DW1, args.epilogue)
        torch.cuda.synchronize()
        c = 0
        for _ in range(args.iters + 1):
            for i in [w for _ in range(args.calls) for w in range(wl.W)]:
                if args.batch > 1:
                    lo = (c * args.batch) % 8 if 8 % args.batch == 0 else 0
                    eng.accumulate_mlp_batch(i, args.batch, xs_d[lo:lo + args.batch], ys_d[lo:lo + args.batch])
                else:
                    eng.accumulate_mlp(i, xs_d[c % 8], ys_d[c % 8])
                c += 1
            eng.sync_step()
        eng.check()
        eng.destroy()
    print("done", args.case)
    return 0


def timeline(args, B, wlm, dev):
    """Workload 4 (3072-4096-10, W = 4, b_i ~ U{1..8}), pipelined, with every worker's calls on its own streams:
    six warm-up iterations, then `--iters` iterations with abs_profile(ctx, 2); prints every timed kernel's span
    (start, stop, stream) and, per kernel, the mean duration while the workers' calls overlap."""
    wl = wlm.config(4, T=6 + args.iters)
    d = wl.mlp
    x0 = torch.from_numpy(wlm.params0(wl)).to(dev)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).to(dev), torch.from_numpy(ys).to(dev)
    sched = wlm.schedule(wl)
    eng = B.AbsSgd(x0, wl.W, wl.lr, wl.momentum, pipelined=True, mlp=(d.d_in, d.d_hidden, d.d_out, d.mb), mlp_defer=args.defer)
    torch.cuda.synchronize()
    n = 0

    def run(rows):
        nonlocal n
        with torch.cuda.stream(eng.stream_acc):
            for b_row in rows:
                if args.batch > 1:
                    for i, b in enumerate(b_row):
                        left = int(b)
                        while left > 0:
                            k = min(args.batch, left)
                            lo = (n * 7) % (wl.mlp_pool - args.batch)
                            eng.accumulate_mlp_batch(i, k, xs_d[lo:lo + k], ys_d[lo:lo + k]); left -= k; n += k
                else:
                    for (i, k) in wlm.call_order(b_row):
                        eng.accumulate_mlp(i, xs_d[n % wl.mlp_pool], ys_d[n % wl.mlp_pool]); n += 1
                eng.sync_step()
            eng.wait()
        torch.cuda.synchronize()

    run(sched[:6])
    eng.profile(2)
    run(sched[6:])
    spans = eng.profile_timeline()
    eng.profile(False)
    names = {("mlp_fwd", 0): "cast", ("mlp_fwd", 1): "forward GEMM", ("mlp_fwd", 2): "bias/ReLU/logits", ("mlp_bwd", 0): "backward",
             ("mlp_dw1", 0): "dW1", ("sync", 0): "fused step"}
    print(f"b of the timed iterations: {sched[6:].tolist()}; calls of up to {args.batch} micro-batches")
    stat = {}
    for (cls, part, stream, t0, t1) in sorted(spans, key=lambda r: r[3]):
        nm = names.get((cls, part), cls)
        print(f"  {t0:9.1f} .. {t1:9.1f} us  ({t1 - t0:6.1f})  stream {stream:2d}  {nm}")
        stat.setdefault(nm, []).append(t1 - t0)
    last = max(t1 for (_, _, _, _, t1) in spans)
    print(f"{len(spans)} spans over {last:.1f} us")
    for nm, v in stat.items():
        print(f"  {nm:18s} n = {len(v):3d}  mean {np.mean(v):6.1f} us  min {np.min(v):6.1f}  max {np.max(v):6.1f}")
    eng.check()
    eng.destroy()
    print("done timeline")
    return 0


if __name__ == "__main__":
    sys.exit(main())
