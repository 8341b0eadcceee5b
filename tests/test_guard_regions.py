"""No kernel writes outside the workspace it was given: the workspace sits between two 64 KiB guard regions
filled with a pattern, the library is driven through its streaming, MLP and multi-GPU paths (sizes with ragged
tails), and the guards are compared afterwards.  (compute-sanitizer is not available to these tests; this is
the out-of-bounds check they can make.)"""

import numpy as np
import pytest

from paper_2308_15164_b200 import workloads as wlm

pytestmark = pytest.mark.gpu

GUARD = 64 * 1024


class Guarded:
    def __init__(self, nbytes, dev):
        import torch

        self.n = (nbytes + 255) // 256 * 256
        self.buf = torch.full((GUARD + self.n + GUARD,), 0xA5, dtype=torch.uint8, device=dev)
        assert self.buf.data_ptr() % 256 == 0
        self.workspace = self.buf[GUARD:GUARD + self.n]

    def intact(self):
        lo, hi = self.buf[:GUARD], self.buf[GUARD + self.n:]
        return bool((lo == 0xA5).all().item()) and bool((hi == 0xA5).all().item())


def _make(x0_d, W, wl, dev, **kw):
    from paper_2308_15164_b200 import binding as B

    flags = (B.FLAG_PIPELINED if kw.get("pipelined") else 0) | (B.FLAG_MLP if kw.get("mlp") else 0) | \
            (B.FLAG_OVERWRITE_FIRST if kw.get("overwrite_first") else 0) | (B.FLAG_MLP_COALESCE if kw.get("mlp_coalesce") else 0) | \
            (B.FLAG_MLP_DEFER if kw.get("mlp_defer") else 0)
    gd = kw.get("grad_dtype", B.GRAD_F32)
    cfg = B.make_config(x0_d.numel(), W, wl.lr, wl.momentum, wl.weight_decay, 0.0, gd, flags, kw.get("mlp"), 1, 2 if kw.get("pipelined") else 0)
    g = Guarded(B.abs_workspace_bytes(cfg), dev)
    eng = B.AbsSgd(x0_d, W, wl.lr, wl.momentum, wl.weight_decay, workspace=g.workspace, **kw)
    return eng, g


@pytest.mark.parametrize("P", [1, 1023, 4097, 65537, 670_504])
@pytest.mark.parametrize("pipelined", [False, True], ids=["eager", "pipelined"])
def test_streaming_path_stays_inside_its_workspace(P, pipelined):
    import torch

    from paper_2308_15164_b200 import binding as B

    dev = torch.device("cuda:0")
    wl = wlm.config(2, small=True, T=3)
    gen = torch.Generator(device=dev).manual_seed(P)
    for dtype, gd in ((torch.float32, B.GRAD_F32), (torch.bfloat16, B.GRAD_BF16)):
        x0 = torch.randn(P, device=dev, generator=gen)
        grads = [torch.randn((P + 7) // 8 * 8, device=dev, generator=gen).to(dtype) for _ in range(3)]
        for W in (1, 4, 9):
            eng, g = _make(x0, W, wl, dev, pipelined=pipelined, grad_dtype=gd)
            for t in range(3):
                for i in range(W):
                    eng.accumulate(i, grads[(t + i) % 3])
                    if i % 2:
                        eng.accumulate_batch(i, [grads[0], grads[1], grads[2]])
                eng.sync_step()
            eng.check()
            eng.synchronize()
            assert g.intact(), (P, W, dtype)
            eng.destroy()


def test_mlp_and_multi_gpu_paths_stay_inside_their_workspaces():
    import torch

    from paper_2308_15164_b200 import dist as D

    dev = torch.device("cuda:0")
    wl = wlm.config(4, small=True, T=3)
    d = wl.mlp
    mlp = (d.d_in, d.d_hidden, d.d_out, d.mb)
    x0 = torch.from_numpy(wlm.params0(wl)).to(dev)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).to(dev), torch.from_numpy(ys).to(dev)
    torch.cuda.synchronize()
    pairs = [_make(x0, 2, wl, dev, pipelined=True, mlp=mlp, mlp_coalesce=(r == 0)) for r in range(2)]
    ranks = [p[0] for p in pairs]
    grp = D.LocalRanks(ranks)
    for t in range(3):
        for r, e in enumerate(ranks):
            for i in range(2):
                for k in range(3):
                    e.accumulate_mlp(i, xs_d[(t + i + k) % 8], ys_d[(t + i + k) % 8])
                e.accumulate_mlp_batch(i, 3, xs_d[8:11], ys_d[8:11])
        grp.sync_step()
    for e, g in pairs:
        e.check()
        e.synchronize()
        assert g.intact()
    blob = ranks[0].state_export()
    ranks[0].state_import(blob)
    assert pairs[0][1].intact()
    for e in ranks:
        e.destroy()


@pytest.mark.parametrize("pipelined", [False, True], ids=["eager", "pipelined"])
def test_deferred_mlp_mode_stays_inside_its_workspace(pipelined):
    """ABS_FLAG_MLP_DEFER: the operand pools are the last regions of the workspace, right in front of the upper guard.
    Single, gathered and batch calls (up to eight micro-batches), a pool that overflows, the step from the pooled
    operands and the one from the rows, a read of the rows and an export."""
    import torch

    from paper_2308_15164_b200 import binding as B

    dev = torch.device("cuda:0")
    wl = wlm.config(4, small=True, T=3)
    d = wl.mlp
    mlp = (d.d_in, d.d_hidden, d.d_out, d.mb)
    x0 = torch.from_numpy(wlm.params0(wl)).to(dev)
    xs, ys = wlm.mlp_batches(wl)
    xs_d, ys_d = torch.from_numpy(xs).to(dev), torch.from_numpy(ys).to(dev)
    torch.cuda.synchronize()
    for coalesce in (False, True):
        eng, g = _make(x0, 2, wl, dev, pipelined=pipelined, mlp=mlp, mlp_defer=True, mlp_coalesce=coalesce)
        for t in range(4):
            if t == 2:
                eng.set_launch(B.K_MLP_BWD, 1)       # rows first from here on
            for i in range(2):
                for k in range(3):
                    eng.accumulate_mlp(i, xs_d[(t + i + k) % 8], ys_d[(t + i + k) % 8])
                eng.accumulate_mlp_batch(i, 8, xs_d[8:16], ys_d[8:16])
                eng.accumulate_mlp_batch(i, 5, xs_d[3:8], ys_d[3:8])
            if t == 1:                               # 32 slots: this iteration overflows the pool
                for k in range(6):
                    eng.accumulate_mlp(k % 2, xs_d[k], ys_d[k])
                eng.accumulator(eng.counters()[1], 0)
            eng.sync_step()
        eng.check()
        eng.synchronize()
        assert g.intact(), coalesce
        blob = eng.state_export()
        eng.state_import(blob)
        assert g.intact()
        eng.destroy()
