"""Seeded synthetic workloads for the delayed synchronous step.

This module only *generates inputs* (initial parameters, per-iteration micro-batch
counts b_i, the order in which workers' micro-batches arrive, gradient vectors and MLP
micro-batches).  It holds none of the optimiser's arithmetic, so both the CPU oracle's
tests and the CUDA path's tests/benchmark may draw their inputs from it.

The five workloads follow the shapes of the paper's experiments (Section 6: ResNet18,
4 workers, static / dynamic heterogeneity) and of larger flat models:

  1  tiny      P=4096,        W=2,  b=(3,1) fixed,          fresh N(0,1) gradients
  2  resnet18  P=11,689,512,  W=4,  b=(2,2,4,8) fixed,      per-tensor N(0, var 1/fan_in)
  3  resnet50  P=25,557,032,  W=8,  b~round(LogNormal),     N(0, std 0.1)
  4  mlp       3072-4096-10,  W=4,  b~U{1..8},              gradients computed from (x, y)
  5  gpt2s     P=124,439,808, W=16, b~U{1..12},             bf16 N(0, std 0.02)

Workloads 2, 3 and 5 draw their micro-batch gradients from a seeded *pool* of R vectors
(larger than the GPU's L2); the micro-batch with global call index c uses pool[c mod R].
Every random draw comes from a Philox generator keyed by (seed, stream id), so any piece
can be regenerated independently.
"""

from __future__ import annotations

import dataclasses
import math
from typing import Iterator, List, Optional, Sequence, Tuple

import numpy as np

# --------------------------------------------------------------------------- rng ---------

_KIND_PARAMS, _KIND_GRAD, _KIND_SCHED, _KIND_X, _KIND_Y, _KIND_POOL = range(6)


def _rng(seed: int, kind: int, a: int = 0, b: int = 0, c: int = 0) -> np.random.Generator:
    """Philox generator for stream (seed; kind, a, b, c)."""
    stream = (kind & 0xFF) << 56 | (a & 0xFFFFFF) << 32 | (b & 0xFFFF) << 16 | (c & 0xFFFF)
    return np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, stream]))


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (nearest, ties to even) and return the 16-bit patterns.

    Used only to *prepare inputs* that are specified as bf16 tensors.
    """
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to the fp32 values they denote (exact)."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------- layouts -----

def resnet18_tensors(num_classes: int = 1000) -> List[Tuple[str, Tuple[int, ...]]]:
    """The 62 parameter tensors of ResNet18 in network order (conv, bn weight, bn bias, fc)."""
    out: List[Tuple[str, Tuple[int, ...]]] = []

    def conv(name, co, ci, k):
        out.append((name, (co, ci, k, k)))

    def bn(name, c):
        out.append((name + ".weight", (c,)))
        out.append((name + ".bias", (c,)))

    conv("conv1", 64, 3, 7)
    bn("bn1", 64)
    widths = [64, 128, 256, 512]
    cin = 64
    for s, w in enumerate(widths):
        for blk in range(2):
            pre = f"layer{s + 1}.{blk}"
            conv(pre + ".conv1", w, cin if blk == 0 else w, 3)
            bn(pre + ".bn1", w)
            conv(pre + ".conv2", w, w, 3)
            bn(pre + ".bn2", w)
            if blk == 0 and s > 0:
                conv(pre + ".downsample.0", w, cin, 1)
                bn(pre + ".downsample.1", w)
        cin = w
    out.append(("fc.weight", (num_classes, 512)))
    out.append(("fc.bias", (num_classes,)))
    return out


def _fan_in(shape: Tuple[int, ...]) -> int:
    if len(shape) == 1:
        return shape[0]
    return int(np.prod(shape[1:]))


@dataclasses.dataclass(frozen=True)
class MlpDims:
    d_in: int
    d_hidden: int
    d_out: int
    mb: int  # samples per micro-batch (the paper's reference batch size M_r)

    @property
    def P(self) -> int:
        return self.d_in * self.d_hidden + self.d_hidden + self.d_hidden * self.d_out + self.d_out

    @property
    def offsets(self) -> Tuple[int, int, int, int]:
        """Flat offsets of W1 [d_in, d_hidden], b1, W2 [d_hidden, d_out], b2 (all row-major)."""
        o_w1 = 0
        o_b1 = o_w1 + self.d_in * self.d_hidden
        o_w2 = o_b1 + self.d_hidden
        o_b2 = o_w2 + self.d_hidden * self.d_out
        return o_w1, o_b1, o_w2, o_b2


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    cfg: int
    seed: int
    P: int
    W: int
    T: int
    lr: float
    momentum: float
    weight_decay: float
    grad_dtype: str = "f32"          # "f32" or "bf16": element type handed to abs_accumulate
    pool_size: int = 0               # 0: a fresh gradient vector per micro-batch
    init_std: float = 0.0
    grad_std: float = 0.0
    tensors: Optional[Tuple[Tuple[str, Tuple[int, ...]], ...]] = None
    mlp: Optional[MlpDims] = None
    sched: str = "fixed"             # fixed | lognormal | uniform
    sched_arg: Tuple[int, ...] = ()
    mlp_pool: int = 64

    @property
    def mean_calls_per_iter(self) -> float:
        return float(schedule(self).sum(axis=1).mean())


# --------------------------------------------------------------------------- configs -----

def config(n: int, small: bool = False, T: Optional[int] = None) -> Workload:
    """Workload ``n`` (1..5).  ``small=True`` gives the same recipe at a size a CPU finishes
    in seconds (several tiles and a ragged tail); ``T`` overrides the iteration count."""
    if n == 1:
        wl = Workload("tiny", 1, 0, 4096, 2, 5, 0.1, 0.9, 0.0, init_std=0.01, grad_std=1.0,
                      sched="fixed", sched_arg=(3, 1))
    elif n == 2:
        tens = resnet18_tensors()
        if small:  # stem + first stage + classifier: same tensor kinds, 670,504 params
            tens = [t for t in tens if t[0].startswith(("conv1", "bn1", "layer1", "fc"))]
        P = sum(int(np.prod(s)) for _, s in tens)
        wl = Workload("resnet18" + ("-small" if small else ""), 2, 2, P, 4, 100, 0.1, 0.9, 5e-4,
                      pool_size=16, tensors=tuple(tens), sched="fixed", sched_arg=(2, 2, 4, 8))
    elif n == 3:
        P = 1_000_003 if small else 25_557_032
        wl = Workload("resnet50" + ("-small" if small else ""), 3, 3, P, 8, 200, 0.05, 0.9, 1e-4,
                      pool_size=8, init_std=0.02, grad_std=0.1, sched="lognormal", sched_arg=(0, 16))
    elif n == 4:
        dims = MlpDims(384, 512, 10, 64) if small else MlpDims(3072, 4096, 10, 64)
        wl = Workload("mlp" + ("-small" if small else ""), 4, 4, dims.P, 4, 50, 0.05, 0.9, 0.0,
                      mlp=dims, sched="uniform", sched_arg=(1, 8))
    elif n == 5:
        P = 2_000_005 if small else 124_439_808
        wl = Workload("gpt2s" + ("-small" if small else ""), 5, 5, P, 16, 20, 3e-4, 0.9, 0.01,
                      grad_dtype="bf16", pool_size=8, init_std=0.02, grad_std=0.02,
                      sched="uniform", sched_arg=(1, 12))
    else:
        raise ValueError(f"no workload {n}")
    if T is not None:
        wl = dataclasses.replace(wl, T=T)
    return wl


# --------------------------------------------------------------------------- inputs ------

def params0(wl: Workload) -> np.ndarray:
    """Initial parameters x_0, fp32 vector of length P."""
    if wl.tensors is not None:
        # conv / fc weights: Kaiming normal, std = sqrt(2 / fan_in); bn weight 1; biases 0.
        rng = _rng(wl.seed, _KIND_PARAMS)
        parts = []
        for name, shape in wl.tensors:
            n = int(np.prod(shape))
            if len(shape) >= 2:
                parts.append(rng.standard_normal(n, dtype=np.float32)
                             * np.float32(math.sqrt(2.0 / _fan_in(shape))))
            elif "bn" in name or "downsample" in name:
                parts.append(np.full(n, 1.0 if name.endswith("weight") else 0.0, dtype=np.float32))
            else:
                parts.append(np.zeros(n, dtype=np.float32))
        return np.concatenate(parts)
    if wl.mlp is not None:
        d = wl.mlp
        rng = _rng(wl.seed, _KIND_PARAMS)
        x = np.zeros(d.P, dtype=np.float32)
        o_w1, o_b1, o_w2, o_b2 = d.offsets
        x[o_w1:o_b1] = rng.standard_normal(d.d_in * d.d_hidden, dtype=np.float32) * np.float32(
            math.sqrt(2.0 / d.d_in))
        x[o_w2:o_b2] = rng.standard_normal(d.d_hidden * d.d_out, dtype=np.float32) * np.float32(
            math.sqrt(2.0 / d.d_hidden))
        return x
    rng = _rng(wl.seed, _KIND_PARAMS)
    return rng.standard_normal(wl.P, dtype=np.float32) * np.float32(wl.init_std)


def grad_scale(wl: Workload) -> np.ndarray:
    """Per-element standard deviation of the synthetic gradients (fp32, length P)."""
    if wl.tensors is not None:
        parts = [np.full(int(np.prod(s)), _fan_in(s) ** -0.5, dtype=np.float32) for _, s in wl.tensors]
        return np.concatenate(parts)
    return np.full(wl.P, wl.grad_std, dtype=np.float32)


def schedule(wl: Workload) -> np.ndarray:
    """Micro-batch counts b_i^t, int32 array [T, W].

    fixed:      the same tuple every iteration (static heterogeneity).
    lognormal:  clip(rint(LogNormal(ln 4, 0.6)), lo, hi) i.i.d. per (t, i) (dynamic
                heterogeneity); additionally, every 10th iteration (t % 10 == 7) worker
                (t // 10) % W is forced to 0 so that idle workers are exercised.
    uniform:    integers uniform on [lo, hi] inclusive.
    """
    if wl.sched == "fixed":
        row = np.asarray(wl.sched_arg, dtype=np.int32)
        assert row.shape == (wl.W,)
        return np.tile(row, (wl.T, 1))
    rng = _rng(wl.seed, _KIND_SCHED)
    lo, hi = wl.sched_arg
    if wl.sched == "lognormal":
        draw = rng.lognormal(mean=math.log(4.0), sigma=0.6, size=(wl.T, wl.W))
        b = np.clip(np.rint(draw), lo, hi).astype(np.int32)
        for t in range(7, wl.T, 10):
            b[t, (t // 10) % wl.W] = 0
        return b
    if wl.sched == "uniform":
        return rng.integers(lo, hi + 1, size=(wl.T, wl.W)).astype(np.int32)
    raise ValueError(wl.sched)


def call_order(b_row: Sequence[int]) -> List[Tuple[int, int]]:
    """Arrival order of one iteration's micro-batches as (worker, k) pairs.

    Workers run concurrently; worker i finishes its k-th micro-batch (k = 0..b_i-1) at
    virtual time (k+1)/b_i of the iteration.  Calls are ordered by that time, ties by
    worker index, which interleaves fast and slow workers the way a real cluster would.
    """
    ev = []
    for i, b in enumerate(b_row):
        for k in range(int(b)):
            ev.append(((k + 1) / float(b), i, k))
    ev.sort()
    return [(i, k) for _, i, k in ev]


def iter_calls(wl: Workload) -> Iterator[List[Tuple[int, int, int]]]:
    """For each iteration t yield the list of (worker, k, c) in arrival order, where c is
    the global call index (counts every micro-batch of the run from 0)."""
    c = 0
    for b_row in schedule(wl):
        calls = []
        for (i, k) in call_order(b_row):
            calls.append((i, k, c))
            c += 1
        yield calls


def fresh_grad(wl: Workload, t: int, i: int, k: int) -> np.ndarray:
    """Gradient of micro-batch (t, i, k) for pool-less workloads: fp32 N(0, grad_std)."""
    rng = _rng(wl.seed, _KIND_GRAD, t, i, k)
    return rng.standard_normal(wl.P, dtype=np.float32) * np.float32(wl.grad_std)


def grad_pool(wl: Workload, columns: Optional[np.ndarray] = None) -> np.ndarray:
    """Gradient pool [R, P]: fp32 values, or bf16 bit patterns (uint16) when grad_dtype is bf16.

    ``columns`` (sorted indices) restricts the result to those parameter positions while
    drawing the same numbers as the full pool.
    """
    assert wl.pool_size > 0
    scale = grad_scale(wl)
    rows = []
    for r in range(wl.pool_size):
        rng = _rng(wl.seed, _KIND_POOL, r)
        g = rng.standard_normal(wl.P, dtype=np.float32) * scale
        if wl.grad_dtype == "bf16":
            g = f32_to_bf16_bits(g)
        rows.append(g if columns is None else g[columns])
    return np.stack(rows)


def grad_for_call(wl: Workload, pool: Optional[np.ndarray], t: int, i: int, k: int, c: int) -> np.ndarray:
    """The gradient vector the micro-batch with global call index c carries."""
    if wl.pool_size:
        return pool[c % wl.pool_size]
    return fresh_grad(wl, t, i, k)


def mlp_batches(wl: Workload) -> Tuple[np.ndarray, np.ndarray]:
    """Pool of MLP micro-batches: x fp32 [R, mb, d_in] ~ N(0,1), y int32 [R, mb] uniform classes."""
    d = wl.mlp
    assert d is not None
    rx = _rng(wl.seed, _KIND_X)
    ry = _rng(wl.seed, _KIND_Y)
    x = rx.standard_normal((wl.mlp_pool, d.mb, d.d_in), dtype=np.float32)
    y = ry.integers(0, d.d_out, size=(wl.mlp_pool, d.mb)).astype(np.int32)
    return x, y


def sample_columns(P: int, n_random: int = 100_000, window: int = 4096, seed: int = 1234) -> np.ndarray:
    """Sorted parameter indices used to check a full-size run element by element on a sample:
    windows at the start, around every quarter point and at the very end, plus random picks."""
    idx = [np.arange(0, min(window, P))]
    for q in (1, 2, 3):
        c = (P * q) // 4
        idx.append(np.arange(max(0, c - window // 2), min(P, c + window // 2)))
    idx.append(np.arange(max(0, P - window), P))
    rng = _rng(seed, _KIND_GRAD, 999)
    idx.append(rng.integers(0, P, size=min(n_random, P)))
    return np.unique(np.concatenate(idx))
