"""ctypes binding of the C ABI declared in include/abs_sgd.h.

Argument marshalling only: every step of the delayed synchronous step runs in the CUDA
kernels of libabs_sgd.so.  PyTorch is used for device memory and stream handles.  There is
no CPU fallback: if the shared library is missing this module raises at import.
"""

from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libabs_sgd.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} not found: build it with `python -m paper_2308_15164_b200.build` "
        "(nvcc, sm_100a).  There is no CPU fallback.")

lib = ctypes.CDLL(LIB_PATH)

OK, EINVAL, ESTATE, ECUDA, ENOMEM, ETIMEOUT, ELIMIT = 0, -1, -2, -3, -4, -5, -6
GRAD_F32, GRAD_BF16 = 0, 1
FLAG_PIPELINED, FLAG_MLP, FLAG_HOST_INPUT, FLAG_OVERWRITE_FIRST, FLAG_MLP_COALESCE, FLAG_GRAD_NORM, FLAG_MLP_X_BF16, FLAG_MLP_DEFER = 1, 2, 4, 8, 16, 32, 64, 128
K_ACCUMULATE, K_SYNC, K_MLP_FWD, K_MLP_BWD, K_MLP_DW1, K_CHAIN = range(6)
MAX_WORKERS, MAX_RANKS, IPC_HANDLE_BYTES = 64, 16, 64
KERNEL_NAMES = ["accumulate", "sync", "mlp_fwd", "mlp_bwd", "mlp_dw1"]


class AbsConfig(ctypes.Structure):
    _fields_ = [
        ("P", ctypes.c_uint64), ("W", ctypes.c_uint32),
        ("lr", ctypes.c_float), ("momentum", ctypes.c_float), ("weight_decay", ctypes.c_float),
        ("lambda_dc", ctypes.c_float),
        ("grad_dtype", ctypes.c_uint32), ("flags", ctypes.c_uint32),
        ("mlp_in", ctypes.c_uint32), ("mlp_hidden", ctypes.c_uint32), ("mlp_out", ctypes.c_uint32),
        ("mlp_mb", ctypes.c_uint32),
        ("stream_acc", ctypes.c_void_p), ("stream_sync", ctypes.c_void_p),
    ]


class AbsSpan(ctypes.Structure):
    _fields_ = [("kernel_class", ctypes.c_int32), ("stream", ctypes.c_int32), ("part", ctypes.c_int32),
                ("start_us", ctypes.c_float), ("stop_us", ctypes.c_float)]


class AbsPeerTable(ctypes.Structure):
    _fields_ = [("n_ranks", ctypes.c_uint32), ("rank", ctypes.c_uint32), ("workspace_dev", ctypes.c_void_p * MAX_RANKS)]


_vp, _u32, _u64 = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64
_sig = {
    "abs_workspace_bytes": (ctypes.c_size_t, [ctypes.POINTER(AbsConfig)]),
    "abs_init": (ctypes.c_int, [ctypes.POINTER(_vp), ctypes.POINTER(AbsConfig), _vp, ctypes.c_size_t, _vp]),
    "abs_accumulate": (ctypes.c_int, [_vp, _u32, _vp]),
    "abs_accumulate_batch": (ctypes.c_int, [_vp, _u32, _u32, ctypes.POINTER(ctypes.c_void_p)]),
    "abs_accumulate_host": (ctypes.c_int, [_vp, _u32, _vp]),
    "abs_accumulate_mlp": (ctypes.c_int, [_vp, _u32, _vp, _vp]),
    "abs_accumulate_mlp_batch": (ctypes.c_int, [_vp, _u32, _u32, _vp, _vp]),
    "abs_accumulate_mlp_list": (ctypes.c_int, [_vp, _u32, _u32, ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_void_p)]),
    "abs_sync_step": (ctypes.c_int, [_vp]),
    "abs_params": (ctypes.c_int, [_vp, ctypes.POINTER(_vp)]),
    "abs_params_host": (ctypes.c_int, [_vp, _vp]),
    "abs_momentum": (ctypes.c_int, [_vp, ctypes.POINTER(_vp)]),
    "abs_accumulator": (ctypes.c_int, [_vp, _u32, _u32, ctypes.POINTER(_vp)]),
    "abs_counters": (ctypes.c_int, [_vp, _vp, ctypes.POINTER(_u32), ctypes.POINTER(_u64)]),
    "abs_consumed": (ctypes.c_int, [_vp, _u64, _vp]),
    "abs_grad_norm2": (ctypes.c_int, [_vp, _u64, ctypes.POINTER(ctypes.c_double)]),
    "abs_set_lr": (ctypes.c_int, [_vp, ctypes.c_float]),
    "abs_step1_finished": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_int)]),
    "abs_wait": (ctypes.c_int, [_vp]),
    "abs_check": (ctypes.c_int, [_vp]),
    "abs_selftest_timeout": (ctypes.c_int, [_vp]),
    "abs_set_launch": (ctypes.c_int, [_vp, ctypes.c_int, ctypes.c_int]),
    "abs_profile": (ctypes.c_int, [_vp, ctypes.c_int]),
    "abs_kernel_stats": (ctypes.c_int, [_vp, ctypes.c_int, ctypes.POINTER(_u64), ctypes.POINTER(ctypes.c_double)]),
    "abs_profile_timeline": (ctypes.c_int, [_vp, ctypes.POINTER(AbsSpan), ctypes.c_size_t, ctypes.POINTER(ctypes.c_size_t)]),
    "abs_launch_count": (ctypes.c_uint64, [_vp]),
    "abs_last_error": (ctypes.c_char_p, [_vp]),
    "abs_destroy": (ctypes.c_int, [_vp]),
    "abs_global_attach": (ctypes.c_int, [_vp, ctypes.POINTER(AbsPeerTable)]),
    "abs_global_begin": (ctypes.c_int, [_vp, ctypes.POINTER(_vp), ctypes.POINTER(_u32)]),
    "abs_global_step": (ctypes.c_int, [_vp]),
    "abs_global_end": (ctypes.c_int, [_vp]),
    "abs_global_slice": (ctypes.c_int, [_vp, ctypes.POINTER(_u64), ctypes.POINTER(_u64)]),
    "abs_global_consumed": (ctypes.c_int, [_vp, _u64, _vp]),
    "abs_global_partition": (ctypes.c_int, [_u64, _u32, _u32, ctypes.POINTER(_u64), ctypes.POINTER(_u64)]),
    "abs_ipc_export": (ctypes.c_int, [_vp, _vp, ctypes.POINTER(_u64)]),
    "abs_ipc_open": (ctypes.c_int, [_vp, _u64, ctypes.POINTER(_vp)]),
    "abs_ipc_close": (ctypes.c_int, [_vp, _u64]),
    "abs_state_bytes": (ctypes.c_size_t, [_vp]),
    "abs_state_export": (ctypes.c_int, [_vp, _vp, ctypes.c_size_t]),
    "abs_state_import": (ctypes.c_int, [_vp, _vp, ctypes.c_size_t]),
    "abs_sync_step_noalloc": (ctypes.c_int, [_vp, _vp, _vp, _u64, _u64, _u32, _vp, ctypes.c_float, ctypes.c_float,
                                             ctypes.c_float, _vp]),
}
for _name, (_res, _args) in _sig.items():
    _fn = getattr(lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args


class AbsError(RuntimeError):
    def __init__(self, code, text):
        super().__init__(f"abs_sgd status {code}: {text}")
        self.code = code


def _ptr(t) -> int:
    """Raw address of a torch tensor / numpy array / int."""
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return int(t) if t is not None else 0


def make_config(P, W, lr, momentum=0.0, weight_decay=0.0, lambda_dc=0.0, grad_dtype=GRAD_F32, flags=0,
                mlp=None, stream_acc=0, stream_sync=0) -> AbsConfig:
    c = AbsConfig()
    c.P, c.W = int(P), int(W)
    c.lr, c.momentum, c.weight_decay, c.lambda_dc = lr, momentum, weight_decay, lambda_dc
    c.grad_dtype, c.flags = grad_dtype, flags
    if mlp is not None:
        c.mlp_in, c.mlp_hidden, c.mlp_out, c.mlp_mb = mlp
    c.stream_acc, c.stream_sync = stream_acc or None, stream_sync or None
    return c


def abs_workspace_bytes(cfg: AbsConfig) -> int:
    return int(lib.abs_workspace_bytes(ctypes.byref(cfg)))


class AbsSgd:
    """Thin object wrapper: one method per C entry point, same names without the ``abs_`` prefix."""

    def __init__(self, params0: torch.Tensor, W: int, lr: float, momentum=0.0, weight_decay=0.0, lambda_dc=0.0,
                 grad_dtype=GRAD_F32, pipelined=False, mlp=None, host_input=False, overwrite_first=False,
                 mlp_coalesce=False, grad_norm=False, mlp_x_bf16=False, mlp_defer=False, stream_acc: Optional[torch.cuda.Stream] = None, stream_sync: Optional[torch.cuda.Stream] = None,
                 workspace: Optional[torch.Tensor] = None):
        assert params0.is_cuda and params0.dtype == torch.float32 and params0.is_contiguous()
        self.device = params0.device
        self.P, self.W = params0.numel(), W
        # An MLP context's own stream_acc is a high-priority stream: the operand cast of a gradient call runs there and
        # would otherwise queue behind the thousands of CTAs of earlier calls' dW1 GEMMs.  (Streaming contexts keep
        # the default priority: their accumulate kernels must not starve the fused step on stream_sync.)
        self.stream_acc = stream_acc or torch.cuda.Stream(device=self.device, priority=-1 if mlp else 0)
        self.stream_sync = stream_sync or (torch.cuda.Stream(device=self.device) if pipelined else None)
        flags = (FLAG_PIPELINED if pipelined else 0) | (FLAG_MLP if mlp else 0) | (FLAG_HOST_INPUT if host_input else 0) | (FLAG_OVERWRITE_FIRST if overwrite_first else 0) | (FLAG_MLP_COALESCE if mlp_coalesce else 0) | (FLAG_GRAD_NORM if grad_norm else 0) | (FLAG_MLP_X_BF16 if mlp_x_bf16 else 0) | (FLAG_MLP_DEFER if mlp_defer else 0)
        self.cfg = make_config(self.P, W, lr, momentum, weight_decay, lambda_dc, grad_dtype, flags, mlp,
                               self.stream_acc.cuda_stream, self.stream_sync.cuda_stream if self.stream_sync else 0)
        nbytes = abs_workspace_bytes(self.cfg)
        if nbytes == 0:
            raise AbsError(EINVAL, "invalid configuration")
        if workspace is None:
            workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        assert workspace.dtype == torch.uint8 and workspace.is_cuda and workspace.numel() >= nbytes
        self.workspace = workspace            # caller-provided memory is used as it is (abs_init checks the alignment)
        self._h = _vp()
        # params0 may have been produced on another stream: make it visible to stream_acc.
        self.stream_acc.wait_stream(torch.cuda.current_stream(self.device))
        with torch.cuda.device(self.device):
            rc = lib.abs_init(ctypes.byref(self._h), ctypes.byref(self.cfg), self.workspace.data_ptr(), nbytes,
                              params0.data_ptr())
        if rc != OK:
            raise AbsError(rc, lib.abs_last_error(None).decode())
        self._keep = params0

    def _ck(self, rc):
        if rc != OK:
            raise AbsError(rc, lib.abs_last_error(self._h).decode())

    def accumulate(self, worker: int, grad):
        self._ck(lib.abs_accumulate(self._h, worker, _ptr(grad)))

    def accumulate_batch(self, worker: int, grads):
        """grads: sequence of 1..8 device tensors (or raw device addresses), added in this order."""
        arr = (ctypes.c_void_p * len(grads))(*[_ptr(g) for g in grads])
        self._ck(lib.abs_accumulate_batch(self._h, worker, len(grads), arr))

    def accumulate_host(self, worker: int, grad_host):
        self._ck(lib.abs_accumulate_host(self._h, worker, _ptr(grad_host)))

    def accumulate_mlp(self, worker: int, x, y):
        self._ck(lib.abs_accumulate_mlp(self._h, worker, _ptr(x), _ptr(y)))

    def accumulate_mlp_batch(self, worker: int, n: int, x, y):
        self._ck(lib.abs_accumulate_mlp_batch(self._h, worker, n, _ptr(x), _ptr(y)))

    def accumulate_mlp_list(self, worker: int, xs, ys):
        """n separate micro-batches (tensors or raw device addresses) in one call."""
        n = len(xs)
        assert n == len(ys)
        xa = (ctypes.c_void_p * n)(*[_ptr(x) for x in xs])
        ya = (ctypes.c_void_p * n)(*[_ptr(y) for y in ys])
        self._ck(lib.abs_accumulate_mlp_list(self._h, worker, n, xa, ya))

    def sync_step(self):
        self._ck(lib.abs_sync_step(self._h))

    def params(self) -> torch.Tensor:
        """The published parameters as a tensor aliasing library memory (valid until the next sync_step)."""
        p = _vp()
        self._ck(lib.abs_params(self._h, ctypes.byref(p)))
        return _alias(p.value, self.P, torch.float32, self.device)

    def params_host(self, out: Optional[np.ndarray] = None) -> np.ndarray:
        if out is None:
            out = np.empty(self.P, dtype=np.float32)
        self._ck(lib.abs_params_host(self._h, _ptr(out)))
        return out

    def momentum(self) -> torch.Tensor:
        p = _vp()
        self._ck(lib.abs_momentum(self._h, ctypes.byref(p)))
        return _alias(p.value, self.P, torch.float32, self.device)

    def accumulator(self, set_index: int, worker: int) -> torch.Tensor:
        p = _vp()
        self._ck(lib.abs_accumulator(self._h, set_index, worker, ctypes.byref(p)))
        return _alias(p.value, self.P, torch.float32, self.device)

    def counters(self):
        cnt = np.zeros((2, self.W), dtype=np.int32)
        cur, t = _u32(0), _u64(0)
        self._ck(lib.abs_counters(self._h, cnt.ctypes.data, ctypes.byref(cur), ctypes.byref(t)))
        return cnt, int(cur.value), int(t.value)

    def consumed(self, step: int) -> np.ndarray:
        b = np.zeros(self.W, dtype=np.int32)
        self._ck(lib.abs_consumed(self._h, step, b.ctypes.data))
        return b

    # ---- Step 1 across GPUs (one context per rank) ----
    def global_attach(self, rank: int, workspaces):
        """workspaces: device address of every rank's workspace as mapped in this process (own one at [rank])."""
        tab = AbsPeerTable()
        tab.n_ranks, tab.rank = len(workspaces), rank
        for q, w in enumerate(workspaces):
            tab.workspace_dev[q] = _ptr(w)
        self._ck(lib.abs_global_attach(self._h, ctypes.byref(tab)))
        self.n_ranks = len(workspaces)

    def global_begin(self) -> torch.Tensor:
        """Returns the int32 exchange vector (aliasing library memory) that the caller sums over all ranks."""
        p, n = _vp(), _u32(0)
        self._ck(lib.abs_global_begin(self._h, ctypes.byref(p), ctypes.byref(n)))
        return _alias(p.value, int(n.value), torch.int32, self.device)

    def global_step(self):
        self._ck(lib.abs_global_step(self._h))

    def global_end(self):
        self._ck(lib.abs_global_end(self._h))

    def global_slice(self):
        first, count = _u64(0), _u64(0)
        self._ck(lib.abs_global_slice(self._h, ctypes.byref(first), ctypes.byref(count)))
        return int(first.value), int(count.value)

    def global_consumed(self, step: int) -> np.ndarray:
        b = np.zeros(self.n_ranks * self.W, dtype=np.int32)
        self._ck(lib.abs_global_consumed(self._h, step, b.ctypes.data))
        return b

    # ---- checkpoint / resume ----
    def state_export(self) -> np.ndarray:
        buf = np.empty(int(lib.abs_state_bytes(self._h)), dtype=np.uint8)
        self._ck(lib.abs_state_export(self._h, buf.ctypes.data, buf.nbytes))
        return buf

    def state_import(self, buf: np.ndarray):
        buf = np.ascontiguousarray(buf, dtype=np.uint8)
        self._ck(lib.abs_state_import(self._h, buf.ctypes.data, buf.nbytes))

    def grad_norm2(self, step: int) -> float:
        out = ctypes.c_double(0.0)
        self._ck(lib.abs_grad_norm2(self._h, step, ctypes.byref(out)))
        return float(out.value)

    def step1_finished(self) -> bool:
        done = ctypes.c_int(1)
        self._ck(lib.abs_step1_finished(self._h, ctypes.byref(done)))
        return bool(done.value)

    def set_lr(self, lr: float):
        self._ck(lib.abs_set_lr(self._h, lr))

    def wait(self):
        self._ck(lib.abs_wait(self._h))

    def check(self):
        self._ck(lib.abs_check(self._h))

    def selftest_timeout(self):
        self._ck(lib.abs_selftest_timeout(self._h))

    def set_launch(self, kernel_class: int, ctas_per_sm: int):
        self._ck(lib.abs_set_launch(self._h, kernel_class, ctas_per_sm))

    def profile(self, enable):
        """False / True: per-kernel totals; 2: the timeline of the timed launches as well (profile_timeline)."""
        self._ck(lib.abs_profile(self._h, int(enable)))

    def profile_timeline(self):
        """[(kernel class name, part, stream, start_us, stop_us), ...] of the launches timed since profile(2)."""
        n = ctypes.c_size_t(0)
        self._ck(lib.abs_profile_timeline(self._h, None, 0, ctypes.byref(n)))
        buf = (AbsSpan * max(n.value, 1))()
        self._ck(lib.abs_profile_timeline(self._h, buf, n.value, ctypes.byref(n)))
        return [(KERNEL_NAMES[b.kernel_class], b.part, b.stream, b.start_us, b.stop_us) for b in buf[:n.value]]

    def kernel_stats(self, kernel_class: int):
        n, ms = _u64(0), ctypes.c_double(0.0)
        self._ck(lib.abs_kernel_stats(self._h, kernel_class, ctypes.byref(n), ctypes.byref(ms)))
        return int(n.value), float(ms.value)

    def launch_count(self) -> int:
        return int(lib.abs_launch_count(self._h))

    def synchronize(self):
        self.stream_acc.synchronize()
        if self.stream_sync is not None:
            self.stream_sync.synchronize()

    def destroy(self):
        if self._h:
            lib.abs_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def sync_step_noalloc(x: torch.Tensor, v: torch.Tensor, acc: torch.Tensor, cnt: torch.Tensor, lr: float,
                      momentum: float = 0.0, weight_decay: float = 0.0, stream: Optional[torch.cuda.Stream] = None) -> int:
    """abs_sync_step_noalloc on caller-owned tensors: x, v fp32 [P]; acc fp32 [W, row_stride]; cnt int32 [W].
    Returns the status code (no exception), so callers can test for ELIMIT / EINVAL."""
    s = stream.cuda_stream if stream is not None else torch.cuda.current_stream(x.device).cuda_stream
    with torch.cuda.device(x.device):             # the entry point works on the current device
        return int(lib.abs_sync_step_noalloc(x.data_ptr(), v.data_ptr(), acc.data_ptr(), acc.stride(0), x.numel(),
                                             acc.shape[0], cnt.data_ptr(), lr, momentum, weight_decay, s))


def global_partition(P: int, n_ranks: int, rank: int) -> tuple:
    """(first, count): the slice of the flat vector that `rank` of `n_ranks` reduces in multi-GPU mode."""
    first, count = _u64(0), _u64(0)
    rc = lib.abs_global_partition(P, n_ranks, rank, ctypes.byref(first), ctypes.byref(count))
    if rc != OK:
        raise AbsError(rc, "abs_global_partition: bad arguments")
    return int(first.value), int(count.value)


def ipc_export(dev_ptr) -> tuple:
    """(handle bytes, offset) naming the device allocation that holds ``dev_ptr``, for abs_ipc_open in another process."""
    buf = ctypes.create_string_buffer(IPC_HANDLE_BYTES)
    off = _u64(0)
    rc = lib.abs_ipc_export(_ptr(dev_ptr), buf, ctypes.byref(off))
    if rc != OK:
        raise AbsError(rc, "abs_ipc_export failed (memory not from cudaMalloc?)")
    return bytes(buf.raw), int(off.value)


def ipc_open(handle: bytes, offset: int) -> int:
    p = _vp()
    rc = lib.abs_ipc_open(ctypes.c_char_p(handle), offset, ctypes.byref(p))
    if rc != OK:
        raise AbsError(rc, "abs_ipc_open failed")
    return int(p.value)


def ipc_close(dev_ptr: int, offset: int):
    lib.abs_ipc_close(dev_ptr, offset)


def _alias(addr: int, n: int, dtype, device) -> torch.Tensor:
    """A tensor viewing ``n`` elements of library-owned device memory at ``addr`` (no copy)."""
    itemsize = torch.empty(0, dtype=dtype).element_size()

    class _Mem:
        __cuda_array_interface__ = {
            "shape": (n,), "typestr": {torch.float32: "<f4", torch.int32: "<i4"}.get(dtype, "<u2"), "data": (addr, False),
            "version": 2,
        }

    return torch.as_tensor(_Mem(), device=device)
