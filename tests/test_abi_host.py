"""CPU-only checks of the C-ABI library: it loads without a GPU, exports every symbol the public
header declares, and rejects bad arguments before touching the device."""

import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2308_15164_b200 import build

    build.build()
    from paper_2308_15164_b200 import binding

    return binding


def _declared_functions():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names.update(re.findall(r"\b(abs_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(B):
    names = _declared_functions()
    assert {"abs_init", "abs_accumulate", "abs_accumulate_mlp", "abs_sync_step", "abs_params"} <= set(names)
    for n in names:
        assert hasattr(B.lib, n), f"{n} declared in include/ but not exported"
        assert n in B._sig, f"{n} has no binding signature"


def test_workspace_bytes_host_side(B):
    cfg = B.make_config(P=4096, W=2, lr=0.1, stream_acc=1)
    n = B.abs_workspace_bytes(cfg)
    # x, v, acc[2][W][P] at least
    assert n >= 4096 * 4 * (2 + 2 * 2)
    cfgp = B.make_config(P=4096, W=2, lr=0.1, flags=B.FLAG_PIPELINED, stream_acc=1, stream_sync=2)
    assert B.abs_workspace_bytes(cfgp) >= n + 4096 * 4
    big = B.make_config(P=124_439_808, W=16, lr=3e-4, grad_dtype=B.GRAD_BF16, flags=B.FLAG_PIPELINED, stream_acc=1, stream_sync=2)
    nb = B.abs_workspace_bytes(big)
    assert 124_439_808 * 4 * 35 <= nb < 124_439_808 * 4 * 35 + (1 << 22)


@pytest.mark.parametrize("kw", [
    dict(P=0, W=2), dict(P=16, W=0), dict(P=16, W=65), dict(P=16, W=2, grad_dtype=7), dict(P=16, W=2, flags=256),
    dict(P=16, W=2, flags=128), dict(P=16, W=2, flags=64), dict(P=16, W=2, flags=16),
    dict(P=16, W=2, lr=float("nan")), dict(P=16, W=2, flags=1, stream_acc=5, stream_sync=5),
    dict(P=16, W=2, flags=2, mlp=(100, 128, 10, 64)), dict(P=16, W=2, flags=2, mlp=(128, 128, 10, 64)),
    dict(P=128 * 128 + 128 + 1280 + 10, W=2, flags=2, mlp=(128, 128, 10, 32)),
    dict(P=128 * 128 + 128 + 128 * 17 + 17, W=2, flags=2, mlp=(128, 128, 17, 64)),
])
def test_invalid_configs_are_rejected(B, kw):
    kw.setdefault("lr", 0.1)
    cfg = B.make_config(**kw)
    assert B.abs_workspace_bytes(cfg) == 0
    h = ctypes.c_void_p()
    rc = B.lib.abs_init(ctypes.byref(h), ctypes.byref(cfg), 256, 1 << 30, 256)
    assert rc == B.EINVAL and not h.value
    assert B.lib.abs_last_error(None) != b""


def test_init_pointer_checks_happen_before_any_device_work(B):
    cfg = B.make_config(P=4096, W=2, lr=0.1)
    h = ctypes.c_void_p()
    need = B.abs_workspace_bytes(cfg)
    assert B.lib.abs_init(None, ctypes.byref(cfg), 256, need, 256) == B.EINVAL
    assert B.lib.abs_init(ctypes.byref(h), None, 256, need, 256) == B.EINVAL
    assert B.lib.abs_init(ctypes.byref(h), ctypes.byref(cfg), None, need, 256) == B.EINVAL
    assert B.lib.abs_init(ctypes.byref(h), ctypes.byref(cfg), 257, need, 256) == B.EINVAL      # misaligned
    assert B.lib.abs_init(ctypes.byref(h), ctypes.byref(cfg), 256, need, None) == B.EINVAL
    assert B.lib.abs_init(ctypes.byref(h), ctypes.byref(cfg), 256, need, 260) == B.EINVAL      # misaligned
    assert B.lib.abs_init(ctypes.byref(h), ctypes.byref(cfg), 256, need - 1, 256) == B.ENOMEM


def test_dead_context_is_rejected(B):
    for name in ("abs_sync_step", "abs_wait", "abs_destroy"):
        assert getattr(B.lib, name)(None) == B.ESTATE
    assert B.lib.abs_accumulate(None, 0, 256) == B.ESTATE
    assert B.lib.abs_accumulate_mlp(None, 0, 256, 256) == B.ESTATE
    bogus = ctypes.create_string_buffer(4096)        # not a context the library created
    assert B.lib.abs_sync_step(ctypes.addressof(bogus)) == B.ESTATE
    assert B.lib.abs_launch_count(None) == 0


@pytest.mark.parametrize("P", [1, 1023, 1024, 1025, 4096, 11_689_512, 25_557_032, 124_439_808])
@pytest.mark.parametrize("G", [1, 2, 3, 4, 7, 8, 16])
def test_multi_gpu_partition_covers_the_vector_once(B, P, G):
    """Slices of ranks 0..G-1 are consecutive, disjoint, cover [0, P), start on 1024-element boundaries
    (whole 256-vector tiles) and differ in length by at most one tile, except that trailing ranks take
    what is left."""
    at = 0
    sizes = []
    for r in range(G):
        first, count = B.global_partition(P, G, r)
        assert first == min(at, P) and first % 1024 == 0 or count == 0
        at = first + count
        sizes.append(count)
    assert at == P and sum(sizes) == P
    full = [s for s in sizes if s and s % 1024 == 0]
    assert len(set(full)) <= 1 or max(full) == sizes[0]
    assert sizes == sorted(sizes, reverse=True)


def test_multi_gpu_entry_points_reject_bad_arguments_on_the_host(B):
    assert B.lib.abs_global_partition(0, 2, 0, None, None) == B.EINVAL
    assert B.lib.abs_global_partition(16, 0, 0, None, None) == B.EINVAL
    assert B.lib.abs_global_partition(16, 17, 0, None, None) == B.EINVAL
    assert B.lib.abs_global_partition(16, 2, 2, None, None) == B.EINVAL
    for name in ("abs_global_step", "abs_global_end"):
        assert getattr(B.lib, name)(None) == B.ESTATE
    assert B.lib.abs_global_attach(None, None) == B.ESTATE
    assert B.lib.abs_global_begin(None, None, None) == B.ESTATE
    assert B.lib.abs_ipc_export(None, None, None) == B.EINVAL
    assert B.lib.abs_ipc_open(None, 0, None) == B.EINVAL
    assert B.lib.abs_ipc_close(None, 0) == B.EINVAL


def test_workspace_of_the_deferred_mlp_mode_grows_by_its_operand_pools(B):
    """ABS_FLAG_MLP_DEFER adds one operand pool per accumulator set: max(32, 16 W) slots, at most 128, of
    (3 d_in + 2 d_hidden) * 128 bytes of bf16 operands, the labels and the micro-batch's db1 | dW2 | db2."""
    d_in, d_h, d_out = 256, 384, 10
    P = d_in * d_h + d_h + d_h * d_out + d_out

    def extra(W):
        kw = dict(P=P, W=W, lr=0.1, mlp=(d_in, d_h, d_out, 64))
        plain = B.abs_workspace_bytes(B.make_config(flags=B.FLAG_MLP, **kw))
        defer = B.abs_workspace_bytes(B.make_config(flags=B.FLAG_MLP | B.FLAG_MLP_DEFER, **kw))
        assert plain > 0 and defer > plain
        return defer - plain

    def up(v, a):
        return (v + a - 1) // a * a

    def pools(cap):
        part = up(d_h + d_h * d_out + d_out, 32) * 4
        one = 2 * up(cap * d_in * 64 * 2, 1024) + up(cap * d_h * 64 * 2, 1024) + up(cap * 64 * 4, 1024) + up(cap * part, 1024)
        return 2 * up(one, 4096)

    assert extra(1) == pools(32)
    assert extra(4) == pools(64)
    assert extra(8) == pools(128)
    assert extra(40) == pools(128)                   # capped
