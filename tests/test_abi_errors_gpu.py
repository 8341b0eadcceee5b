"""GPU: argument errors on a live context are reported as status codes before anything is enqueued, and a
destroyed context is rejected."""

import ctypes

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_runtime_argument_errors_and_use_after_destroy():
    import torch

    from paper_2308_15164_b200 import binding as B

    P, W = 10_000, 3
    x0 = torch.zeros(P, device="cuda")
    eng = B.AbsSgd(x0, W, 0.1, 0.9)
    g = torch.ones(P + 8, device="cuda")
    h = eng._h
    n0 = eng.launch_count()
    assert B.lib.abs_accumulate(h, W, g.data_ptr()) == B.EINVAL                 # worker out of range
    assert B.lib.abs_accumulate(h, 0, None) == B.EINVAL                         # null gradient
    assert B.lib.abs_accumulate(h, 0, g.data_ptr() + 4) == B.EINVAL             # misaligned gradient
    assert B.lib.abs_accumulate_mlp(h, 0, g.data_ptr(), g.data_ptr()) == B.EINVAL   # not an MLP context
    assert B.lib.abs_accumulate_host(h, 0, g.data_ptr()) == B.EINVAL            # no host-input staging reserved
    assert B.lib.abs_params(h, None) == B.EINVAL
    assert B.lib.abs_consumed(h, 0, None) == B.EINVAL
    b = np.zeros(W, dtype=np.int32)
    assert B.lib.abs_consumed(h, 5, b.ctypes.data) == B.EINVAL                  # step not reached yet
    assert B.lib.abs_set_lr(h, float("inf")) == B.EINVAL
    assert B.lib.abs_set_launch(h, 99, 1) == B.EINVAL
    assert B.lib.abs_last_error(h) != b""
    assert eng.launch_count() == n0                                             # nothing was launched
    eng.accumulate(1, g)                                                        # the context is still usable
    eng.sync_step(); eng.sync_step()
    assert np.allclose(eng.params_host(), -0.1)
    assert eng.consumed(1).tolist() == [0, 1, 0]
    eng.check()
    raw = ctypes.c_void_p(h.value)
    eng.destroy()
    assert B.lib.abs_sync_step(raw) == B.ESTATE                                 # use after destroy
    assert B.lib.abs_accumulate(raw, 0, g.data_ptr()) == B.ESTATE
    assert B.lib.abs_destroy(raw) == B.ESTATE


def test_workspace_too_small_and_inconsistent_mlp_shape_rejected():
    import torch

    from paper_2308_15164_b200 import binding as B

    cfg = B.make_config(P=4096, W=2, lr=0.1)
    need = B.abs_workspace_bytes(cfg)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    x0 = torch.zeros(4096, device="cuda")
    h = ctypes.c_void_p()
    assert B.lib.abs_init(ctypes.byref(h), ctypes.byref(cfg), ws.data_ptr(), need - 1, x0.data_ptr()) == B.ENOMEM
    assert not h.value
    bad = B.make_config(P=128 * 128 + 128 + 1280 + 10 + 1, W=2, lr=0.1, flags=B.FLAG_MLP, mlp=(128, 128, 10, 64))
    assert B.abs_workspace_bytes(bad) == 0                     # P does not match the MLP shape


def test_a_wait_that_runs_out_is_reported_and_leaves_the_context_usable():
    """The bounded device-side wait: a barrier that nothing completes makes the polling loop give up; the host
    reads ABS_ETIMEOUT from abs_check once, and the same context then runs a normal step with correct results."""
    import numpy as np
    import torch

    from paper_2308_15164_b200 import binding as B

    dev = torch.device("cuda:0")
    P = 5000
    x0 = torch.ones(P, device=dev)
    g = torch.full((P + 8,), 2.0, device=dev)
    eng = B.AbsSgd(x0, 5, 0.1, pipelined=True)
    eng.set_launch(B.K_SYNC, -2)                         # the fused step as the bulk-copy pipeline
    eng.check()
    eng.selftest_timeout()
    with pytest.raises(B.AbsError) as e:
        eng.check()
    assert e.value.code == B.ETIMEOUT
    eng.check()                                          # reported once
    for i in range(5):
        eng.accumulate(i, g)
    eng.sync_step(); eng.sync_step()
    eng.check()
    got = eng.params_host()
    assert np.allclose(got, 1.0 - 0.1 * 2.0, rtol=0, atol=1e-6)
    eng.destroy()


def test_mlp_batch_call_argument_checks():
    """abs_accumulate_mlp_batch takes 1..8 micro-batches, aligned non-null device pointers and a worker in range;
    a rejected call launches nothing and counts nothing."""
    import torch

    from paper_2308_15164_b200 import binding as B
    from paper_2308_15164_b200 import workloads as wlm

    wl = wlm.config(4, small=True)
    d = wl.mlp
    x0 = torch.from_numpy(wlm.params0(wl)).cuda()
    x = torch.zeros((9, d.mb, d.d_in), device="cuda")
    y = torch.zeros((9, d.mb), dtype=torch.int32, device="cuda")
    for defer in (False, True):
        eng = B.AbsSgd(x0, wl.W, wl.lr, mlp=(d.d_in, d.d_hidden, d.d_out, d.mb), mlp_defer=defer)
        h = eng._h
        n0 = eng.launch_count()
        assert B.lib.abs_accumulate_mlp_batch(h, 0, 0, x.data_ptr(), y.data_ptr()) == B.EINVAL
        assert B.lib.abs_accumulate_mlp_batch(h, 0, 9, x.data_ptr(), y.data_ptr()) == B.EINVAL
        assert B.lib.abs_accumulate_mlp_batch(h, wl.W, 1, x.data_ptr(), y.data_ptr()) == B.EINVAL
        assert B.lib.abs_accumulate_mlp_batch(h, 0, 1, None, y.data_ptr()) == B.EINVAL
        assert B.lib.abs_accumulate_mlp_batch(h, 0, 1, x.data_ptr() + 4, y.data_ptr()) == B.EINVAL
        assert B.lib.abs_accumulate_mlp_batch(h, 0, 1, x.data_ptr(), None) == B.EINVAL
        assert eng.launch_count() == n0 and not eng.counters()[0].any()
        assert B.lib.abs_accumulate_mlp_batch(h, 0, 8, x.data_ptr(), y.data_ptr()) == B.OK
        assert eng.counters()[0][eng.counters()[1]].tolist() == [8, 0, 0, 0]
        eng.check()
        eng.destroy()
