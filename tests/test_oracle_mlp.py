"""CPU-only pins for the MLP part of the oracle (the gradient of one reference batch, Step 2 of
Algorithm 1, for the 2-layer ReLU network with mean softmax cross-entropy)."""

import numpy as np
import pytest

from oracle.abs_oracle import bf16_round, mlp_loss_and_grad, mlp_split


def _problem(rng, d_in, d_h, d_out, mb, scale=1.0):
    P = d_in * d_h + d_h + d_h * d_out + d_out
    p = (rng.standard_normal(P) * scale).astype(np.float32)
    X = rng.standard_normal((mb, d_in)).astype(np.float32)
    y = rng.integers(0, d_out, size=mb)
    return p, X, y


def _loss64(p64, X, y, dims):
    """Mean softmax cross-entropy written independently of the oracle (fp64, from the definition)."""
    d_in, d_h, d_out = dims
    W1, b1, W2, b2 = mlp_split(p64, d_in, d_h, d_out)
    H = np.maximum(X.astype(np.float64) @ W1 + b1, 0.0)
    L = H @ W2 + b2
    tot = 0.0
    for r in range(X.shape[0]):
        tot += np.log(np.sum(np.exp(L[r] - L[r].max()))) + L[r].max() - L[r, y[r]]
    return tot / X.shape[0]


def test_gradient_matches_finite_differences_exhaustively_on_tiny_net():
    rng = np.random.default_rng(0)
    dims = (7, 5, 3)
    p, X, y = _problem(rng, *dims, mb=4, scale=0.7)
    loss, grad, _ = mlp_loss_and_grad(p, X, y, *dims, mode="exact")
    p64 = p.astype(np.float64)
    assert abs(loss - _loss64(p64, X, y, dims)) < 1e-12
    h = 1e-6
    for j in range(p.size):
        e = np.zeros_like(p64); e[j] = h
        fd = (_loss64(p64 + e, X, y, dims) - _loss64(p64 - e, X, y, dims)) / (2 * h)
        assert abs(fd - grad[j]) < 1e-7 + 1e-6 * abs(grad[j]), (j, fd, grad[j])


def test_gradient_matches_finite_differences_on_sampled_coordinates():
    rng = np.random.default_rng(1)
    dims = (96, 128, 10)
    p, X, y = _problem(rng, *dims, mb=16, scale=0.15)
    _, grad, _ = mlp_loss_and_grad(p, X, y, *dims, mode="exact")
    p64 = p.astype(np.float64)
    h = 1e-6
    o_b1 = dims[0] * dims[1]; o_w2 = o_b1 + dims[1]; o_b2 = o_w2 + dims[1] * dims[2]
    picks = np.concatenate([rng.integers(0, o_b1, 60), rng.integers(o_b1, o_w2, 30),
                            rng.integers(o_w2, o_b2, 40), np.arange(o_b2, p.size)])
    for j in picks:
        e = np.zeros_like(p64); e[j] = h
        fd = (_loss64(p64 + e, X, y, dims) - _loss64(p64 - e, X, y, dims)) / (2 * h)
        assert abs(fd - grad[j]) < 1e-7 + 1e-5 * abs(grad[j]), (j, fd, grad[j])


@pytest.mark.parametrize("dims,mb", [((96, 128, 10), 16), ((3072, 4096, 10), 64)])
def test_gradient_matches_autograd(dims, mb):
    import torch

    rng = np.random.default_rng(2)
    p, X, y = _problem(rng, *dims, mb=mb, scale=0.02)
    loss, grad, _ = mlp_loss_and_grad(p, X, y, *dims, mode="exact")
    d_in, d_h, d_out = dims
    tp = torch.tensor(p.astype(np.float64), requires_grad=True)
    o = 0
    W1 = tp[o:o + d_in * d_h].view(d_in, d_h); o += d_in * d_h
    b1 = tp[o:o + d_h]; o += d_h
    W2 = tp[o:o + d_h * d_out].view(d_h, d_out); o += d_h * d_out
    b2 = tp[o:o + d_out]
    H = torch.relu(torch.tensor(X.astype(np.float64)) @ W1 + b1)
    L = H @ W2 + b2
    tl = torch.nn.functional.cross_entropy(L, torch.tensor(y), reduction="mean")
    tl.backward()
    ref = tp.grad.numpy()
    assert abs(float(tl.detach()) - loss) < 1e-10
    np.testing.assert_allclose(grad, ref, rtol=1e-9, atol=1e-12)


def test_bf16_round_is_nearest_even():
    # Exactly representable values are unchanged; halfway cases go to the even mantissa.
    assert bf16_round(np.array([1.0, -2.5, 0.0]))[0] == 1.0
    one_ulp = 2.0 ** -7                       # bf16 spacing in [1, 2)
    x = np.array([1.0 + one_ulp / 2, 1.0 + 3 * one_ulp / 2, 1.0 + one_ulp * 0.49, 1.0 + one_ulp * 0.51])
    r = bf16_round(x)
    assert r.tolist() == [1.0, 1.0 + 2 * one_ulp, 1.0, 1.0 + one_ulp]
    # against torch's bfloat16 conversion (library routine)
    import torch

    v = np.random.default_rng(3).standard_normal(10000).astype(np.float32) * 3
    ref = torch.tensor(v).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(bf16_round(v), ref)


def test_bf16_mode_stays_close_to_exact_mode():
    """Rounding the GEMM operands to bf16 (relative error 2^-9 each) moves every gradient
    tensor by a few 1e-3 of its scale at most -- a sanity bound that pins the emulation."""
    rng = np.random.default_rng(4)
    dims = (384, 512, 10)
    d_in, d_h, d_out = dims
    p, X, y = _problem(rng, *dims, mb=64, scale=0.0)
    p[: d_in * d_h] = rng.standard_normal(d_in * d_h) * np.sqrt(2.0 / d_in)
    o_w2 = d_in * d_h + d_h
    p[o_w2: o_w2 + d_h * d_out] = rng.standard_normal(d_h * d_out) * np.sqrt(2.0 / d_h)
    _, g_exact, aux_e = mlp_loss_and_grad(p, X, y, *dims, mode="exact")
    _, g_bf16, aux_b = mlp_loss_and_grad(p, X, y, *dims, mode="bf16")
    # Operand rounding moves pre-activations near zero across the ReLU threshold; those few
    # gates are a separate, discrete effect, so compare at equal gates.
    flips = [tuple(f) for f in np.argwhere((aux_e["Z"] > 0) != (aux_b["Z"] > 0))]
    assert 0 < len(flips) < 0.005 * aux_e["Z"].size
    assert np.abs(aux_e["Z"][tuple(np.array(flips).T)]).max() < 0.05
    _, g_same_gate, _ = mlp_loss_and_grad(p, X, y, *dims, mode="bf16", relu_flip=flips)
    for a, b in zip(mlp_split(g_exact, *dims), mlp_split(g_same_gate, *dims)):
        assert np.linalg.norm(a - b) / np.linalg.norm(a) < 6e-3
        assert np.abs(a - b).max() / np.abs(a).max() < 6e-3
    assert not np.array_equal(g_exact, g_same_gate)


def test_relu_flip_changes_only_that_hidden_unit():
    """For a pre-activation at (numerically) zero, inverting its gate changes only column h of
    dW1 and entry h of db1 -- the two valid outcomes a mixed-precision path may produce."""
    rng = np.random.default_rng(6)
    dims = (12, 9, 4)
    p, X, y = _problem(rng, *dims, mb=5, scale=0.5)
    _, _, aux = mlp_loss_and_grad(p, X, y, *dims, mode="bf16")
    p[dims[0] * dims[1] + 3] -= np.float32(aux["Z"][2, 3])        # push Z[2,3] to ~0 via b1[3]
    _, g0, aux = mlp_loss_and_grad(p, X, y, *dims, mode="bf16")
    assert abs(aux["Z"][2, 3]) < 1e-6
    _, g1, _ = mlp_loss_and_grad(p, X, y, *dims, mode="bf16", relu_flip=[(2, 3)])
    dW1a, db1a, dW2a, db2a = mlp_split(g0, *dims)
    dW1b, db1b, dW2b, db2b = mlp_split(g1, *dims)
    changed = np.where(np.abs(dW1a - dW1b).max(axis=0) > 1e-6)[0]
    assert changed.tolist() == [3]
    assert np.where(np.abs(db1a - db1b) > 1e-6)[0].tolist() == [3]
    assert np.abs(dW2a - dW2b).max() < 1e-6 and np.abs(db2a - db2b).max() < 1e-6
    # the difference is exactly X[r,:] * bf16(dH[r,h])
    from oracle.abs_oracle import bf16_round as rnd
    r, h = 2, 3
    np.testing.assert_allclose(np.abs(dW1a[:, h] - dW1b[:, h]), np.abs(aux["X"][r] * rnd(aux["dH"][r, h])), atol=1e-6)


# ------------------------------------------------------------------------------------------
# Where the bf16 roundings sit.  The mixed-precision path rounds exactly six tensors to bf16 before they
# enter a product: X, W1, W2 (forward), H (before the second layer and before dW2), dL (before dH and dW2)
# and dZ (before dW1); bias gradients, ReLU, softmax and the loss gradient use the unrounded values.
# The restatement below spells that out with torch's own bfloat16 conversion and fp64 matmuls; the oracle
# must agree with it to rounding error of the fp64 sums, and dropping any ONE of the six roundings in the
# oracle must break that agreement.
# ------------------------------------------------------------------------------------------
def _restated_with_torch_bfloat16(p, X, y, dims):
    import torch

    def q(t):                                   # fp64 -> fp32 -> bf16 (nearest even) -> fp64
        return t.to(torch.float32).to(torch.bfloat16).to(torch.float64)

    d_in, d_h, d_out = dims
    t = torch.tensor(np.asarray(p, dtype=np.float32).astype(np.float64))
    o = 0
    W1 = t[o:o + d_in * d_h].view(d_in, d_h); o += d_in * d_h
    b1 = t[o:o + d_h]; o += d_h
    W2 = t[o:o + d_h * d_out].view(d_h, d_out); o += d_h * d_out
    b2 = t[o:o + d_out]
    Xt = torch.tensor(np.asarray(X, dtype=np.float64))
    mb = Xt.shape[0]
    Xq, W1q, W2q = q(Xt), q(W1), q(W2)
    Z = Xq @ W1q + b1
    gate = Z > 0
    H = torch.where(gate, Z, torch.zeros_like(Z))
    Hq = q(H)
    L = Hq @ W2q + b2
    prob = torch.softmax(L, dim=1)
    dL = prob.clone()
    dL[torch.arange(mb), torch.tensor(np.asarray(y, dtype=np.int64))] -= 1.0
    dL = dL / mb
    dLq = q(dL)
    dW2 = Hq.T @ dLq
    db2 = dL.sum(dim=0)                         # unrounded
    dH = dLq @ W2q.T
    dZ = torch.where(gate, dH, torch.zeros_like(dH))
    db1 = dZ.sum(dim=0)                         # unrounded
    dW1 = Xq.T @ q(dZ)
    return torch.cat([dW1.reshape(-1), db1, dW2.reshape(-1), db2]).numpy()


_ROUNDING_POINTS = ["X", "W1", "W2", "H", "dL", "dZ"]      # the order in which the oracle rounds them


def _rounding_problem():
    rng = np.random.default_rng(8)
    dims = (96, 128, 10)
    d_in, d_h, d_out = dims
    p, X, y = _problem(rng, *dims, mb=64, scale=0.0)
    p[: d_in * d_h] = rng.standard_normal(d_in * d_h) * np.sqrt(2.0 / d_in)
    o_b1 = d_in * d_h
    p[o_b1: o_b1 + d_h] = rng.standard_normal(d_h) * 0.1
    o_w2 = o_b1 + d_h
    p[o_w2: o_w2 + d_h * d_out] = rng.standard_normal(d_h * d_out) * np.sqrt(2.0 / d_h)
    p[o_w2 + d_h * d_out:] = rng.standard_normal(d_out) * 0.1
    return p, X, y, dims


def _agrees(g, ref, dims):
    return all(np.abs(a - b).max() <= 1e-12 * max(np.abs(b).max(), 1e-300)
               for a, b in zip(mlp_split(g, *dims), mlp_split(ref, *dims)))


def test_bf16_rounding_points_match_a_restatement_with_torch_bfloat16():
    p, X, y, dims = _rounding_problem()
    _, g, _ = mlp_loss_and_grad(p, X, y, *dims, mode="bf16")
    ref = _restated_with_torch_bfloat16(p, X, y, dims)
    for name, a, b in zip(("dW1", "db1", "dW2", "db2"), mlp_split(g, *dims), mlp_split(ref, *dims)):
        assert np.abs(a - b).max() <= 1e-12 * np.abs(b).max(), name
    # and at the size of workload 4's small form, with the generator's own inputs
    from paper_2308_15164_b200 import workloads as wlm

    wl = wlm.config(4, small=True)
    d = wl.mlp
    xs, ys = wlm.mlp_batches(wl)
    x0 = wlm.params0(wl)
    _, g, _ = mlp_loss_and_grad(x0, xs[0], ys[0], d.d_in, d.d_hidden, d.d_out, mode="bf16")
    assert _agrees(g, _restated_with_torch_bfloat16(x0, xs[0], ys[0], (d.d_in, d.d_hidden, d.d_out)), (d.d_in, d.d_hidden, d.d_out))


@pytest.mark.parametrize("k", range(6), ids=_ROUNDING_POINTS)
def test_dropping_one_rounding_point_in_the_oracle_is_caught(k, monkeypatch):
    """Planted mistake, in the oracle: its k-th bf16 rounding (order X, W1, W2, H, dL, dZ) is skipped."""
    import oracle.abs_oracle as O

    p, X, y, dims = _rounding_problem()
    ref = _restated_with_torch_bfloat16(p, X, y, dims)
    real = O.bf16_round
    calls = []

    def skip_kth(a):
        calls.append(np.shape(a))
        return np.asarray(a, dtype=np.float64) if len(calls) - 1 == k else real(a)

    monkeypatch.setattr(O, "bf16_round", skip_kth)
    _, g_bad, _ = O.mlp_loss_and_grad(p, X, y, *dims, mode="bf16")
    monkeypatch.setattr(O, "bf16_round", real)
    mb, (d_in, d_h, d_out) = X.shape[0], dims
    assert calls == [(mb, d_in), (d_in, d_h), (d_h, d_out), (mb, d_h), (mb, d_out), (mb, d_h)]   # X W1 W2 H dL dZ
    assert not _agrees(g_bad, ref, dims), f"the restatement does not notice a missing rounding of {_ROUNDING_POINTS[k]}"
    _, g_good, _ = O.mlp_loss_and_grad(p, X, y, *dims, mode="bf16")
    assert _agrees(g_good, ref, dims)


@pytest.mark.parametrize("what", ["db1 from rounded dZ", "db2 from rounded dL", "dH from unrounded dL", "dW2 from unrounded H"])
def test_a_rounding_in_the_wrong_place_is_caught(what):
    """Planted mistakes of the other kind: a value used rounded where the path keeps it exact, or the other way
    round.  Each is a copy of the restatement with one line changed; the oracle must disagree with every one."""
    import torch

    p, X, y, dims = _rounding_problem()
    _, g, _ = mlp_loss_and_grad(p, X, y, *dims, mode="bf16")
    good = _restated_with_torch_bfloat16(p, X, y, dims)
    dW1, db1, dW2, db2 = [a.copy() for a in mlp_split(good, *dims)]
    aux = mlp_loss_and_grad(p, X, y, *dims, mode="bf16")[2]
    q = lambda a: torch.tensor(a).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    W2 = mlp_split(np.asarray(p, dtype=np.float32).astype(np.float64), *dims)[2]
    Z = aux["Z"]
    gate = Z > 0
    H = np.where(gate, Z, 0.0)
    L = q(H) @ q(W2) + mlp_split(np.asarray(p, dtype=np.float32).astype(np.float64), *dims)[3]
    e = np.exp(L - L.max(axis=1, keepdims=True))
    dL = e / e.sum(axis=1, keepdims=True)
    dL[np.arange(X.shape[0]), y] -= 1.0
    dL /= X.shape[0]
    if what == "db1 from rounded dZ":
        db1 = q(np.where(gate, q(dL) @ q(W2).T, 0.0)).sum(axis=0)
    elif what == "db2 from rounded dL":
        db2 = q(dL).sum(axis=0)
    elif what == "dH from unrounded dL":
        dZ = np.where(gate, dL @ q(W2).T, 0.0)
        db1 = dZ.sum(axis=0)
        dW1 = q(X).T @ q(dZ)
    else:
        dW2 = H.T @ q(dL)
    wrong = np.concatenate([dW1.ravel(), db1, dW2.ravel(), db2])
    assert not _agrees(g, wrong, dims)
    assert _agrees(g, good, dims)
