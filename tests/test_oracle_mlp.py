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
