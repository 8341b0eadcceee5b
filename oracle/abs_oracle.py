"""CPU oracle for the delayed synchronous step of ABS-SGD (arXiv 2308.15164, Algorithm 1).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, obviously-correct restatement of what
the hot path computes.  It shares no code with the CUDA path and imports nothing from it;
only tests, the smoke check and the benchmark's CPU-baseline leg may use it.

State (Algorithm 1, "Initialization" and Step 2):
    x          parameters x_t                         (held in fp64)
    v          momentum buffer, v_0 = 0               (held in fp64; not in the paper)
    acc[2][W]  per-worker accumulated gradients G^i   (fp32, added in call order)
    cnt[2][W]  per-worker micro-batch counts b_i      (integers; M^i = b_i * M_r)
    cur        which of the two sets the current iteration fills
    t          iteration counter

One iteration t of Algorithm 1:
    accumulate(i, g)  once per reference batch a worker finishes while Step 1 runs
                      (Step 2: G_t^i += g, M_t^i += M_r),
    sync_step()       Step 1 + "Update parameters": the weighted average of the DELAYED
                      set G_{t-1} (Section 5, weighted gradient averaging mechanism)
                      is applied to x_t, giving x_{t+1}; the delayed set is cleared and
                      becomes the target of iteration t+1.

Readings where the paper is silent (also listed in the design notes):
  * A micro-batch gradient g is the MEAN over the M_r samples of the reference batch, so
    sum_i G^i / sum_i M^i (per-sample sums over sample counts) equals sum_i G^i / sum_i b_i
    (per-micro-batch means over micro-batch counts).
  * If sum_i b_i = 0 for the delayed set (always true at t = 0, where G_{-1} = 0) the
    step leaves x and v untouched; counters/buffers still clear and swap, t still advances.
  * Momentum and weight decay are not in the paper (its update is plain SGD).  They follow
    the common convention: g = Gbar + wd * x ; v = mu * v + g ; x = x - lr * v.
    With mu = wd = 0 this is exactly "x_{t+1} = x_t - gamma * Gbar_{t-1}".
  * Delayed-gradient compensation (Eq. 6): Gtilde = Gbar + lambda * Gbar*Gbar*(x_t - x_{t-1}),
    applied to the averaged gradient before weight decay and momentum.  x_{-1} := x_0.
"""

from __future__ import annotations

import numpy as np


class AbsSgdOracle:
    """Sequential reference of the delayed synchronous step (Algorithm 1)."""

    def __init__(self, x0, W, lr, momentum=0.0, weight_decay=0.0, lambda_dc=0.0):
        x0 = np.asarray(x0)
        assert x0.ndim == 1 and W >= 1
        self.P = x0.shape[0]
        self.W = int(W)
        self.lr = float(lr)
        self.momentum = float(momentum)
        self.weight_decay = float(weight_decay)
        self.lambda_dc = float(lambda_dc)
        self.x = x0.astype(np.float64).copy()
        self.x_prev = self.x.copy()                       # x_{t-1}, for Eq. 6
        self.v = np.zeros(self.P, dtype=np.float64)
        self.acc = np.zeros((2, self.W, self.P), dtype=np.float32)   # G_{-1}^i = 0
        self.cnt = np.zeros((2, self.W), dtype=np.int64)
        self.cur = 0
        self.t = 0
        self.consumed = []                                # b_i used by each sync step
        self.gnorm2 = []                                  # |Gbar|^2 applied by each sync step (0: nothing applied)

    # Step 2 of Algorithm 1: G_t^i = G_t^i + g ; M_t^i = M_t^i + M_r
    def accumulate(self, i, g):
        assert 0 <= i < self.W
        g = np.asarray(g)
        assert g.shape == (self.P,)
        if g.dtype == np.uint16:                          # bf16 bit patterns: widen (exact)
            g = (g.astype(np.uint32) << np.uint32(16)).view(np.float32)
        # fp32 accumulation in call order (the accumulator is an fp32 buffer).
        self.acc[self.cur, i] += g.astype(np.float32)
        self.cnt[self.cur, i] += 1

    # Step 1 of Algorithm 1 on the delayed set, then "Update parameters".
    def sync_step(self):
        d = self.cur ^ 1                                  # the set filled during iteration t-1
        b = self.cnt[d].copy()
        B = int(b.sum())                                  # sum_i M_{t-1}^i / M_r
        self.consumed.append(b.astype(np.int32))
        x_old = self.x.copy()
        if B > 0:
            G = np.zeros(self.P, dtype=np.float64)
            for i in range(self.W):                       # sum_i G_{t-1}^i, worker order
                G += self.acc[d, i].astype(np.float64)
            Gbar = G / B                                  # weighted average (Algorithm 1, Step 1)
            self.gnorm2.append(float(np.dot(Gbar, Gbar)))  # a logged metric; takes no part in the update
            if self.lambda_dc != 0.0:                     # Eq. 6, delayed-gradient compensation
                Gbar = Gbar + self.lambda_dc * Gbar * Gbar * (self.x - self.x_prev)
            g = Gbar + self.weight_decay * self.x
            self.v = self.momentum * self.v + g
            self.x = self.x - self.lr * self.v            # x_{t+1} = x_t - gamma * Gtilde_t
        else:
            self.gnorm2.append(0.0)
        self.x_prev = x_old
        self.acc[d].fill(0.0)                             # Step 2 "Initialization" of the next
        self.cnt[d].fill(0)                               # iteration's G and M
        self.cur = d
        self.t += 1
        return B

    def params(self):
        """Current parameters rounded to fp32 (the storage type of the hot path)."""
        return self.x.astype(np.float32)

    def counters(self):
        return self.cnt.astype(np.int32).copy(), self.cur, self.t


# ------------------------------------------------------------------------------------------
# Two-layer MLP workload: the "compute the gradients of a reference batch" of Step 2 for a
# 3072-4096-10 ReLU network with softmax cross-entropy (mean over the micro-batch).
# ------------------------------------------------------------------------------------------

def bf16_round(a):
    """Round to the nearest bf16 value (ties to even), starting from the fp32 rounding of
    ``a``; returns fp64 holding bf16-representable numbers."""
    f = np.asarray(a, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = ((u + 0x7FFF + lsb) >> 16) << 16
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(a))


def mlp_split(flat, d_in, d_hidden, d_out):
    """Views of W1 [d_in, d_hidden], b1 [d_hidden], W2 [d_hidden, d_out], b2 [d_out] in a flat vector."""
    o = 0
    W1 = flat[o:o + d_in * d_hidden].reshape(d_in, d_hidden); o += d_in * d_hidden
    b1 = flat[o:o + d_hidden]; o += d_hidden
    W2 = flat[o:o + d_hidden * d_out].reshape(d_hidden, d_out); o += d_hidden * d_out
    b2 = flat[o:o + d_out]; o += d_out
    assert o == flat.shape[0]
    return W1, b1, W2, b2


def mlp_loss_and_grad(flat_params, X, y, d_in, d_hidden, d_out, mode="exact", relu_flip=()):
    """Mean softmax cross-entropy of one micro-batch and its gradient w.r.t. the flat params.

    mode "exact": everything in fp64.
    mode "bf16":  GEMM operands are rounded to bf16 at the points where the mixed-precision
                  path rounds them (X, W1, W2, H, dL, dZ); every product is accumulated in
                  fp64; bias adds, ReLU, softmax and the gradient of the loss are not rounded.
    relu_flip:    (row, hidden) entries whose ReLU gate is inverted.  Tests use it to
                  enumerate the valid outcomes when a pre-activation is so close to zero
                  that fp32 and fp64 accumulation may disagree about its sign.
    Returns (loss, grad_flat fp64, aux); aux holds intermediates (Z: pre-activations, dL: gradient of the loss
    w.r.t. the logits, dH: gradient w.r.t. the hidden activations, X: the first-layer operand as used).
    """
    p = np.asarray(flat_params, dtype=np.float32).astype(np.float64)   # fp32 master weights
    W1, b1, W2, b2 = mlp_split(p, d_in, d_hidden, d_out)
    X = np.asarray(X, dtype=np.float64)
    y = np.asarray(y).astype(np.int64)
    mb = X.shape[0]
    rnd = bf16_round if mode == "bf16" else (lambda a: a)

    Xo, W1o, W2o = rnd(X), rnd(W1), rnd(W2)
    Z = Xo @ W1o + b1                                   # [mb, hidden]
    gate = Z > 0.0
    for (r, h) in relu_flip:
        gate[r, h] = ~gate[r, h]
    H = np.where(gate, Z, 0.0)
    Ho = rnd(H)
    L = Ho @ W2o + b2                                   # logits [mb, out]
    Lm = L - L.max(axis=1, keepdims=True)
    e = np.exp(Lm)
    prob = e / e.sum(axis=1, keepdims=True)
    loss = float(-(Lm[np.arange(mb), y] - np.log(e.sum(axis=1))).mean())
    dL = prob.copy()
    dL[np.arange(mb), y] -= 1.0
    dL /= mb                                            # mean over the micro-batch
    dLo = rnd(dL)
    dW2 = Ho.T @ dLo
    db2 = dL.sum(axis=0)
    dH = dLo @ W2o.T
    dZ = np.where(gate, dH, 0.0)
    db1 = dZ.sum(axis=0)
    dZo = rnd(dZ)
    dW1 = Xo.T @ dZo
    grad = np.concatenate([dW1.ravel(), db1, dW2.ravel(), db2])
    return loss, grad, {"Z": Z, "dH": dH, "X": Xo, "dL": dL}
