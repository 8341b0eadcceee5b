"""CPU-only: the oracle against closed forms, invariants, a library optimiser and hand-worked
examples; plus deliberately broken oracles, each of which at least one pin must catch."""

import numpy as np
import pytest

from oracle.abs_oracle import AbsSgdOracle
from oracle.c_oracle import AbsSgdOracleC
from tests.oracle_pins import ALL_PINS


def make_np(x0, W, lr, mu, wd, lam):
    return AbsSgdOracle(x0, W, lr, mu, wd, lam)


def make_c(x0, W, lr, mu, wd, lam):
    return AbsSgdOracleC(x0, W, lr, mu, wd, lam)


@pytest.mark.parametrize("pin", ALL_PINS, ids=lambda p: p.__name__)
@pytest.mark.parametrize("make", [make_np, make_c], ids=["numpy", "c"])
def test_pin(make, pin):
    pin(make)


# ------------------------------------------------------------------------------------------
# Two plain implementations agree (NumPy oracle vs C oracle), including bf16 inputs, idle
# workers, weight decay, momentum and compensation.
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("lam", [0.0, 0.5])
@pytest.mark.parametrize("bf16", [False, True])
def test_numpy_and_c_oracles_agree(lam, bf16):
    rng = np.random.default_rng(5)
    P, W, T = 1003, 5, 9
    x0 = (rng.standard_normal(P) * 0.1).astype(np.float32)
    a = AbsSgdOracle(x0, W, 0.05, 0.9, 1e-3, lam)
    b = AbsSgdOracleC(x0, W, 0.05, 0.9, 1e-3, lam)
    for t in range(T):
        counts = rng.integers(0, 4, size=W)
        for i in range(W):
            for _ in range(counts[i]):
                g = rng.standard_normal(P).astype(np.float32)
                if bf16:
                    g = (g.view(np.uint32) >> 16).astype(np.uint16)
                a.accumulate(i, g)
                b.accumulate(i, g)
        ca, cb = a.counters(), b.counters()
        assert np.array_equal(ca[0], cb[0]) and ca[1:] == cb[1:]
        assert a.sync_step() == b.sync_step()
        np.testing.assert_allclose(a.params(), b.params(), rtol=0, atol=1e-7)
        np.testing.assert_allclose(a.v, b.v, rtol=1e-12, atol=1e-12)
    assert [c.tolist() for c in a.consumed] == [c.tolist() for c in b.consumed]


# ------------------------------------------------------------------------------------------
# Planted mistakes.  Each mutant re-implements sync_step/accumulate with one plausible error.
# ------------------------------------------------------------------------------------------
class Mutant(AbsSgdOracle):
    def __init__(self, bug, *a):
        super().__init__(*a)
        self.bug = bug

    def accumulate(self, i, g):
        if self.bug == "count_not_incremented_for_worker0" and i == 0 and self.cnt[self.cur, 0] >= 1:
            g = np.asarray(g)
            self.acc[self.cur, i] += g.astype(np.float32)
            return
        if self.bug == "bf16_bits_taken_as_integers" and np.asarray(g).dtype == np.uint16:
            g = np.asarray(g).astype(np.float32)
        super().accumulate(i, g)

    def sync_step(self):
        bug = self.bug
        d = self.cur if bug == "no_delay" else self.cur ^ 1
        b = self.cnt[d].copy()
        B = int(b.sum())
        self.consumed.append(b.astype(np.int32))
        x_old = self.x.copy()
        if B > 0 or bug == "noop_step_still_decays":
            G = np.zeros(self.P)
            for i in range(self.W):
                if bug == "drops_last_worker" and i == self.W - 1 and self.W > 1:
                    continue
                G += self.acc[d, i].astype(np.float64)
            if bug == "uniform_average":
                act = [i for i in range(self.W) if b[i] > 0]
                Gbar = sum(self.acc[d, i].astype(np.float64) / b[i] for i in act) / len(act)
            elif bug == "divide_by_workers":
                Gbar = G / self.W
            elif bug == "divide_by_active_workers":
                Gbar = G / max(1, int((b > 0).sum()))
            else:
                Gbar = G / max(B, 1)
            if self.lambda_dc != 0.0:
                disp = (self.x - self.x_prev)
                if bug == "compensation_sign":
                    disp = -disp
                if bug == "compensation_linear":
                    Gbar = Gbar + self.lambda_dc * Gbar * disp
                else:
                    Gbar = Gbar + self.lambda_dc * Gbar * Gbar * disp
            wdx = self.weight_decay * self.x
            if bug == "weight_decay_sign":
                wdx = -wdx
            g = Gbar + wdx
            if bug == "dampened_momentum":
                self.v = self.momentum * self.v + (1 - self.momentum) * g
            else:
                self.v = self.momentum * self.v + g
            if bug == "nesterov":
                self.x = self.x - self.lr * (g + self.momentum * self.v)
            elif bug == "lr_inside_momentum":
                # v accumulates lr*g; same as the rule only while lr is constant -- caught by
                # nothing here unless lr changes, so make it visibly different: decay by lr too.
                self.x = self.x - self.lr * self.lr * self.v
            else:
                self.x = self.x - self.lr * self.v
        if bug != "stale_previous_params":
            self.x_prev = x_old
        if bug != "accumulator_not_cleared":
            self.acc[d].fill(0.0)
        if bug != "counters_not_cleared":
            self.cnt[d].fill(0)
        if bug != "no_delay":
            self.cur = d
        else:
            self.acc[d].fill(0.0); self.cnt[d].fill(0)
        self.t += 1
        return B


MUTANTS = [
    "no_delay", "uniform_average", "divide_by_workers", "divide_by_active_workers", "drops_last_worker",
    "weight_decay_sign", "dampened_momentum", "nesterov", "lr_inside_momentum", "noop_step_still_decays",
    "accumulator_not_cleared", "counters_not_cleared", "compensation_sign", "compensation_linear",
    "stale_previous_params", "count_not_incremented_for_worker0", "bf16_bits_taken_as_integers",
]


@pytest.mark.parametrize("bug", MUTANTS)
def test_planted_mistake_is_caught(bug):
    def make(x0, W, lr, mu, wd, lam):
        return Mutant(bug, x0, W, lr, mu, wd, lam)

    caught = []
    for pin in ALL_PINS:
        try:
            pin(make)
        except AssertionError:
            caught.append(pin.__name__)
        except Exception:           # a crash also counts as detection
            caught.append(pin.__name__)
    assert caught, f"no pin detects the planted mistake '{bug}'"


def test_unbroken_mutant_passes():
    def make(x0, W, lr, mu, wd, lam):
        return Mutant("none", x0, W, lr, mu, wd, lam)

    for pin in ALL_PINS:
        pin(make)


def test_logged_gradient_norm_closed_form():
    """|Gbar|^2 for constant-per-worker gradients c_i: P * (sum_i b_i c_i / sum_i b_i)^2, logged one step late
    (the delayed gradients), 0 for steps that applied nothing; Eq. 6 and weight decay do not enter it."""
    P, W = 37, 3
    o = AbsSgdOracle(np.ones(P, dtype=np.float32), W, 0.1, 0.9, 0.01, 0.5)
    b, c = (3, 0, 2), (2.0, 100.0, -1.0)
    for i in range(W):
        for _ in range(b[i]):
            o.accumulate(i, np.full(P, c[i], dtype=np.float32))
    o.sync_step()                                      # applies G_{-1} = 0: nothing
    o.sync_step()                                      # applies the set above
    o.sync_step()                                      # nothing again
    want = P * ((3 * 2.0 + 2 * -1.0) / 5.0) ** 2
    assert o.gnorm2[0] == 0.0 and o.gnorm2[2] == 0.0
    assert abs(o.gnorm2[1] - want) <= 1e-12 * want
