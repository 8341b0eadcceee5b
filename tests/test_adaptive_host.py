"""Host logic of the adaptive batch size driver and of the paper's heterogeneity simulation (Section 6.1),
against a stand-in engine that needs no GPU: Step 1 "finishes" after a fixed number of polls."""

import numpy as np
import pytest

from paper_2308_15164_b200.adaptive import heterogeneity, run_adaptive


class FakeEngine:
    def __init__(self, W, polls_per_step1):
        self.W, self.polls_per_step1 = W, polls_per_step1
        self.calls, self.syncs, self._polls = [], 0, 0

    def accumulate(self, worker, grad):
        self.calls.append((self.syncs, worker, grad))

    def step1_finished(self):
        self._polls += 1
        return self._polls >= self.polls_per_step1

    def sync_step(self):
        self.syncs += 1
        self._polls = 0


def test_presets_follow_the_paper():
    assert heterogeneity("static", 4) == ([0.0, 1.0, 2.0, 3.0], 0.0)        # +0 %, 100 %, 200 %, 300 %
    assert heterogeneity("dynamic", 4) == ([0.0] * 4, 0.5)                   # +U(0 %, 50 %)
    assert heterogeneity("both", 6) == ([0.0, 1.0, 2.0, 3.0, 0.0, 1.0], 0.5)
    with pytest.raises(ValueError):
        heterogeneity("other", 4)


def test_static_heterogeneity_gives_iteration_times_1_2_3_4():
    # the driver starts polling once every worker has contributed (round 4 here): 9 polls end round 12
    eng = FakeEngine(4, polls_per_step1=9)
    static, dyn = heterogeneity("static", 4)
    sched = run_adaptive(eng, lambda t, i, k: (t, i, k), 3, static=static, dynamic=dyn)
    assert sched == [[12, 6, 4, 3]] * 3                                     # 12 rounds: 12/1, 12/2, 12/3, 12/4 batches
    assert eng.syncs == 3 and len(eng.calls) == 3 * 25
    # same thing expressed as periods
    eng2 = FakeEngine(4, polls_per_step1=9)
    assert run_adaptive(eng2, lambda t, i, k: (t, i, k), 3, period=(1, 2, 3, 4)) == sched
    assert eng2.calls == eng.calls                                          # same arrival order


def test_every_worker_contributes_and_the_cap_holds():
    eng = FakeEngine(4, polls_per_step1=1)                                  # Step 1 is over at the first poll
    sched = run_adaptive(eng, lambda t, i, k: None, 2, period=(1, 1, 2, 4), min_batches=2)
    assert sched == [[8, 8, 4, 2]] * 2                                      # runs on until the slowest has 2
    eng = FakeEngine(2, polls_per_step1=10 ** 9)                            # Step 1 never reports: the cap ends it
    assert run_adaptive(eng, lambda t, i, k: None, 1, period=(1, 3), max_batches=5) == [[5, 5]]


def test_dynamic_heterogeneity_is_seeded_bounded_and_traced():
    runs = []
    for seed in (5, 5, 6):
        eng, trace = FakeEngine(4, polls_per_step1=40), []
        sched = run_adaptive(eng, lambda t, i, k: (t, i, k), 4, dynamic=0.5, seed=seed, trace=trace)
        assert [c[1:] for c in eng.calls] == [(i, (t, i, k)) for (t, i, k) in trace]
        runs.append((sched, trace))
        for counts in sched:                                                # durations in [1, 1.5] rounds
            assert all(40 / 1.5 - 1 <= c <= 42 for c in counts)
        for t in range(4):                                                  # k counts up per worker
            for i in range(4):
                ks = [k for (tt, ii, k) in trace if tt == t and ii == i]
                assert ks == list(range(sched[t][i]))
    assert runs[0] == runs[1] and runs[0] != runs[2]
    arr = np.array(runs[0][0])
    assert arr.min() < arr.max()                                            # the counts do fluctuate


def test_argument_errors():
    eng = FakeEngine(2, 3)
    with pytest.raises(ValueError):
        run_adaptive(eng, lambda t, i, k: None, 1, period=(1, 2), static=(0.0, 1.0))
    with pytest.raises(ValueError):
        run_adaptive(eng, lambda t, i, k: None, 1, static=(0.0,))
    with pytest.raises(ValueError):
        run_adaptive(eng, lambda t, i, k: None, 1, dynamic=-0.1)
