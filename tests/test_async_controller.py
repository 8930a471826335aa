"""The asynchronous stage controller (host only) against the oracle's event simulation of Appendix B's three rules
and against the library's C simulator, on the same verdict streams."""
import numpy as np
import pytest

from oracle import lr_cycles as C
from paper_2506_19830_b200 import binding as B
from paper_2506_19830_b200.async_cycle import AsyncStageController, StageExecutor
from paper_2506_19830_b200.build import build_library


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()


class _Stream(StageExecutor):
    """Feeds verdicts from a fixed 0/1 stream in the order the controller asks for them."""

    def __init__(self, verdicts):
        self.v, self.k = list(verdicts), 0
        self.open_starts = []

    def start_position(self, i, now):
        self.open_starts.append((i, now))

    def target_done(self, i, now):
        v = self.v[self.k]
        self.k += 1
        return v


def _run(gamma, num, den, verdicts):
    ctl = AsyncStageController(gamma, num, den)
    ex = _Stream(verdicts)
    n_zero = int(sum(1 for v in verdicts if not v))
    for _ in range(n_zero):  # one stage per rejection in the stream; what follows the last 0 belongs to no whole stage
        assert ctl.run_stage(ex) is not None
    return ctl


CASES = [(1, 1, 3), (2, 1, 10), (3, 1, 4), (4, 1, 3), (8, 1, 2), (5, 2, 9), (6, 1, 100), (3, 3, 10), (2, 0, 5), (7, 5, 5)]


@pytest.mark.parametrize("gamma,num,den", CASES)
@pytest.mark.parametrize("alpha", [0.0, 0.3, 0.7, 0.9])
def test_controller_matches_the_oracle_and_the_c_simulator(gamma, num, den, alpha):
    for n in (1, 7, 400):
        v = (np.random.Generator(np.random.PCG64(31 * gamma + n)).random(n) < alpha).astype(np.uint8)
        ref = C.simulate_async(gamma, num, den, v.tolist())
        ctl = _run(gamma, num, den, v.tolist())
        for key in ("stages", "steps", "time", "verdicts_used"):
            assert ctl.stats[key] == ref[key], key
        lib = B.lr_cycle_simulate_async(gamma, num, den, v)
        assert {k: lib[k] for k in ("stages", "steps", "time", "verdicts_used")} == {k: ref[k] for k in ("stages", "steps", "time", "verdicts_used")}
        # the controller also starts positions behind the rejected one (it cannot know yet): never more than gamma at once
        assert ref["peak_in_flight"] <= ctl.stats["peak_in_flight"] <= gamma


def test_event_order_follows_the_three_rules():
    gamma, num, den = 3, 2, 7
    v = [1, 1, 1, 1, 0, 1, 0, 0]
    ctl = _run(gamma, num, den, v)
    starts, finished = {}, {}
    stage_t0, stage = 0, 0
    for t, ev, i in ctl.log:
        if ev == "start":
            # rule 1: after the previous draft, and once generation i - gamma is done; rule 2: draft and target start together
            lo = stage_t0 if i == 0 else starts[(stage, i - 1)] + num
            if i >= gamma:
                lo = max(lo, starts[(stage, i - gamma)] + den)
            assert t == lo, (stage, i, t, lo)
            starts[(stage, i)] = t
        elif ev in ("accept", "reject"):
            assert t == starts[(stage, i)] + den  # rule 3: the verdict is read when the target's step is done
            finished[(stage, i)] = ev
            if ev == "reject":
                stage += 1
                stage_t0 = t
    assert [e for e in finished.values()] == ["accept", "accept", "accept", "accept", "reject", "accept", "reject", "reject"]
    assert ctl.stats["steps"] == 5 + 2 + 1 and ctl.stats["stages"] == 3


def test_a_stage_without_a_rejection_stays_open():
    ctl = AsyncStageController(2, 1, 3)
    ex = _Stream([1, 1, 1])
    assert ctl.run_stage(ex, max_positions=3) is None
    assert ctl.stats["stages"] == 0 and ex.k == 3
