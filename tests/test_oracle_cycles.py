"""Pins of the cycle-timing oracle: the closed forms of Section 3.2 / Appendix B and the cases that fix them."""
import math

import numpy as np
import pytest

from oracle import lr_cycles as C


def _verdicts(alpha, n, seed):
    return (np.random.Generator(np.random.PCG64(seed)).random(n) < alpha).astype(np.uint8)


# per-stage wall time, as the appendix states it ------------------------------------------------------------------
@pytest.mark.parametrize("gamma,num,den", [(4, 1, 3), (5, 2, 5), (8, 1, 2), (3, 1, 3), (2, 7, 10)])
def test_async_stage_time_when_the_draft_model_is_the_limit(gamma, num, den):
    assert gamma >= math.ceil(den / num)  # case 1: never more than ceil(1/c) generations in flight
    for x in range(0, 30):
        r = C.simulate_async(gamma, num, den, [1] * x + [0])
        assert r["stages"] == 1 and r["steps"] == x + 1
        assert r["time"] == den + num * x  # T + c T X
        assert r["peak_in_flight"] <= math.ceil(den / num)


@pytest.mark.parametrize("gamma,num,den", [(2, 1, 10), (3, 1, 4), (4, 1, 5), (1, 1, 3), (6, 1, 100)])
def test_async_stage_time_when_the_depth_is_the_limit(gamma, num, den):
    assert gamma < math.ceil(den / num)  # case 2
    for x in range(0, 40):
        r = C.simulate_async(gamma, num, den, [1] * x + [0])
        assert r["time"] == math.ceil((x + 1) / gamma) * den + num * (x % gamma)
        assert r["steps"] == x + 1 and r["peak_in_flight"] <= gamma


def test_async_by_hand():
    # gamma 2, draft 1 unit, target 10 units; verdicts 1 1 1 0: positions start at 0, 1, 10 (position 0 must
    # finish), 11 (position 1 must finish); draft 3 is rejected when its target step is done at 21
    r = C.simulate_async(2, 1, 10, [1, 1, 1, 0])
    assert (r["steps"], r["time"], r["stages"], r["peak_in_flight"]) == (4, 21, 1, 2)
    # two stages: reject at once (10 units, 1 step), then accept one and reject (1 + 10 units, 2 steps)
    r = C.simulate_async(2, 1, 10, [0, 1, 0, 1, 1])  # the last two verdicts open a stage that never ends: dropped
    assert (r["steps"], r["time"], r["stages"], r["verdicts_used"]) == (3, 21, 2, 3)


def test_sync_by_hand():
    # gamma 3: two drafts (2 units each) then the parallel target steps (7 units) = 11 units a cycle
    r = C.simulate_sync(3, 2, 7, [1, 1, 0, 1, 1, 0])
    assert (r["stages"], r["time"], r["steps"]) == (3, 33, 3 + 1 + 2)
    assert C.simulate_sync(1, 2, 7, [0, 0])["steps"] == 2  # no drafts: the target alone, speedup 1
    assert C.speedup(C.simulate_sync(1, 2, 7, [0, 0]), 7) == 1.0


# the closed forms, by the law of large numbers -----------------------------------------------------------------------
@pytest.mark.parametrize("alpha", [0.3, 0.6, 0.8])
@pytest.mark.parametrize("gamma,num,den", [(2, 1, 4), (4, 1, 3), (5, 1, 10), (3, 3, 10)])
def test_sync_speedup_converges_to_f_sync(alpha, gamma, num, den):
    r = C.simulate_sync(gamma, num, den, _verdicts(alpha, 400_000, 1))
    assert abs(C.speedup(r, den) / C.f_sync(gamma, alpha, num / den) - 1) < 6e-3


@pytest.mark.parametrize("alpha", [0.3, 0.6, 0.8])
@pytest.mark.parametrize("gamma,num,den", [(4, 1, 3), (8, 1, 4), (3, 1, 3), (5, 2, 9)])
def test_async_speedup_converges_to_s1(alpha, gamma, num, den):
    c = num / den
    assert gamma >= math.ceil(1 / c)
    r = C.simulate_async(gamma, num, den, _verdicts(alpha, 400_000, 2))
    s1 = 1 / (c + (1 - c) * (1 - alpha))
    assert abs(C.speedup(r, den) / s1 - 1) < 6e-3
    assert C.f_async(gamma, alpha, c) == s1


@pytest.mark.parametrize("alpha", [0.3, 0.6, 0.8])
@pytest.mark.parametrize("gamma,num,den", [(2, 1, 10), (3, 1, 4), (4, 1, 5), (6, 1, 100)])
def test_async_speedup_converges_to_s2(alpha, gamma, num, den):
    c = num / den
    assert gamma < math.ceil(1 / c)
    r = C.simulate_async(gamma, num, den, _verdicts(alpha, 400_000, 3))
    s2 = (1 - alpha ** gamma) / ((1 - alpha) + c * (alpha - alpha ** (gamma + 1) - gamma * (1 - alpha) * alpha ** gamma))
    assert abs(C.speedup(r, den) / s2 - 1) < 6e-3
    assert C.f_async(gamma, alpha, c) == s2


def test_limits():
    # nothing is ever accepted: every stage is one target step, speedup exactly 1 in the async version
    assert C.speedup(C.simulate_async(4, 1, 5, [0] * 100), 5) == 1.0
    # a free draft model and everything accepted up to the depth: the sync version emits gamma steps per T
    assert C.speedup(C.simulate_sync(5, 0, 3, [1] * 400), 3) == 5.0
    assert C.f_sync(1, 0.7, 0.2) == 1.0 and C.f_token(1, 0.7, 0.2) == 1.0


# Eq. 1 and the hybrid-optimality theorem ---------------------------------------------------------------------------------
def test_best_strategy_is_hybrid_in_the_theorems_range():
    for a1 in (0.53, 0.65, 0.79):
        for a2 in (0.53, 0.65, 0.79):
            for c1 in (0.05, 0.2, 0.33):
                for c2 in (0.02, 0.1, 0.19):
                    for M in (16, 24, 64):
                        k1, k2, h = C.best_strategy(M, a1, c1, a2, c2)
                        assert k1 >= 2 and k2 >= 2, (a1, a2, c1, c2, M)
                        # and it beats both pure strategies
                        pure_token = max(C.f_token(k, a2, c2) for k in range(1, M + 1))
                        pure_step = max(C.f_async(k, a1, c1) for k in range(1, M + 1))
                        assert h > pure_token and h > pure_step


def test_best_strategy_respects_the_budget_and_finds_the_maximum():
    M, a1, c1, a2, c2 = 12, 0.6, 0.25, 0.7, 0.1
    k1, k2, h = C.best_strategy(M, a1, c1, a2, c2, asynchronous=False)
    assert k1 * k2 <= M
    for x in range(1, M + 1):
        for y in range(1, M // x + 1):
            assert C.f_sync(x, a1, c1) * C.f_token(y, a2, c2) <= h + 1e-15
