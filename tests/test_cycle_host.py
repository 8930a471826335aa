"""The library's host-side cycle model against the oracle (CPU only: these entry points use no device)."""
import math

import numpy as np
import pytest

from oracle import lr_cycles as C
from paper_2506_19830_b200 import binding as B
from paper_2506_19830_b200.build import build_library


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()


def _verdicts(alpha, n, seed):
    return (np.random.Generator(np.random.PCG64(seed)).random(n) < alpha).astype(np.uint8)


CASES = [(1, 1, 3), (2, 1, 10), (3, 1, 4), (4, 1, 3), (8, 1, 2), (5, 2, 9), (6, 1, 100), (3, 3, 10), (2, 0, 5), (7, 5, 5)]


@pytest.mark.parametrize("gamma,num,den", CASES)
@pytest.mark.parametrize("alpha", [0.0, 0.3, 0.7, 1.0])
def test_simulators_match_the_oracle_exactly(gamma, num, den, alpha):
    for n in (0, 1, 7, 1000, 20_000):
        v = _verdicts(alpha, n, 11 * gamma + n)
        got = B.lr_cycle_simulate_async(gamma, num, den, v)
        assert got == C.simulate_async(gamma, num, den, v.tolist())
        got = B.lr_cycle_simulate_sync(gamma, num, den, v)
        ref = C.simulate_sync(gamma, num, den, v.tolist())
        assert {k: got[k] for k in ref} == ref


def test_closed_forms_match():
    for k in (1, 2, 3, 5, 9, 40):
        for a in (0.1, 0.52, 0.8, 0.97):
            for c in (0.01, 0.2, 1 / 3, 0.5, 0.9):
                assert math.isclose(B.lr_cycle_speedup(0, k, a, c), C.f_sync(k, a, c), rel_tol=1e-13)
                assert math.isclose(B.lr_cycle_speedup(1, k, a, c), C.f_async(k, a, c), rel_tol=1e-13)
                assert math.isclose(B.lr_cycle_speedup(2, k, a, c), C.f_token(k, a, c), rel_tol=1e-13)
    assert math.isnan(B.lr_cycle_speedup(0, 0, 0.5, 0.5)) and math.isnan(B.lr_cycle_speedup(1, 2, 1.0, 0.5))


@pytest.mark.parametrize("asynchronous", [True, False])
def test_strategy_search_matches(asynchronous):
    rng = np.random.Generator(np.random.PCG64(5))
    for _ in range(60):
        M = int(rng.integers(1, 65))
        a1, a2 = rng.uniform(0.05, 0.95, 2)
        c1, c2 = rng.uniform(0.02, 0.6, 2)
        k1, k2, h = B.lr_cycle_best_strategy(M, a1, c1, a2, c2, asynchronous)
        r1, r2, rh = C.best_strategy(M, a1, c1, a2, c2, asynchronous)
        assert math.isclose(h, rh, rel_tol=1e-12)
        if (k1, k2) != (r1, r2):  # only a tie within rounding may be resolved differently
            f = C.f_async if asynchronous else C.f_sync
            assert math.isclose(f(k1, a1, c1) * C.f_token(k2, a2, c2), rh, rel_tol=1e-12)


def test_bad_arguments():
    for args in ((0, 1, 3), (2, -1, 3), (2, 1, 0)):
        with pytest.raises(B.LrError):
            B.lr_cycle_simulate_async(*args, np.zeros(4, np.uint8))
        with pytest.raises(B.LrError):
            B.lr_cycle_simulate_sync(*args, np.zeros(4, np.uint8))
    with pytest.raises(B.LrError):
        B.lr_cycle_best_strategy(0, 0.5, 0.5, 0.5, 0.5)
    with pytest.raises(B.LrError):
        B.lr_cycle_best_strategy(8, 1.5, 0.5, 0.5, 0.5)
