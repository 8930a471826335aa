"""CPU oracle for the timing model of Lookahead Reasoning cycles -- test infrastructure only.

Only ``tests/`` and the benchmark's CPU legs may import this module; the product never does.

What is modelled (Section 3.2 "Theoretical Speedup Analysis" and Appendix B "speedup proof"): the target model
needs T time units for one reasoning step, the draft model c1*T, verification is free, one draft per position,
and every draft step is accepted independently.  Time is kept in integer units: T = ``den`` and a draft step
costs ``num`` units (c1 = num / den), so every event time is an exact integer.  The accept/reject outcomes are
inputs (a 0/1 stream), not drawn here.

``simulate_sync``   Algorithm 1: per cycle gamma - 1 drafts one after another, then gamma target steps in parallel;
                    the cycle emits the accepted run of drafts plus the target's step after it.
``simulate_async``  Appendix B's three rules, as an event simulation with a cap on target generations in flight.
``f_token``         g(k2) of Section 3.3, the token-level speculative decoding speedup.
``best_strategy``   Eq. 1 (Section 3.3) by exhaustive search.
"""
from __future__ import annotations

import math
from typing import Dict, Sequence, Tuple


def simulate_sync(gamma: int, num: int, den: int, verdicts: Sequence[int]) -> Dict[str, int]:
    """Whole cycles of the synchronous algorithm that the verdict stream allows.

    One cycle: the draft model writes gamma - 1 steps in sequence (num units each), then the target writes its
    gamma steps in parallel (den units), one after every draft prefix.  Drafts are checked in order; the cycle
    emits the drafts before the first rejected one and the target's own step at that position (after gamma - 1
    accepted drafts: the target's step after the last of them).  A cycle reads gamma - 1 verdicts; with
    gamma = 1 (no drafts at all) it reads none and one cycle is run per entry of the stream.
    """
    assert gamma >= 1 and num >= 0 and den >= 1
    time = steps = used = 0
    n_cycles = len(verdicts) // (gamma - 1) if gamma > 1 else len(verdicts)
    for _ in range(n_cycles):
        accepted = 0
        for v in verdicts[used:used + gamma - 1]:
            if not v:
                break
            accepted += 1
        used += gamma - 1
        time += (gamma - 1) * num + den
        steps += accepted + 1
    cycles = n_cycles
    return {"stages": cycles, "steps": steps, "time": time, "verdicts_used": used}


def simulate_async(gamma: int, num: int, den: int, verdicts: Sequence[int]) -> Dict[str, int]:
    """Whole stages of the asynchronous algorithm that the verdict stream allows.

    Within a stage, position i = 0, 1, ...: (rule 1) the draft model writes draft i as soon as it has finished
    draft i - 1 and fewer than gamma target generations are in flight; (rule 2) at the moment draft i is started
    the target starts its own step for position i, which takes den units; (rule 3) when the target's step i is
    done draft i is checked, and a rejected draft ends the stage there: the stage emits drafts 0..i-1 and the
    target's step i, everything later in flight is dropped, and the next stage starts at that moment.
    A stage reads verdicts up to and including its first 0.
    """
    assert gamma >= 1 and num >= 0 and den >= 1
    time = steps = stages = used = 0
    peak = 0
    while True:
        # the stage's verdicts: everything up to the first rejection
        end = used
        while end < len(verdicts) and verdicts[end]:
            end += 1
        if end >= len(verdicts):
            break  # the stream ends inside this stage: drop it
        x = end - used  # drafts accepted before the rejected one
        used = end + 1
        start = []  # start[i]: when draft i and the target's step i begin, relative to the stage
        for i in range(x + 1):
            t = 0 if i == 0 else start[i - 1] + num  # the draft model is free
            if i >= gamma:
                t = max(t, start[i - gamma] + den)  # generation i - gamma has to finish first
            start.append(t)
            peak = max(peak, sum(1 for s in start if s + den > t))
        time += start[x] + den
        steps += x + 1
        stages += 1
    return {"stages": stages, "steps": steps, "time": time, "verdicts_used": used, "peak_in_flight": peak}


def speedup(result: Dict[str, int], den: int) -> float:
    """Steps emitted per step the target alone would have written in the same time."""
    return result["steps"] / (result["time"] / den)


def f_sync(k1: int, alpha: float, c: float) -> float:
    """Step-level speedup of the synchronous version (Section 3.2)."""
    return (1 - alpha ** k1) / ((1 - alpha) * (1 - c + c * k1))


def f_async(k1: int, alpha: float, c: float) -> float:
    """Step-level speedup of the asynchronous version: S_1 or S_2 of Section 3.2 by the case."""
    if k1 >= math.ceil(1 / c):
        return 1 / (c + (1 - c) * (1 - alpha))
    return (1 - alpha ** k1) / ((1 - alpha) + c * (alpha - alpha ** (k1 + 1) - k1 * (1 - alpha) * alpha ** k1))


def f_token(k2: int, alpha: float, c: float) -> float:
    """g(k2), Section 3.3."""
    return (1 - alpha ** k2) / ((1 - alpha) * (1 - c + c * k2))


def best_strategy(budget: int, alpha1: float, c1: float, alpha2: float, c2: float, asynchronous: bool = True
                  ) -> Tuple[int, int, float]:
    """(k1, k2, h) maximising h = f(k1) * g(k2) under ParallelDim_f * ParallelDim_g <= budget (Eq. 1), where
    ParallelDim_g = k2 and ParallelDim_f = k1 (sync) or min(ceil(1 / c1), k1) (async).  Ties go to the smaller
    k1, then the smaller k2; k1 and k2 range over 1..budget."""
    best = (1, 1, -1.0)
    for k1 in range(1, budget + 1):
        dim_f = min(math.ceil(1 / c1), k1) if asynchronous else k1
        for k2 in range(1, budget + 1):
            if dim_f * k2 > budget:
                continue
            h = (f_async(k1, alpha1, c1) if asynchronous else f_sync(k1, alpha1, c1)) * f_token(k2, alpha2, c2)
            if h > best[2]:
                best = (k1, k2, h)
    return best
