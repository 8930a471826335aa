"""Pins for the oracle's stochastic acceptance (rejection sampling for point-mass drafts).

The pins do not retype the oracle's arithmetic: a hand-computed example, the exactness theorem of
speculative sampling checked by integrating over the random inputs, the greedy limit (which must agree
with the separately pinned greedy acceptance), scipy's softmax, and structural invariants.
"""
import numpy as np
import pytest

from lr_workloads import bf16_round
from oracle import lr_oracle as O


def _bits(x):
    return bf16_round(np.asarray(x, dtype=np.float32))


def test_hand_computed_example():
    # logits ln(1), ln(2), ln(3), ln(2) at T = 1 would give P = (1, 2, 3, 2) / 8; bf16 rounds ln 3 and ln 2,
    # so use exact powers of two: logits 0, 1, 2, 1 (base-e) are not dyadic either -- take T = 1/ln 2 with
    # logits 0, 1, 2, 1: P = 2^x / sum = (1, 2, 4, 2) / 9.
    T = 1.0 / np.log(2.0)
    rows = _bits([[0, 1, 2, 1], [0, 1, 2, 1], [2, 1, 0, 1]])
    cu = np.array([0, 2], dtype=np.int32)
    drafts = np.array([2, 1], dtype=np.int32)  # P_0(2) = 4/9, P_1(1) = 2/9
    # accept first (u < 4/9), reject second (u >= 2/9): residual of row 1 = (1, 0, 4, 2)/7; u_final = 0.5 -> cum (1, 1, 5, 7)/7, 3.5 -> index 2
    n, f, p = O.accept_sample(rows, drafts, cu, T, np.array([0.4, 0.3]), np.array([0.5]))
    assert (n[0], f[0]) == (1, 2)
    assert p == pytest.approx([4 / 9, 2 / 9], rel=1e-12)
    # both accepted: final from row 2, P = (4, 2, 1, 2)/9, u_final = 0.7 -> 6.3 -> cum 4, 6, 7, 9 -> index 2
    n, f, _ = O.accept_sample(rows, drafts, cu, T, np.array([0.4, 0.2]), np.array([0.7]))
    assert (n[0], f[0]) == (2, 2)
    # first rejected: later uniforms are irrelevant; residual of row 0 = (1, 2, 0, 2)/5, u_final = 0.1 -> 0.5 -> index 0
    n, f, _ = O.accept_sample(rows, drafts, cu, T, np.array([0.45, 0.0]), np.array([0.1]))
    assert (n[0], f[0]) == (0, 0)
    # the resampled token is never the rejected one
    for u in np.linspace(0, 0.999, 50):
        n, f, _ = O.accept_sample(rows, drafts, cu, T, np.array([0.99, 0.0]), np.array([u]))
        assert n[0] == 0 and f[0] != 2


def test_probabilities_agree_with_scipy_softmax():
    from scipy.special import softmax

    rng = np.random.default_rng(1)
    bits = _bits(rng.standard_normal(300) * 3)
    x = O.bf16_bits_to_f64(bits)
    for T in (0.6, 1.0, 2.5):
        assert O.target_probs(bits, T) == pytest.approx(softmax(x / T), rel=1e-12)


def test_output_distribution_equals_the_target_distribution():
    """Exactness of speculative sampling: with one draft, whatever the drafted token, the emitted token
    (the draft if accepted, else the resampled one) is distributed exactly as P.  Integrated over a fine
    grid of (u_accept, u_final)."""
    rng = np.random.default_rng(2)
    V, T = 6, 0.8
    rows = _bits(rng.standard_normal((2, V)) * 1.5)
    P = O.target_probs(rows[0], T)
    cu = np.array([0, 1], dtype=np.int32)
    G = 400
    grid = (np.arange(G) + 0.5) / G
    for d in (0, 3, 5):
        counts = np.zeros(V)
        for ua in grid:
            # for a fixed u_accept the decision is one of two; integrate u_final on the grid only when rejected
            n, f, _ = O.accept_sample(rows, np.array([d], dtype=np.int32), cu, T, np.array([ua]), np.array([0.0]))
            if n[0] == 1:
                counts[d] += 1.0
            else:
                for uf in grid:
                    _, f, _ = O.accept_sample(rows, np.array([d], dtype=np.int32), cu, T, np.array([ua]), np.array([uf]))
                    counts[f[0]] += 1.0 / G
        assert counts / G == pytest.approx(P, abs=3.0 / G)


def test_greedy_limit_agrees_with_greedy_acceptance():
    """T -> 0: P concentrates on the argmax, so a draft is accepted iff it is the argmax and the final
    token is the argmax of the stop row -- the separately pinned greedy rule (rows without ties)."""
    rng = np.random.default_rng(3)
    V, B, L = 64, 6, 5
    x = rng.permuted(np.tile(np.arange(V, dtype=np.float32) / 4.0, (B * (L + 1), 1)), axis=1)  # distinct values per row
    bits = _bits(x)
    cu = np.arange(0, B * L + 1, L, dtype=np.int32)
    arg = O.row_argmax(bits)
    drafts = np.concatenate([arg[b * (L + 1) : b * (L + 1) + L] for b in range(B)]).astype(np.int32)
    for b in range(B):  # plant a mismatch at position b (branch 5: none)
        if b < L:
            drafts[b * L + b] = (drafts[b * L + b] + 1) % V
    ng, bg, _ = O.accept_greedy(bits, drafts, cu)
    ns, fs, _ = O.accept_sample(bits, drafts, cu, 0.01, rng.uniform(0.01, 0.99, B * L), rng.uniform(0.0, 0.99, B))
    assert np.array_equal(ns, ng) and np.array_equal(fs, bg)


def test_structural_invariants():
    rng = np.random.default_rng(4)
    V, B, L = 50, 8, 4
    bits = _bits(rng.standard_normal((B * (L + 1), V)))
    cu = np.arange(0, B * L + 1, L, dtype=np.int32)
    drafts = rng.integers(0, V, B * L).astype(np.int32)
    drafts[3] = -1
    drafts[7] = V  # outside the vocabulary: probability 0, always rejected
    uf = rng.uniform(0, 1, B)
    n0, _, p = O.accept_sample(bits, drafts, cu, 0.7, np.zeros(B * L), uf)
    assert n0[0] == 3 and n0[1] == 3 and all(n0[2:] == L)  # u = 0 accepts everything with P > 0
    assert p[3] == 0.0 and p[7] == 0.0
    n1, f1, _ = O.accept_sample(bits, drafts, cu, 0.7, np.full(B * L, 0.999999), uf)
    assert all(n1 == 0)  # u ~ 1 rejects everything
    assert all(f1[b] != drafts[b * L] for b in range(B))
    # only the uniforms up to the first rejection matter
    ua = rng.uniform(0, 1, B * L)
    n, f, _ = O.accept_sample(bits, drafts, cu, 0.7, ua, uf)
    ub = ua.copy()
    for b in range(B):
        ub[b * L + n[b] + 1 : (b + 1) * L] = rng.uniform(0, 1, max(0, L - n[b] - 1))
    n2, f2, _ = O.accept_sample(bits, drafts, cu, 0.7, ub, uf)
    assert np.array_equal(n, n2) and np.array_equal(f, f2)
    assert all(0 <= n[b] <= L for b in range(B)) and all(0 <= f[b] < V for b in range(B))


# ---- the sampling filters (top_k, top_p) ---------------------------------------------------------------
def test_filter_hand_computed_examples():
    P = np.array([1 / 16, 1 / 2, 1 / 8, 1 / 4, 1 / 16])  # ranking: 1, 3, 2, then 0 before 4 (equal: lower index first)
    # top_p = 0.8: ranks 0, 1, 2 have 0, 1/2, 3/4 ahead of them (< 0.8), rank 3 has 7/8: three tokens stay
    assert O.filter_probs(P, 0, 0.8) == pytest.approx([0, 4 / 7, 1 / 7, 2 / 7, 0], abs=1e-15)
    # exactly at a step: the tokens before rank 2 hold 3/4, which is not less than 3/4
    assert O.filter_probs(P, 0, 0.75) == pytest.approx([0, 2 / 3, 0, 1 / 3, 0], abs=1e-15)
    # top_k = 4 cuts between the two equal tokens: the lower index stays
    assert O.filter_probs(P, 4, 1.0) == pytest.approx([1 / 15, 8 / 15, 2 / 15, 4 / 15, 0], abs=1e-15)
    # both: after top_k = 2 the masses are 2/3, 1/3; top_p = 0.6 keeps only the first
    assert O.filter_probs(P, 2, 0.6) == pytest.approx([0, 1, 0, 0, 0], abs=1e-15)
    # no filter
    assert np.array_equal(O.filter_probs(P, 0, 1.0), P)


def test_filter_is_the_smallest_leading_set_that_reaches_top_p():
    """Declarative check by brute force over sorted prefixes (independent of how the oracle walks the ranking)."""
    rng = np.random.default_rng(5)
    for trial in range(200):
        V = int(rng.integers(2, 40))
        P = rng.dirichlet(np.full(V, rng.choice([0.05, 0.3, 2.0])))
        if trial % 3 == 0:  # ties
            P = np.round(P * 16) + 1
            P = P / P.sum()
        k = int(rng.integers(0, V + 2))
        p = float(rng.choice([0.3, 0.6, 0.9, 0.95, 0.999, 1.0]))
        F = O.filter_probs(P, k, p)
        kept = np.flatnonzero(F > 0)
        ranked = sorted(range(V), key=lambda v: (-P[v], v))
        n_k = min(k, V) if k > 0 else V
        top = ranked[:n_k]
        mass_k = sum(P[v] for v in top)
        # smallest n with mass(first n) >= p * mass_k (all of them if none reaches it)
        n_p = n_k
        acc = 0.0
        for n, v in enumerate(top, start=1):
            acc += P[v]
            if p < 1.0 and acc / mass_k >= p - 1e-15:
                n_p = n
                break
        expect = sorted(top[:n_p])
        if abs(sum(P[v] for v in top[:n_p - 1]) / mass_k - p) < 1e-12 or abs(acc / mass_k - p) < 1e-12:
            continue  # a prefix mass within rounding of top_p: either side is a valid reading
        assert list(kept) == expect, (trial, k, p)
        assert F[kept] == pytest.approx(P[kept] / P[kept].sum(), rel=1e-12)  # renormalised, proportions unchanged


def test_top_k_one_is_the_greedy_rule():
    rng = np.random.default_rng(6)
    V, L = 50, 5
    rows = _bits(np.round(rng.standard_normal((L + 1, V)) * 2) / 2)  # coarse values: ties at the maximum happen
    arg = O.row_argmax(rows)
    cu = np.array([0, L], dtype=np.int32)
    for trial in range(30):
        drafts = arg[:L].astype(np.int32).copy()
        miss = int(rng.integers(0, L + 1))
        if miss < L:
            drafts[miss] = (drafts[miss] + 1 + int(rng.integers(0, V - 1))) % V
        ua, uf = rng.uniform(0, 0.999, L), rng.uniform(0, 1, 1)
        n, f, p = O.accept_sample(rows, drafts, cu, 0.7, ua, uf, top_k=1)
        n_ref, bonus_ref, _ = O.accept_greedy(rows, drafts, cu)
        assert (n[0], f[0]) == (n_ref[0], bonus_ref[0])


def test_filtered_output_distribution_equals_the_filtered_target():
    """Exactness of speculative sampling with the filters on: the emitted token is distributed as the filtered P."""
    rng = np.random.default_rng(7)
    V, T = 7, 0.8
    rows = _bits(rng.standard_normal((2, V)) * 1.5)
    F = O.filter_probs(O.target_probs(rows[0], T), 5, 0.9)
    assert 1 < (F > 0).sum() < V
    cu = np.array([0, 1], dtype=np.int32)
    n_grid = 2000
    us = (np.arange(n_grid) + 0.5) / n_grid
    kw = dict(top_k=5, top_p=0.9)
    for d in range(V):
        dd = np.array([d], dtype=np.int32)
        # the acceptance decision depends on u_accept alone, the resampled token on u_final alone
        acc = np.mean([O.accept_sample(rows, dd, cu, T, np.array([ua]), np.array([0.5]), **kw)[0][0] for ua in us])
        hist = np.zeros(V)
        for uf in us:
            n, f, _ = O.accept_sample(rows, dd, cu, T, np.array([1.0]), np.array([uf]), **kw)
            assert n[0] == 0
            hist[f[0]] += 1
        emitted = (1 - acc) * hist / n_grid
        emitted[d] += acc
        assert emitted == pytest.approx(F, abs=2e-3), d
