"""Pins for the greedy-acceptance oracle."""
import itertools

import numpy as np
import pytest

from lr_workloads import Model, bf16_round, bf16_to_f32, build_batch, fill_logits_and_drafts, make_config, make_random_small
from oracle import lr_oracle as O


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def _py_first_max(row_f32):
    """First strict maximum by a plain left-to-right scan (NaN ranks as -inf)."""
    best, best_i = None, 0
    for i, x in enumerate(row_f32):
        x = float(x)
        if x != x:
            x = float("-inf")
        if best is None or x > best:
            best, best_i = x, i
    return best_i


def test_row_argmax_matches_a_plain_scan_with_natural_ties():
    rng = _rng(1)
    # coarse values -> many natural ties at the maximum
    x = np.round(rng.standard_normal((40, 997)).astype(np.float32) * 2) / 2
    bits = bf16_round(x)
    got = O.row_argmax(bits)
    for r in range(bits.shape[0]):
        assert got[r] == _py_first_max(bf16_to_f32(bits[r]))
    # ties exist in this data
    assert any((bf16_to_f32(bits[r]) == bf16_to_f32(bits[r]).max()).sum() > 1 for r in range(40))


@pytest.mark.parametrize("positions", [(0, 5), (7, 8), (15, 16), (255, 256), (1022, 1023), (3, 1023), (0, 1023)])
def test_constructed_ties_pick_the_lowest_index(positions):
    x = np.zeros((1, 1024), dtype=np.float32) - 1.0
    for p in positions:
        x[0, p] = 3.0
    assert O.row_argmax(bf16_round(x))[0] == positions[0]


def test_signed_zero_nan_and_inf_rules():
    x = np.full((5, 16), -0.0, dtype=np.float32)
    x[0, 9] = 0.0  # +0 == -0: index 0 still wins
    x[1, :] = np.nan  # all NaN -> 0
    x[2, :] = np.nan
    x[2, 11] = -np.inf  # NaN ranks as -inf: tie with a real -inf resolved by index
    x[3, :] = -np.inf
    x[3, 4] = np.nan
    x[4, 3] = np.inf
    x[4, 2] = np.nan
    bits = bf16_round(x)
    bits[0, 0] = 0x8000  # make sure -0 survived the rounding helper
    assert list(O.row_argmax(bits)) == [0, 0, 0, 0, 3]


def _one_branch_logits(L, V, targets):
    x = np.zeros((L + 1, V), dtype=np.float32)
    for i, t in enumerate(targets):
        x[i, t] = 5.0
    return bf16_round(x)


def test_all_match_gives_L_plus_one_and_first_mismatch_gives_zero():
    L, V = 6, 50
    targets = [3, 9, 9, 41, 0, 49, 17]
    logits = _one_branch_logits(L, V, targets)
    cu = np.array([0, L], dtype=np.int32)
    n, bonus, _ = O.accept_greedy(logits, np.array(targets[:L], dtype=np.int32), cu)
    assert n[0] == L and n[0] + 1 == L + 1 and bonus[0] == targets[L]
    drafts = np.array(targets[:L], dtype=np.int32)
    drafts[0] = 4
    n, bonus, _ = O.accept_greedy(logits, drafts, cu)
    assert n[0] == 0 and bonus[0] == targets[0]


@pytest.mark.parametrize("L", [1, 2, 3, 4])
def test_every_match_pattern(L):
    """All 2^L match/mismatch patterns: n = number of leading matches; later matches are ignored."""
    V = 11
    targets = list(range(1, L + 2))
    logits = _one_branch_logits(L, V, targets)
    cu = np.array([0, L], dtype=np.int32)
    for pattern in itertools.product([True, False], repeat=L):
        drafts = np.array([targets[i] if pattern[i] else 0 for i in range(L)], dtype=np.int32)
        n, bonus, _ = O.accept_greedy(logits, drafts, cu)
        lead = 0
        for ok in pattern:
            if not ok:
                break
            lead += 1
        assert n[0] == lead
        assert bonus[0] == targets[lead]


def test_out_of_range_draft_never_matches():
    logits = _one_branch_logits(2, 8, [0, 1, 2])
    cu = np.array([0, 2], dtype=np.int32)
    for bad in (-1, 8, 2**31 - 1):
        n, bonus, _ = O.accept_greedy(logits, np.array([bad, 1], dtype=np.int32), cu)
        assert n[0] == 0 and bonus[0] == 0


def test_several_branches_use_their_own_rows():
    # branch 0: L=2 rows 0..2 ; branch 1: L=1 rows 3..4 ; branch 2: L=3 rows 5..8
    targets = [[4, 5, 6], [7, 8], [1, 2, 3, 9]]
    rows = [t for br in targets for t in br]
    logits = _one_branch_logits(len(rows) - 1, 16, rows)
    cu = np.array([0, 2, 3, 6], dtype=np.int32)
    drafts = np.array([4, 5, 0, 1, 2, 0], dtype=np.int32)
    n, bonus, _ = O.accept_greedy(logits, drafts, cu)
    assert list(n) == [2, 0, 2] and list(bonus) == [6, 7, 3]


def test_generator_match_lengths_are_recovered():
    """The generator plants peaks so that branch b matches exactly match_len[b] drafts."""
    for seed in range(6):
        w = make_random_small(100 + seed)
        n, _, _ = O.accept_greedy(w.tensors.logits, w.tensors.draft_ids, w.batch.cu_draft)
        assert np.array_equal(n, w.tensors.match_len)
    w = make_config(1)
    n, _, _ = O.accept_greedy(w.tensors.logits, w.tensors.draft_ids, w.batch.cu_draft)
    assert np.array_equal(n, w.tensors.match_len)


def test_mean_emitted_tokens_follows_the_geometric_model():
    """E[n+1] = (1 - a^(L+1)) / (1 - a) for per-token acceptance rate a (Background, g(gamma) numerator)."""
    rng = _rng(2024)
    L, V, B = 8, 64, 12000
    p = 0.3
    model = Model(1, 1, 64, V)
    batch = build_batch(model, [{"P": 0, "segs": [], "branches": [(0, L, L, L)] * B}], rng)
    logits, drafts, m = fill_logits_and_drafts(batch, rng, p, p_decoy=0.25, p_tie=0.25)
    n, _, _ = O.accept_greedy(logits, drafts, batch.cu_draft)
    a = 1 - p
    expect = (1 - a ** (L + 1)) / (1 - a)
    # the mismatch row's random draft hits the background argmax with probability 1/V, which
    # lengthens a run slightly; allow for it plus sampling noise
    assert abs((n + 1).mean() - expect) < 0.08
