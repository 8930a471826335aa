"""Pins for the step-level commit oracle."""
import numpy as np
import pytest

from lr_workloads import Model, build_batch, make_config, make_random_small
from oracle import lr_oracle as O

PAGE = 16


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def _token_list_model(batch, verdict, n_accept, r):
    """Independent list model on *tokens*: build the output token sequence of
    Algorithm 1 (accepted draft steps, then the decisive target step's kept tokens)
    as a list of (physical page, in-page offset) and derive everything from it."""
    s0, s1 = int(batch.req_span_off[r]), int(batch.req_span_off[r + 1])
    gamma = s1 - s0 - 1
    cu_v, cu_d = batch.cu_verdict, batch.cu_draft
    j_star = gamma
    for j in range(gamma):
        if not verdict[cu_v[r] + j]:
            j_star = j
            break

    def tokens(slot, n):
        return [(int(batch.page_ids[slot + t // PAGE]), t % PAGE) for t in range(n)]

    seq = tokens(int(batch.span_slot[s0]), int(batch.span_len[s0]))
    for c in range(1, j_star + 1):
        seq += tokens(int(batch.span_slot[s0 + c]), int(batch.span_len[s0 + c]))
    surv = -1
    for b in range(batch.n_branch):
        if batch.br_req[b] == r and batch.br_depth[b] == j_star:
            surv = b
            break
    if surv >= 0:
        L = int(cu_d[surv + 1] - cu_d[surv])
        seq += tokens(int(batch.br_own_slot[surv]), int(batch.br_own_len[surv]) - L + int(n_accept[surv]))
    keep = []
    for pg, _ in seq:
        if not keep or keep[-1][0] != pg:
            keep.append([pg, 0])
        keep[-1][1] += 1
    all_pages = []
    for c in range(gamma + 1):
        all_pages += [int(batch.page_ids[int(batch.span_slot[s0 + c]) + p]) for p in range((int(batch.span_len[s0 + c]) + 15) // 16)]
    for b in range(batch.n_branch):
        if batch.br_req[b] == r:
            all_pages += [int(batch.page_ids[int(batch.br_own_slot[b]) + p]) for p in range((int(batch.br_own_len[b]) + 15) // 16)]
    kept = {k[0] for k in keep}
    free = [p for p in all_pages if p not in kept]  # canonical order = table order of what is left
    return j_star, surv, len(seq), keep, free, all_pages


@pytest.mark.parametrize("seed", list(range(12)))
def test_commit_matches_the_token_list_model(seed):
    w = make_random_small(200 + seed)
    b_, t = w.batch, w.tensors
    rng = _rng(seed)
    n_accept = np.array([rng.integers(0, L + 1) for L in b_.br_n_draft], dtype=np.int32)
    c = O.commit(b_, t.verdict, n_accept)
    for r in range(b_.n_req):
        j_star, surv, length, keep, free, all_pages = _token_list_model(b_, t.verdict, n_accept, r)
        assert c["n_steps_accepted"][r] == j_star
        assert c["survivor"][r] == surv
        assert c["committed_len"][r] == length
        k0, k1 = c["keep_off"][r], c["keep_off"][r + 1]
        f0, f1 = c["free_off"][r], c["free_off"][r + 1]
        assert [list(x) for x in zip(c["keep_pages"][k0:k1], c["keep_valid"][k0:k1])] == keep
        assert list(c["free_pages"][f0:f1]) == free
        # partition: keep + free = every page slot of the request exactly once
        assert sorted(list(c["keep_pages"][k0:k1]) + list(c["free_pages"][f0:f1])) == sorted(all_pages)
        assert int(c["keep_valid"][k0:k1].sum()) == length


def _simple(gamma=3, L=4, P=40, seg=20):
    rng = _rng(0)
    model = Model(2, 1, 64, 16)
    req = {"P": P, "segs": [seg] * gamma, "branches": [(j, L, L, L) for j in range(0, gamma + 1)]}
    return build_batch(model, [req], rng, shuffle=False)


def test_all_accepted_first_rejected_and_later_ones_ignored():
    b_ = _simple()
    L = 4
    n_accept = np.array([1, 2, 3, 4], dtype=np.int32)
    c = O.commit(b_, np.array([1, 1, 1], dtype=np.uint8), n_accept)
    assert c["n_steps_accepted"][0] == 3 and c["survivor"][0] == 3
    assert c["committed_len"][0] == 40 + 3 * 20 + (L - L + 4)
    c = O.commit(b_, np.array([0, 1, 1], dtype=np.uint8), n_accept)
    assert c["n_steps_accepted"][0] == 0 and c["survivor"][0] == 0
    assert c["committed_len"][0] == 40 + 1
    c2 = O.commit(b_, np.array([0, 0, 0], dtype=np.uint8), n_accept)
    for key in c:
        assert np.array_equal(c[key], c2[key])  # verdicts after the first False change nothing
    c = O.commit(b_, np.array([1, 0, 1], dtype=np.uint8), n_accept)
    assert c["n_steps_accepted"][0] == 1 and c["survivor"][0] == 1
    assert c["committed_len"][0] == 40 + 20 + 2
    # pages: prefix 3 pages (16,16,8), segment 1: 2 pages (16,4), tail: 1 page with 2 valid tokens
    assert list(c["keep_valid"]) == [16, 16, 8, 16, 4, 2]
    assert list(c["keep_pages"]) == [0, 1, 2, 3, 4, 10]
    assert list(c["free_pages"]) == [5, 6, 7, 8, 9, 11, 12]


def test_no_branch_at_decisive_depth_keeps_only_the_chain():
    # benchmark indexing: branches have depth 1..gamma, so j* = 0 has no decisive branch in the pass
    w = make_config(1, with_logits=False, with_kv=False)
    b_ = w.batch
    c = O.commit(b_, np.array([0, 1], dtype=np.uint8), np.array([3, 3], dtype=np.int32))
    assert c["survivor"][0] == -1 and c["committed_len"][0] == 256
    assert len(c["keep_pages"]) == 16 and len(c["free_pages"]) == 2 * 2 + 2


def test_kept_tail_zero_frees_the_whole_tail():
    b_ = _simple(gamma=1, L=4)
    c = O.commit(b_, np.array([1], dtype=np.uint8), np.array([0, 0], dtype=np.int32))
    assert c["survivor"][0] == 1 and c["committed_len"][0] == 60
    assert list(c["free_pages"]) == [5, 6]


def test_mean_accepted_steps_follows_the_geometric_model():
    """E[j*] = a (1 - a^gamma) / (1 - a) for i.i.d. step verdicts with rate a (geometric run, capped)."""
    rng = _rng(7)
    gamma, R, a = 6, 3000, 0.6
    model = Model(1, 1, 64, 16)
    req = {"P": 1, "segs": [1] * gamma, "branches": [(0, 1, 1, 1)]}
    b_ = build_batch(model, [req] * R, rng, shuffle=False)
    verdict = (rng.random(R * gamma) < a).astype(np.uint8)
    c = O.commit(b_, verdict, np.zeros(R, dtype=np.int32))
    expect = a * (1 - a**gamma) / (1 - a)
    assert abs(c["n_steps_accepted"].mean() - expect) < 0.08
