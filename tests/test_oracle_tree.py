"""Pins of the oracle's multi-branch (tree) drafting readings (Section 3, "Multi-Branch Drafting"): which draft
steps a branch sees, and which steps the commit walks through.  None of the checks re-uses the oracle's own walk."""
import dataclasses

import numpy as np
import pytest
import torch

from lr_workloads import Model, bf16_round, bf16_to_f32, build_batch, fill_kv, fill_q, make_random_small, make_random_tree
from lr_workloads.gen import _tree_request
from oracle import lr_oracle as O

PAGE = 16


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def _as_tree(batch):
    """The same chain, written with explicit parents."""
    parent = np.concatenate([np.arange(-1, batch.req_span_off[r + 1] - batch.req_span_off[r] - 1, dtype=np.int32)
                             for r in range(batch.n_req)])
    return dataclasses.replace(batch, seg_parent=parent)


def _ancestor_matrix(batch, r):
    """anc[a, c]: segment a lies on the way from the prefix to segment c (or is c).  By transitive closure of the
    parent relation with matrix powers -- not by walking up."""
    s0, s1 = int(batch.req_span_off[r]), int(batch.req_span_off[r + 1])
    n = s1 - s0
    step = np.eye(n, dtype=np.int64)
    for c in range(1, n):
        step[int(batch.seg_parent[s0 + c]), c] = 1
    reach = np.linalg.matrix_power(step, max(1, n))
    return reach > 0


def _tokens(batch, slot, n):
    return [(int(batch.page_ids[slot + t // PAGE]), t % PAGE) for t in range(n)]


# (i) a chain written as a tree is the chain -------------------------------------------------------
@pytest.mark.parametrize("seed", [1, 2, 3, 4])
def test_chain_written_with_parents_gives_the_chain_results(seed):
    w = make_random_small(seed)
    b, t = w.batch, w.tensors
    bt = _as_tree(b)
    o0, l0 = O.verify_attention(b, t.q, t.k_pool, t.v_pool)
    o1, l1 = O.verify_attention(bt, t.q, t.k_pool, t.v_pool)
    assert np.array_equal(o0, o1) and np.array_equal(l0, l1)
    n_acc = _rng(seed).integers(0, b.br_n_draft + 1).astype(np.int32)
    c0, c1 = O.commit(b, t.verdict, n_acc), O.commit(bt, t.verdict, n_acc)
    for k in c0:
        assert np.array_equal(c0[k], c1[k]), k


# (ii) every branch is plain causal attention over prefix + its ancestors + its tail ------------------
@pytest.mark.parametrize("seed", range(8))
def test_each_branch_is_causal_attention_over_its_ancestor_sequence(seed):
    w = make_random_tree(seed)
    b_, t = w.batch, w.tensors
    out, _ = O.verify_attention(b_, t.q, t.k_pool, t.v_pool)
    G, m = b_.model.group, b_.model
    qf = torch.from_numpy(bf16_to_f32(t.q).astype(np.float64))
    for b in range(b_.n_branch):
        r = int(b_.br_req[b])
        s0 = int(b_.req_span_off[r])
        anc = _ancestor_matrix(b_, r)
        node = int(b_.br_depth[b])
        seen = [c for c in range(anc.shape[0]) if anc[c, node]]  # ascending index = sequence order (parent < child)
        toks = []
        for c in seen:
            toks += _tokens(b_, int(b_.span_slot[s0 + c]), int(b_.span_len[s0 + c]))
        toks += _tokens(b_, int(b_.br_own_slot[b]), int(b_.br_own_len[b]))
        K = np.stack([bf16_to_f32(t.k_pool[p, :, o, :]).astype(np.float64) for p, o in toks])
        V = np.stack([bf16_to_f32(t.v_pool[p, :, o, :]).astype(np.float64) for p, o in toks])
        n = len(toks)
        r0, r1 = int(b_.cu_q[b]), int(b_.cu_q[b + 1])
        q_len = r1 - r0
        Qfull = torch.zeros(n, m.n_q_heads, m.head_dim, dtype=torch.float64)
        Qfull[n - q_len:] = qf[r0:r1]
        Kt = torch.from_numpy(K).repeat_interleave(G, dim=1)
        Vt = torch.from_numpy(V).repeat_interleave(G, dim=1)
        ref = torch.nn.functional.scaled_dot_product_attention(
            Qfull.permute(1, 0, 2)[None], Kt.permute(1, 0, 2)[None], Vt.permute(1, 0, 2)[None], is_causal=True
        )[0].permute(1, 0, 2)[n - q_len:]
        np.testing.assert_allclose(out[r0:r1], ref.numpy(), rtol=1e-9, atol=1e-11)


# (iii) closed form with hand-written visible sets: siblings and cousins contribute exactly nothing ------------
HAND = {"P": 19, "segs": [5, 17, 3, 9, 4], "parents": [0, 0, 1, 1, 3],
        "branches": [(0, 4, 2, 2), (2, 3, 3, 3), (3, 6, 2, 2), (4, 1, 1, 1), (5, 2, 2, 2), (5, 5, 1, 1)]}
HAND_SEEN = {0: [0], 2: [0, 2], 3: [0, 1, 3], 4: [0, 1, 4], 5: [0, 1, 3, 5]}  # by node: spans seen (0 = prefix)


def test_span_indicator_values_give_the_share_of_each_seen_span_and_zero_elsewhere():
    rng = _rng(5)
    model = Model(4, 2, 64, 32)
    batch = build_batch(model, [HAND], rng)
    k, v = fill_kv(batch, rng)
    q = fill_q(batch, rng)
    kc = bf16_round(np.full(k.shape, 0.5, dtype=np.float32))  # equal keys: uniform weights over what is seen
    vf = np.zeros(v.shape, dtype=np.float32)
    for s in range(batch.n_span):
        for p in range((int(batch.span_len[s]) + PAGE - 1) // PAGE):
            vf[batch.page_ids[int(batch.span_slot[s]) + p], :, :, s] = 1.0
    for b in range(batch.n_branch):
        for p in range((int(batch.br_own_len[b]) + PAGE - 1) // PAGE):
            vf[batch.page_ids[int(batch.br_own_slot[b]) + p], :, :, batch.n_span + b] = 1.0
    out, _ = O.verify_attention(batch, q, kc, bf16_round(vf))
    for b in range(batch.n_branch):
        seen = HAND_SEEN[int(batch.br_depth[b])]
        q_len = int(batch.cu_q[b + 1] - batch.cu_q[b])
        for i in range(q_len):
            tail_vis = int(batch.br_own_len[b]) - q_len + i + 1
            n_vis = sum(int(batch.span_len[c]) for c in seen) + tail_vis
            expect = np.zeros(model.head_dim)
            for c in seen:
                expect[c] = int(batch.span_len[c]) / n_vis
            expect[batch.n_span + b] = tail_vis / n_vis
            row = int(batch.cu_q[b]) + i
            for h in range(model.n_q_heads):
                np.testing.assert_allclose(out[row, h], expect, rtol=0, atol=1e-13)
                assert (out[row, h, expect == 0.0] == 0.0).all()


# (iv) commit: a worked example --------------------------------------------------------------------------------
def _worked_batch():
    req = {"P": 20, "segs": [5, 17, 3, 16, 2], "parents": [0, 0, 2, 2, 4],
           "branches": [(0, 4, 4, 4), (2, 3, 3, 3), (4, 20, 3, 3), (4, 2, 2, 2), (5, 1, 1, 1), (1, 2, 2, 2)]}
    # page slots, in order: prefix 0 1 | steps: 2 | 3 4 | 5 | 6 | 7 | tails: 8 | 9 | 10 11 | 12 | 13 | 14
    return build_batch(Model(4, 1, 64, 64), [req], _rng(0), shuffle=False)


def test_worked_example_first_agreeing_child_at_every_level():
    b = _worked_batch()
    n_acc = np.array([0, 0, 1, 0, 0, 0], dtype=np.int32)
    c = O.commit(b, np.array([0, 1, 0, 1, 0], dtype=np.uint8), n_acc)
    # prefix -> step 2 (step 1 disagrees) -> step 4 (step 3 disagrees) -> stop (step 5 disagrees)
    assert c["n_steps_accepted"].tolist() == [2] and c["survivor"].tolist() == [2]
    assert c["committed_len"].tolist() == [20 + 17 + 16 + (20 - 3 + 1)]
    assert c["keep_pages"].tolist() == [0, 1, 3, 4, 6, 10, 11] and c["keep_valid"].tolist() == [16, 4, 16, 1, 16, 16, 2]
    assert c["free_pages"].tolist() == [2, 5, 7, 8, 9, 12, 13, 14]
    assert c["keep_off"].tolist() == [0, 7] and c["free_off"].tolist() == [0, 8]


def test_worked_example_lowest_numbered_agreeing_sibling_wins_and_a_leaf_ends_the_walk():
    b = _worked_batch()
    c = O.commit(b, np.ones(5, dtype=np.uint8), np.zeros(6, dtype=np.int32))
    # steps 1 and 2 both agree: step 1 is taken, it has no children
    assert c["n_steps_accepted"].tolist() == [1] and c["survivor"].tolist() == [5]
    assert c["committed_len"].tolist() == [25]
    assert c["keep_pages"].tolist() == [0, 1, 2] and c["keep_valid"].tolist() == [16, 4, 5]
    assert c["free_pages"].tolist() == [3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13, 14]


# (v) commit against a declarative model, token by token ---------------------------------------------------------
def _alive(batch, r, verdict):
    """Steps the commit walks through, without walking: a step is alive iff it agrees, what it continues is alive
    (the prefix always is) and no lower-numbered step continuing the same thing agrees."""
    s0, s1 = int(batch.req_span_off[r]), int(batch.req_span_off[r + 1])
    v0 = int(batch.cu_verdict[r])
    alive = {0}
    for c in range(1, s1 - s0):  # parents come first, so one pass settles it
        par = int(batch.seg_parent[s0 + c])
        rivals = [x for x in range(1, c) if int(batch.seg_parent[s0 + x]) == par and verdict[v0 + x - 1]]
        if verdict[v0 + c - 1] and par in alive and not rivals:
            alive.add(c)
    return sorted(alive)


@pytest.mark.parametrize("seed", range(12))
def test_commit_lists_hold_exactly_the_walked_sequence(seed):
    w = make_random_tree(100 + seed)
    b, t = w.batch, w.tensors
    n_acc = _rng(seed).integers(0, b.br_n_draft + 1).astype(np.int32)
    c = O.commit(b, t.verdict, n_acc)
    for r in range(b.n_req):
        s0 = int(b.req_span_off[r])
        alive = _alive(b, r, t.verdict)
        assert c["n_steps_accepted"][r] == len(alive) - 1
        at = [x for x in range(b.n_branch) if b.br_req[x] == r and b.br_depth[x] == alive[-1]]
        assert c["survivor"][r] == (at[0] if at else -1)
        seq = []
        for s in alive:
            seq += _tokens(b, int(b.span_slot[s0 + s]), int(b.span_len[s0 + s]))
        if at:
            seq += _tokens(b, int(b.br_own_slot[at[0]]), int(b.br_own_len[at[0]] - b.br_n_draft[at[0]] + n_acc[at[0]]))
        kept = []
        for i in range(c["keep_off"][r], c["keep_off"][r + 1]):
            kept += [(int(c["keep_pages"][i]), o) for o in range(int(c["keep_valid"][i]))]
        assert kept == seq and c["committed_len"][r] == len(seq)
        # keep and free together are every page slot of the request, once
        mine = []
        for s in range(s0, int(b.req_span_off[r + 1])):
            mine += [int(b.page_ids[int(b.span_slot[s]) + p]) for p in range((int(b.span_len[s]) + PAGE - 1) // PAGE)]
        for x in range(b.n_branch):
            if b.br_req[x] == r:
                mine += [int(b.page_ids[int(b.br_own_slot[x]) + p]) for p in range((int(b.br_own_len[x]) + PAGE - 1) // PAGE)]
        both = list(c["keep_pages"][c["keep_off"][r]:c["keep_off"][r + 1]]) + list(c["free_pages"][c["free_off"][r]:c["free_off"][r + 1]])
        assert sorted(both) == sorted(mine) and len(set(both)) == len(both)


@pytest.mark.parametrize("seed", range(6))
def test_verdicts_off_the_walk_change_nothing(seed):
    w = make_random_tree(200 + seed)
    b, t = w.batch, w.tensors
    n_acc = np.zeros(b.n_branch, dtype=np.int32)
    ref = O.commit(b, t.verdict, n_acc)
    v = t.verdict.copy()
    for r in range(b.n_req):
        s0, s1 = int(b.req_span_off[r]), int(b.req_span_off[r + 1])
        alive = set(_alive(b, r, t.verdict))
        for c in range(1, s1 - s0):
            par = int(b.seg_parent[s0 + c])
            later_sibling_of_alive = any(x in alive and x < c and int(b.seg_parent[s0 + x]) == par for x in range(1, c))
            if par not in alive or later_sibling_of_alive:
                v[int(b.cu_verdict[r]) + c - 1] ^= 1
    got = O.commit(b, v, n_acc)
    for k in ref:
        assert np.array_equal(ref[k], got[k]), k


# (vi) accepted steps per cycle with W candidates per position ------------------------------------------------------
@pytest.mark.parametrize("W,gamma,p", [(1, 4, 0.6), (2, 3, 0.5), (4, 2, 0.3)])
def test_mean_accepted_steps_follows_the_any_of_w_acceptance_rate(W, gamma, p):
    # one position is passed iff any of its W candidates agrees: a = 1 - (1 - p)^W; the walk is then the chain's
    # with step acceptance a: E[j*] = a (1 - a^gamma) / (1 - a)
    R = 3000
    rng = _rng(7 * W + gamma)
    req = _tree_request(1, W, gamma, lambda i: 1, 1)
    req["branches"] = [(0, 1, 1, 1)]
    b = build_batch(Model(1, 1, 64, 8), [dict(req) for _ in range(R)], rng, shuffle=False)
    verdict = (rng.random(int(b.cu_verdict[-1])) < p).astype(np.uint8)
    c = O.commit(b, verdict, np.zeros(b.n_branch, dtype=np.int32))
    a = 1 - (1 - p) ** W
    mean = a * (1 - a ** gamma) / (1 - a)
    sd = gamma / 2  # a bound on the standard deviation of a variable in [0, gamma]
    assert abs(c["n_steps_accepted"].mean() - mean) < 4 * sd / np.sqrt(R)


# (vii) the pins notice a wrong visibility rule ---------------------------------------------------------------------
@pytest.mark.parametrize("wrong", ["chain", "no_self"])
def test_visibility_pins_catch_planted_mistakes(monkeypatch, wrong):
    right = O.node_path
    if wrong == "chain":  # every earlier-numbered step, as if the steps were nested
        monkeypatch.setattr(O, "node_path", lambda batch, r, node: list(range(1, node + 1)))
    else:  # the node's own step left out
        monkeypatch.setattr(O, "node_path", lambda batch, r, node: right(batch, r, node)[:-1])
    with pytest.raises(AssertionError):
        test_span_indicator_values_give_the_share_of_each_seen_span_and_zero_elsewhere()
    with pytest.raises(AssertionError):
        for seed in range(8):
            test_each_branch_is_causal_attention_over_its_ancestor_sequence(seed)
