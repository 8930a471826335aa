"""Asynchronous Lookahead Reasoning stages on one paged cache: every target generation is a verify pass of its own,
issued when the controller starts its position; results against the oracle per position, the schedule against the
oracle's event simulation, and the cache against a model without pages (a plain token array that grows by what each
stage commits)."""
import numpy as np
import pytest

from lr_workloads import Model, bf16_round, bf16_to_f32, build_batch, fill_logits_and_drafts
from oracle import lr_cycles as C
from oracle import lr_oracle as O
from paper_2506_19830_b200.async_cycle import AsyncCycleEngine, PositionInput
from paper_2506_19830_b200.cycle import BranchInput
from gpu_util import REL_LARGE, assert_attention_close

pytestmark = pytest.mark.gpu
PAGE = 16


def _tokens(rng, n, model):
    """n tokens of finite bf16 K and V bits, [n, H_kv, D]."""
    shape = (n, model.n_kv_heads, model.head_dim)
    return bf16_round(rng.standard_normal(shape).astype(np.float32)), bf16_round(rng.standard_normal(shape).astype(np.float32))


def _oracle_position(model, rng, seq_k, seq_v, segs, x: PositionInput):
    """The same pass on a cache built from scratch: the logical context, the draft steps before the position, its tail."""
    i = len(segs)
    spec = {"P": len(seq_k), "segs": [len(k) for k, _ in segs], "branches": [(i, len(x.branch.k_tail), x.branch.q_len, x.branch.n_draft)]}
    b = build_batch(model, [spec], rng)
    k = np.zeros((b.n_pool_pages, model.n_kv_heads, PAGE, model.head_dim), dtype=np.uint16)
    v = np.zeros_like(k)

    def put(slot, ks, vs):
        for t in range(len(ks)):
            pg = int(b.page_ids[slot + t // PAGE])
            k[pg, :, t % PAGE, :], v[pg, :, t % PAGE, :] = ks[t], vs[t]

    put(int(b.span_slot[0]), seq_k, seq_v)
    for c, (ks, vs) in enumerate(segs):
        put(int(b.span_slot[1 + c]), ks, vs)
    put(int(b.br_own_slot[0]), x.branch.k_tail, x.branch.v_tail)
    o_ref, _ = O.verify_attention(b, x.q, k, v)
    n_ref, bonus_ref, _ = O.accept_greedy(x.logits, x.draft_ids, b.cu_draft)
    return o_ref, int(n_ref[0]), int(bonus_ref[0])


@pytest.mark.parametrize("head_dim,gamma,num,den,alpha", [(128, 3, 1, 3, 0.7), (64, 2, 1, 4, 0.5), (128, 4, 2, 5, 0.8)])
def test_stages_follow_the_schedule_and_keep_the_cache_equal_to_the_logical_sequence(head_dim, gamma, num, den, alpha):
    rng = np.random.Generator(np.random.PCG64(1000 * gamma + head_dim))
    model = Model(8, 2, head_dim, 1000)
    eng = AsyncCycleEngine(model, 700, gamma, num, den)
    seq_k, seq_v = _tokens(rng, int(rng.choice([37, 130])), model)
    assert eng.add_request(seq_k, seq_v) == 0
    verdict_stream = []
    for stage in range(5):
        made = {}

        def source(i):
            L = int(rng.integers(1, 9))
            own = L + int(rng.choice([0, 1, 5]))
            tk, tv = _tokens(rng, own, model)
            sk, sv = _tokens(rng, int(rng.integers(3, 45)), model)
            fake = build_batch(model, [{"P": 0, "segs": [], "branches": [(0, own, L, L)]}], rng)  # row bookkeeping for the logits
            logits, drafts, _ = fill_logits_and_drafts(fake, rng, 0.3)
            q = bf16_round(rng.standard_normal((L, model.n_q_heads, model.head_dim)).astype(np.float32))
            x = PositionInput(sk, sv, BranchInput(i, tk, tv, L, L), q, logits, drafts, int(rng.random() < alpha))
            made[i] = x
            return x

        res = eng.run_stage(source)
        xr = res["rejected_at"]
        assert xr is not None
        verdict_stream += [1] * xr + [0]
        # every finished position: attention and acceptance against the oracle on the logical prefix
        segs = []
        for i in range(xr + 1):
            o_ref, n_ref, bonus_ref = _oracle_position(model, rng, seq_k, seq_v, segs, made[i])
            got = res["positions"][i]
            err = np.abs(bf16_to_f32(got["out"]).astype(np.float64) - o_ref)
            assert_attention_close(err, o_ref, REL_LARGE)
            assert (got["n_accept"], got["bonus_id"]) == (n_ref, bonus_ref), (stage, i)
            segs.append((made[i].seg_k, made[i].seg_v))
        # the stage's output: drafts 0..xr-1 and the kept part of the target's step at xr
        keep_tail = len(made[xr].branch.k_tail) - made[xr].branch.n_draft + res["positions"][xr]["n_accept"]
        for i in range(xr):
            seq_k, seq_v = np.concatenate([seq_k, made[i].seg_k]), np.concatenate([seq_v, made[i].seg_v])
        seq_k = np.concatenate([seq_k, made[xr].branch.k_tail[:keep_tail]])
        seq_v = np.concatenate([seq_v, made[xr].branch.v_tail[:keep_tail]])
        assert res["n_steps_accepted"] == xr and res["committed_len"] == len(seq_k)
        gk, gv = eng.sequence(0)
        assert eng.length[0] == len(seq_k) and np.array_equal(gk, seq_k) and np.array_equal(gv, seq_v), stage
        assert sorted(eng.pages[0] + eng.free) == list(range(700))  # every page owned once or free once
    ref = C.simulate_async(gamma, num, den, verdict_stream)
    for key in ("stages", "steps", "time", "verdicts_used"):
        assert eng.controller.stats[key] == ref[key], key
    assert ref["peak_in_flight"] <= eng.controller.stats["peak_in_flight"] <= gamma
