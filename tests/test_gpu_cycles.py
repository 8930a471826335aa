"""Several synchronous cycles in a row on one paged cache (verify -> commit -> compact -> next cycle), against a
model without pages: per request a plain token array that grows by what the oracle's pass commits."""
import numpy as np
import pytest

from lr_workloads import Model, bf16_to_f32, build_batch, fill_kv, fill_logits_and_drafts, fill_q, fill_verdicts
from oracle import lr_oracle as O
from paper_2506_19830_b200.cycle import BranchInput, PagedCycleEngine, RequestInput
from gpu_util import REL_LARGE, assert_attention_close

pytestmark = pytest.mark.gpu
PAGE = 16


def _span_tokens(batch, pool, slot, n):
    pg = np.array([batch.page_ids[slot + t // PAGE] for t in range(n)], dtype=np.int64)
    return pool[pg, :, np.arange(n) % PAGE, :] if n else np.zeros((0,) + pool.shape[1:2] + pool.shape[3:], dtype=pool.dtype)


@pytest.mark.parametrize("head_dim,tree", [(128, False), (64, False), (128, True)])
def test_cycles_keep_the_cache_equal_to_the_logical_sequences(head_dim, tree):
    rng = np.random.Generator(np.random.PCG64(77 + head_dim + tree))
    model = Model(8, 2, head_dim, 1000)
    n_req, n_pool = 3, 600
    eng = PagedCycleEngine(model, n_pool)
    seq = []
    for r in range(n_req):
        n0 = int(rng.choice([0, 16, 37, 130]))
        k0 = rng.integers(0x3C00, 0x4000, size=(n0, model.n_kv_heads, head_dim)).astype(np.uint16)  # finite bf16 in [0.0078, 2)
        v0 = rng.integers(0x3C00, 0x4000, size=(n0, model.n_kv_heads, head_dim)).astype(np.uint16)
        seq.append((k0, v0))
        assert eng.add_request(k0, v0) == r
    for cycle in range(6):
        specs = []
        for r in range(n_req):
            n_seg = int(rng.integers(1, 5))
            segs = [int(x) for x in rng.integers(3, 45, size=n_seg)]
            parents = [int(rng.integers(0, c + 1)) for c in range(n_seg)] if tree else None
            branches = []
            for node in range(0, n_seg + 1):
                L = int(rng.integers(1, 9))
                branches.append((node, L + int(rng.choice([0, 1, 5])), L, L))
            spec = {"P": len(seq[r][0]), "segs": segs, "branches": branches}
            if tree:
                spec["parents"] = parents
            specs.append(spec)
        b = build_batch(model, specs, rng)
        k, v = fill_kv(b, rng, poison="nan")
        for r in range(n_req):  # the prefix of the oracle's cache is the logical sequence so far
            s0 = int(b.req_span_off[r])
            for t in range(len(seq[r][0])):
                pg = int(b.page_ids[int(b.span_slot[s0]) + t // PAGE])
                k[pg, :, t % PAGE, :] = seq[r][0][t]
                v[pg, :, t % PAGE, :] = seq[r][1][t]
        q = fill_q(b, rng)
        logits, drafts, _ = fill_logits_and_drafts(b, rng, 0.3)
        verdict = fill_verdicts(b, rng, 0.6)
        ref = O.verify_pass(b, q, k, v, logits, drafts, verdict)
        # the same cycle on the GPU engine: only the new tokens travel
        inputs = []
        for r in range(n_req):
            s0, s1 = int(b.req_span_off[r]), int(b.req_span_off[r + 1])
            segs = [(_span_tokens(b, k, int(b.span_slot[s]), int(b.span_len[s])), _span_tokens(b, v, int(b.span_slot[s]), int(b.span_len[s])))
                    for s in range(s0 + 1, s1)]
            brs = [BranchInput(int(b.br_depth[i]), _span_tokens(b, k, int(b.br_own_slot[i]), int(b.br_own_len[i])),
                               _span_tokens(b, v, int(b.br_own_slot[i]), int(b.br_own_len[i])),
                               int(b.cu_q[i + 1] - b.cu_q[i]), int(b.br_n_draft[i]))
                   for i in range(b.n_branch) if b.br_req[i] == r]
            inputs.append(RequestInput(segs, brs, specs[r].get("parents", ())))
        got = eng.run_cycle(inputs, q, logits, drafts, verdict)
        for key in ("n_accept", "bonus_id", "n_steps_accepted", "survivor", "committed_len"):
            assert np.array_equal(got[key], ref[key]), (cycle, key)
        err = np.abs(bf16_to_f32(got["out"]).astype(np.float64) - ref["out"])
        assert_attention_close(err, ref["out"], REL_LARGE)  # random ragged cycles: the random generators' bound
        # grow the logical sequences by what was committed, token by token from the oracle's cache
        for r in range(n_req):
            s0 = int(b.req_span_off[r])
            kept = [int(p) for p in ref["keep_pages"][ref["keep_off"][r]:ref["keep_off"][r + 1]]]
            valid = [int(x) for x in ref["keep_valid"][ref["keep_off"][r]:ref["keep_off"][r + 1]]]
            ks = np.concatenate([k[p, :, :n, :].transpose(1, 0, 2) for p, n in zip(kept, valid)] or [seq[r][0][:0]])
            vs = np.concatenate([v[p, :, :n, :].transpose(1, 0, 2) for p, n in zip(kept, valid)] or [seq[r][1][:0]])
            assert len(ks) == ref["committed_len"][r] and np.array_equal(ks[: len(seq[r][0])], seq[r][0])
            seq[r] = (ks, vs)
            gk, gv = eng.sequence(r)
            assert eng.length[r] == len(ks) and np.array_equal(gk, ks) and np.array_equal(gv, vs), (cycle, r)
        # every page is owned once or free once
        owned = [p for pages in eng.pages for p in pages]
        assert sorted(owned + eng.free) == list(range(n_pool))
