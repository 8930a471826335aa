"""GPU parity with multi-branch (tree) drafting: the same three calls on batches whose draft steps form a tree."""
import dataclasses

import numpy as np
import pytest
import torch

from lr_workloads import Model, build_batch, make_config, make_random_small, make_random_tree, make_tree
from oracle import lr_oracle as O
from paper_2506_19830_b200 import binding as B
from paper_2506_19830_b200 import runner as R
from gpu_util import REL_LARGE, attention_path_for, check_commit, run_and_check_pass

pytestmark = pytest.mark.gpu


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


@pytest.mark.parametrize("seed", list(range(12)))
def test_whole_pass_random_trees(seed):
    run_and_check_pass(make_random_tree(500 + seed), rel_large=REL_LARGE)


@pytest.mark.parametrize("seed", list(range(4)))
def test_whole_pass_random_trees_tensor_core_path(seed):
    run_and_check_pass(make_random_tree(600 + seed, head_dim=128), rel_large=REL_LARGE)


def test_many_small_passes_on_the_tensor_core_path():
    """Tiny passes put several one-tile pieces into one CTA, where one of its two streams has nothing to do: the
    piece-by-piece barrier phases must still line up (seed 5000 once ran into an expired wait)."""
    for seed in [5000] + list(range(5100, 5140)):
        run_and_check_pass(make_random_tree(seed, head_dim=128), rel_large=REL_LARGE)
        run_and_check_pass(make_random_small(seed, head_dim=128), rel_large=REL_LARGE)


@pytest.mark.parametrize("seed", list(range(4)))
def test_whole_pass_random_trees_generic_path(seed):
    run_and_check_pass(make_random_tree(700 + seed), path=B.PATH_GENERIC, rel_large=REL_LARGE)


@pytest.mark.parametrize("W,gamma,size", [(2, 2, "tiny"), (3, 2, "tiny"), (2, 3, "layer"), (4, 2, "layer"), (2, 2, "serving")])
def test_whole_pass_full_trees(W, gamma, size):
    run_and_check_pass(make_tree(W, gamma, size=size))


@pytest.mark.parametrize("make", [lambda: make_config(2), lambda: make_random_small(5, head_dim=128), lambda: make_random_small(6, head_dim=64)])
def test_a_chain_written_with_parents_gives_the_same_bits(make):
    w = make()
    b, t = w.batch, w.tensors
    parent = np.concatenate([np.arange(-1, b.req_span_off[r + 1] - b.req_span_off[r] - 1, dtype=np.int32) for r in range(b.n_req)])
    results = []
    for batch in (b, dataclasses.replace(b, seg_parent=parent)):
        ctx = B.Context(batch.model, 0)
        plan = B.Plan(ctx, batch)
        plan.lr_plan_set_attention_path(attention_path_for(batch.model))
        x, y = R.DeviceInputs(batch, t), R.PassOutputs(batch)
        R.run_pass(ctx, plan, x, y)
        assert plan.lr_poll_status() == 0
        results.append((R.bf16_bits(y.out).copy(), y.lse.cpu().numpy().copy(), y.commit_dict()))
        plan.close()
        ctx.close()
    assert np.array_equal(results[0][0], results[1][0]) and np.array_equal(results[0][1], results[1][1])
    check_commit(results[1][2], results[0][2])


def _commit_only(b, verdict, n_accept):
    ctx = B.Context(b.model, 0)
    plan = B.Plan(ctx, b)
    y = R.PassOutputs(b, n_rows=1)
    dev = "cuda:0"
    v = verdict if len(verdict) else np.zeros(1, dtype=np.uint8)
    plan.lr_commit(torch.from_numpy(v).to(dev), torch.from_numpy(n_accept).to(dev), y.n_steps_accepted, y.survivor,
                   y.committed_len, y.keep_off, y.keep_pages, y.keep_valid, y.free_off, y.free_pages)
    assert plan.lr_poll_status() == 0
    check_commit(y.commit_dict(), O.commit(b, verdict, n_accept))
    return ctx, plan, y


@pytest.mark.parametrize("seed", list(range(10)))
def test_commit_on_random_trees_with_arbitrary_acceptance_counts(seed):
    w = make_random_tree(900 + seed)
    b = w.batch
    n_accept = _rng(seed).integers(0, b.br_n_draft + 1).astype(np.int32)
    for p in (0.0, 0.6, 1.0):
        verdict = (_rng(seed + 50).random(len(w.tensors.verdict)) < p).astype(np.uint8)
        _commit_only(b, verdict, n_accept)


def test_commit_many_tree_requests():
    rng = _rng(2)
    model = Model(2, 1, 64, 16)
    reqs = []
    for _ in range(600):
        n = int(rng.integers(0, 9))
        parents = [int(rng.integers(0, c + 1)) for c in range(n)]
        segs = [int(x) for x in rng.integers(1, 50, size=n)]
        brs = [(int(rng.integers(0, n + 1)), 5, 3, 4) for _ in range(int(rng.integers(1, 4)))]
        reqs.append({"P": int(rng.integers(0, 90)), "segs": segs, "parents": parents, "branches": brs})
    b = build_batch(model, reqs, rng)
    verdict = (rng.random(int(b.cu_verdict[-1])) < 0.6).astype(np.uint8)
    _commit_only(b, verdict, rng.integers(0, 5, size=b.n_branch).astype(np.int32))


@pytest.mark.parametrize("seed", list(range(4)))
def test_compaction_after_a_tree_commit(seed):
    w = make_random_tree(1100 + seed)
    b, t = w.batch, w.tensors
    n_accept = _rng(seed).integers(0, b.br_n_draft + 1).astype(np.int32)
    ctx, plan, y = _commit_only(b, t.verdict, n_accept)
    dev = "cuda:0"
    x = R.DeviceInputs(b, t, dev, with_logits=False)
    new_len = torch.empty(b.n_req, dtype=torch.int32, device=dev)
    n_kept = torch.empty(b.n_req, dtype=torch.int32, device=dev)
    plan.lr_compact(y.keep_off, y.keep_pages, y.keep_valid, x.k_pool, x.v_pool, new_len, n_kept, plan.compact_scratch())
    assert plan.lr_poll_status() == 0
    c = O.commit(b, t.verdict, n_accept)
    len_ref, kept_ref, k_ref, v_ref = O.compact(c["keep_off"], c["keep_pages"], c["keep_valid"], t.k_pool, t.v_pool)
    assert np.array_equal(new_len.cpu().numpy(), len_ref) and np.array_equal(n_kept.cpu().numpy(), kept_ref)
    k_gpu, v_gpu = R.bf16_bits(x.k_pool), R.bf16_bits(x.v_pool)
    for r in range(b.n_req):
        pages = c["keep_pages"][c["keep_off"][r]:c["keep_off"][r + 1]]
        for i in range(int(kept_ref[r])):
            n = min(16, int(len_ref[r]) - 16 * i)
            assert np.array_equal(k_gpu[pages[i], :, :n], k_ref[pages[i], :, :n])
            assert np.array_equal(v_gpu[pages[i], :, :n], v_ref[pages[i], :, :n])
