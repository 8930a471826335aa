"""Device-side error paths, reached without faulting the GPU: a corrupted page id or acceptance count in device memory
is met by a kernel's own bounds check, which substitutes a safe value, raises the plan's status word and carries on; and
the per-pass request limits of lr_commit / lr_compact are refused on the host before anything is launched."""
import numpy as np
import pytest
import torch

from lr_workloads import Model, build_batch, fill_kv, make_config, make_random_small
from oracle import lr_oracle as O
from paper_2506_19830_b200 import binding as B
from paper_2506_19830_b200 import runner as R

from gpu_util import check_attention, check_commit

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _guarded_out(b):
    n = b.n_q_rows * b.model.n_q_heads * b.model.head_dim
    guard = 4096
    buf = torch.full((n + 2 * guard,), -7.0, dtype=torch.bfloat16, device=DEV)
    return buf, buf[guard : guard + n].view(b.n_q_rows, b.model.n_q_heads, b.model.head_dim), guard, n


def _expect_bounds(plan, details):
    with pytest.raises(B.LrError) as e:
        plan.lr_poll_status()
    assert e.value.status == -5, e.value  # LR_EBOUNDS
    assert any(f"detail {d})" in str(e.value) for d in details), str(e.value)
    assert plan.lr_poll_status() == 0  # the status word was cleared by the poll that reported it


@pytest.mark.parametrize("cfg,path,details,slot_of", [
    (1, B.PATH_GENERIC, (100,), lambda b: int(b.span_slot[0]) + 3),
    (2, B.PATH_GENERIC, (100,), lambda b: int(b.span_slot[0]) + 100),
    (2, B.PATH_TENSOR_CORE, (200, 201), lambda b: int(b.span_slot[0]) + 100),   # deep inside the prefix
    (2, B.PATH_TENSOR_CORE, (200, 201), lambda b: int(b.span_slot[0])),         # the first page a CTA fetches
    (2, B.PATH_TENSOR_CORE, (200, 201), lambda b: int(b.br_own_slot[1])),       # a branch tail
    (2, B.PATH_PAIR, (200, 201), lambda b: int(b.span_slot[0]) + 100),
    (2, B.PATH_PAIR, (200, 201), lambda b: int(b.span_slot[0])),
])
def test_a_page_id_outside_the_pool_is_reported_not_dereferenced(cfg, path, details, slot_of):
    w = make_config(cfg, with_logits=False)
    b, t = w.batch, w.tensors
    ctx = B.Context(b.model, 0)
    plan = B.Plan(ctx, b)
    plan.lr_plan_set_attention_path(path)
    x = R.DeviceInputs(b, t, DEV, with_logits=False)
    buf, out, guard, n = _guarded_out(b)
    slot = slot_of(b)
    good = int(b.page_ids[slot])
    plan.lr_plan_debug_set_page(slot, int(b.n_pool_pages) + 5)
    plan.lr_verify_attention(x.q, x.k_pool, x.v_pool, out, None)
    _expect_bounds(plan, details)
    assert bool((buf[:guard] == -7.0).all()) and bool((buf[guard + n :] == -7.0).all())
    # the context and the plan stay usable: with the page put back the pass is correct again
    plan.lr_plan_debug_set_page(slot, good)
    plan.lr_verify_attention(x.q, x.k_pool, x.v_pool, out, None)
    assert plan.lr_poll_status() == 0
    o_ref, _ = O.verify_attention(b, t.q, t.k_pool, t.v_pool)
    check_attention(out, None, o_ref, None)
    plan.close()
    ctx.close()


def test_an_acceptance_count_outside_its_range_is_reported_by_commit():
    w = make_config(1, with_logits=False)
    b, t = w.batch, w.tensors
    ctx = B.Context(b.model, 0)
    plan = B.Plan(ctx, b)
    y = R.PassOutputs(b, DEV, n_rows=1)
    verdict = np.ones(len(t.verdict), dtype=np.uint8)  # every step accepted: the deepest branch decides
    bad = np.asarray(b.br_n_draft, dtype=np.int32) + 3
    plan.lr_commit(torch.from_numpy(verdict).to(DEV), torch.from_numpy(bad).to(DEV), y.n_steps_accepted, y.survivor,
                   y.committed_len, y.keep_off, y.keep_pages, y.keep_valid, y.free_off, y.free_pages)
    _expect_bounds(plan, (300, 301))
    # the count was clamped to L: the lists are those of a full match
    check_commit(y.commit_dict(), O.commit(b, verdict, np.asarray(b.br_n_draft, dtype=np.int32)))
    plan.close()
    ctx.close()


def test_a_keep_list_page_outside_the_pool_is_reported_by_compact():
    w = make_random_small(8003, head_dim=64)
    b, t = w.batch, w.tensors
    ctx = B.Context(b.model, 0)
    plan = B.Plan(ctx, b)
    n_accept = np.asarray(b.br_n_draft, dtype=np.int32)
    verdict = np.ones(len(t.verdict), dtype=np.uint8)
    c = O.commit(b, verdict, n_accept)
    # the last kept page of a request whose list has a partly filled page before it is one that must move
    target = None
    for r in range(b.n_req):
        v = c["keep_valid"][c["keep_off"][r] : c["keep_off"][r + 1]]
        if len(v) >= 2 and (v[:-1] != 16).any():
            target = int(c["keep_off"][r + 1]) - 1
            break
    assert target is not None, "the seed must give a request whose commit displaces tokens"
    x = R.DeviceInputs(b, t, DEV, with_logits=False)
    k_before, v_before = R.bf16_bits(x.k_pool).copy(), R.bf16_bits(x.v_pool).copy()
    pages = c["keep_pages"].astype(np.int32).copy()
    pages[target] = int(b.n_pool_pages) + 9
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)  # noqa: E731
    new_len = torch.empty(b.n_req, dtype=torch.int32, device=DEV)
    n_kept = torch.empty(b.n_req, dtype=torch.int32, device=DEV)
    plan.lr_compact(i32(c["keep_off"]), i32(pages), i32(c["keep_valid"]), x.k_pool, x.v_pool, new_len, n_kept, plan.compact_scratch())
    _expect_bounds(plan, (400, 401))
    # pages outside the keep lists are untouched
    touched = set(int(p) for p in c["keep_pages"])
    others = np.array([p for p in range(b.n_pool_pages) if p not in touched], dtype=np.int64)
    assert np.array_equal(R.bf16_bits(x.k_pool)[others], k_before[others])
    assert np.array_equal(R.bf16_bits(x.v_pool)[others], v_before[others])
    plan.close()
    ctx.close()


def _many_requests(n_req, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    model = Model(2, 1, 64, 16)
    reqs = []
    for _ in range(n_req):
        gamma = int(rng.integers(0, 3))
        segs = [int(x) for x in rng.integers(1, 20, size=gamma)]
        reqs.append({"P": int(rng.integers(0, 20)), "segs": segs, "branches": [(int(rng.integers(0, gamma + 1)), 4, 2, 3)]})
    b = build_batch(model, reqs, rng)
    verdict = (rng.random(int(b.cu_verdict[-1])) < 0.6).astype(np.uint8)
    n_accept = rng.integers(0, 4, size=b.n_branch).astype(np.int32)
    return model, b, verdict, n_accept, rng


@pytest.mark.parametrize("n_req,ok", [(B.COMMIT_MAX_REQUESTS, True), (B.COMMIT_MAX_REQUESTS + 1, False)])
def test_commit_request_limit(n_req, ok):
    model, b, verdict, n_accept, _ = _many_requests(n_req, 21)
    ctx = B.Context(model, 0)
    plan = B.Plan(ctx, b)  # the plan itself has no such limit
    y = R.PassOutputs(b, DEV, n_rows=1)
    y.keep_off.fill_(-7)
    args = (torch.from_numpy(verdict).to(DEV), torch.from_numpy(n_accept).to(DEV), y.n_steps_accepted, y.survivor,
            y.committed_len, y.keep_off, y.keep_pages, y.keep_valid, y.free_off, y.free_pages)
    if ok:
        plan.lr_commit(*args)
        assert plan.lr_poll_status() == 0
        check_commit(y.commit_dict(), O.commit(b, verdict, n_accept))
    else:
        with pytest.raises(B.LrError) as e:
            plan.lr_commit(*args)
        assert e.value.status == -2  # LR_EUNSUPPORTED, nothing launched
        torch.cuda.synchronize()
        assert bool((y.keep_off == -7).all())
    plan.close()
    ctx.close()


@pytest.mark.parametrize("n_req,ok", [(B.COMPACT_MAX_REQUESTS, True), (B.COMPACT_MAX_REQUESTS + 1, False)])
def test_compact_request_limit(n_req, ok):
    model, b, verdict, n_accept, rng = _many_requests(n_req, 22)
    c = O.commit(b, verdict, n_accept)
    k, v = fill_kv(b, rng, poison="nan")
    ctx = B.Context(model, 0)
    plan = B.Plan(ctx, b)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)  # noqa: E731
    kd, vd = R.bf16_tensor(k, DEV), R.bf16_tensor(v, DEV)
    new_len = torch.full((b.n_req,), -7, dtype=torch.int32, device=DEV)
    n_kept = torch.full((b.n_req,), -7, dtype=torch.int32, device=DEV)
    args = (i32(c["keep_off"]), i32(c["keep_pages"]), i32(c["keep_valid"]), kd, vd, new_len, n_kept, plan.compact_scratch())
    if ok:
        plan.lr_compact(*args)
        assert plan.lr_poll_status() == 0
        len_ref, kept_ref, k_ref, v_ref = O.compact(c["keep_off"], c["keep_pages"], c["keep_valid"], k, v)
        assert np.array_equal(new_len.cpu().numpy(), len_ref) and np.array_equal(n_kept.cpu().numpy(), kept_ref)
        kg = R.bf16_bits(kd)
        for r in range(0, b.n_req, 97):  # a sample of requests, token by token
            pages = c["keep_pages"][c["keep_off"][r] : c["keep_off"][r + 1]]
            n = int(len_ref[r])
            for i in range(int(kept_ref[r])):
                nv = min(16, n - i * 16)
                assert np.array_equal(kg[int(pages[i]), :, :nv, :], k_ref[int(pages[i]), :, :nv, :]), (r, i)
    else:
        with pytest.raises(B.LrError) as e:
            plan.lr_compact(*args)
        assert e.value.status == -2
        torch.cuda.synchronize()
        assert bool((new_len == -7).all()) and bool((n_kept == -7).all())  # refused before the first launch
    plan.close()
    ctx.close()


@pytest.mark.parametrize("path", [B.PATH_TENSOR_CORE, B.PATH_PAIR])
def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(path):
    """One barrier of the first CTA is made to expect bytes that never arrive, and the waits are given 3 ms instead of a
    second: the CTA must give up, record LR_ETIMEOUT, drain what it has in flight and leave; the other CTAs finish;
    the next pass on the same plan is correct."""
    w = make_config(2, with_logits=False)
    b, t = w.batch, w.tensors
    ctx = B.Context(b.model, 0)
    plan = B.Plan(ctx, b)
    plan.lr_plan_set_attention_path(path)
    x = R.DeviceInputs(b, t, DEV, with_logits=False)
    buf, out, guard, n = _guarded_out(b)
    plan.lr_plan_debug_set_wait_limit(3000)
    plan.lr_plan_debug_set_phantom_bytes(4096)
    plan.lr_verify_attention(x.q, x.k_pool, x.v_pool, out, None)
    with pytest.raises(B.LrError) as e:
        plan.lr_poll_status()
    assert e.value.status == -4, e.value  # LR_ETIMEOUT
    assert bool((buf[:guard] == -7.0).all()) and bool((buf[guard + n :] == -7.0).all())
    plan.lr_plan_debug_set_phantom_bytes(0)
    plan.lr_plan_debug_set_wait_limit(1_000_000)
    for _ in range(2):
        plan.lr_verify_attention(x.q, x.k_pool, x.v_pool, out, None)
        assert plan.lr_poll_status() == 0
    o_ref, _ = O.verify_attention(b, t.q, t.k_pool, t.v_pool)
    check_attention(out, None, o_ref, None)
    plan.close()
    ctx.close()
