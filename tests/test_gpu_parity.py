"""GPU parity: every step of the verify pass, through the C ABI, against the fp64 oracle."""
import copy

import numpy as np
import pytest
import torch

from lr_workloads import Model, bf16_round, build_batch, fill_kv, fill_q, make_config, make_random_mid, make_random_small
from oracle import lr_oracle as O
from paper_2506_19830_b200 import binding as B
from paper_2506_19830_b200 import runner as R

from gpu_util import REL_LARGE, attention_path_for, check_attention, check_commit, run_and_check_pass

pytestmark = pytest.mark.gpu


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def test_library_is_the_in_tree_build():
    import os

    assert os.path.exists(B.LIB_PATH)
    B.lib()


@pytest.mark.parametrize("cfg", [1, 2])
def test_whole_pass_small_configs(cfg):
    run_and_check_pass(make_config(cfg))


@pytest.mark.parametrize("cfg", [3, 4, 5])
def test_whole_pass_full_size_configs(cfg):
    run_and_check_pass(make_config(cfg))


@pytest.mark.parametrize("cfg", [1, 2, 5])
def test_whole_pass_with_the_carry_in_token_as_a_query(cfg):
    """q_len = L + 1: the last accepted token and the L drafts are the queries, one per logits row."""
    w = make_config(cfg, carry_in=True)
    assert w.batch.n_q_rows == w.batch.n_logit_rows
    run_and_check_pass(w)


@pytest.mark.parametrize("seed", list(range(16)))
def test_whole_pass_ragged_small(seed):
    run_and_check_pass(make_random_small(1000 + seed), rel_large=REL_LARGE)


@pytest.mark.parametrize("seed", list(range(10)))
def test_whole_pass_mid_size_batches(seed):
    """Both sides of the attention plan's switch between pairing query tiles and taking them one by one; attention is
    compared on a sample of branches (the oracle is slow), acceptance and commit in full."""
    w = make_random_mid(seed)
    rng = _rng(seed)
    pick = sorted(set(int(x) for x in rng.integers(0, w.batch.n_branch, size=min(4, w.batch.n_branch))))
    run_and_check_pass(w, check_rows_of_branches=pick, rel_large=REL_LARGE)


def test_overlapped_pass_gives_the_same_results():
    """Attention on one stream, acceptance -> commit on another (they share no data): same outputs."""
    w = make_config(2)
    b, t = w.batch, w.tensors
    ctx = B.Context(b.model, 0)
    plan = B.Plan(ctx, b)
    plan.lr_plan_set_attention_path(attention_path_for(b.model))
    x = R.DeviceInputs(b, t)
    y = R.PassOutputs(b)
    side = torch.cuda.Stream()
    for _ in range(3):
        R.run_pass_overlapped(ctx, plan, x, y, side)
    torch.cuda.synchronize()
    assert plan.lr_poll_status() == 0
    o_ref, _ = O.verify_attention(b, t.q, t.k_pool, t.v_pool)
    check_attention(y.out, None, o_ref, None)
    n_ref, bonus_ref, _ = O.accept_greedy(t.logits, t.draft_ids, b.cu_draft)
    assert np.array_equal(y.n_accept.cpu().numpy(), n_ref) and np.array_equal(y.bonus_id.cpu().numpy(), bonus_ref)
    check_commit(y.commit_dict(), O.commit(b, t.verdict, n_ref))


@pytest.mark.parametrize("cfg", [1, 2])
def test_generic_attention_path(cfg):
    run_and_check_pass(make_config(cfg), path=B.PATH_GENERIC)


@pytest.mark.parametrize("poison", ["nan", "big"])
def test_poison_in_slack_and_unreferenced_pages_changes_nothing(poison):
    """Same seed, different bytes in every location no visible token owns: bit-identical output."""
    outs = []
    for p in (poison, "zero"):
        w = make_random_small(77, poison=p)
        ctx = B.Context(w.batch.model, 0)
        plan = B.Plan(ctx, w.batch)
        plan.lr_plan_set_attention_path(attention_path_for(w.batch.model))
        x = R.DeviceInputs(w.batch, w.tensors)
        y = R.PassOutputs(w.batch)
        plan.lr_verify_attention(x.q, x.k_pool, x.v_pool, y.out, y.lse)
        assert plan.lr_poll_status() == 0
        outs.append((R.bf16_bits(y.out), y.lse.cpu().numpy()))
    assert np.array_equal(outs[0][0], outs[1][0])
    assert np.array_equal(outs[0][1], outs[1][1])


def test_attention_is_deterministic_and_does_not_write_outside_its_output():
    w = make_config(2)
    b, t = w.batch, w.tensors
    ctx = B.Context(b.model, 0)
    plan = B.Plan(ctx, b)
    plan.lr_plan_set_attention_path(B.PATH_TENSOR_CORE)
    x = R.DeviceInputs(b, t)
    n = b.n_q_rows * b.model.n_q_heads * b.model.head_dim
    guard = 4096
    buf = torch.full((n + 2 * guard,), -7.0, dtype=torch.bfloat16, device="cuda:0")
    out = buf[guard : guard + n].view(b.n_q_rows, b.model.n_q_heads, b.model.head_dim)
    plan.lr_verify_attention(x.q, x.k_pool, x.v_pool, out, None)
    first = R.bf16_bits(out).copy()
    plan.lr_verify_attention(x.q, x.k_pool, x.v_pool, out, None)
    assert plan.lr_poll_status() == 0
    assert np.array_equal(first, R.bf16_bits(out))
    assert bool((buf[:guard] == -7.0).all()) and bool((buf[guard + n :] == -7.0).all())


def test_increasing_scores_force_running_max_updates():
    """Keys whose scores grow along the sequence: the running maximum changes at every tile."""
    rng = _rng(3)
    model = Model(8, 2, 128, 64)
    P = 1500
    batch = build_batch(model, [{"P": P, "segs": [40, 24], "branches": [(1, 16, 16, 16), (2, 9, 9, 9)]}], rng)
    k, v = fill_kv(batch, rng, poison="nan")
    q = fill_q(batch, rng)
    # overwrite K so that score ~ position: k = (pos / 40) * sign pattern of q's first row ... simpler: all queries = ones
    q = bf16_round(np.ones(q.shape, dtype=np.float32))
    kf = np.zeros((batch.n_pool_pages, 2, 16, 128), dtype=np.float32)
    pos = 0
    for s in range(batch.n_span):
        for tok in range(int(batch.span_len[s])):
            pg = batch.page_ids[int(batch.span_slot[s]) + tok // 16]
            kf[pg, :, tok % 16, :] = (pos / 25.0) / 128 * np.sqrt(128)
            pos += 1
    k2 = bf16_round(kf)
    nan = np.isnan(np.asarray(k.view(np.uint16) == 0x7FC0))  # keep the poison where the generator put it
    k2[k == 0x7FC0] = 0x7FC0
    ctx = B.Context(model, 0)
    plan = B.Plan(ctx, batch)
    plan.lr_plan_set_attention_path(B.PATH_TENSOR_CORE)
    x = R.DeviceInputs(batch, type("T", (), dict(q=q, k_pool=k2, v_pool=v, logits=None, draft_ids=None, verdict=None)), with_logits=False)
    y = R.PassOutputs(batch)
    plan.lr_verify_attention(x.q, x.k_pool, x.v_pool, y.out, y.lse)
    assert plan.lr_poll_status() == 0
    o_ref, l_ref = O.verify_attention(batch, q, k2, v)
    check_attention(y.out, y.lse, o_ref, l_ref)


def test_score_jumps_force_the_exact_redo_of_a_half_unit():
    """A few late keys score ~70 nats above everything before them (more than 2^64 in the kernel's log2
    units): the sweep that runs against the stale reference exponent must notice and redo the half-unit
    with its own maximum.  One jump sits in the prefix, one in a segment, one in a branch tail."""
    rng = _rng(11)
    model = Model(8, 2, 128, 64)
    batch = build_batch(model, [{"P": 1100, "segs": [40, 24], "branches": [(1, 20, 16, 16), (2, 9, 9, 9)]}], rng)
    k, v = fill_kv(batch, rng, poison="nan")
    q = bf16_round(np.ones((batch.n_q_rows, 8, 128), dtype=np.float32))
    kf = bf16_round(np.zeros(k.shape, dtype=np.float32))
    big = np.float32(70.0 * np.sqrt(128) / 128)  # q . k * scale = 70
    spans = [(int(batch.span_slot[0]), 700), (int(batch.span_slot[0]), 1000), (int(batch.span_slot[1]), 17),
             (int(batch.br_own_slot[0]), 3), (int(batch.br_own_slot[1]), 8)]
    for n, (slot, tok) in enumerate(spans):
        pg = batch.page_ids[slot + tok // 16]
        kf[pg, :, tok % 16, :] = bf16_round(np.full((2, 128), big * (1 + 0.5 * n), dtype=np.float32))
    kf[k == 0x7FC0] = 0x7FC0  # keep the poison where the generator put it
    ctx = B.Context(model, 0)
    plan = B.Plan(ctx, batch)
    plan.lr_plan_set_attention_path(B.PATH_TENSOR_CORE)
    x = R.DeviceInputs(batch, type("T", (), dict(q=q, k_pool=kf, v_pool=v, logits=None, draft_ids=None, verdict=None)), with_logits=False)
    y = R.PassOutputs(batch)
    plan.lr_verify_attention(x.q, x.k_pool, x.v_pool, y.out, y.lse)
    assert plan.lr_poll_status() == 0
    o_ref, l_ref = O.verify_attention(batch, q, kf, v)
    check_attention(y.out, y.lse, o_ref, l_ref)


def test_accept_special_rows_and_ties():
    """Natural ties, ties across vector / chunk boundaries, -0/+0, NaN, inf, and a vocab that is not a multiple of 8."""
    rng = _rng(5)
    for vocab, stride in ((8192 * 2 + 24, 8192 * 2 + 24), (1003, 1008), (5, 8)):
        n_rows = 24
        x = np.round(rng.standard_normal((n_rows, stride)).astype(np.float32) * 2) / 2  # coarse: many ties
        x[0, :] = -np.inf
        x[1, :] = np.nan
        x[2, :] = -0.0
        x[2, vocab - 1] = 0.0
        x[3, :] = np.nan
        x[3, vocab - 1] = -np.inf
        x[4, :] = 1.0  # everything ties: index 0
        x[5, :] = -1.0
        x[5, vocab - 1] = 4.0  # maximum in the ragged end
        if vocab > 8200:
            x[6, :] = -1.0
            x[6, 8191] = 9.0
            x[6, 8192] = 9.0  # tie across the chunk boundary
            x[7, :] = -1.0
            x[7, 8199] = 9.0
            x[7, 8200] = 9.0
        x[8, : vocab] = np.inf
        x[:, vocab:] = 99.0  # padding beyond vocab must be ignored
        bits = bf16_round(x)
        bits[2, : vocab - 1] = 0x8000
        ref = O.row_argmax(bits[:, :vocab])
        model = Model(1, 1, 64, vocab)
        ctx = B.Context(model, 0)
        # branches: 8 branches of L = 2 (3 rows each)
        cu = np.arange(0, 17, 2, dtype=np.int32)
        drafts = ref.reshape(8, 3)[:, :2].copy()
        drafts[1, 0] = -1
        drafts[2, 1] = vocab  # out of range never matches
        drafts[3, 0] = (drafts[3, 0] + 1) % vocab
        drafts = drafts.reshape(-1).astype(np.int32)
        n_ref, b_ref, _ = O.accept_greedy(bits[:, :vocab], drafts, cu)
        dev = "cuda:0"
        lg = R.bf16_tensor(bits, dev)
        n_acc = torch.empty(8, dtype=torch.int32, device=dev)
        bonus = torch.empty(8, dtype=torch.int32, device=dev)
        arg = torch.empty(n_rows, dtype=torch.int32, device=dev)
        scratch = B.Context.accept_scratch(n_rows, dev)
        for _ in range(2):  # twice: the scratch must come back zeroed
            ctx.lr_accept_greedy(lg, torch.from_numpy(drafts).to(dev), torch.from_numpy(cu).to(dev), n_acc, bonus, scratch, arg)
            assert np.array_equal(arg.cpu().numpy(), ref), (vocab, arg.cpu().numpy(), ref)
            assert np.array_equal(n_acc.cpu().numpy(), n_ref)
            assert np.array_equal(bonus.cpu().numpy(), b_ref)
        ctx.close()


def test_accept_background_rows_with_many_ties_at_the_maximum():
    """bf16 N(0,1) rows over the full vocabulary, half of them clipped at 3.0 so that hundreds of
    entries scattered over the row tie at the maximum; the lowest index must win."""
    rng = _rng(8)
    vocab, n_rows = 152064, 12
    x = rng.standard_normal((n_rows, vocab)).astype(np.float32)
    x[::2] = np.minimum(x[::2], 3.0)
    bits = bf16_round(x)
    ref = O.row_argmax(bits)
    f = (bits.astype(np.uint32) << 16).view(np.float32)
    assert all((f[r] == f[r].max()).sum() > 50 for r in range(0, n_rows, 2))
    ctx = B.Context(Model(1, 1, 64, vocab), 0)
    dev = "cuda:0"
    cu = np.array([0, n_rows - 1], dtype=np.int32)
    drafts = ref[:-1].astype(np.int32).copy()
    n_acc = torch.empty(1, dtype=torch.int32, device=dev)
    bonus = torch.empty(1, dtype=torch.int32, device=dev)
    arg = torch.empty(n_rows, dtype=torch.int32, device=dev)
    ctx.lr_accept_greedy(R.bf16_tensor(bits, dev), torch.from_numpy(drafts).to(dev), torch.from_numpy(cu).to(dev), n_acc, bonus,
                         B.Context.accept_scratch(n_rows, dev), arg)
    assert np.array_equal(arg.cpu().numpy(), ref)
    assert int(n_acc.item()) == n_rows - 1 and int(bonus.item()) == int(ref[-1])


@pytest.mark.parametrize("seed", list(range(8)))
def test_commit_with_arbitrary_acceptance_counts(seed):
    w = make_random_small(3000 + seed)
    b, t = w.batch, w.tensors
    rng = _rng(seed)
    n_accept = np.array([rng.integers(0, L + 1) for L in b.br_n_draft], dtype=np.int32)
    ctx = B.Context(b.model, 0)
    plan = B.Plan(ctx, b)
    y = R.PassOutputs(b)
    dev = "cuda:0"
    v = t.verdict if len(t.verdict) else np.zeros(1, dtype=np.uint8)
    plan.lr_commit(torch.from_numpy(v).to(dev), torch.from_numpy(n_accept).to(dev), y.n_steps_accepted, y.survivor,
                   y.committed_len, y.keep_off, y.keep_pages, y.keep_valid, y.free_off, y.free_pages)
    assert plan.lr_poll_status() == 0
    check_commit(y.commit_dict(), O.commit(b, t.verdict, n_accept))


def test_commit_many_requests():
    """More requests than threads in a CTA and more page slots than one CTA's share."""
    rng = _rng(1)
    model = Model(2, 1, 64, 16)
    reqs = []
    for _ in range(700):
        gamma = int(rng.integers(0, 5))
        segs = [int(x) for x in rng.integers(1, 50, size=gamma)]
        brs = [(int(rng.integers(0, gamma + 1)), 5, 3, 4) for _ in range(int(rng.integers(1, 4)))]
        reqs.append({"P": int(rng.integers(0, 90)), "segs": segs, "branches": brs})
    b = build_batch(model, reqs, rng)
    verdict = (rng.random(int(b.cu_verdict[-1])) < 0.6).astype(np.uint8)
    n_accept = rng.integers(0, 5, size=b.n_branch).astype(np.int32)
    ctx = B.Context(model, 0)
    plan = B.Plan(ctx, b)
    y = R.PassOutputs(b, n_rows=1)
    dev = "cuda:0"
    plan.lr_commit(torch.from_numpy(verdict).to(dev), torch.from_numpy(n_accept).to(dev), y.n_steps_accepted, y.survivor,
                   y.committed_len, y.keep_off, y.keep_pages, y.keep_valid, y.free_off, y.free_pages)
    assert plan.lr_poll_status() == 0
    check_commit(y.commit_dict(), O.commit(b, verdict, n_accept))


def test_host_buffer_pass_matches_the_device_pass():
    import ctypes as C

    w = make_config(1)
    b, t = w.batch, w.tensors
    ctx = B.Context(b.model, 0)
    plan = B.Plan(ctx, b)
    x = R.DeviceInputs(b, t)
    staging = plan.pass_staging()
    m = b.model
    host = {
        "q_h": torch.from_numpy(t.q.view(np.int16)).pin_memory(),
        "logits_h": torch.from_numpy(t.logits.view(np.int16)).pin_memory(),
        "draft_ids_h": torch.from_numpy(t.draft_ids).pin_memory(),
        "verdict_h": torch.from_numpy(t.verdict).pin_memory(),
        "out_h": torch.empty((b.n_q_rows, m.n_q_heads, m.head_dim), dtype=torch.int16).pin_memory(),
        "n_accept_h": torch.empty(b.n_branch, dtype=torch.int32).pin_memory(),
        "bonus_id_h": torch.empty(b.n_branch, dtype=torch.int32).pin_memory(),
        "n_steps_accepted_h": torch.empty(b.n_req, dtype=torch.int32).pin_memory(),
        "survivor_h": torch.empty(b.n_req, dtype=torch.int32).pin_memory(),
        "committed_len_h": torch.empty(b.n_req, dtype=torch.int32).pin_memory(),
        "keep_off_h": torch.empty(b.n_req + 1, dtype=torch.int32).pin_memory(),
        "free_off_h": torch.empty(b.n_req + 1, dtype=torch.int32).pin_memory(),
        "keep_pages_h": torch.empty(b.n_page_slots, dtype=torch.int32).pin_memory(),
        "keep_valid_h": torch.empty(b.n_page_slots, dtype=torch.int32).pin_memory(),
        "free_pages_h": torch.empty(b.n_page_slots, dtype=torch.int32).pin_memory(),
    }
    io = B.lr_pass_host_io(**{k: v.data_ptr() for k, v in host.items()})
    for _ in range(2):
        plan.lr_verify_pass_host(io, x.k_pool, x.v_pool, staging)
    o_ref, _ = O.verify_attention(b, t.q, t.k_pool, t.v_pool)
    from gpu_util import assert_attention_close, attention_errors

    assert_attention_close(attention_errors(host["out_h"].numpy().view(np.uint16), o_ref), o_ref)
    n_ref, bonus_ref, _ = O.accept_greedy(t.logits, t.draft_ids, b.cu_draft)
    assert np.array_equal(host["n_accept_h"].numpy(), n_ref) and np.array_equal(host["bonus_id_h"].numpy(), bonus_ref)
    c = O.commit(b, t.verdict, n_ref)
    nk, nf = int(c["keep_off"][-1]), int(c["free_off"][-1])
    assert np.array_equal(host["keep_pages_h"].numpy()[:nk], c["keep_pages"])
    assert np.array_equal(host["keep_valid_h"].numpy()[:nk], c["keep_valid"])
    assert np.array_equal(host["free_pages_h"].numpy()[:nf], c["free_pages"])
    assert np.array_equal(host["committed_len_h"].numpy(), c["committed_len"])


def test_bad_arguments_are_errors_not_faults():
    w = make_random_small(9)
    b = w.batch
    ctx = B.Context(b.model, 0)
    bad = copy.copy(b)
    bad.page_ids = b.page_ids.copy()
    bad.page_ids[0] = b.n_pool_pages + 5
    with pytest.raises(B.LrError) as e:
        B.Plan(ctx, bad)
    assert e.value.status == -1
    bad = copy.copy(b)
    bad.br_own_len = b.br_own_len.copy()
    bad.br_own_len[0] = 0
    with pytest.raises(B.LrError):
        B.Plan(ctx, bad)
    plan = B.Plan(ctx, b)
    x = R.DeviceInputs(b, w.tensors)
    y = R.PassOutputs(b)
    with pytest.raises(B.LrError):
        plan.lr_verify_attention(x.q, x.k_pool, None, y.out)
    with pytest.raises(B.LrError):  # misaligned output
        plan.lr_verify_attention(x.q, x.k_pool, x.v_pool, y.out.view(-1)[1:])
    with pytest.raises(B.LrError) as e:
        B.Context(Model(6, 4, 128, 100), 0)
    assert e.value.status == -2
    with pytest.raises(B.LrError):
        B.Context(Model(4, 4, 96, 100), 0)
