"""GPU parity of lr_accept_sample_filtered (top-k / top-p filters, then rejection-sampling acceptance) against the
fp64 oracle, through the C ABI.

The kernel works on masses rounded from fp32 exponentials, the oracle in fp64, so the kernel's kept set is the
oracle's for a top_p within CUT_EPS (relative) of the one given: its size must lie between the oracle's sizes at
top_p (1 - CUT_EPS) and top_p (1 + CUT_EPS) -- equal to the oracle's wherever those two agree -- and a token
between the two cuts may be in or out.  A branch whose draft is such a token, whose acceptance uniform lies
within 1e-5 of P'(draft), or whose final draw lies within rounding of a CDF step, may go either way: such branches
are counted (they must be rare) and checked for validity; all others match exactly.  Where the tokens between the two
cuts hold more than 1e-4 of the kept mass (few, nearly equal tokens and a top_p that falls on a step between them),
both readings are right and differ in every probability of the row: there only what holds for both is checked."""
import numpy as np
import pytest
import torch

from lr_workloads import Model, bf16_round, make_config, make_random_small
from oracle import lr_oracle as O
from paper_2506_19830_b200 import binding as B
from paper_2506_19830_b200 import runner as R

pytestmark = pytest.mark.gpu
EPS = 1e-5
CUT_EPS = 2e-5


def _f32(x):
    return float(np.float32(x))


def _run(model, logits_bits, drafts, cu, T, top_k, top_p, ua, uf, dev="cuda:0", repeats=2):
    ctx = B.Context(model, 0)
    n_rows, vocab = logits_bits.shape
    stride = (vocab + 7) // 8 * 8
    padded = np.full((n_rows, stride), 0x7F80, dtype=np.uint16)  # +inf beyond the vocabulary: must be ignored
    padded[:, :vocab] = logits_bits
    lg = R.bf16_tensor(padded, dev)[:, :vocab]
    nb = len(cu) - 1
    t = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).to(dev)  # noqa: E731
    outs = []
    scratch = ctx.accept_sample_filtered_scratch(n_rows)
    for _ in range(repeats):  # on the same scratch
        n_acc = torch.full((nb,), -7, dtype=torch.int32, device=dev)
        fin = torch.full((nb,), -7, dtype=torch.int32, device=dev)
        pd = torch.full((max(1, len(drafts)),), -1.0, dtype=torch.float32, device=dev)
        kept = torch.full((n_rows,), -7, dtype=torch.int32, device=dev)
        ctx.lr_accept_sample_filtered(lg, t(drafts, np.int32), t(cu, np.int32), T, top_k, top_p, t(ua, np.float32),
                                      t(uf, np.float32), n_acc, fin, scratch, pd, kept)
        torch.cuda.synchronize()
        outs.append((n_acc.cpu().numpy(), fin.cpu().numpy(), pd.cpu().numpy(), kept.cpu().numpy()))
    ctx.close()
    for o in outs[1:]:  # same inputs, same outputs, bit for bit
        for a, b in zip(outs[0], o):
            assert np.array_equal(a, b)
    return outs[0]


HEAVY = 1e-4  # a token between the two cuts with more than this share of the kept mass changes every P' noticeably


def _check(logits_bits, drafts, cu, T, top_k, top_p, ua, uf, got, max_ambiguous_frac=0.05, rows_to_check=None):
    ua32, uf32 = ua.astype(np.float32).astype(np.float64), uf.astype(np.float32).astype(np.float64)
    p32 = _f32(top_p)
    n_ref, f_ref, p_ref = O.accept_sample(logits_bits, drafts, cu, T, ua32, uf32, top_k=top_k, top_p=p32)
    n_gpu, f_gpu, p_gpu, kept_gpu = got
    V = logits_bits.shape[1]
    filters_off = (top_k <= 0 or top_k >= V) and p32 >= 1.0
    cache = {}

    def row_info(row):  # filtered distribution at top_p; kept sets at top_p (1 -+ CUT_EPS); is the edge heavy?
        if row not in cache:
            P = O.target_probs(logits_bits[row], T)
            F = O.filter_probs(P, top_k, p32)
            lo = hi = F > 0
            heavy = False
            if p32 < 1.0:
                lo = O.filter_probs(P, top_k, p32 * (1 - CUT_EPS)) > 0
                F_hi = O.filter_probs(P, top_k, min(1.0, p32 * (1 + CUT_EPS)))
                hi = F_hi > 0
                heavy = float(F_hi[hi & ~lo].sum()) > HEAVY
            cache[row] = (F, lo, hi, heavy)
        return cache[row]

    # kept-set sizes, on every row or on a sample of them
    n_rows = logits_bits.shape[0]
    rows = range(n_rows) if rows_to_check is None else rows_to_check
    for row in rows:
        F, lo, hi, _ = row_info(row)
        if filters_off:
            assert kept_gpu[row] == V, f"row {row}"  # nothing is cut: every token counts, whatever its probability
        elif top_k > 0 and p32 >= 1.0:
            # tokens of probability 0 inside the cut (top_k reaching into the -inf entries) count for the kernel
            assert int((F > 0).sum()) <= kept_gpu[row] <= min(top_k, V), f"row {row}"
        else:
            assert int(lo.sum()) <= kept_gpu[row] <= int(hi.sum()), f"row {row}: kept {kept_gpu[row]} vs {(F > 0).sum()}"

    ambiguous = 0
    for b in range(len(cu) - 1):
        d0, L = int(cu[b]), int(cu[b + 1] - cu[b])
        n = int(n_ref[b])
        visited = [d0 + b + i for i in range(min(n + 1, L + 1))]
        if any(row_info(r)[3] for r in visited):
            # a heavy token on the edge of a kept set: with it or without it every probability of the row is
            # different, and both readings are right.  Only what holds for both is checked.
            ambiguous += 1
            assert 0 <= n_gpu[b] <= L
            g, ng = int(f_gpu[b]), int(n_gpu[b])
            assert 0 <= g < V and row_info(d0 + b + ng)[2][g], f"branch {b}: final token {g} is outside the kept set"
            continue
        close = False
        for i in range(min(n + 1, L)):
            F, lo, hi, _ = row_info(d0 + b + i)
            d = int(drafts[d0 + i])
            if 0 <= d < V and lo[d] != hi[d]:  # the draft sits on the edge of the kept set: either 0 or about P / Z
                close = True
                continue
            assert p_gpu[d0 + i] == pytest.approx(p_ref[d0 + i], rel=2e-4 + 2 * HEAVY, abs=1e-7), f"branch {b} draft {i}"
            close = close or abs(ua32[d0 + i] - p_ref[d0 + i]) < EPS + 2 * HEAVY * p_ref[d0 + i]
        if n_gpu[b] != n:
            assert close, f"branch {b}: n_accept {n_gpu[b]} vs {n} with no uniform near its threshold"
            ambiguous += 1
            continue
        F, lo, hi, _ = row_info(d0 + b + n)
        P = F.copy()
        dead = int(drafts[d0 + n]) if n < L else -1
        if 0 <= dead < V:
            P[dead] = 0.0
        c = np.cumsum(P)
        target = uf32[b] * c[-1]
        g = int(f_gpu[b])
        assert 0 <= g < V and hi[g] and g != dead, f"branch {b}: final token {g} is outside the kept set"
        if g != f_ref[b]:
            tol = (EPS + 2 * CUT_EPS + 2 * HEAVY) * c[-1]  # tokens on the edge of the kept set shift every cumulative mass a little
            lo_c = c[g - 1] if g > 0 else 0.0
            assert lo_c - tol <= target <= c[g] + tol, f"branch {b}: final token {g} vs {f_ref[b]} not within rounding"
            ambiguous += 1
    assert ambiguous <= max(1, int(max_ambiguous_frac * (len(cu) - 1))), f"{ambiguous} ambiguous branches"


# the paper's settings (Section 4, "Setup"): temperature 0.6 with top-p 0.95, and with top-k 20 besides
@pytest.mark.parametrize("cfg,T,top_k,top_p", [(1, 0.6, 0, 0.95), (1, 0.6, 20, 0.95), (2, 0.6, 20, 0.95), (2, 0.6, 0, 0.95),
                                               (2, 1.0, 50, 1.0), (3, 0.6, 0, 0.95), (5, 0.6, 20, 0.95)])
def test_configs(cfg, T, top_k, top_p):
    w = make_config(cfg, with_kv=False)
    b, t = w.batch, w.tensors
    rng = np.random.default_rng(300 + cfg)
    ua, uf = rng.uniform(0, 1, len(t.draft_ids)), rng.uniform(0, 1, b.n_branch)
    got = _run(b.model, t.logits, t.draft_ids, b.cu_draft, T, top_k, top_p, ua, uf)
    n_rows = t.logits.shape[0]
    rows = None if n_rows <= 48 else sorted(set(np.random.default_rng(1).integers(0, n_rows, 40).tolist()))
    _check(t.logits, t.draft_ids, b.cu_draft, T, top_k, top_p, ua, uf, got, rows_to_check=rows)


@pytest.mark.parametrize("seed", range(6))
def test_ragged_small(seed):
    w = make_random_small(5000 + seed)
    b, t = w.batch, w.tensors
    rng = np.random.default_rng(seed)
    ua, uf = rng.uniform(0, 1, len(t.draft_ids)), rng.uniform(0, 1, b.n_branch)
    ua[::3] = 0.0
    top_k, top_p = [(0, 0.9), (5, 1.0), (40, 0.8), (1, 1.0), (0, 0.5), (10 ** 6, 0.99)][seed]
    got = _run(b.model, t.logits, t.draft_ids, b.cu_draft, 0.8, top_k, top_p, ua, uf)
    _check(t.logits, t.draft_ids, b.cu_draft, 0.8, top_k, top_p, ua, uf, got)


@pytest.mark.parametrize("top_k,top_p", [(0, 0.3), (777, 1.0), (5000, 0.7), (0, 0.999), (20000, 1.0), (20000, 0.9)])
def test_ties_special_values_and_long_chains(top_k, top_p):
    """Flat rows (the cut splits one large group of equal logits: the kept ones are the lowest indices), coarse rows
    (many groups of equal logits), -inf and NaN entries, out-of-range drafts, a vocabulary that is not a multiple of
    8 and chains of 40 drafts."""
    rng = np.random.default_rng(9)
    vocab, L, nb = 20011, 40, 5
    n_rows = nb * (L + 1)
    x = np.zeros((n_rows, vocab), dtype=np.float32)
    x[1::3] = rng.standard_normal((len(x[1::3]), vocab)).astype(np.float32) * 2
    x[2::3] = np.round(rng.standard_normal((len(x[2::3]), vocab)) * 2) / 2
    x[:, 100:300] = -np.inf
    bits = bf16_round(x)
    bits[:, 500:520] = 0x7FC0  # NaN: counts as -inf
    bits[:, 600:610] = 0x8000  # -0: equal to +0
    cu = np.arange(0, nb * L + 1, L, dtype=np.int32)
    drafts = rng.integers(0, vocab, nb * L).astype(np.int32)
    drafts[5] = 150  # a token with probability 0
    drafts[L + 3] = vocab + 7
    ua = rng.uniform(0, 1, nb * L)
    ua[2 * L : 3 * L] = 0.0
    ua[:5] = 0.0
    uf = np.array([0.0, 0.999999, 0.5, 0.25, 0.75])
    got = _run(Model(1, 1, 64, vocab), bits, drafts, cu, 1.0, top_k, top_p, ua, uf)
    _check(bits, drafts, cu, 1.0, top_k, top_p, ua, uf, got, max_ambiguous_frac=0.4)
    if top_k == 777:  # flat rows: exactly the 777 lowest indices with a finite logit stay, each with mass 1/777
        assert got[3][0] == 777


def test_top_k_one_is_greedy():
    w = make_config(1, with_kv=False)
    b, t = w.batch, w.tensors
    rng = np.random.default_rng(4)
    ua, uf = rng.uniform(0, 1, len(t.draft_ids)), rng.uniform(0, 1, b.n_branch)
    n, f, p, kept = _run(b.model, t.logits, t.draft_ids, b.cu_draft, 0.6, 1, 1.0, ua, uf)
    n_ref, bonus_ref, _ = O.accept_greedy(t.logits, t.draft_ids, b.cu_draft)
    assert np.array_equal(n, n_ref) and np.array_equal(f, bonus_ref) and (kept == 1).all()
    assert set(np.unique(p[: len(t.draft_ids)])) <= {0.0, 1.0}


def test_filters_off_match_the_unfiltered_call():
    w = make_random_small(5003)
    b, t = w.batch, w.tensors
    rng = np.random.default_rng(8)
    ua, uf = rng.uniform(0, 1, len(t.draft_ids)), rng.uniform(0, 1, b.n_branch)
    got = _run(b.model, t.logits, t.draft_ids, b.cu_draft, 0.7, 0, 1.0, ua, uf)
    assert (got[3] == t.logits.shape[1]).all()
    _check(t.logits, t.draft_ids, b.cu_draft, 0.7, 0, 1.0, ua, uf, got)


def test_bad_arguments():
    model = Model(1, 1, 64, 4096)
    ctx = B.Context(model, 0)
    dev = "cuda:0"
    lg = torch.zeros((2, 4096), dtype=torch.bfloat16, device=dev)
    z = lambda n, dt: torch.zeros(n, dtype=dt, device=dev)  # noqa: E731
    cu = torch.tensor([0, 1], dtype=torch.int32, device=dev)
    scratch = ctx.accept_sample_filtered_scratch(2)
    for T, k, p in [(0.0, 0, 0.9), (0.6, -1, 0.9), (0.6, 0, 0.0), (0.6, 0, 1.5), (0.6, 0, float("nan"))]:
        with pytest.raises(B.LrError) as e:
            ctx.lr_accept_sample_filtered(lg, z(1, torch.int32), cu, T, k, p, z(1, torch.float32), z(1, torch.float32),
                                          z(1, torch.int32), z(1, torch.int32), scratch)
        assert e.value.status == -1  # LR_EINVAL
    ctx.close()


@pytest.mark.parametrize("vocab,top_k,top_p", [(72, 8, 0.9), (72, 0, 0.5), (1000, 1024, 0.97), (3000, 1024, 1.0), (3000, 1025, 1.0),
                                               (3000, 0, 1e-6), (40000, 2, 0.999)])
def test_small_vocabularies_and_limits_of_the_bound(vocab, top_k, top_p):
    """Vocabularies with fewer tokens than the filter kernel has threads (most threads see no token), top_k at and
    just past the number of threads (the lower bound from the threads' maxima applies up to it), and a top_p so small
    that only the most likely token stays."""
    rng = np.random.default_rng(vocab + top_k)
    L, nb = 6, 4
    n_rows = nb * (L + 1)
    bits = bf16_round((rng.standard_normal((n_rows, vocab)) * 3).astype(np.float32))
    cu = np.arange(0, nb * L + 1, L, dtype=np.int32)
    arg = O.row_argmax(bits)
    drafts = np.where(rng.uniform(size=nb * L) < 0.6, np.concatenate([arg[b * (L + 1): b * (L + 1) + L] for b in range(nb)]),
                      rng.integers(0, vocab, nb * L)).astype(np.int32)
    ua, uf = rng.uniform(0, 1, nb * L), rng.uniform(0, 1, nb)
    got = _run(Model(1, 1, 64, vocab), bits, drafts, cu, 0.7, top_k, top_p, ua, uf)
    _check(bits, drafts, cu, 0.7, top_k, top_p, ua, uf, got, max_ambiguous_frac=0.5)
    if top_p == 1e-6:
        assert (got[3] == 1).all()


@pytest.mark.parametrize("seed", range(12))
def test_logit_shapes_that_move_the_window(seed):
    """Rows whose kept set does not lie in the first window of keys below the maximum, or lies across several: logits
    spread over many octaves with both signs, all-negative rows, a few large tokens over a flat sea 40 below them,
    nearly flat rows and coarse rows with many ties -- with top_k and top_p drawn to put the cuts at either end."""
    rng = np.random.default_rng(90000 + seed)
    vocab = int(rng.choice([257, 5003, 20000, 70001]))
    L, nb = int(rng.integers(1, 6)), int(rng.integers(1, 4))
    n_rows = nb * (L + 1)
    kind = seed % 6
    if kind == 0:
        x = rng.standard_normal((n_rows, vocab)) * 8
    elif kind == 1:
        x = np.sign(rng.standard_normal((n_rows, vocab))) * np.exp2(rng.uniform(-30, 6, (n_rows, vocab)))
    elif kind == 2:
        x = -np.exp2(rng.uniform(-20, 5, (n_rows, vocab)))
    elif kind == 3:
        x = np.round(rng.standard_normal((n_rows, vocab)) * 3) / 4
    elif kind == 4:
        x = np.full((n_rows, vocab), -40.0) + rng.standard_normal((n_rows, vocab)) * 0.01
        for r in range(n_rows):
            x[r, rng.integers(0, vocab, 3)] = rng.uniform(0, 3, 3)
    else:
        x = rng.standard_normal((n_rows, vocab)) * 1e-3
    bits = bf16_round(x.astype(np.float32))
    if seed % 3 == 0:
        bits[:, rng.integers(0, vocab, max(1, vocab // 50))] = 0xFF80
    T = float(rng.choice([0.3, 0.6, 1.0, 2.0]))
    top_k = int(rng.choice([0, 2, 20, 1024, 1025, vocab // 2]))
    top_p = float(rng.choice([1.0, 0.999, 0.95, 0.5, 0.1]))
    cu = np.arange(0, nb * L + 1, L, dtype=np.int32)
    arg = O.row_argmax(bits)
    drafts = np.where(rng.uniform(size=nb * L) < 0.6, np.concatenate([arg[b * (L + 1): b * (L + 1) + L] for b in range(nb)]),
                      rng.integers(0, vocab, nb * L)).astype(np.int32)
    ua, uf = rng.uniform(0, 1, nb * L), rng.uniform(0, 1, nb)
    got = _run(Model(1, 1, 64, vocab), bits, drafts, cu, T, top_k, top_p, ua, uf)
    _check(bits, drafts, cu, T, top_k, top_p, ua, uf, got, max_ambiguous_frac=1.0)
