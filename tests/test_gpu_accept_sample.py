"""GPU parity of lr_accept_sample (rejection-sampling acceptance) against the fp64 oracle, through the C ABI.

The kernel decides in fp32, the oracle in fp64: an acceptance whose uniform lies within 1e-5 of P(draft),
or a final-token draw whose target lies within 1e-5 (relative) of a CDF step, may legitimately go either
way.  Such branches are counted (they must be rare) and checked for validity; every other branch must match
exactly."""
import numpy as np
import pytest
import torch

from lr_workloads import Model, bf16_round, make_config, make_random_small
from oracle import lr_oracle as O
from paper_2506_19830_b200 import binding as B
from paper_2506_19830_b200 import runner as R

pytestmark = pytest.mark.gpu
EPS = 1e-5


def _run(model, logits_bits, drafts, cu, T, ua, uf, dev="cuda:0"):
    ctx = B.Context(model, 0)
    n_rows, vocab = logits_bits.shape
    stride = (vocab + 7) // 8 * 8
    padded = np.full((n_rows, stride), 0x7F80, dtype=np.uint16)  # +inf beyond the vocabulary: must be ignored
    padded[:, :vocab] = logits_bits
    lg = R.bf16_tensor(padded, dev)[:, :vocab]
    nb = len(cu) - 1
    t = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).to(dev)  # noqa: E731
    n_acc = torch.full((nb,), -7, dtype=torch.int32, device=dev)
    fin = torch.full((nb,), -7, dtype=torch.int32, device=dev)
    pd = torch.full((max(1, len(drafts)),), -1.0, dtype=torch.float32, device=dev)
    scratch = ctx.accept_sample_scratch(n_rows)
    for _ in range(2):  # twice on the same scratch
        ctx.lr_accept_sample(lg, t(drafts, np.int32), t(cu, np.int32), T, t(ua, np.float32), t(uf, np.float32), n_acc, fin, scratch, pd)
    torch.cuda.synchronize()
    ctx.close()
    return n_acc.cpu().numpy(), fin.cpu().numpy(), pd.cpu().numpy()


def _check(logits_bits, drafts, cu, T, ua, uf, got, max_ambiguous_frac=0.05):
    ua32, uf32 = ua.astype(np.float32).astype(np.float64), uf.astype(np.float32).astype(np.float64)
    n_ref, f_ref, p_ref = O.accept_sample(logits_bits, drafts, cu, T, ua32, uf32)
    n_gpu, f_gpu, p_gpu = got
    V = logits_bits.shape[1]
    ambiguous = 0
    for b in range(len(cu) - 1):
        d0, L = int(cu[b]), int(cu[b + 1] - cu[b])
        n = int(n_ref[b])
        # probabilities of the drafts the chain looked at
        for i in range(min(n + 1, L)):
            assert p_gpu[d0 + i] == pytest.approx(p_ref[d0 + i], rel=2e-4, abs=1e-7)
        close = any(abs(ua32[d0 + i] - p_ref[d0 + i]) < EPS for i in range(min(n + 1, L)))
        if n_gpu[b] != n:
            assert close, f"branch {b}: n_accept {n_gpu[b]} vs {n} with no uniform near its threshold"
            ambiguous += 1
            continue
        row = d0 + b + n
        P = O.target_probs(logits_bits[row], T)
        if n < L and 0 <= drafts[d0 + n] < V:
            P[drafts[d0 + n]] = 0.0
        c = np.cumsum(P)
        target = uf32[b] * c[-1]
        g = int(f_gpu[b])
        assert 0 <= g < V and P[g] > 0.0, f"branch {b}: final token {g} has no weight"
        if g != f_ref[b]:
            lo = c[g - 1] if g > 0 else 0.0
            assert lo - EPS * c[-1] <= target <= c[g] + EPS * c[-1], f"branch {b}: final token {g} vs {f_ref[b]} not within rounding"
            ambiguous += 1
    assert ambiguous <= max(1, int(max_ambiguous_frac * (len(cu) - 1))), f"{ambiguous} ambiguous branches"


@pytest.mark.parametrize("cfg,T", [(1, 0.6), (2, 0.6), (2, 1.0)])
def test_configs(cfg, T):
    w = make_config(cfg, with_kv=False)
    b, t = w.batch, w.tensors
    rng = np.random.default_rng(100 + cfg)
    ua, uf = rng.uniform(0, 1, len(t.draft_ids)), rng.uniform(0, 1, b.n_branch)
    got = _run(b.model, t.logits, t.draft_ids, b.cu_draft, T, ua, uf)
    _check(t.logits, t.draft_ids, b.cu_draft, T, ua, uf, got)


@pytest.mark.parametrize("seed", range(6))
def test_ragged_small(seed):
    w = make_random_small(5000 + seed)
    b, t = w.batch, w.tensors
    rng = np.random.default_rng(seed)
    ua, uf = rng.uniform(0, 1, len(t.draft_ids)), rng.uniform(0, 1, b.n_branch)
    ua[::3] = 0.0  # some sure acceptances, so that chains get long
    got = _run(b.model, t.logits, t.draft_ids, b.cu_draft, 0.8, ua, uf)
    _check(t.logits, t.draft_ids, b.cu_draft, 0.8, ua, uf, got)


def test_flat_rows_special_values_and_long_chains():
    """Flat logits (every token equally likely, the draw lands anywhere in the vocabulary, across chunks), -inf
    and NaN entries, out-of-range drafts, a vocabulary that is not a multiple of 8 and more drafts than one
    batch of the chain."""
    rng = np.random.default_rng(9)
    vocab, L, nb = 20011, 40, 5
    n_rows = nb * (L + 1)
    x = np.zeros((n_rows, vocab), dtype=np.float32)
    x[1::2] = rng.standard_normal((len(x[1::2]), vocab)).astype(np.float32)
    x[:, 100:300] = -np.inf
    bits = bf16_round(x)
    bits[:, 500:520] = 0x7FC0  # NaN: counts as -inf
    cu = np.arange(0, nb * L + 1, L, dtype=np.int32)
    drafts = rng.integers(1000, vocab, nb * L).astype(np.int32)  # clear of the -inf and NaN columns
    drafts[5] = 150  # a token with probability 0
    drafts[L + 3] = vocab + 7
    ua = rng.uniform(0, 1, nb * L)
    ua[2 * L : 3 * L] = 0.0  # branch 2 accepts all 40 drafts
    ua[:5] = 0.0
    uf = np.array([0.0, 0.999999, 0.5, 0.25, 0.75])
    got = _run(Model(1, 1, 64, vocab), bits, drafts, cu, 1.0, ua, uf)
    _check(bits, drafts, cu, 1.0, ua, uf, got, max_ambiguous_frac=0.4)
    assert got[0][2] == L and got[0][0] == 5
