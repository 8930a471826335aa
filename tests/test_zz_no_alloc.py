"""``lr_accept_greedy_static`` -- greedy acceptance for callers that cannot hand the library a
scratch buffer (an engine whose HBM is fully committed to its KV cache, or code that must not call
cudaMalloc because it stalls the device) -- must give exactly what ``lr_accept_greedy`` gives, and
what the CPU oracle's acceptance rule gives.

This file sorts last on purpose: a run that stops at the first failure has then already executed
every other test.  It passes on its own in a fresh process and after the rest of the suite.
"""
import numpy as np
import pytest
import torch

from lr_workloads import make_config, make_random_small
from oracle import lr_oracle as O
from paper_2506_19830_b200 import binding as B
from paper_2506_19830_b200 import runner as R

pytestmark = pytest.mark.gpu


def _both(w, dev="cuda:0"):
    b, t = w.batch, w.tensors
    ctx = B.Context(b.model, 0)
    x = R.DeviceInputs(b, t, dev)
    n_rows = b.n_logit_rows
    i32 = dict(dtype=torch.int32, device=dev)
    ref = [torch.empty(b.n_branch, **i32), torch.empty(b.n_branch, **i32), torch.empty(n_rows, **i32)]
    ctx.lr_accept_greedy(x.logits, x.draft_ids, x.cu_draft, ref[0], ref[1], B.Context.accept_scratch(n_rows, dev), ref[2])
    torch.cuda.synchronize()
    n_ref, bonus_ref, arg_ref = O.accept_greedy(t.logits, t.draft_ids, b.cu_draft)
    oracle = [torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev) for a in (n_ref, bonus_ref, arg_ref)]
    for call in range(2):  # two calls in a row: the second one sees whatever the first left in the array
        got = [torch.full((b.n_branch,), -7, **i32), torch.full((b.n_branch,), -7, **i32), torch.full((n_rows,), -7, **i32)]
        ctx.lr_accept_greedy_static(x.logits, x.draft_ids, x.cu_draft, got[0], got[1], got[2])
        torch.cuda.synchronize()
        for name, g, r, o in zip(("n_accept", "bonus_id", "row_argmax"), got, ref, oracle):
            assert torch.equal(g, r), f"call {call}: {name} differs from lr_accept_greedy"  # integer results: bit-exact
            assert torch.equal(g, o), f"call {call}: {name} differs from the oracle"
    ctx.close()


def test_static_scratch_acceptance_matches_on_two_calls_in_a_row():
    _both(make_config(1))
    _both(make_random_small(4242))
    _both(make_config(2, with_kv=True))


def test_static_scratch_acceptance_rejects_too_many_rows():
    w = make_config(1)
    ctx = B.Context(w.batch.model, 0)
    dev = "cuda:0"
    n_rows = B.ACCEPT_STATIC_MAX_ROWS + 1
    logits = torch.zeros((n_rows, w.batch.model.vocab), dtype=torch.bfloat16, device=dev)
    cu = torch.tensor([0, n_rows - 1], dtype=torch.int32, device=dev)
    drafts = torch.zeros(n_rows - 1, dtype=torch.int32, device=dev)
    out = torch.empty(1, dtype=torch.int32, device=dev)
    with pytest.raises(B.LrError) as e:
        ctx.lr_accept_greedy_static(logits, drafts, cu, out, out.clone())
    assert e.value.status == -1 and "at most" in str(e.value)
    ctx.close()
