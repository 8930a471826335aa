"""GPU parity of lr_compact against the oracle, through the C ABI: lr_commit's keep lists in, pools moved in place."""
import numpy as np
import pytest
import torch

from lr_workloads import make_config, make_random_small
from oracle import lr_oracle as O
from paper_2506_19830_b200 import binding as B
from paper_2506_19830_b200 import runner as R

pytestmark = pytest.mark.gpu
PAGE = 16


def _run_and_check(w, n_accept):
    b, t = w.batch, w.tensors
    dev = "cuda:0"
    ctx = B.Context(b.model, 0)
    plan = B.Plan(ctx, b)
    x = R.DeviceInputs(b, t, dev, with_logits=False)
    y = R.PassOutputs(b, dev, n_rows=1)
    verdict = t.verdict if len(t.verdict) else np.zeros(1, dtype=np.uint8)
    plan.lr_commit(torch.from_numpy(verdict).to(dev), torch.from_numpy(n_accept).to(dev), y.n_steps_accepted, y.survivor,
                   y.committed_len, y.keep_off, y.keep_pages, y.keep_valid, y.free_off, y.free_pages)
    new_len = torch.full((b.n_req,), -7, dtype=torch.int32, device=dev)
    n_kept = torch.full((b.n_req,), -7, dtype=torch.int32, device=dev)
    scratch = plan.compact_scratch()
    plan.lr_compact(y.keep_off, y.keep_pages, y.keep_valid, x.k_pool, x.v_pool, new_len, n_kept, scratch)
    assert plan.lr_poll_status() == 0
    c = O.commit(b, t.verdict, n_accept)
    len_ref, kept_ref, k_ref, v_ref = O.compact(c["keep_off"], c["keep_pages"], c["keep_valid"], t.k_pool, t.v_pool)
    assert np.array_equal(new_len.cpu().numpy(), len_ref) and np.array_equal(n_kept.cpu().numpy(), kept_ref)
    k_gpu, v_gpu = R.bf16_bits(x.k_pool), R.bf16_bits(x.v_pool)
    touched = set()
    for r in range(b.n_req):
        pages = c["keep_pages"][c["keep_off"][r] : c["keep_off"][r + 1]]
        touched.update(int(p) for p in pages)
        n = int(len_ref[r])
        for i in range(int(kept_ref[r])):  # the committed sequence, page by page, bit for bit
            v = min(PAGE, n - i * PAGE)
            pg = int(pages[i])
            assert np.array_equal(k_gpu[pg, :, :v, :], k_ref[pg, :, :v, :]), (r, i)
            assert np.array_equal(v_gpu[pg, :, :v, :], v_ref[pg, :, :v, :]), (r, i)
    others = np.array([p for p in range(b.n_pool_pages) if p not in touched], dtype=np.int64)
    assert np.array_equal(k_gpu[others], t.k_pool[others]) and np.array_equal(v_gpu[others], t.v_pool[others])
    plan.close()
    ctx.close()


@pytest.mark.parametrize("seed", range(10))
def test_ragged_small(seed):
    w = make_random_small(8000 + seed)
    rng = np.random.default_rng(seed)
    n_accept = np.array([rng.integers(0, L + 1) for L in w.batch.br_n_draft], dtype=np.int32)
    _run_and_check(w, n_accept)


@pytest.mark.parametrize("cfg", [1, 2, 5])
def test_configs(cfg):
    w = make_config(cfg, with_logits=False)
    rng = np.random.default_rng(cfg)
    n_accept = np.array([rng.integers(0, L + 1) for L in w.batch.br_n_draft], dtype=np.int32)
    _run_and_check(w, n_accept)
