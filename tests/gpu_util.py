"""Helpers shared by the GPU parity tests (the CUDA path is reached only through the C-ABI binding)."""
import numpy as np
import torch

from lr_workloads import bf16_to_f32
from oracle import lr_oracle as O
from paper_2506_19830_b200 import binding as B
from paper_2506_19830_b200 import runner as R

# attention tolerance versus the fp64 oracle (bf16 inputs, fp32 accumulate, bf16 output)
MAX_ABS = 1.5e-2
MEAN_ABS = 2e-3
LSE_ABS = 2e-3
# The output is bf16 and so are the softmax weights that enter the PV product: each rounding is worth up to half an ulp,
# 2^-9 of the value.  For |O| above about 2 that alone reaches MAX_ABS (spacing 2^-6 in [2, 4), 2^-5 in [4, 8)), so large
# elements are held to a relative bound instead: 2^-7 |O| (output rounding + weight rounding + as much again for the
# fp32 accumulation and the exp2 approximation).  Below |O| = 1.92 the absolute bound is the binding one.
MAX_REL_LARGE = 2.0 ** -7


def check_attention(out_gpu: torch.Tensor, lse_gpu, out_ref: np.ndarray, lse_ref, rows=None):
    got = bf16_to_f32(R.bf16_bits(out_gpu)).astype(np.float64)
    if rows is not None:
        got, out_ref = got[rows], out_ref[rows]
    assert not np.isnan(got).any(), "NaN in attention output"
    err = np.abs(got - out_ref)
    over = err - np.maximum(MAX_ABS, MAX_REL_LARGE * np.abs(out_ref))
    assert over.max() <= 0, f"max-abs {err.max():.4g} (largest excess {over.max():.3g} at reference {out_ref.flat[over.argmax()]:.4g})"
    assert err.mean() <= MEAN_ABS, f"mean-abs {err.mean():.4g}"
    if lse_gpu is not None:
        l = lse_gpu.cpu().numpy().astype(np.float64)
        if rows is not None:
            l, lse_ref = l[rows], lse_ref[rows]
        assert np.abs(l - lse_ref).max() <= LSE_ABS, f"lse max-abs {np.abs(l - lse_ref).max():.4g}"
    return float(err.max()), float(err.mean())


def check_commit(got: dict, ref: dict):
    for k in ("n_steps_accepted", "survivor", "committed_len", "keep_off", "free_off", "keep_pages", "keep_valid", "free_pages"):
        assert np.array_equal(got[k], ref[k]), f"commit field {k} differs"


def run_and_check_pass(w, path=B.PATH_AUTO, check_rows_of_branches=None):
    """Whole pass through the C ABI on workload w, compared with the oracle."""
    b, t = w.batch, w.tensors
    ctx = B.Context(b.model, 0)
    plan = B.Plan(ctx, b)
    plan.lr_plan_set_attention_path(path)
    x = R.DeviceInputs(b, t)
    y = R.PassOutputs(b)
    y.out.fill_(float("nan"))
    R.run_pass(ctx, plan, x, y)
    assert plan.lr_poll_status() == 0
    o_ref, l_ref = O.verify_attention(b, t.q, t.k_pool, t.v_pool, branches=check_rows_of_branches)
    rows = None
    if check_rows_of_branches is not None:
        rows = np.concatenate([np.arange(b.cu_q[i], b.cu_q[i + 1]) for i in check_rows_of_branches])
    errs = check_attention(y.out, y.lse, o_ref, l_ref, rows)
    n_ref, bonus_ref, arg_ref = O.accept_greedy(t.logits, t.draft_ids, b.cu_draft)
    assert np.array_equal(y.n_accept.cpu().numpy(), n_ref)
    assert np.array_equal(y.bonus_id.cpu().numpy(), bonus_ref)
    assert np.array_equal(y.row_argmax.cpu().numpy(), arg_ref)
    check_commit(y.commit_dict(), O.commit(b, t.verdict, n_ref))
    # the scratch must be left zeroed for the next call
    assert int(y.scratch.abs().sum().item()) == 0
    plan.close()
    ctx.close()
    return errs
