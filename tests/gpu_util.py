"""Helpers shared by the GPU parity tests (the CUDA path is reached only through the C-ABI binding)."""
import numpy as np
import torch

from lr_workloads import bf16_to_f32
from oracle import lr_oracle as O
from paper_2506_19830_b200 import binding as B
from paper_2506_19830_b200 import runner as R

# Attention tolerance versus the fp64 oracle (bf16 inputs, fp32 accumulate, bf16 output): max-abs 1.5e-2 and mean-abs
# 2e-3, with no other clause, on the five named configurations (chain and carry-in).
MAX_ABS = 1.5e-2
MEAN_ABS = 2e-3
LSE_ABS = 2e-3
# The random and degenerate generators produce rows that see one or two keys and return a V value of magnitude 2..5.
# The output is bf16 and so are the softmax weights that enter the PV product: each rounding is worth up to half an ulp,
# 2^-9 of the value, so for |O| >= 3.84 the two roundings alone reach MAX_ABS (bf16 spacing is 2^-6 in [2, 4) and 2^-5 in
# [4, 8)).  For those generators only, an element may use the relative bound 2^-8 |O| (output rounding + weight
# rounding) where that is the larger one.
REL_LARGE = 2.0 ** -8


def attention_errors(got_bits: np.ndarray, out_ref: np.ndarray):
    got = bf16_to_f32(got_bits).astype(np.float64)
    assert not np.isnan(got).any(), "NaN in attention output"
    return np.abs(got - out_ref)


def assert_attention_close(err: np.ndarray, out_ref: np.ndarray, rel_large: float = 0.0):
    """max-abs / mean-abs check; rel_large > 0 lets elements with large |reference| use rel_large * |reference|."""
    bound = np.maximum(MAX_ABS, rel_large * np.abs(out_ref)) if rel_large > 0 else np.full(err.shape, MAX_ABS)
    over = err - bound
    assert over.max() <= 0, f"max-abs {err.max():.4g} (largest excess {over.max():.3g} at reference {out_ref.flat[over.argmax()]:.4g})"
    assert err.mean() <= MEAN_ABS, f"mean-abs {err.mean():.4g}"


def check_attention(out_gpu: torch.Tensor, lse_gpu, out_ref: np.ndarray, lse_ref, rows=None, rel_large: float = 0.0):
    bits = R.bf16_bits(out_gpu)
    if rows is not None:
        bits, out_ref = bits[rows], out_ref[rows]
    err = attention_errors(bits, out_ref)
    assert_attention_close(err, out_ref, rel_large)
    if lse_gpu is not None:
        l = lse_gpu.cpu().numpy().astype(np.float64)
        if rows is not None:
            l, lse_ref = l[rows], lse_ref[rows]
        assert np.abs(l - lse_ref).max() <= LSE_ABS, f"lse max-abs {np.abs(l - lse_ref).max():.4g}"
    return float(err.max()), float(err.mean())


def check_commit(got: dict, ref: dict):
    for k in ("n_steps_accepted", "survivor", "committed_len", "keep_off", "free_off", "keep_pages", "keep_valid", "free_pages"):
        assert np.array_equal(got[k], ref[k]), f"commit field {k} differs"


def attention_path_for(model):
    """The tensor-core path, named explicitly, wherever the head size allows it: a plan that cannot take it then fails
    with LR_EUNSUPPORTED instead of passing on the CUDA-core kernel."""
    return B.PATH_TENSOR_CORE if model.head_dim == 128 else B.PATH_GENERIC


def run_and_check_pass(w, path=None, check_rows_of_branches=None, rel_large: float = 0.0):
    """Whole pass through the C ABI on workload w, compared with the oracle.  path None = the tensor-core kernel
    for head_dim 128 (forced, so a silent fall-back is an error), the CUDA-core kernel otherwise."""
    b, t = w.batch, w.tensors
    ctx = B.Context(b.model, 0)
    plan = B.Plan(ctx, b)
    if path is None:
        path = attention_path_for(b.model)
    plan.lr_plan_set_attention_path(path)
    info = plan.lr_plan_describe()
    assert info["uses_tensor_core"] == (1 if path in (B.PATH_TENSOR_CORE, B.PATH_PAIR) else 0), info
    x = R.DeviceInputs(b, t)
    y = R.PassOutputs(b)
    y.out.fill_(float("nan"))
    R.run_pass(ctx, plan, x, y)
    assert plan.lr_poll_status() == 0
    o_ref, l_ref = O.verify_attention(b, t.q, t.k_pool, t.v_pool, branches=check_rows_of_branches)
    rows = None
    if check_rows_of_branches is not None:
        rows = np.concatenate([np.arange(b.cu_q[i], b.cu_q[i + 1]) for i in check_rows_of_branches])
    errs = check_attention(y.out, y.lse, o_ref, l_ref, rows, rel_large)
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
