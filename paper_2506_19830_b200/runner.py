"""Device-side buffers for one verify pass and the three C-ABI calls in order.

Marshalling only: uploads host arrays as torch tensors, allocates outputs and
calls ``lr_verify_attention`` -> ``lr_accept_greedy`` -> ``lr_commit``.
"""
from __future__ import annotations

from typing import Optional

import numpy as np
import torch

from . import binding as B


def bf16_tensor(bits: np.ndarray, device) -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor on ``device`` (no value conversion)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class DeviceInputs:
    def __init__(self, batch, tensors, device="cuda:0", with_logits=True):
        self.device = device
        self.q = bf16_tensor(tensors.q, device)
        self.k_pool = bf16_tensor(tensors.k_pool, device)
        self.v_pool = bf16_tensor(tensors.v_pool, device)
        self.cu_draft = torch.from_numpy(np.ascontiguousarray(batch.cu_draft, dtype=np.int32)).to(device)
        self.logits = None
        if with_logits and tensors.logits is not None:
            n_rows, vocab = tensors.logits.shape
            stride = (vocab + 7) // 8 * 8  # the C ABI wants a row stride that is a multiple of 8 elements
            if stride == vocab:
                self.logits = bf16_tensor(tensors.logits, device)
            else:
                # padding columns hold +inf: they lie beyond `vocab` and must never be looked at
                padded = np.full((n_rows, stride), 0x7F80, dtype=np.uint16)
                padded[:, :vocab] = tensors.logits
                self.logits = bf16_tensor(padded, device)[:, :vocab]
        self.draft_ids = (torch.from_numpy(np.ascontiguousarray(tensors.draft_ids, dtype=np.int32)).to(device)
                          if tensors.draft_ids is not None else None)
        v = tensors.verdict if tensors.verdict is not None and len(tensors.verdict) else np.zeros(1, dtype=np.uint8)
        self.verdict = torch.from_numpy(np.ascontiguousarray(v, dtype=np.uint8)).to(device)


class PassOutputs:
    def __init__(self, batch, device="cuda:0", n_rows: Optional[int] = None):
        m = batch.model
        i32 = dict(dtype=torch.int32, device=device)
        self.out = torch.empty((batch.n_q_rows, m.n_q_heads, m.head_dim), dtype=torch.bfloat16, device=device)
        self.lse = torch.empty((batch.n_q_rows, m.n_q_heads), dtype=torch.float32, device=device)
        self.n_accept = torch.empty(batch.n_branch, **i32)
        self.bonus_id = torch.empty(batch.n_branch, **i32)
        n_rows = batch.n_logit_rows if n_rows is None else n_rows
        self.row_argmax = torch.empty(n_rows, **i32)
        self.scratch = B.Context.accept_scratch(n_rows, device)
        self.n_steps_accepted = torch.empty(batch.n_req, **i32)
        self.survivor = torch.empty(batch.n_req, **i32)
        self.committed_len = torch.empty(batch.n_req, **i32)
        self.keep_off = torch.empty(batch.n_req + 1, **i32)
        self.free_off = torch.empty(batch.n_req + 1, **i32)
        self.keep_pages = torch.full((batch.n_page_slots,), -1, **i32)
        self.keep_valid = torch.full((batch.n_page_slots,), -1, **i32)
        self.free_pages = torch.full((batch.n_page_slots,), -1, **i32)

    def commit_dict(self):
        d = {k: getattr(self, k).cpu().numpy() for k in
             ("n_steps_accepted", "survivor", "committed_len", "keep_off", "keep_pages", "keep_valid", "free_off", "free_pages")}
        nk, nf = int(d["keep_off"][-1]), int(d["free_off"][-1])
        d["keep_pages"], d["keep_valid"], d["free_pages"] = d["keep_pages"][:nk], d["keep_valid"][:nk], d["free_pages"][:nf]
        return d


def run_pass(ctx: B.Context, plan: B.Plan, x: DeviceInputs, y: PassOutputs, stream=None, want_lse=True, want_row_argmax=True):
    """One whole verify pass on device-resident inputs (three kernel launches)."""
    plan.lr_verify_attention(x.q, x.k_pool, x.v_pool, y.out, y.lse if want_lse else None, 0.0, stream)
    ctx.lr_accept_greedy(x.logits, x.draft_ids, x.cu_draft, y.n_accept, y.bonus_id, y.scratch,
                         y.row_argmax if want_row_argmax else None, stream)
    plan.lr_commit(x.verdict, y.n_accept, y.n_steps_accepted, y.survivor, y.committed_len, y.keep_off, y.keep_pages,
                   y.keep_valid, y.free_off, y.free_pages, stream)


def run_pass_overlapped(ctx: B.Context, plan: B.Plan, x: DeviceInputs, y: PassOutputs, side: torch.cuda.Stream,
                        k_pool=None, v_pool=None, logits=None):
    """One whole verify pass with the two independent chains on two streams: attention on the current
    stream, acceptance -> commit (which need nothing from attention) on ``side``; both are joined back
    into the current stream.  Works under CUDA-graph capture (fork/join through events)."""
    main = torch.cuda.current_stream()
    k_pool = x.k_pool if k_pool is None else k_pool
    v_pool = x.v_pool if v_pool is None else v_pool
    logits = x.logits if logits is None else logits
    fork = torch.cuda.Event()
    fork.record(main)
    side.wait_event(fork)
    with torch.cuda.stream(side):
        ctx.lr_accept_greedy(logits, x.draft_ids, x.cu_draft, y.n_accept, y.bonus_id, y.scratch, None, None)
        plan.lr_commit(x.verdict, y.n_accept, y.n_steps_accepted, y.survivor, y.committed_len, y.keep_off, y.keep_pages,
                       y.keep_valid, y.free_off, y.free_pages, None)
        join = torch.cuda.Event()
        join.record(side)
    plan.lr_verify_attention(x.q, k_pool, v_pool, y.out, None, 0.0, None)
    main.wait_event(join)
