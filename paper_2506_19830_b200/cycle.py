"""A synchronous Lookahead Reasoning cycle loop over a paged KV cache (Algorithm 1, one iteration per call).

Host bookkeeping only -- which physical pages a request owns, a free list, where new tokens go -- around the
library calls that do the work: ``lr_plan_create``, ``lr_verify_attention``, ``lr_accept_greedy``, ``lr_commit``
and ``lr_compact``.  The models are not here: the caller hands in, per cycle, the K/V of the drafted steps and of
every branch's tail, the queries, the logits and the step verdicts, as a serving engine would after running its
draft model, target model and verifier.

Invariant between cycles: request r's committed sequence of ``length[r]`` tokens sits densely in ``pages[r]``
(token k at slot k % 16 of page k // 16), which is what ``lr_compact`` leaves behind and what the next cycle's
prefix span needs.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence, Tuple

import numpy as np
import torch

from . import binding as B
from . import runner as R

PAGE = 16


@dataclass
class BranchInput:
    node: int  # number of leading draft steps the branch sees (the node it continues, with a tree)
    k_tail: np.ndarray  # uint16 [own_len, H_kv, D] bf16 bits of the branch's private tokens
    v_tail: np.ndarray
    q_len: int  # the last q_len tail tokens are queries
    n_draft: int  # token-level drafts verified for the branch


@dataclass
class RequestInput:
    segs: List[Tuple[np.ndarray, np.ndarray]]  # per draft step: (K, V) bits [len, H_kv, D]
    branches: List[BranchInput]
    parents: Sequence[int] = ()  # multi-branch drafting: the step each draft step continues (0 = prefix); empty = chain


class _HostBatch:
    """The fields ``binding.HostBatch`` reads."""

    def __init__(self, model, **kw):
        self.model = model
        self.__dict__.update(kw)


class PagedCycleEngine:
    def __init__(self, model, n_pool_pages: int, device: str = "cuda:0"):
        self.model, self.device = model, device
        self.ctx = B.Context(model, torch.device(device).index or 0)
        shape = (n_pool_pages, model.n_kv_heads, PAGE, model.head_dim)
        self.k_pool = torch.zeros(shape, dtype=torch.bfloat16, device=device)
        self.v_pool = torch.zeros(shape, dtype=torch.bfloat16, device=device)
        self.free: List[int] = list(range(n_pool_pages - 1, -1, -1))  # a stack: pop() hands out the lowest first
        self.pages: List[List[int]] = []
        self.length: List[int] = []

    # ---- page bookkeeping -------------------------------------------------------------------------------
    def _alloc(self, n_tokens: int) -> List[int]:
        n = (n_tokens + PAGE - 1) // PAGE
        if n > len(self.free):
            raise RuntimeError(f"KV pool exhausted: {n} pages wanted, {len(self.free)} free")
        return [self.free.pop() for _ in range(n)]

    def _write(self, pages: List[int], k_bits: np.ndarray, v_bits: np.ndarray) -> None:
        """Token t of the span goes to slot t % 16 of pages[t // 16]."""
        n = len(k_bits)
        if n == 0:
            return
        idx_page = torch.tensor([pages[t // PAGE] for t in range(n)], device=self.device)
        idx_slot = torch.arange(n, device=self.device) % PAGE
        self.k_pool[idx_page, :, idx_slot, :] = R.bf16_tensor(k_bits, self.device)
        self.v_pool[idx_page, :, idx_slot, :] = R.bf16_tensor(v_bits, self.device)

    def add_request(self, k_bits: np.ndarray, v_bits: np.ndarray) -> int:
        """A new request whose context so far is the given tokens; returns its index."""
        pages = self._alloc(len(k_bits))
        self._write(pages, k_bits, v_bits)
        self.pages.append(pages)
        self.length.append(len(k_bits))
        return len(self.pages) - 1

    def sequence(self, r: int) -> Tuple[np.ndarray, np.ndarray]:
        """The committed tokens of request r, gathered from its pages: two uint16 arrays [length, H_kv, D]."""
        n = self.length[r]
        idx_page = torch.tensor([self.pages[r][t // PAGE] for t in range(n)], device=self.device, dtype=torch.long)
        idx_slot = torch.arange(n, device=self.device) % PAGE
        return R.bf16_bits(self.k_pool[idx_page, :, idx_slot, :]), R.bf16_bits(self.v_pool[idx_page, :, idx_slot, :])

    # ---- one cycle ------------------------------------------------------------------------------------------
    def run_cycle(self, reqs: Sequence[RequestInput], q_bits: np.ndarray, logits_bits: np.ndarray, draft_ids: np.ndarray,
                  verdict: np.ndarray) -> dict:
        """Verify, commit and compact one cycle for every request (``reqs[r]`` belongs to request r; queries, logits
        rows, drafts and verdicts are packed in request, branch order as the C ABI wants them)."""
        assert len(reqs) == len(self.pages)
        page_ids: List[int] = []
        req_span_off, span_len, span_slot, seg_parent = [0], [], [], []
        br = {k: [] for k in ("br_req", "br_depth", "br_own_len", "br_own_slot", "br_n_draft")}
        cu_q = [0]
        tree = any(len(x.parents) for x in reqs)

        def place(pages: List[int]) -> int:
            first = len(page_ids)
            page_ids.extend(pages)
            return first

        for r, x in enumerate(reqs):
            span_len.append(self.length[r])
            span_slot.append(place(self.pages[r][: (self.length[r] + PAGE - 1) // PAGE]))
            seg_parent.append(-1)
            for c, (k, v) in enumerate(x.segs):
                pages = self._alloc(len(k))
                self._write(pages, k, v)
                span_len.append(len(k))
                span_slot.append(place(pages))
                seg_parent.append(int(x.parents[c]) if len(x.parents) else c)
            req_span_off.append(len(span_len))
            for b in x.branches:
                pages = self._alloc(len(b.k_tail))
                self._write(pages, b.k_tail, b.v_tail)
                br["br_req"].append(r)
                br["br_depth"].append(b.node)
                br["br_own_len"].append(len(b.k_tail))
                br["br_own_slot"].append(place(pages))
                br["br_n_draft"].append(b.n_draft)
                cu_q.append(cu_q[-1] + b.q_len)
        i32 = lambda a: np.asarray(a, dtype=np.int32)  # noqa: E731
        batch = _HostBatch(self.model, req_span_off=i32(req_span_off), span_len=i32(span_len), span_slot=i32(span_slot),
                           cu_q=i32(cu_q), page_ids=i32(page_ids), n_pool_pages=self.k_pool.shape[0],
                           seg_parent=i32(seg_parent) if tree else None, **{k: i32(v) for k, v in br.items()})
        n_req, n_branch, n_slots = len(reqs), len(br["br_req"]), len(page_ids)
        plan = B.Plan(self.ctx, batch)
        dev, i32t = self.device, dict(dtype=torch.int32, device=self.device)
        q = R.bf16_tensor(q_bits, dev)
        vocab = logits_bits.shape[1]
        stride = (vocab + 7) // 8 * 8
        logits = torch.zeros((logits_bits.shape[0], stride), dtype=torch.bfloat16, device=dev)
        logits[:, :vocab] = R.bf16_tensor(logits_bits, dev)
        cu_draft = torch.from_numpy(np.concatenate([[0], np.cumsum(br["br_n_draft"])]).astype(np.int32)).to(dev)
        out = torch.empty((cu_q[-1], self.model.n_q_heads, self.model.head_dim), dtype=torch.bfloat16, device=dev)
        n_accept, bonus = torch.empty(n_branch, **i32t), torch.empty(n_branch, **i32t)
        steps, surv, clen = (torch.empty(n_req, **i32t) for _ in range(3))
        keep_off, free_off = torch.empty(n_req + 1, **i32t), torch.empty(n_req + 1, **i32t)
        keep_pages, keep_valid, free_pages = (torch.empty(n_slots, **i32t) for _ in range(3))
        new_len, n_kept = torch.empty(n_req, **i32t), torch.empty(n_req, **i32t)
        v = verdict if len(verdict) else np.zeros(1, dtype=np.uint8)
        plan.lr_verify_attention(q, self.k_pool, self.v_pool, out, None, 0.0, None)
        self.ctx.lr_accept_greedy(logits[:, :vocab], torch.from_numpy(i32(draft_ids)).to(dev), cu_draft, n_accept, bonus,
                                  B.Context.accept_scratch(logits_bits.shape[0], dev), None, None)
        plan.lr_commit(torch.from_numpy(np.ascontiguousarray(v, dtype=np.uint8)).to(dev), n_accept, steps, surv, clen,
                       keep_off, keep_pages, keep_valid, free_off, free_pages, None)
        plan.lr_compact(keep_off, keep_pages, keep_valid, self.k_pool, self.v_pool, new_len, n_kept, plan.compact_scratch(), None)
        status = plan.lr_poll_status()  # synchronises the stream
        if status != 0:
            raise RuntimeError(f"device status {status} after the cycle")
        # the new page lists: the leading kept pages hold the sequence; everything else goes back to the free list
        ko, kp, fo, fp = (t.cpu().numpy() for t in (keep_off, keep_pages, free_off, free_pages))
        nl, nk = new_len.cpu().numpy(), n_kept.cpu().numpy()
        for r in range(n_req):
            kept = [int(p) for p in kp[ko[r]:ko[r + 1]]]
            self.pages[r] = kept[: int(nk[r])]
            self.length[r] = int(nl[r])
            self.free.extend(kept[int(nk[r]):])
            self.free.extend(int(p) for p in fp[fo[r]:fo[r + 1]])
        plan.close()
        return {"out": R.bf16_bits(out), "n_accept": n_accept.cpu().numpy(), "bonus_id": bonus.cpu().numpy(),
                "n_steps_accepted": steps.cpu().numpy(), "survivor": surv.cpu().numpy(), "committed_len": clen.cpu().numpy()}
