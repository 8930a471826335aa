"""The asynchronous variant of Lookahead Reasoning (Section 3.1, "Asynchronous Generation"; Appendix B, the three
rules of a stage) as a controller around the verify-pass library.

``AsyncStageController`` is the schedule alone, on the host: an event loop over an integer clock in which a target
step costs ``den`` units and a draft step ``num``.  Position i of a stage is started -- the draft model begins draft
step i and, at the same moment, the target model begins its own step i on the prefix that ends with draft i - 1 --
as soon as the draft model is free and fewer than gamma target generations are in flight; when the target's step i is
done the verifier's verdict for draft i is read, and the first rejected draft ends the stage: drafts 0..i-1 and the
target's step i are the output, whatever was started later is dropped.  It calls back into an executor at every event.

``AsyncCycleEngine`` is that executor on the paged KV cache: a target generation in flight is one verify pass for a
single branch (nested-prefix attention over the committed context, the draft steps before it and its own tail, then
greedy token-level acceptance), issued on a CUDA stream of its own the moment the controller starts the position
and read back when the controller says it is done; a finished draft step is written into fresh pages; the end of a
stage is ``lr_commit`` + ``lr_compact`` over everything the stage wrote, and the pages of dropped positions go back
to the free list.  The models are not here: the caller supplies, per position, the K/V of the draft step, the
branch's tail, queries, logits and draft ids, and the verifier's verdict, as the sync engine's caller does.
"""
from __future__ import annotations

import heapq
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Tuple

import numpy as np
import torch

from . import binding as B
from . import runner as R
from .cycle import PAGE, BranchInput, PagedCycleEngine, _HostBatch


class StageExecutor:
    """What the controller calls; every time is on the controller's integer clock."""

    def start_position(self, i: int, now: int) -> None:  # draft i and the target's step i begin
        pass

    def draft_done(self, i: int, now: int) -> None:  # draft step i exists (and its KV)
        pass

    def target_done(self, i: int, now: int) -> int:  # the target's step i is complete; returns the verdict for draft i
        raise NotImplementedError

    def end_stage(self, rejected_at: int, started: int, now: int) -> None:  # drafts 0..rejected_at-1 + target step rejected_at
        pass


class AsyncStageController:
    """Appendix B's three rules as an event loop.  ``run_stage`` returns when a draft has been rejected."""

    def __init__(self, gamma: int, num: int, den: int):
        assert gamma >= 1 and num >= 0 and den >= 1
        self.gamma, self.num, self.den = gamma, num, den
        self.now = 0
        self.stats = {"stages": 0, "steps": 0, "time": 0, "verdicts_used": 0, "peak_in_flight": 0}
        self.log: List[Tuple[int, str, int]] = []  # (time, event, position)

    def run_stage(self, ex: StageExecutor, max_positions: Optional[int] = None) -> Optional[int]:
        """One stage.  Returns the position whose draft was rejected, or None when ``max_positions`` positions were
        all accepted (the caller has no more drafts to offer: the stage is left open and nothing is committed)."""
        gamma, num, den = self.gamma, self.num, self.den
        t0 = self.now
        events: List[Tuple[int, int, int]] = []  # (time, kind, position); kind 0 = draft done, 1 = target done
        in_flight = 0
        next_pos = 0
        draft_free_at = t0
        verdicts_read = 0
        while True:
            # rule 1 and 2: start positions while the draft model is free and fewer than gamma generations are in flight
            while in_flight < gamma and draft_free_at <= self.now and (max_positions is None or next_pos < max_positions):
                ex.start_position(next_pos, self.now)
                self.log.append((self.now, "start", next_pos))
                heapq.heappush(events, (self.now + num, 0, next_pos))
                heapq.heappush(events, (self.now + den, 1, next_pos))
                draft_free_at = self.now + num
                in_flight += 1
                self.stats["peak_in_flight"] = max(self.stats["peak_in_flight"], in_flight)
                next_pos += 1
            if not events:
                return None
            t, kind, i = heapq.heappop(events)
            self.now = t
            if kind == 0:
                ex.draft_done(i, t)
                self.log.append((t, "draft", i))
                continue
            # rule 3: the target's step i is done, the verifier looks at draft i
            in_flight -= 1
            v = ex.target_done(i, t)
            verdicts_read += 1
            self.log.append((t, "accept" if v else "reject", i))
            if v:
                continue
            ex.end_stage(i, next_pos, t)
            self.stats["stages"] += 1
            self.stats["steps"] += i + 1
            self.stats["time"] += t - t0
            self.stats["verdicts_used"] += verdicts_read
            return i


@dataclass
class PositionInput:
    """What the caller's models produce for one position of a stage."""
    seg_k: np.ndarray  # draft step i: uint16 [len, H_kv, D] bf16 bits (K of its tokens under the target model)
    seg_v: np.ndarray
    branch: BranchInput  # the target's step i: its tail so far and the token-level drafts being verified
    q: np.ndarray  # uint16 [q_len, H_q, D]
    logits: np.ndarray  # uint16 [n_draft + 1, vocab]
    draft_ids: np.ndarray  # int32 [n_draft]
    verdict: int  # the verifier's verdict for draft step i against the target's step i


@dataclass
class _InFlight:
    plan: B.Plan
    stream: torch.cuda.Stream
    out: torch.Tensor
    n_accept: torch.Tensor
    bonus: torch.Tensor
    keep: tuple  # device tensors the pass reads, kept alive until it is read back
    tail_pages: List[int] = field(default_factory=list)
    own_len: int = 0
    n_draft: int = 0


class AsyncCycleEngine(PagedCycleEngine, StageExecutor):
    """One request on a paged cache, advanced stage by stage under ``AsyncStageController``."""

    def __init__(self, model, n_pool_pages: int, gamma: int, num: int, den: int, device: str = "cuda:0"):
        PagedCycleEngine.__init__(self, model, n_pool_pages, device)
        self.controller = AsyncStageController(gamma, num, den)
        self.streams = [torch.cuda.Stream(device=device) for _ in range(gamma)]  # one per generation in flight
        self._source: Optional[Callable[[int], PositionInput]] = None
        self.results: Dict[int, dict] = {}

    # ---- one stage --------------------------------------------------------------------------------------
    def run_stage(self, source: Callable[[int], PositionInput], max_positions: Optional[int] = None) -> dict:
        """Runs one stage of request 0.  ``source(i)`` is asked for position i when the controller starts it (its
        draft step may depend on nothing the stage has not produced yet).  Returns per-position results of the
        positions that finished and ``rejected_at``."""
        assert len(self.pages) == 1, "the asynchronous engine advances one request"
        self._source = source
        self._inputs: Dict[int, PositionInput] = {}
        self._seg_pages: Dict[int, List[int]] = {}
        self._flight: Dict[int, _InFlight] = {}
        self.results = {}
        self._stage: dict = {}
        rejected = self.controller.run_stage(self, max_positions)
        return {"rejected_at": rejected, "positions": self.results, **self._stage}

    # ---- StageExecutor -----------------------------------------------------------------------------------
    def start_position(self, i: int, now: int) -> None:
        x = self._source(i)
        self._inputs[i] = x
        # the target's step i: one branch over the committed context and draft steps 0..i-1 (all written by now: draft
        # i - 1 finished before this position could start)
        tail_pages = self._alloc(len(x.branch.k_tail))
        stream = self.streams[i % len(self.streams)]
        page_ids = list(self.pages[0][: (self.length[0] + PAGE - 1) // PAGE])
        span_len, span_slot = [self.length[0]], [0]
        for c in range(i):
            span_slot.append(len(page_ids))
            span_len.append(len(self._inputs[c].seg_k))
            page_ids.extend(self._seg_pages[c])
        own_slot = len(page_ids)
        page_ids.extend(tail_pages)
        i32 = lambda a: np.asarray(a, dtype=np.int32)  # noqa: E731
        batch = _HostBatch(self.model, req_span_off=i32([0, len(span_len)]), span_len=i32(span_len), span_slot=i32(span_slot),
                           cu_q=i32([0, x.branch.q_len]), page_ids=i32(page_ids), n_pool_pages=self.k_pool.shape[0], seg_parent=None,
                           br_req=i32([0]), br_depth=i32([i]), br_own_len=i32([len(x.branch.k_tail)]), br_own_slot=i32([own_slot]),
                           br_n_draft=i32([x.branch.n_draft]))
        dev = self.device
        main = torch.cuda.current_stream()
        stream.wait_stream(main)  # the draft steps before this position were written on the main stream
        with torch.cuda.stream(stream):
            self._write(tail_pages, x.branch.k_tail, x.branch.v_tail)
            plan = B.Plan(self.ctx, batch, stream)
            q = R.bf16_tensor(x.q, dev)
            vocab = x.logits.shape[1]
            stride = (vocab + 7) // 8 * 8
            logits = torch.zeros((x.logits.shape[0], stride), dtype=torch.bfloat16, device=dev)
            logits[:, :vocab] = R.bf16_tensor(x.logits, dev)
            drafts = torch.from_numpy(np.ascontiguousarray(x.draft_ids, dtype=np.int32)).to(dev)
            cu_draft = torch.tensor([0, x.branch.n_draft], dtype=torch.int32, device=dev)
            out = torch.empty((x.branch.q_len, self.model.n_q_heads, self.model.head_dim), dtype=torch.bfloat16, device=dev)
            n_accept = torch.empty(1, dtype=torch.int32, device=dev)
            bonus = torch.empty(1, dtype=torch.int32, device=dev)
            scratch = B.Context.accept_scratch(x.logits.shape[0], dev)
            plan.lr_verify_attention(q, self.k_pool, self.v_pool, out, None, 0.0, stream)
            self.ctx.lr_accept_greedy(logits[:, :vocab], drafts, cu_draft, n_accept, bonus, scratch, None, stream)
        self._flight[i] = _InFlight(plan, stream, out, n_accept, bonus, (q, logits, drafts, cu_draft, scratch), tail_pages,
                                    len(x.branch.k_tail), x.branch.n_draft)

    def draft_done(self, i: int, now: int) -> None:
        x = self._inputs[i]
        pages = self._alloc(len(x.seg_k))
        self._write(pages, x.seg_k, x.seg_v)  # on the main stream; later positions wait for it before they start
        self._seg_pages[i] = pages

    def target_done(self, i: int, now: int) -> int:
        f = self._flight[i]
        status = f.plan.lr_poll_status(f.stream)  # waits for this generation only
        if status != 0:
            raise RuntimeError(f"device status {status} in the pass of position {i}")
        self.results[i] = {"out": R.bf16_bits(f.out), "n_accept": int(f.n_accept.item()), "bonus_id": int(f.bonus.item()),
                           "finished_at": now}
        return int(self._inputs[i].verdict)

    def end_stage(self, rejected_at: int, started: int, now: int) -> None:
        """Commit the accepted drafts and the target's step at the rejected position; drop everything later."""
        dev = self.device
        for f in self._flight.values():  # generations still in flight are dropped, but their pages are reused below
            f.stream.synchronize()
        torch.cuda.current_stream().synchronize()
        # one batch over everything the stage wrote: the chain of draft steps written so far, one branch per started position
        n_seg = len(self._seg_pages)
        page_ids = list(self.pages[0][: (self.length[0] + PAGE - 1) // PAGE])
        span_len, span_slot = [self.length[0]], [0]
        for c in range(n_seg):
            span_slot.append(len(page_ids))
            span_len.append(len(self._inputs[c].seg_k))
            page_ids.extend(self._seg_pages[c])
        branches = [p for p in range(started) if p <= n_seg]  # a branch needs its draft prefix as segments
        br_slot, cu_q = [], [0]
        for p in branches:
            br_slot.append(len(page_ids))
            page_ids.extend(self._flight[p].tail_pages)
            cu_q.append(cu_q[-1] + self._inputs[p].branch.q_len)
        i32 = lambda a: np.asarray(a, dtype=np.int32)  # noqa: E731
        batch = _HostBatch(self.model, req_span_off=i32([0, len(span_len)]), span_len=i32(span_len), span_slot=i32(span_slot),
                           cu_q=i32(cu_q), page_ids=i32(page_ids), n_pool_pages=self.k_pool.shape[0], seg_parent=None,
                           br_req=i32([0] * len(branches)), br_depth=i32(branches),
                           br_own_len=i32([self._flight[p].own_len for p in branches]), br_own_slot=i32(br_slot),
                           br_n_draft=i32([self._flight[p].n_draft for p in branches]))
        plan = B.Plan(self.ctx, batch)
        i32t = dict(dtype=torch.int32, device=dev)
        # verdicts of the chain: drafts before the rejected one were accepted; the rest are not read by the commit
        verdict = np.zeros(max(1, n_seg), dtype=np.uint8)
        verdict[: min(rejected_at, n_seg)] = 1
        n_accept = torch.zeros(len(branches), **i32t)
        for k, p in enumerate(branches):
            if p in self.results:  # a pass that was read back; dropped generations contribute nothing
                n_accept[k] = self.results[p]["n_accept"]
        steps, surv, clen = (torch.empty(1, **i32t) for _ in range(3))
        keep_off, free_off = torch.empty(2, **i32t), torch.empty(2, **i32t)
        n_slots = len(page_ids)
        keep_pages, keep_valid, free_pages = (torch.empty(n_slots, **i32t) for _ in range(3))
        new_len, n_kept = torch.empty(1, **i32t), torch.empty(1, **i32t)
        plan.lr_commit(torch.from_numpy(verdict).to(dev), n_accept, steps, surv, clen, keep_off, keep_pages, keep_valid, free_off,
                       free_pages, None)
        plan.lr_compact(keep_off, keep_pages, keep_valid, self.k_pool, self.v_pool, new_len, n_kept, plan.compact_scratch(), None)
        if plan.lr_poll_status() != 0:
            raise RuntimeError("device status after the commit of a stage")
        ko, kp, fo, fp = (t.cpu().numpy() for t in (keep_off, keep_pages, free_off, free_pages))
        kept = [int(p) for p in kp[ko[0]:ko[1]]]
        nk = int(n_kept.item())
        self.pages[0] = kept[:nk]
        self.length[0] = int(new_len.item())
        self.free.extend(kept[nk:])
        self.free.extend(int(p) for p in fp[fo[0]:fo[1]])
        # tails of positions that had no segment prefix in the batch (started after the last finished draft) were never listed
        for p in range(started):
            if p not in branches:
                self.free.extend(self._flight[p].tail_pages)
        self._stage = {"n_steps_accepted": int(steps.item()), "survivor": int(surv.item()), "committed_len": int(clen.item())}
        plan.close()
        for f in self._flight.values():
            f.plan.close()
        self._flight = {}
