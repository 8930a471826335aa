"""Seeded workload generator for the Lookahead Reasoning verify pass.

One verify pass (Algorithm 1, the "in parallel do" block) sees, per request, a
shared token prefix x_{1:t}, a nested chain of gamma drafted reasoning steps
(segments S_1..S_gamma) and a set of branches; branch b sees the prefix, the
first ``depth`` segments and its own private tail, whose last ``q_len`` tokens
are the queries being verified.  This module produces that structure, a paged
bf16 KV cache with a shuffled page table, vocab-wide bf16 logits, draft ids and
step verdicts -- all from one ``numpy`` generator, in a fixed order.

Nothing here computes what the pass computes.  In particular the logits/draft
generator never takes an argmax: where a draft token is meant to match the
target's greedy token it *plants* a peak (a value above the clip range of the
background noise) at the draft id instead.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

PAGE = 16

CONFIG_NAMES = {
    1: "tiny",
    2: "32b_layer",
    3: "long_context",
    4: "tensor_core_regime",
    5: "ragged_serving",
}

# bf16 bit patterns used as poison in memory no visible token owns.
POISON_NAN = np.uint16(0x7FC0)
POISON_BIG = np.uint16(0x7F00)  # 1.7e38, finite
PEAK_VALUE = 8.0  # planted logit; background is clipped to +-CLIP
CLIP = 7.5


# --------------------------------------------------------------------------
# bf16 helpers (storage format only)
# --------------------------------------------------------------------------
def bf16_round(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round to nearest even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    out = (r >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = POISON_NAN
    return out


def bf16_to_f32(u: np.ndarray) -> np.ndarray:
    """bf16 bit pattern (uint16) -> float32, exact."""
    return (np.ascontiguousarray(u, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------
# containers
# --------------------------------------------------------------------------
@dataclass
class Model:
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    vocab: int
    page_size: int = PAGE

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


@dataclass
class Batch:
    """Integer description of one verify pass (all arrays int32, host)."""

    model: Model
    req_span_off: np.ndarray  # [R+1] chain spans of request r: span 0 = prefix, span c = segment c
    span_len: np.ndarray  # [n_span] tokens in the span
    span_slot: np.ndarray  # [n_span] first index into page_ids (ceil(len/16) slots)
    br_req: np.ndarray  # [B] owning request (non-decreasing)
    br_depth: np.ndarray  # [B] number of leading segments the branch sees
    br_own_len: np.ndarray  # [B] private-tail tokens (>= q_len)
    br_own_slot: np.ndarray  # [B] first index into page_ids for the tail
    br_n_draft: np.ndarray  # [B] L_b: token-level draft tokens verified for the branch
    cu_q: np.ndarray  # [B+1] query-row offsets
    page_ids: np.ndarray  # [n_page_slots] physical page numbers
    n_pool_pages: int
    # Multi-branch (tree) drafting: [n_span], for segment c of a request the local index (0 = prefix, else an
    # earlier segment) of the segment it continues; -1 at the prefix spans.  None = the nested chain (parent c - 1).
    # With a tree, br_depth[b] is the local index of the node branch b continues (0 = the prefix alone).
    seg_parent: Optional[np.ndarray] = None

    @property
    def n_req(self) -> int:
        return len(self.req_span_off) - 1

    @property
    def n_branch(self) -> int:
        return len(self.br_req)

    @property
    def n_span(self) -> int:
        return len(self.span_len)

    @property
    def n_page_slots(self) -> int:
        return len(self.page_ids)

    @property
    def n_q_rows(self) -> int:
        return int(self.cu_q[-1])

    @property
    def cu_draft(self) -> np.ndarray:
        out = np.zeros(self.n_branch + 1, dtype=np.int32)
        np.cumsum(self.br_n_draft, out=out[1:])
        return out

    @property
    def cu_verdict(self) -> np.ndarray:
        """Offsets of each request's gamma_r verdicts in the packed verdict vector."""
        return (self.req_span_off - np.arange(self.n_req + 1, dtype=np.int32)).astype(np.int32)

    @property
    def n_logit_rows(self) -> int:
        return int(self.br_n_draft.sum()) + self.n_branch

    @property
    def n_verified_tokens(self) -> int:
        return int(self.br_n_draft.sum())

    def kv_tokens(self) -> int:
        return int(self.span_len.sum() + self.br_own_len.sum())


@dataclass
class Tensors:
    q: Optional[np.ndarray] = None  # uint16 [n_q_rows, H_q, D]
    k_pool: Optional[np.ndarray] = None  # uint16 [n_pool_pages, H_kv, 16, D]
    v_pool: Optional[np.ndarray] = None
    logits: Optional[np.ndarray] = None  # uint16 [n_logit_rows, V]
    draft_ids: Optional[np.ndarray] = None  # int32 [sum L_b]
    verdict: Optional[np.ndarray] = None  # uint8 [sum gamma_r]
    match_len: Optional[np.ndarray] = None  # int32 [B]: match length the drafts were built to have


@dataclass
class Workload:
    name: str
    seed: int
    batch: Batch
    tensors: Tensors
    recipe: dict = field(default_factory=dict)


# --------------------------------------------------------------------------
# structure
# --------------------------------------------------------------------------
def _pages(n_tokens: int) -> int:
    return (int(n_tokens) + PAGE - 1) // PAGE


def build_batch(
    model: Model,
    requests: Sequence[dict],
    rng: np.random.Generator,
    shuffle: bool = True,
    extra_page_frac: float = 0.25,
) -> Batch:
    """Lay out page slots and tables.

    ``requests[r]`` = ``{"P": int, "segs": [len...], "branches": [(depth, own_len, q_len, n_draft), ...]}``,
    plus ``"parents": [parent of segment 1, ...]`` (0 = prefix) when any request is a tree.
    Every span (prefix, segment, tail) owns whole pages and starts at slot 0 of
    its first page; a physical page belongs to at most one span.
    """
    req_span_off = [0]
    span_len: List[int] = []
    span_slot: List[int] = []
    br_req: List[int] = []
    br_depth: List[int] = []
    br_own_len: List[int] = []
    br_own_slot: List[int] = []
    br_n_draft: List[int] = []
    cu_q = [0]
    slot = 0
    tree = any("parents" in req for req in requests)
    seg_parent: List[int] = []
    for r, req in enumerate(requests):
        seg_parent += [-1] + [int(v) for v in req.get("parents", range(len(req["segs"])))]
        for ln in [req["P"]] + list(req["segs"]):
            span_len.append(int(ln))
            span_slot.append(slot)
            slot += _pages(ln)
        req_span_off.append(len(span_len))
        for depth, own_len, q_len, n_draft in req["branches"]:
            br_req.append(r)
            br_depth.append(int(depth))
            br_own_len.append(int(own_len))
            br_own_slot.append(slot)
            br_n_draft.append(int(n_draft))
            cu_q.append(cu_q[-1] + int(q_len))
            slot += _pages(own_len)
    n_slots = slot
    n_pool = max(1, int(np.ceil(n_slots * (1.0 + extra_page_frac))))
    if shuffle:
        page_ids = rng.permutation(n_pool)[:n_slots].astype(np.int32)
    else:
        page_ids = np.arange(n_slots, dtype=np.int32)
    i32 = lambda a: np.asarray(a, dtype=np.int32)  # noqa: E731
    return Batch(
        model=model,
        req_span_off=i32(req_span_off),
        span_len=i32(span_len),
        span_slot=i32(span_slot),
        br_req=i32(br_req),
        br_depth=i32(br_depth),
        br_own_len=i32(br_own_len),
        br_own_slot=i32(br_own_slot),
        br_n_draft=i32(br_n_draft),
        cu_q=i32(cu_q),
        page_ids=page_ids,
        n_pool_pages=n_pool,
        seg_parent=i32(seg_parent) if tree else None,
    )


def _slot_tables(batch: Batch):
    """Per page slot: owning request and number of valid tokens."""
    n = batch.n_page_slots
    slot_req = np.zeros(n, dtype=np.int32)
    slot_valid = np.zeros(n, dtype=np.int32)

    def put(first, length, r):
        npg = _pages(length)
        if npg == 0:
            return
        slot_req[first : first + npg] = r
        slot_valid[first : first + npg] = PAGE
        rem = length - (npg - 1) * PAGE
        slot_valid[first + npg - 1] = rem

    for r in range(batch.n_req):
        for s in range(batch.req_span_off[r], batch.req_span_off[r + 1]):
            put(int(batch.span_slot[s]), int(batch.span_len[s]), r)
    for b in range(batch.n_branch):
        put(int(batch.br_own_slot[b]), int(batch.br_own_len[b]), int(batch.br_req[b]))
    return slot_req, slot_valid


def fill_kv(
    batch: Batch,
    rng: np.random.Generator,
    k_head_scale: Optional[np.ndarray] = None,
    poison: str = "nan",
):
    """K/V pools ``[n_pool_pages, H_kv, 16, D]`` as bf16 bit patterns.

    Valid tokens ~ N(0,1) (K optionally multiplied per (request, kv head) by
    ``k_head_scale[r, h]``); page slack beyond a span's length and pages no span
    references are filled with ``poison`` ("nan", "big" or "zero").
    """
    m = batch.model
    pv = {"nan": POISON_NAN, "big": POISON_BIG, "zero": np.uint16(0)}[poison]
    shape = (batch.n_pool_pages, m.n_kv_heads, PAGE, m.head_dim)
    slot_req, slot_valid = _slot_tables(batch)
    n = batch.n_page_slots
    tok = np.arange(PAGE, dtype=np.int32)
    slack = tok[None, :] >= slot_valid[:, None]  # [n_slots, 16]
    pools = []
    for which in ("k", "v"):
        pool = np.full(shape, pv, dtype=np.uint16)
        if n:
            x = rng.standard_normal((n, m.n_kv_heads, PAGE, m.head_dim), dtype=np.float32)
            if which == "k" and k_head_scale is not None:
                x *= k_head_scale[slot_req][:, :, None, None].astype(np.float32)
            xb = bf16_round(x)
            del x
            xb[np.broadcast_to(slack[:, None, :, None], xb.shape)] = pv
            pool[batch.page_ids] = xb
        pools.append(pool)
    return pools[0], pools[1]


def fill_q(batch: Batch, rng: np.random.Generator) -> np.ndarray:
    m = batch.model
    x = rng.standard_normal((batch.n_q_rows, m.n_q_heads, m.head_dim), dtype=np.float32)
    return bf16_round(x)


def fill_logits_and_drafts(
    batch: Batch,
    rng: np.random.Generator,
    p_mismatch: float,
    p_decoy: float = 0.25,
    p_tie: float = 0.25,
):
    """Background N(0,1) logits (clipped to +-7.5, bf16) with planted peaks.

    Per branch with L drafts (L+1 logits rows) a match length m is drawn with
    P(m = k) = (1-p)^k p, truncated at L (the geometric acceptance model of the
    paper's analysis, alpha = 1-p).  Rows i < m get a peak of 8.0 planted at a
    random id which becomes draft i (with probability ``p_tie`` a second, equal
    peak at a *higher* id, so only a lowest-index tie-break still matches).
    Row m is left as pure background and its draft id is a random id, so the
    target's greedy token there almost surely differs.  Rows after the mismatch
    get random drafts, a fraction ``p_decoy`` of them with a planted peak at the
    draft id (they would match, but lie behind the first mismatch).  The last
    row (no draft) is pure background.
    """
    V = batch.model.vocab
    n_rows = batch.n_logit_rows
    x = rng.standard_normal((n_rows, V), dtype=np.float32)
    np.clip(x, -CLIP, CLIP, out=x)
    logits = bf16_round(x)
    del x
    peak = bf16_round(np.array([PEAK_VALUE], dtype=np.float32))[0]
    cu = batch.cu_draft
    drafts = np.zeros(int(cu[-1]), dtype=np.int32)
    match_len = np.zeros(batch.n_branch, dtype=np.int32)
    for b in range(batch.n_branch):
        L = int(batch.br_n_draft[b])
        row0 = int(cu[b]) + b
        m = int(rng.geometric(p_mismatch)) - 1  # numpy counts trials, we count successes before failure
        m = min(m, L)
        match_len[b] = m
        for i in range(L):
            t = int(rng.integers(0, V))
            drafts[cu[b] + i] = t
            u_tie = rng.random()
            u_decoy = rng.random()
            if i < m:
                logits[row0 + i, t] = peak
                if u_tie < p_tie and t < V - 1:
                    t2 = int(rng.integers(t + 1, V))
                    logits[row0 + i, t2] = peak
            elif i > m and u_decoy < p_decoy:
                logits[row0 + i, t] = peak
    return logits, drafts, match_len


def fill_verdicts(batch: Batch, rng: np.random.Generator, p_accept: float) -> np.ndarray:
    n = int(batch.cu_verdict[-1])
    return (rng.random(n) < p_accept).astype(np.uint8)


# --------------------------------------------------------------------------
# the five configurations
# --------------------------------------------------------------------------
def _chain_request(P: int, segs: Sequence[int], L: int, carry_in: bool = False) -> dict:
    """Branch j (j = 1..gamma) sees segments 1..j; own_len = q_len = n_draft = L.  With ``carry_in`` the
    tail also holds the last accepted token in front of the L drafts and it is a query too (own_len = q_len
    = L + 1): the L + 1 query rows are then exactly the rows whose logits the acceptance step reads."""
    q = L + 1 if carry_in else L
    return {"P": P, "segs": list(segs), "branches": [(j, q, q, L) for j in range(1, len(segs) + 1)]}


def make_config(idx: int, seed: Optional[int] = None, with_logits: bool = True, with_kv: bool = True,
                poison: str = "nan", carry_in: bool = False) -> Workload:
    """Workload ``idx`` (1..5) of the benchmark suite; seed defaults to 20250619 + idx."""
    if seed is None:
        seed = 20250619 + idx
    rng = np.random.Generator(np.random.PCG64(seed))
    k_scale = None
    if idx == 1:
        model = Model(4, 1, 64, 1024)
        reqs = [_chain_request(256, [24, 24], 8, carry_in)]
        p_geo, p_ver = 0.3, 0.7
    elif idx == 2:
        model = Model(40, 8, 128, 152064)
        reqs = [_chain_request(4096, [32] * 3, 16, carry_in)]
        p_geo, p_ver = 0.25, 0.6
    elif idx == 3:
        model = Model(40, 8, 128, 152064)
        reqs = [_chain_request(16384, [48] * 4, 8, carry_in) for _ in range(4)]
        p_geo, p_ver = 0.25, 0.6
    elif idx == 4:
        model = Model(32, 8, 128, 152064)
        reqs = [_chain_request(32768, [40] * 6, 16, carry_in)]
        p_geo, p_ver = 0.2, 0.6
    elif idx == 5:
        model = Model(40, 8, 128, 152064)
        reqs = []
        for _ in range(16):
            P = int(rng.integers(1024, 16384 + 1))
            gamma = int(rng.integers(2, 6 + 1))
            segs = [int(v) for v in rng.integers(16, 64 + 1, size=gamma)]
            L = int(rng.choice([4, 8, 16]))
            reqs.append(_chain_request(P, segs, L, carry_in))
        p_geo, p_ver = 0.25, 0.6
    else:
        raise ValueError("config index must be 1..5")
    batch = build_batch(model, reqs, rng, shuffle=True)
    if idx == 3:
        k_scale = rng.uniform(0.5, 2.0, size=(batch.n_req, model.n_kv_heads)).astype(np.float32)
    t = Tensors()
    if with_kv:
        t.k_pool, t.v_pool = fill_kv(batch, rng, k_head_scale=k_scale, poison=poison)
        t.q = fill_q(batch, rng)
    if with_logits:
        t.logits, t.draft_ids, t.match_len = fill_logits_and_drafts(batch, rng, p_geo)
    t.verdict = fill_verdicts(batch, rng, p_ver)
    recipe = {"p_mismatch": p_geo, "p_step_accept": p_ver, "poison": poison, "carry_in": carry_in}
    return Workload(CONFIG_NAMES[idx], seed, batch, t, recipe)


def make_random_small(seed: int, head_dim: Optional[int] = None, max_prefix: int = 200,
                      vocab: Optional[int] = None, poison: str = "nan", shuffle: bool = True) -> Workload:
    """A small ragged batch that exercises the degenerate shapes.

    Random request count, prefix lengths including 0, zero to four segments with
    ragged lengths, branches of any depth 0..gamma (not necessarily distinct or
    ordered), tails longer than the query block, and draft counts that differ
    from the query count.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    if head_dim is None:
        head_dim = int(rng.choice([64, 128]))
    h_kv = int(rng.choice([1, 2, 4]))
    group = int(rng.choice([1, 2, 4, 5, 8]))
    if vocab is None:
        vocab = int(rng.choice([1000, 1024, 4099, 8192]))
    model = Model(h_kv * group, h_kv, head_dim, vocab)
    reqs = []
    for _ in range(int(rng.integers(1, 4))):
        P = int(rng.choice([0, 1, 15, 16, 17, int(rng.integers(0, max_prefix + 1))]))
        gamma = int(rng.integers(0, 5))
        segs = [int(v) for v in rng.integers(1, 41, size=gamma)]
        branches = []
        for _ in range(int(rng.integers(1, gamma + 3))):
            depth = int(rng.integers(0, gamma + 1))
            q_len = int(rng.integers(1, 10))
            own_len = q_len + int(rng.choice([0, 0, 1, 7, 20]))
            n_draft = int(rng.choice([q_len, max(1, q_len - 1), int(rng.integers(1, 9))]))
            n_draft = min(n_draft, own_len)  # drafts are tail tokens
            branches.append((depth, own_len, q_len, n_draft))
        reqs.append({"P": P, "segs": segs, "branches": branches})
    batch = build_batch(model, reqs, rng, shuffle=shuffle)
    t = Tensors()
    k_scale = rng.uniform(0.5, 2.0, size=(batch.n_req, model.n_kv_heads)).astype(np.float32)
    t.k_pool, t.v_pool = fill_kv(batch, rng, k_head_scale=k_scale, poison=poison)
    t.q = fill_q(batch, rng)
    t.logits, t.draft_ids, t.match_len = fill_logits_and_drafts(batch, rng, 0.3)
    t.verdict = fill_verdicts(batch, rng, 0.6)
    return Workload(f"random_small_{seed}", seed, batch, t, {"p_mismatch": 0.3, "p_step_accept": 0.6})


# --------------------------------------------------------------------------
# multi-branch (tree) drafting
# --------------------------------------------------------------------------
def _tree_request(P: int, W: int, gamma: int, seg_len, L: int) -> dict:
    """Full W-ary tree of draft steps, gamma levels deep, numbered level by level (so a parent precedes its
    children); one branch per node, the prefix alone included: the target continues every draft prefix."""
    parents: List[int] = []
    level = [0]
    for _ in range(gamma):
        nxt = []
        for node in level:
            for _ in range(W):
                parents.append(node)
                nxt.append(len(parents))
        level = nxt
    segs = [int(seg_len(i)) for i in range(len(parents))]
    return {"P": P, "segs": segs, "parents": parents, "branches": [(n, L, L, L) for n in range(len(parents) + 1)]}


def _finish(name: str, seed: int, model: Model, reqs, rng, p_geo: float, p_ver: float, with_logits: bool,
            with_kv: bool, poison: str) -> Workload:
    batch = build_batch(model, reqs, rng, shuffle=True)
    t = Tensors()
    if with_kv:
        k_scale = rng.uniform(0.5, 2.0, size=(batch.n_req, model.n_kv_heads)).astype(np.float32)
        t.k_pool, t.v_pool = fill_kv(batch, rng, k_head_scale=k_scale, poison=poison)
        t.q = fill_q(batch, rng)
    if with_logits:
        t.logits, t.draft_ids, t.match_len = fill_logits_and_drafts(batch, rng, p_geo)
    t.verdict = fill_verdicts(batch, rng, p_ver)
    return Workload(name, seed, batch, t, {"p_mismatch": p_geo, "p_step_accept": p_ver, "poison": poison})


def make_tree(W: int, gamma: int, seed: Optional[int] = None, size: str = "layer", with_logits: bool = True,
              with_kv: bool = True, poison: str = "nan") -> Workload:
    """Tree-drafting workloads.  ``size`` "tiny": the geometry of config 1 (prefix 250, ragged segments);
    "layer": the geometry of config 2 (one request, prefix 4096, segments of 32, L = 16);
    "serving": 8 requests with the ragged lengths of config 5."""
    if seed is None:
        seed = 20250700 + 16 * W + gamma
    rng = np.random.Generator(np.random.PCG64(seed))
    if size == "tiny":
        model = Model(4, 1, 64, 1024)
        reqs = [_tree_request(250, W, gamma, lambda i: rng.integers(5, 40), 8)]
    elif size == "layer":
        model = Model(40, 8, 128, 152064)
        reqs = [_tree_request(4096, W, gamma, lambda i: 32, 16)]
    elif size == "serving":
        model = Model(40, 8, 128, 152064)
        reqs = [_tree_request(int(rng.integers(1024, 16384 + 1)), W, gamma, lambda i: rng.integers(16, 64 + 1),
                              int(rng.choice([4, 8, 16]))) for _ in range(8)]
    else:
        raise ValueError("size must be tiny, layer or serving")
    return _finish(f"tree_w{W}_g{gamma}_{size}", seed, model, reqs, rng, 0.25, 0.6, with_logits, with_kv, poison)


def make_random_tree(seed: int, head_dim: Optional[int] = None, poison: str = "nan", max_nodes: int = 8) -> Workload:
    """Small ragged batches of irregular trees: every segment picks any earlier node as its parent (so chains,
    stars and everything between occur), branches hang off arbitrary nodes, some nodes have none, some several;
    one request in three is a plain chain written as a tree."""
    rng = np.random.Generator(np.random.PCG64(seed))
    if head_dim is None:
        head_dim = int(rng.choice([64, 128]))
    h_kv = int(rng.choice([1, 2]))
    group = int(rng.choice([1, 2, 4, 5, 8]))
    model = Model(h_kv * group, h_kv, head_dim, int(rng.choice([1000, 1024, 4099])))
    reqs = []
    for _ in range(int(rng.integers(1, 4))):
        P = int(rng.choice([0, 1, 16, 17, int(rng.integers(0, 201))]))
        n = int(rng.integers(0, max_nodes + 1))
        chain = rng.random() < 1 / 3
        parents = [c if chain else int(rng.integers(0, c + 1)) for c in range(n)]
        segs = [int(v) for v in rng.integers(1, 41, size=n)]
        branches = []
        for _ in range(int(rng.integers(1, n + 3))):
            q_len = int(rng.integers(1, 10))
            own_len = q_len + int(rng.choice([0, 0, 1, 7, 20]))
            n_draft = min(own_len, int(rng.choice([q_len, max(1, q_len - 1), int(rng.integers(1, 9))])))
            branches.append((int(rng.integers(0, n + 1)), own_len, q_len, n_draft))
        reqs.append({"P": P, "segs": segs, "parents": parents, "branches": branches})
    return _finish(f"random_tree_{seed}", seed, model, reqs, rng, 0.3, 0.6, True, True, poison)


def make_random_mid(seed: int) -> Workload:
    """Mid-size ragged batches (1-6 requests, contexts of 100-6000 tokens, 1-5 draft steps as a chain or a tree,
    several head geometries with head_dim 128): a few to a few dozen key tiles per SM, i.e. both sides of the point
    where the attention plan switches between its two ways of grouping query tiles."""
    rng = np.random.Generator(np.random.PCG64(9000 + seed))
    hq, hkv = [(40, 8), (16, 4), (8, 8), (32, 8), (5, 1)][seed % 5]
    model = Model(hq, hkv, 128, int(rng.choice([1000, 4099])))
    reqs = []
    for _ in range(int(rng.integers(1, 7))):
        gamma = int(rng.integers(1, 6))
        L = int(rng.choice([4, 8, 16]))
        req = {"P": int(rng.integers(100, 6000)), "segs": [int(v) for v in rng.integers(8, 80, size=gamma)]}
        if rng.random() < 0.4:
            req["parents"] = [int(rng.integers(0, c + 1)) for c in range(gamma)]
            req["branches"] = ([(n, L + int(rng.choice([0, 3])), L, L) for n in range(gamma + 1) if rng.random() < 0.8]
                               or [(0, L, L, L)])
        else:
            req["branches"] = [(j, L, L, L) for j in range(1, gamma + 1)]
        reqs.append(req)
    if any("parents" in r for r in reqs):  # one batch is a chain batch or a tree batch
        for r in reqs:
            r.setdefault("parents", list(range(len(r["segs"]))))
    return _finish(f"random_mid_{seed}", seed, model, reqs, rng, 0.3, 0.6, True, True, "nan")
