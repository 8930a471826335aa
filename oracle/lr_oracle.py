"""CPU fp64 oracle for the step-parallel verification pass of Lookahead Reasoning.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
verify pass computes; tests, the smoke check and the benchmark's CPU-baseline
leg are its only callers.  It shares no code with the CUDA path and imports
nothing from it.  All floating point is float64; bf16 inputs are widened
exactly.  numpy matmul / argmax serve as steps; there is no tiling, fusion or
reordering.

What is computed, and where the paper fixes it:

* ``verify_attention``  -- Algorithm 1, the "in parallel do" block: target step
  s_j is generated from the prefix x'_j = x_{1:t} (+) s^_0 .. s^_{j-1}.  A
  branch of depth d therefore attends to the shared prefix, the first d draft
  step segments and, causally, its own tokens (the L token-level drafts being
  verified in one forward pass, Background "Speculative Decoding").  The
  attention itself is ordinary softmax(q K^T / sqrt(D)) V with grouped-query
  heads; the paper gives no tensor-level detail, so those are readings
  (documented with the design).
* ``accept_greedy``     -- Background "Speculative Decoding": drafts are checked
  in order, the process halts at the first rejected one and one more token is
  taken from the target distribution at that position.  Greedy reading: a draft
  is accepted iff it equals the argmax of the target logits (lowest index on
  ties); the extra ("bonus") token is the argmax of the row where it halted.
* ``accept_sample``     -- the same passage read literally: rejection sampling with acceptance
  probability min(1, P/Q) and a final token from the residual distribution, for point-mass draft
  distributions (prompt-lookup drafts, the paper's SD method), temperature sampling, random numbers
  passed in.
* ``compact``           -- the step after the output construction: the committed sequence, scattered
  over partly filled pages, rewritten densely into its leading kept pages (no arithmetic on values).
* ``commit``            -- Algorithm 1, last two lines: j* = min({j : V(s_j, s^_j)
  = False} U {gamma}); output = s^_0 .. s^_{j*-1} (+) s_{j*}.  On the KV cache
  this keeps the prefix pages, the pages of the first j* segments and the pages
  holding the kept part of the decisive branch's tail; every other page of the
  request is freed.

Pins (tests/test_oracle_*.py): textbook decode attention, torch SDPA causal
attention on each branch's concatenated sequence, closed forms that expose the
visibility sets, brute force over explicit token lists, LSE merge identity,
page-permutation / poison invariance; acceptance against pure-Python scans,
all 2^L match patterns and the (1-a^{L+1})/(1-a) mean; stochastic acceptance against the
exactness theorem of speculative sampling (output distribution = target distribution, by
integrating over the uniforms), a hand-computed example, its greedy limit and scipy's softmax; commit against an
independent token-level list model and the closed-form E[j*].
"""
from __future__ import annotations

import math
from typing import List, Optional, Tuple

import numpy as np

PAGE = 16


def bf16_bits_to_f64(u: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    u32 = np.ascontiguousarray(u, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u32.view(np.float32).astype(np.float64)


# ---------------------------------------------------------------------------
# a1. nested-prefix attention
# ---------------------------------------------------------------------------
def node_path(batch, r: int, node: int) -> List[int]:
    """Draft steps (local span indices of request ``r``) between the prefix and ``node``, ``node`` included, in
    sequence order.  On the nested chain of Algorithm 1 that is 1..node.  With multi-branch drafting (Section 3,
    "Multi-Branch Drafting") every draft step continues one earlier step, or the prefix, named by ``seg_parent``;
    the draft prefix of a node is then the steps met walking up to the prefix, reversed."""
    parent = getattr(batch, "seg_parent", None)
    if parent is None:
        return list(range(1, node + 1))
    s0 = int(batch.req_span_off[r])
    up = []
    while node != 0:
        up.append(node)
        node = int(parent[s0 + node])
    return up[::-1]


def branch_token_table(batch, b: int) -> Tuple[np.ndarray, np.ndarray, int]:
    """Physical (page, in-page offset) of every token branch ``b`` can ever see, in
    sequence order: prefix, the draft steps in front of it, then its own tail.  Returns
    (pages, offsets, N_b) with N_b the number of chain tokens (prefix+segments).

    Follows x'_j = x_{1:t} (+) s^_0..s^_{j-1} (Algorithm 1) with j = depth; with a tree of
    draft steps the steps are those on the way to the node the branch continues.
    """
    r = int(batch.br_req[b])
    s0 = int(batch.req_span_off[r])
    depth = int(batch.br_depth[b])
    pages: List[np.ndarray] = []
    offs: List[np.ndarray] = []

    def walk(first_slot: int, n_tok: int):
        t = np.arange(n_tok, dtype=np.int64)
        pages.append(np.asarray(batch.page_ids)[first_slot + t // PAGE].astype(np.int64))
        offs.append(t % PAGE)

    for c in [0] + node_path(batch, r, depth):  # span 0 is the prefix, span c is segment c
        walk(int(batch.span_slot[s0 + c]), int(batch.span_len[s0 + c]))
    n_chain = int(sum(len(p) for p in pages))
    walk(int(batch.br_own_slot[b]), int(batch.br_own_len[b]))
    return np.concatenate(pages), np.concatenate(offs), n_chain


def verify_attention(batch, q_bits, k_pool_bits, v_pool_bits, scale: Optional[float] = None,
                     return_weights: bool = False, branches=None):
    """O[row, h, :] and LSE[row, h] for every query row (float64).

    For branch b, query i (i = 0..q_len-1) sits at position
    p_i = N_b + own_len_b - q_len_b + i of the branch's own sequence and sees
    positions 0..p_i.  Rows of branches not in ``branches`` (default: all) are
    left as NaN.  With ``return_weights`` also returns {(row, h): softmax weights}.
    """
    m = batch.model
    H_q, H_kv, D = m.n_q_heads, m.n_kv_heads, m.head_dim
    G = H_q // H_kv
    if scale is None or scale <= 0:
        scale = 1.0 / math.sqrt(D)
    n_rows = int(batch.cu_q[-1])
    out = np.full((n_rows, H_q, D), np.nan, dtype=np.float64)
    lse = np.full((n_rows, H_q), np.nan, dtype=np.float64)
    weights = {}
    q = bf16_bits_to_f64(q_bits).reshape(n_rows, H_q, D)
    todo = range(batch.n_branch) if branches is None else branches
    for b in todo:
        pages, offs, n_chain = branch_token_table(batch, b)
        own_len = int(batch.br_own_len[b])
        row0, row1 = int(batch.cu_q[b]), int(batch.cu_q[b + 1])
        q_len = row1 - row0
        # 1. gather the branch's own contiguous sequence
        K_b = bf16_bits_to_f64(k_pool_bits[pages, :, offs, :])  # [N, H_kv, D]
        V_b = bf16_bits_to_f64(v_pool_bits[pages, :, offs, :])
        n_tot = n_chain + own_len
        pos = n_chain + own_len - q_len + np.arange(q_len)  # p_i
        visible = np.arange(n_tot)[None, :] <= pos[:, None]  # [q_len, N]
        for h in range(H_q):
            kv = h // G
            # 2. scores, softmax, weighted sum
            s = scale * (q[row0:row1, h, :] @ K_b[:, kv, :].T)  # [q_len, N]
            s = np.where(visible, s, -np.inf)
            mx = s.max(axis=1, keepdims=True)
            w = np.exp(s - mx)
            den = w.sum(axis=1, keepdims=True)
            out[row0:row1, h, :] = (w @ V_b[:, kv, :]) / den
            lse[row0:row1, h] = (mx + np.log(den))[:, 0]
            if return_weights:
                for i in range(q_len):
                    weights[(row0 + i, h)] = (w[i] / den[i])[: pos[i] + 1]
    if return_weights:
        return out, lse, weights
    return out, lse


# ---------------------------------------------------------------------------
# a2. greedy token-level acceptance
# ---------------------------------------------------------------------------
def row_argmax(logits_bits: np.ndarray) -> np.ndarray:
    """Greedy target token of every logits row: index of the maximum, lowest index
    on ties, +0 == -0, NaN ranked as -inf (so an all-NaN row gives 0)."""
    x = bf16_bits_to_f64(logits_bits)
    x = np.where(np.isnan(x), -np.inf, x)
    return np.argmax(x, axis=1).astype(np.int32)  # numpy returns the first maximum


def accept_greedy(logits_bits: np.ndarray, draft_ids: np.ndarray, cu_draft: np.ndarray):
    """Per branch b with L_b drafts and L_b+1 logits rows (rows cu_draft[b]+b ...):
    n_b = number of leading drafts equal to the target's greedy token, bonus_b =
    the target's greedy token at row n_b.  Returns (n_accept, bonus_id, row_argmax).
    """
    t = row_argmax(logits_bits)
    B = len(cu_draft) - 1
    n_accept = np.zeros(B, dtype=np.int32)
    bonus = np.zeros(B, dtype=np.int32)
    for b in range(B):
        L = int(cu_draft[b + 1] - cu_draft[b])
        row0 = int(cu_draft[b]) + b
        n = 0
        while n < L and int(draft_ids[cu_draft[b] + n]) == int(t[row0 + n]):
            n += 1  # accepted; move to the next draft
        n_accept[b] = n  # halted at the first mismatch (or ran out of drafts)
        bonus[b] = t[row0 + n]  # one more token from the target at that position
    return n_accept, bonus, t


# ---------------------------------------------------------------------------
# a3. step-level commit
# ---------------------------------------------------------------------------
def commit(batch, verdict: np.ndarray, n_accept: np.ndarray):
    """Step-level output construction on the paged cache.

    Per request with gamma draft steps and verdicts V_0..V_{gamma-1}:
    j* = min({j : V_j False} U {gamma}).  The decisive target step s_{j*} is the
    branch of depth j* (lowest branch index if several, none -> -1).  Kept KV =
    prefix, segments 1..j*, and the first kept_tail = own_len - L + n_accept
    tokens of that branch's tail.  Returns a dict of per-request arrays and CSR
    keep / free page lists:

    keep order: prefix pages, segment pages 1..j*, kept tail pages (table order);
    free order: pages of segments j*+1..gamma, then branch tails in branch order
    (for the decisive branch only the pages past its kept ones).
    """
    if getattr(batch, "seg_parent", None) is not None:
        return _commit_tree(batch, verdict, n_accept)
    R = batch.n_req
    cu_v = batch.cu_verdict
    cu_d = batch.cu_draft
    n_steps = np.zeros(R, dtype=np.int32)
    survivor = np.full(R, -1, dtype=np.int32)
    committed = np.zeros(R, dtype=np.int32)
    keep_off, free_off = [0], [0]
    keep_pages: List[int] = []
    keep_valid: List[int] = []
    free_pages: List[int] = []

    def span_pages(first_slot: int, n_tok: int):
        npg = (n_tok + PAGE - 1) // PAGE
        return [(int(batch.page_ids[first_slot + p]), min(PAGE, n_tok - p * PAGE)) for p in range(npg)]

    for r in range(R):
        s0, s1 = int(batch.req_span_off[r]), int(batch.req_span_off[r + 1])
        gamma = s1 - s0 - 1
        V = [bool(verdict[cu_v[r] + j]) for j in range(gamma)]
        j_star = min([j for j in range(gamma) if not V[j]] + [gamma])
        n_steps[r] = j_star
        branches = [b for b in range(batch.n_branch) if int(batch.br_req[b]) == r]
        decisive = [b for b in branches if int(batch.br_depth[b]) == j_star]
        s = decisive[0] if decisive else -1
        survivor[r] = s
        length = 0
        for c in range(0, j_star + 1):  # prefix and accepted draft steps
            ln = int(batch.span_len[s0 + c])
            length += ln
            for pg, val in span_pages(int(batch.span_slot[s0 + c]), ln):
                keep_pages.append(pg)
                keep_valid.append(val)
        kept_tail = 0
        if s >= 0:
            L = int(cu_d[s + 1] - cu_d[s])
            kept_tail = int(batch.br_own_len[s]) - L + int(n_accept[s])
            length += kept_tail
            for pg, val in span_pages(int(batch.br_own_slot[s]), kept_tail):
                keep_pages.append(pg)
                keep_valid.append(val)
        committed[r] = length
        for c in range(j_star + 1, gamma + 1):  # rejected draft steps
            for pg, _ in span_pages(int(batch.span_slot[s0 + c]), int(batch.span_len[s0 + c])):
                free_pages.append(pg)
        for b in branches:
            pages = span_pages(int(batch.br_own_slot[b]), int(batch.br_own_len[b]))
            skip = (kept_tail + PAGE - 1) // PAGE if b == s else 0
            for pg, _ in pages[skip:]:
                free_pages.append(pg)
        keep_off.append(len(keep_pages))
        free_off.append(len(free_pages))
    i32 = lambda a: np.asarray(a, dtype=np.int32)  # noqa: E731
    return {
        "n_steps_accepted": n_steps,
        "survivor": survivor,
        "committed_len": committed,
        "keep_off": i32(keep_off),
        "keep_pages": i32(keep_pages),
        "keep_valid": i32(keep_valid),
        "free_off": i32(free_off),
        "free_pages": i32(free_pages),
    }


def _commit_tree(batch, verdict: np.ndarray, n_accept: np.ndarray):
    """Commit with multi-branch drafting (Section 3, "Multi-Branch Drafting").

    Verdict c - 1 of a request says whether draft step c agrees with the step the target wrote as the
    continuation of c's parent.  Starting at the prefix, the walk moves to a child whose verdict is True -- the
    lowest-numbered one if several agree; the others are discarded -- and stops where no child agrees.  j* is the
    number of moves, the decisive target step is the branch that continues the node where the walk stopped
    (lowest index; -1 if none), and the kept KV is the prefix, the steps walked through and that branch's
    kept tail.  Lists: keep in sequence order; free = every other draft step in index order, then the tails in
    branch order (the decisive branch: only pages past its kept ones).  On a chain this is Algorithm 1's rule.
    """
    R = batch.n_req
    cu_v, cu_d = batch.cu_verdict, batch.cu_draft
    out = {k: [] for k in ("n_steps_accepted", "survivor", "committed_len")}
    keep_off, free_off = [0], [0]
    keep_pages: List[int] = []
    keep_valid: List[int] = []
    free_pages: List[int] = []

    def span_pages(first_slot: int, n_tok: int):
        npg = (n_tok + PAGE - 1) // PAGE
        return [(int(batch.page_ids[first_slot + p]), min(PAGE, n_tok - p * PAGE)) for p in range(npg)]

    for r in range(R):
        s0, s1 = int(batch.req_span_off[r]), int(batch.req_span_off[r + 1])
        n_seg = s1 - s0 - 1
        node, walked = 0, []
        while True:
            agreeing = [c for c in range(1, n_seg + 1)
                        if int(batch.seg_parent[s0 + c]) == node and bool(verdict[cu_v[r] + c - 1])]
            if not agreeing:
                break
            node = agreeing[0]
            walked.append(node)
        branches = [b for b in range(batch.n_branch) if int(batch.br_req[b]) == r]
        decisive = [b for b in branches if int(batch.br_depth[b]) == node]
        s = decisive[0] if decisive else -1
        length = 0
        for c in [0] + walked:
            ln = int(batch.span_len[s0 + c])
            length += ln
            for pg, val in span_pages(int(batch.span_slot[s0 + c]), ln):
                keep_pages.append(pg)
                keep_valid.append(val)
        kept_tail = 0
        if s >= 0:
            kept_tail = int(batch.br_own_len[s]) - int(cu_d[s + 1] - cu_d[s]) + int(n_accept[s])
            length += kept_tail
            for pg, val in span_pages(int(batch.br_own_slot[s]), kept_tail):
                keep_pages.append(pg)
                keep_valid.append(val)
        for c in range(1, n_seg + 1):
            if c not in walked:
                free_pages += [pg for pg, _ in span_pages(int(batch.span_slot[s0 + c]), int(batch.span_len[s0 + c]))]
        for b in branches:
            pages = span_pages(int(batch.br_own_slot[b]), int(batch.br_own_len[b]))
            skip = (kept_tail + PAGE - 1) // PAGE if b == s else 0
            free_pages += [pg for pg, _ in pages[skip:]]
        out["n_steps_accepted"].append(len(walked))
        out["survivor"].append(s)
        out["committed_len"].append(length)
        keep_off.append(len(keep_pages))
        free_off.append(len(free_pages))
    i32 = lambda a: np.asarray(a, dtype=np.int32)  # noqa: E731
    return {**{k: i32(v) for k, v in out.items()}, "keep_off": i32(keep_off), "keep_pages": i32(keep_pages),
            "keep_valid": i32(keep_valid), "free_off": i32(free_off), "free_pages": i32(free_pages)}


# ---------------------------------------------------------------------------
# a2'. stochastic token-level acceptance (rejection sampling)
# ---------------------------------------------------------------------------
def target_probs(logits_row_bits: np.ndarray, temperature: float) -> np.ndarray:
    """P = softmax(logits / T) of one row, float64 (NaN logits count as -inf)."""
    x = bf16_bits_to_f64(logits_row_bits) / float(temperature)
    x = np.where(np.isnan(x), -np.inf, x)
    w = np.exp(x - x.max())
    return w / w.sum()


def sample_inverse_cdf(weights: np.ndarray, u: float) -> int:
    """Smallest index v with cumsum(weights)[v] > u * sum(weights)  (u in [0, 1))."""
    c = np.cumsum(weights)
    return int(np.searchsorted(c, u * c[-1], side="right"))


def filter_probs(P: np.ndarray, top_k: int = 0, top_p: float = 1.0) -> np.ndarray:
    """The sampling filters of Section 4, "Setup" (top_k 20, top_p 0.95 with the temperature): tokens are ranked by
    probability, highest first, equal probabilities by lower index first.  top_k > 0 keeps the first top_k of the
    ranking and renormalises; top_p < 1 then keeps the shortest leading part of the ranking whose mass reaches top_p
    -- the token of rank r stays iff the tokens ranked before it hold less than top_p -- and renormalises again.
    Returns the filtered distribution (zeros outside the kept set)."""
    V = len(P)
    order = np.lexsort((np.arange(V), -P))  # by probability descending, then index ascending
    keep = np.ones(V, dtype=bool)
    if top_k and top_k > 0:
        keep[order[top_k:]] = False
    P1 = np.where(keep, P, 0.0)
    P1 = P1 / P1.sum()
    if top_p < 1.0:
        ranked = P1[order]
        before = np.concatenate([[0.0], np.cumsum(ranked)[:-1]])  # mass of the tokens ranked ahead
        stay = before < top_p
        stay[0] = True
        keep2 = np.zeros(V, dtype=bool)
        keep2[order[stay]] = True
        P1 = np.where(keep2, P1, 0.0)
        P1 = P1 / P1.sum()
    return P1


def accept_sample(logits_bits: np.ndarray, draft_ids: np.ndarray, cu_draft: np.ndarray, temperature: float,
                  u_accept: np.ndarray, u_final: np.ndarray, top_k: int = 0, top_p: float = 1.0):
    """Rejection sampling of Background, "Speculative Decoding", for drafts whose draft distribution Q
    is a point mass at the drafted token (prompt-lookup / n-gram drafts, the paper's SD method):

    drafts are processed in order; draft i is accepted with probability min(1, P_i(d_i) / Q_i(d_i)) =
    P_i(d_i), here iff u_accept[i] < P_i(d_i); at the first rejection the process halts and the final
    token is sampled from the normalised max(0, P_i - Q_i), i.e. P_i with the rejected token removed;
    if every draft is accepted the final token is sampled from P of the extra row.  Sampling is by
    inverse CDF with u_final[b].  A draft id outside the vocabulary has probability 0.
    With top_k > 0 or top_p < 1 the target distribution P_i is the filtered one (``filter_probs``): a draft
    outside the kept set has probability 0 and is never accepted, and the final token comes from the kept set.
    Returns (n_accept, final_id, p_draft) with p_draft[i] = P_i(d_i).
    """
    filtered = (top_k and top_k > 0) or top_p < 1.0

    def probs(row):
        P = target_probs(logits_bits[row], temperature)
        return filter_probs(P, top_k, top_p) if filtered else P

    V = logits_bits.shape[1]
    B = len(cu_draft) - 1
    n_accept = np.zeros(B, dtype=np.int32)
    final_id = np.zeros(B, dtype=np.int32)
    p_draft = np.zeros(int(cu_draft[-1]), dtype=np.float64)
    for b in range(B):
        d0, L = int(cu_draft[b]), int(cu_draft[b + 1] - cu_draft[b])
        row0 = d0 + b
        n = 0
        residual = None
        while n < L:
            P = probs(row0 + n)
            d = int(draft_ids[d0 + n])
            pd = P[d] if 0 <= d < V else 0.0
            p_draft[d0 + n] = pd
            if float(u_accept[d0 + n]) < pd:
                n += 1  # accepted; next draft
                continue
            residual = P.copy()  # rejected: halt, resample from P with the rejected token removed
            if 0 <= d < V:
                residual[d] = 0.0
            break
        if residual is None:  # all accepted: one more token from the target
            residual = probs(row0 + L)
        n_accept[b] = n
        final_id[b] = sample_inverse_cdf(residual, float(u_final[b]))
    return n_accept, final_id, p_draft


# ---------------------------------------------------------------------------
# a3'. compaction of the committed KV (the step after commit)
# ---------------------------------------------------------------------------
def compact(keep_off: np.ndarray, keep_pages: np.ndarray, keep_valid: np.ndarray, k_pool_bits: np.ndarray,
            v_pool_bits: np.ndarray):
    """After the output construction of Algorithm 1 the committed sequence of a request lies in its kept
    pages, some of them partly filled (the last page of the prefix, of every accepted segment and of the
    kept tail).  Compaction rewrites it densely: token k of the committed sequence goes to slot k % 16 of
    the request's kept page number k // 16, so that the sequence is one span again (the shared prefix of
    the next cycle).  Returns (new_len, n_pages_kept, k_pool, v_pool): per request its length and the number
    of leading pages of its keep list that now hold it (the rest of the list is no longer needed); the
    pools are modified copies.  Bytes outside the first new_len tokens of those pages are unspecified.
    """
    R = len(keep_off) - 1
    k_out, v_out = k_pool_bits.copy(), v_pool_bits.copy()
    new_len = np.zeros(R, dtype=np.int32)
    n_kept = np.zeros(R, dtype=np.int32)
    for r in range(R):
        pages = [int(p) for p in keep_pages[keep_off[r] : keep_off[r + 1]]]
        valid = [int(v) for v in keep_valid[keep_off[r] : keep_off[r + 1]]]
        seq = [(pg, t) for pg, v in zip(pages, valid) for t in range(v)]  # committed tokens in order
        for k, (pg, t) in enumerate(seq):  # read from the ORIGINAL pools: the moves do not see each other
            k_out[pages[k // PAGE], :, k % PAGE, :] = k_pool_bits[pg, :, t, :]
            v_out[pages[k // PAGE], :, k % PAGE, :] = v_pool_bits[pg, :, t, :]
        new_len[r] = len(seq)
        n_kept[r] = (len(seq) + PAGE - 1) // PAGE
    return new_len, n_kept, k_out, v_out


def verify_pass(batch, q_bits, k_pool_bits, v_pool_bits, logits_bits, draft_ids, verdict):
    """All three steps in order, as one pass."""
    o, lse = verify_attention(batch, q_bits, k_pool_bits, v_pool_bits)
    n_acc, bonus, t = accept_greedy(logits_bits, draft_ids, batch.cu_draft)
    c = commit(batch, verdict, n_acc)
    return {"out": o, "lse": lse, "n_accept": n_acc, "bonus_id": bonus, "row_argmax": t, **c}
