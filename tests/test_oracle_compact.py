"""Pins for the oracle's compaction: it moves bytes and must not change what the pass computes.

* attention of a query over the compacted context (one span of new_len tokens in the leading kept pages)
  equals attention over the committed chain as commit described it (prefix + accepted segments + kept tail);
* the committed token sequence read back from the compacted pages is the original one, bit for bit;
* nothing outside the request's kept pages changes; a request whose pages are all full is left untouched.
"""
import numpy as np

from lr_workloads import Model, build_batch, fill_kv, fill_q, make_random_small
from oracle import lr_oracle as O

PAGE = 16


def _sequence(pages, valid, pool):
    return np.concatenate([pool[pg, :, :v, :] for pg, v in zip(pages, valid) if v > 0], axis=1) if len(pages) else None


def _committed(batch, verdict, n_accept):
    return O.commit(batch, verdict, n_accept)


def test_sequence_is_preserved_and_other_pages_untouched():
    for seed in range(12):
        w = make_random_small(7000 + seed)
        b, t = w.batch, w.tensors
        rng = np.random.default_rng(seed)
        n_accept = np.array([rng.integers(0, L + 1) for L in b.br_n_draft], dtype=np.int32)
        c = _committed(b, t.verdict, n_accept)
        new_len, n_kept, k2, v2 = O.compact(c["keep_off"], c["keep_pages"], c["keep_valid"], t.k_pool, t.v_pool)
        assert np.array_equal(new_len, c["committed_len"])
        touched = set()
        for r in range(b.n_req):
            pages = c["keep_pages"][c["keep_off"][r] : c["keep_off"][r + 1]]
            valid = c["keep_valid"][c["keep_off"][r] : c["keep_off"][r + 1]]
            touched.update(int(p) for p in pages)
            n = int(new_len[r])
            assert n_kept[r] == (n + PAGE - 1) // PAGE
            if n == 0:
                continue
            for pool_before, pool_after in ((t.k_pool, k2), (t.v_pool, v2)):
                before = _sequence(pages, valid, pool_before)
                dense_valid = [min(PAGE, n - i * PAGE) for i in range(int(n_kept[r]))]
                after = _sequence(pages[: n_kept[r]], dense_valid, pool_after)
                assert np.array_equal(before, after)
        others = [p for p in range(b.n_pool_pages) if p not in touched]
        assert np.array_equal(t.k_pool[others], k2[others]) and np.array_equal(t.v_pool[others], v2[others])


def test_attention_over_the_compacted_context_is_unchanged():
    rng = np.random.Generator(np.random.PCG64(5))
    model = Model(4, 2, 64, 32)
    batch = build_batch(model, [{"P": 37, "segs": [21, 9, 30], "branches": [(1, 6, 4, 4), (2, 11, 5, 5), (3, 7, 7, 6)]}], rng)
    k, v = fill_kv(batch, rng, poison="zero")
    verdict = np.array([1, 1, 0], dtype=np.uint8)  # two segments accepted: the decisive branch is the one of depth 2
    n_accept = np.array([1, 3, 2], dtype=np.int32)
    c = O.commit(batch, verdict, n_accept)
    assert c["n_steps_accepted"][0] == 2 and c["survivor"][0] == 1
    new_len, n_kept, k2, v2 = O.compact(c["keep_off"], c["keep_pages"], c["keep_valid"], k, v)
    assert new_len[0] == 37 + 21 + 9 + (11 - 5 + 3)
    # a fresh query attending to the whole committed context, described (a) as commit left it and (b) compacted
    kept_tail = 11 - 5 + 3
    free_page = sorted(set(range(batch.n_pool_pages)) - set(int(p) for p in batch.page_ids))[0]  # for the probe query's own token
    # (a): prefix, the two accepted segments, and the kept tail as a third span stored in the decisive branch's tail page
    a = build_batch(model, [{"P": 37, "segs": [21, 9, kept_tail], "branches": [(3, 1, 1, 1)]}], rng, shuffle=False)
    tail_slot = int(batch.br_own_slot[1])
    a.page_ids = np.concatenate([batch.page_ids[0:3], batch.page_ids[3:5], batch.page_ids[5:6],
                                 batch.page_ids[tail_slot : tail_slot + 1], [free_page]]).astype(np.int32)
    a.n_pool_pages = batch.n_pool_pages
    # (b): one span of new_len tokens in the leading kept pages
    bq = build_batch(model, [{"P": int(new_len[0]), "segs": [], "branches": [(0, 1, 1, 1)]}], rng, shuffle=False)
    bq.page_ids = np.concatenate([c["keep_pages"][: n_kept[0]], [free_page]]).astype(np.int32)
    bq.n_pool_pages = batch.n_pool_pages
    q = fill_q(a, rng)
    own = rng.integers(0, 2 ** 14, size=k[free_page].shape).astype(np.uint16)
    for pool in (k, v, k2, v2):
        pool[free_page] = own
    oa, la = O.verify_attention(a, q, k, v)
    ob, lb = O.verify_attention(bq, q, k2, v2)
    assert np.allclose(oa, ob, rtol=0, atol=1e-12) and np.allclose(la, lb, rtol=0, atol=1e-12)


def test_a_request_with_only_full_pages_is_left_alone():
    rng = np.random.Generator(np.random.PCG64(6))
    model = Model(2, 1, 64, 16)
    batch = build_batch(model, [{"P": 64, "segs": [16, 32], "branches": [(2, 16, 16, 16)]}], rng)
    k, v = fill_kv(batch, rng)
    c = O.commit(batch, np.array([1, 1], dtype=np.uint8), np.array([16], dtype=np.int32))
    new_len, n_kept, k2, v2 = O.compact(c["keep_off"], c["keep_pages"], c["keep_valid"], k, v)
    assert new_len[0] == 128 and n_kept[0] == 8
    same = (k == k2) | ((k == 0x7FC0) & (k2 == 0x7FC0))
    assert same.all() and np.array_equal(v, v2)
