"""The seeded generator: shapes of the five configurations, determinism, page-table rules."""
import numpy as np
import pytest

from lr_workloads import make_config, make_random_small, bf16_round, bf16_to_f32


@pytest.mark.parametrize(
    "idx,tokens,pages,q_rows,logit_rows",
    [(1, 320, 22, 16, 18), (2, 4240, 265, 48, 51), (3, 4 * 16608, 4160, 128, 144), (4, 33104, 2072, 96, 102)],
)
def test_config_shapes(idx, tokens, pages, q_rows, logit_rows):
    w = make_config(idx, with_kv=False, with_logits=False)
    b = w.batch
    assert b.kv_tokens() == tokens
    assert b.n_page_slots == pages
    assert b.n_q_rows == q_rows
    assert b.n_logit_rows == logit_rows
    assert len(set(b.page_ids.tolist())) == pages and b.page_ids.max() < b.n_pool_pages
    assert b.n_pool_pages >= int(1.25 * pages)


def test_config5_is_ragged_and_within_the_stated_ranges():
    b = make_config(5, with_kv=False, with_logits=False).batch
    assert b.n_req == 16
    for r in range(16):
        s0, s1 = b.req_span_off[r], b.req_span_off[r + 1]
        assert 1024 <= b.span_len[s0] <= 16384
        assert 2 <= s1 - s0 - 1 <= 6
        assert ((b.span_len[s0 + 1 : s1] >= 16) & (b.span_len[s0 + 1 : s1] <= 64)).all()
    assert set(b.br_n_draft.tolist()) <= {4, 8, 16}
    assert len(set(b.span_len[b.req_span_off[:-1]].tolist())) > 8


def test_same_seed_same_bytes():
    a, b = make_config(1), make_config(1)
    for name in ("q", "k_pool", "v_pool", "logits", "draft_ids", "verdict"):
        assert np.array_equal(getattr(a.tensors, name), getattr(b.tensors, name))
    c = make_config(1, seed=5)
    assert not np.array_equal(a.tensors.q, c.tensors.q)


def test_slack_and_unreferenced_pages_hold_poison_only():
    w = make_random_small(4, poison="nan")
    b, t = w.batch, w.tensors
    ref = np.zeros(b.n_pool_pages, dtype=bool)
    ref[b.page_ids] = True
    assert np.isnan(bf16_to_f32(t.k_pool[~ref])).all()
    assert np.isnan(bf16_to_f32(t.v_pool[~ref])).all()
    # valid tokens are finite
    for s in range(b.n_span):
        for tok in range(int(b.span_len[s])):
            pg = b.page_ids[int(b.span_slot[s]) + tok // 16]
            assert np.isfinite(bf16_to_f32(t.k_pool[pg, :, tok % 16])).all()
        ln = int(b.span_len[s])
        if ln % 16:
            pg = b.page_ids[int(b.span_slot[s]) + ln // 16]
            assert np.isnan(bf16_to_f32(t.v_pool[pg, :, ln % 16 :])).all()


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.0e38], dtype=np.float32)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 ties up to 1 + 2^-6
    got = bf16_to_f32(bf16_round(x))
    assert got[0] == 1.0 and got[1] == 1.0 and got[2] == 1.015625 and got[3] == -2.5
