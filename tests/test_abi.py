"""CPU-side checks of the C-ABI library: it builds, loads, exports every declared symbol,
and its host-only batch validation follows the documented rules."""
import copy
import ctypes
import os
import re

import numpy as np
import pytest

from lr_workloads import make_config, make_random_small
from paper_2506_19830_b200 import binding as B
from paper_2506_19830_b200.build import build_library, LIB_PATH

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()


def _declared_functions():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(lr_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(LIB_PATH)
    names = _declared_functions()
    assert {"lr_verify_attention", "lr_accept_greedy", "lr_commit"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"


def test_strerror_and_status_names():
    lib = B.lib()
    assert lib.lr_strerror(0) == b"ok"
    for code in range(-6, 0):
        assert lib.lr_strerror(code) != b"unknown status"
    assert lib.lr_strerror(-99) == b"unknown status"


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_benchmark_batches_validate(cfg):
    w = make_config(cfg, with_kv=False, with_logits=False)
    B.lr_validate_batch(w.batch.model, w.batch)


def test_random_batches_validate():
    for seed in range(30):
        w = make_random_small(seed)
        B.lr_validate_batch(w.batch.model, w.batch)


def _mut(b, field, idx, value):
    c = copy.copy(b)
    a = getattr(b, field).copy()
    a[idx] = value
    setattr(c, field, a)
    return c


def test_validation_rejects_each_broken_rule():
    w = make_random_small(1)
    b = w.batch
    m = b.model
    assert b.n_span - b.n_req >= 1
    seg = int(b.req_span_off[0]) + 1
    cases = [
        _mut(b, "page_ids", 0, b.n_pool_pages),  # page outside the pool
        _mut(b, "page_ids", 0, -1),
        _mut(b, "page_ids", 0, int(b.page_ids[1])),  # one physical page in two slots
        _mut(b, "br_depth", 0, 200),  # deeper than the chain
        _mut(b, "br_own_len", 0, 0),  # shorter than the query block
        _mut(b, "br_n_draft", 0, int(b.br_own_len[0]) + 1),  # more drafts than tail tokens
        _mut(b, "span_len", seg, 0),  # empty segment
        _mut(b, "span_slot", 0, b.n_page_slots),  # slots out of range
        _mut(b, "br_own_slot", 0, int(b.span_slot[0])) if b.span_len[0] > 0 else _mut(b, "br_own_slot", 0, int(b.span_slot[seg])),
        _mut(b, "cu_q", 0, 1),
        _mut(b, "br_req", 0, 99),
    ]
    for i, bad in enumerate(cases):
        with pytest.raises(B.LrError) as e:
            B.lr_validate_batch(m, bad)
        assert e.value.status == -1, i


def test_tree_batches_validate_and_broken_trees_are_rejected():
    from lr_workloads import Model, build_batch, make_random_tree, make_tree
    for seed in range(10):
        w = make_random_tree(seed)
        B.lr_validate_batch(w.batch.model, w.batch)
    w = make_tree(2, 3, size="tiny", with_logits=False, with_kv=False)
    b = w.batch
    B.lr_validate_batch(b.model, b)
    bad = [
        _mut(b, "seg_parent", 1, 1),  # a segment that continues itself
        _mut(b, "seg_parent", 2, 5),  # ... or a later segment
        _mut(b, "seg_parent", 3, -1),
    ]
    # a chain of nine steps written as a tree is deeper than tree mode allows; as a plain chain it is fine
    rng = np.random.default_rng(0)
    req = {"P": 5, "segs": [3] * 9, "branches": [(9, 2, 2, 2)]}
    B.lr_validate_batch(Model(2, 1, 64, 16), build_batch(Model(2, 1, 64, 16), [req], rng))
    bad.append(build_batch(Model(2, 1, 64, 16), [dict(req, parents=list(range(9)))], rng))
    for i, x in enumerate(bad):
        with pytest.raises(B.LrError) as e:
            B.lr_validate_batch(x.model, x)
        assert e.value.status == -1, i


def test_unsupported_geometry():
    w = make_random_small(2)
    import dataclasses

    for kw in (dict(head_dim=96), dict(page_size=32), dict(n_q_heads=7, n_kv_heads=2), dict(n_q_heads=34, n_kv_heads=2)):
        m = dataclasses.replace(w.batch.model, **kw)
        with pytest.raises(B.LrError) as e:
            B.lr_validate_batch(m, w.batch)
        assert e.value.status == -2


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/liblr_verify.so")
    with pytest.raises(RuntimeError):
        B.lib()
