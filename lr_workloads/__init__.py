"""Seeded synthetic inputs for the step-parallel verification pass.

This package only *shapes* inputs (lengths, page tables, random tensors, draft
ids, verdicts).  It holds none of the method's arithmetic: no attention, no
argmax, no acceptance or commit logic.  Both the CPU oracle's tests and the
CUDA path's tests draw their inputs from here so that they see identical data.
"""
from .gen import (  # noqa: F401
    Model,
    Batch,
    Tensors,
    Workload,
    CONFIG_NAMES,
    bf16_round,
    bf16_to_f32,
    build_batch,
    fill_kv,
    fill_q,
    fill_logits_and_drafts,
    fill_verdicts,
    make_config,
    make_random_small,
    make_tree,
    make_random_tree,
    make_random_mid,
)
