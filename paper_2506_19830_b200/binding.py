"""ctypes binding of ``liblr_verify.so`` with the names of the C ABI.

Argument marshalling only: every step of the verify pass runs in the CUDA
kernels behind ``lr_verify_attention``, ``lr_accept_greedy`` and ``lr_commit``.
torch is used for device memory and streams.  There is no fallback: if the
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
import weakref
from typing import Optional

import numpy as np
import torch

from .build import LIB_PATH

LR_OK = 0
STATUS_NAMES = {0: "LR_OK", -1: "LR_EINVAL", -2: "LR_EUNSUPPORTED", -3: "LR_ECUDA", -4: "LR_ETIMEOUT", -5: "LR_EBOUNDS",
                -6: "LR_ENOMEM"}

PATH_AUTO, PATH_GENERIC, PATH_TENSOR_CORE, PATH_PAIR = 0, 1, 2, 3
ACCEPT_STATIC_MAX_ROWS = 4096  # LR_ACCEPT_STATIC_MAX_ROWS
COMMIT_MAX_REQUESTS = 4096  # LR_COMMIT_MAX_REQUESTS
COMPACT_MAX_REQUESTS = 8192  # LR_COMPACT_MAX_REQUESTS


class LrError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}: {detail}")


class lr_model(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_q_heads", "n_kv_heads", "head_dim", "page_size", "vocab")]


_I32P = C.POINTER(C.c_int32)


class lr_batch(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_req", "n_branch", "n_span", "n_page_slots")] + [
        (n, _I32P)
        for n in ("req_span_off", "span_len", "span_slot", "br_req", "br_depth", "br_own_len", "br_own_slot",
                  "br_n_draft", "cu_q", "page_ids")
    ] + [("n_pool_pages", C.c_int64), ("seg_parent", _I32P)]


class lr_cycle_stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("stages", "steps", "time", "verdicts_used", "peak_in_flight")]


class lr_plan_info(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("tensor_core_ok", "path", "uses_tensor_core", "n_cta", "n_pieces",
                                         "n_merge_targets", "n_partial_slots")]


class lr_pass_host_io(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "q_h", "logits_h", "draft_ids_h", "verdict_h", "out_h", "n_accept_h", "bonus_id_h", "n_steps_accepted_h",
        "survivor_h", "committed_len_h", "keep_off_h", "free_off_h", "keep_pages_h", "keep_valid_h", "free_pages_h")]


_lib = None


def lib() -> C.CDLL:
    """The loaded C-ABI library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2506_19830_b200.build` "
                "(there is no fallback implementation)")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, f32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
        sig = {
            "lr_validate_batch": [C.POINTER(lr_model), C.POINTER(lr_batch)],
            "lr_create": [C.POINTER(vp), C.POINTER(lr_model), C.c_int],
            "lr_destroy": [vp],
            "lr_plan_bytes": [vp, C.POINTER(lr_batch), C.POINTER(sz)],
            "lr_plan_create": [vp, C.POINTER(lr_batch), vp, sz, vp, C.POINTER(vp)],
            "lr_plan_destroy": [vp],
            "lr_plan_set_attention_path": [vp, C.c_int],
            "lr_plan_describe": [vp, C.POINTER(lr_plan_info)],
            "lr_plan_debug_set_page": [vp, i32, i32, vp],
            "lr_plan_debug_set_wait_limit": [vp, C.c_uint32],
            "lr_plan_debug_set_phantom_bytes": [vp, C.c_uint32],
            "lr_verify_attention": [vp, vp, vp, vp, vp, vp, f32, vp],
            "lr_accept_scratch_bytes": [i32, C.POINTER(sz)],
            "lr_accept_greedy": [vp, vp, i64, vp, vp, i32, i32, vp, vp, vp, vp, vp],
            "lr_accept_greedy_static": [vp, vp, i64, vp, vp, i32, i32, vp, vp, vp, vp],
            "lr_accept_sample_scratch_bytes": [vp, i32, C.POINTER(sz)],
            "lr_accept_sample": [vp, vp, i64, vp, vp, i32, i32, f32, vp, vp, vp, vp, vp, vp, vp],
            "lr_accept_sample_filtered_scratch_bytes": [vp, i32, C.POINTER(sz)],
            "lr_accept_sample_filtered": [vp, vp, i64, vp, vp, i32, i32, f32, i32, f32, vp, vp, vp, vp, vp, vp, vp, vp],
            "lr_commit": [vp] + [vp] * 10 + [vp],
            "lr_cycle_simulate_sync": [i32, i64, i64, vp, i64, C.POINTER(lr_cycle_stats)],
            "lr_cycle_simulate_async": [i32, i64, i64, vp, i64, C.POINTER(lr_cycle_stats)],
            "lr_cycle_best_strategy": [i32, C.c_double, C.c_double, C.c_double, C.c_double, i32, C.POINTER(i32),
                                       C.POINTER(i32), C.POINTER(C.c_double)],
            "lr_compact_scratch_bytes": [vp, C.POINTER(sz)],
            "lr_compact": [vp] * 10,
            "lr_pass_staging_bytes": [vp, C.POINTER(sz)],
            "lr_verify_pass_host": [vp, C.POINTER(lr_pass_host_io), vp, vp, vp, sz, f32, vp],
            "lr_poll_status": [vp, vp, C.POINTER(i32)],
        }
        for name, args in sig.items():
            fn = getattr(L, name)
            fn.argtypes = args
            fn.restype = C.c_int
        L.lr_launch_count.argtypes = [vp]
        L.lr_launch_count.restype = C.c_int64
        L.lr_cycle_speedup.argtypes = [i32, i32, C.c_double, C.c_double]
        L.lr_cycle_speedup.restype = C.c_double
        L.lr_strerror.argtypes = [C.c_int]
        L.lr_strerror.restype = C.c_char_p
        L.lr_last_error.argtypes = []
        L.lr_last_error.restype = C.c_char_p
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != LR_OK:
        raise LrError(status, where, lib().lr_last_error().decode(errors="replace"))


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


class HostBatch:
    """Keeps the int32 host tables alive and exposes them as an ``lr_batch``."""

    FIELDS = ("req_span_off", "span_len", "span_slot", "br_req", "br_depth", "br_own_len", "br_own_slot", "br_n_draft",
              "cu_q", "page_ids")

    def __init__(self, batch):
        self.arrays = {f: _i32(getattr(batch, f)) for f in self.FIELDS}
        self.c = lr_batch()
        self.c.n_req = len(self.arrays["req_span_off"]) - 1
        self.c.n_branch = len(self.arrays["br_req"])
        self.c.n_span = len(self.arrays["span_len"])
        self.c.n_page_slots = len(self.arrays["page_ids"])
        for f in self.FIELDS:
            setattr(self.c, f, self.arrays[f].ctypes.data_as(_I32P))
        self.c.n_pool_pages = int(batch.n_pool_pages)
        parent = getattr(batch, "seg_parent", None)  # tree of draft steps; absent = nested chain (NULL)
        if parent is not None:
            self.arrays["seg_parent"] = _i32(parent)
            self.c.seg_parent = self.arrays["seg_parent"].ctypes.data_as(_I32P)


def _model_struct(model) -> lr_model:
    return lr_model(int(model.n_q_heads), int(model.n_kv_heads), int(model.head_dim), int(model.page_size),
                    int(model.vocab))


def lr_validate_batch(model, batch) -> None:
    hb = HostBatch(batch)
    m = _model_struct(model)
    _check(lib().lr_validate_batch(C.byref(m), C.byref(hb.c)), "lr_validate_batch")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


class Context:
    """``lr_ctx``: one per (device, model geometry)."""

    def __init__(self, model, device: int = 0):
        self.model = model
        self.device = device
        h = C.c_void_p()
        m = _model_struct(model)
        _check(lib().lr_create(C.byref(h), C.byref(m), device), "lr_create")
        self.handle = h
        self._plans = weakref.WeakSet()  # plans must be destroyed before their context

    def close(self):
        if self.handle:
            for p in list(self._plans):
                p.close()
            lib().lr_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def launch_count(self) -> int:
        return int(lib().lr_launch_count(self.handle))

    def lr_accept_greedy(self, logits: torch.Tensor, draft_ids: torch.Tensor, cu_draft: torch.Tensor, n_accept: torch.Tensor,
                         bonus_id: torch.Tensor, scratch: torch.Tensor, row_argmax: Optional[torch.Tensor] = None,
                         stream=None) -> None:
        """logits [n_rows, >=vocab] bf16 (row stride = logits.stride(0)); outputs int32 [n_branch]."""
        n_branch = cu_draft.numel() - 1
        n_rows = logits.shape[0]
        _check(lib().lr_accept_greedy(self.handle, _ptr(logits), logits.stride(0), _ptr(draft_ids), _ptr(cu_draft), n_branch,
                                      n_rows, _ptr(n_accept), _ptr(bonus_id), _ptr(row_argmax), _ptr(scratch),
                                      _stream_ptr(stream)), "lr_accept_greedy")

    def lr_accept_greedy_static(self, logits: torch.Tensor, draft_ids: torch.Tensor, cu_draft: torch.Tensor,
                                n_accept: torch.Tensor, bonus_id: torch.Tensor, row_argmax: Optional[torch.Tensor] = None,
                                stream=None) -> None:
        """``lr_accept_greedy`` on the scratch array built into the library: no scratch argument and no
        device allocation; at most ``ACCEPT_STATIC_MAX_ROWS`` logits rows."""
        n_branch = cu_draft.numel() - 1
        _check(lib().lr_accept_greedy_static(self.handle, _ptr(logits), logits.stride(0), _ptr(draft_ids), _ptr(cu_draft),
                                             n_branch, logits.shape[0], _ptr(n_accept), _ptr(bonus_id), _ptr(row_argmax),
                                             _stream_ptr(stream)), "lr_accept_greedy_static")

    def lr_accept_sample(self, logits: torch.Tensor, draft_ids: torch.Tensor, cu_draft: torch.Tensor, temperature: float,
                         u_accept: torch.Tensor, u_final: torch.Tensor, n_accept: torch.Tensor, final_id: torch.Tensor,
                         scratch: torch.Tensor, p_draft: Optional[torch.Tensor] = None, stream=None) -> None:
        """Rejection-sampling acceptance; u_accept [sum L] and u_final [n_branch] are fp32 uniforms in [0, 1)."""
        n_branch = cu_draft.numel() - 1
        _check(lib().lr_accept_sample(self.handle, _ptr(logits), logits.stride(0), _ptr(draft_ids), _ptr(cu_draft), n_branch,
                                      logits.shape[0], float(temperature), _ptr(u_accept), _ptr(u_final), _ptr(n_accept),
                                      _ptr(final_id), _ptr(p_draft), _ptr(scratch), _stream_ptr(stream)), "lr_accept_sample")

    def lr_accept_sample_filtered(self, logits: torch.Tensor, draft_ids: torch.Tensor, cu_draft: torch.Tensor,
                                  temperature: float, top_k: int, top_p: float, u_accept: torch.Tensor, u_final: torch.Tensor,
                                  n_accept: torch.Tensor, final_id: torch.Tensor, scratch: torch.Tensor,
                                  p_draft: Optional[torch.Tensor] = None, n_kept: Optional[torch.Tensor] = None,
                                  stream=None) -> None:
        """``lr_accept_sample`` on the target distribution after the top-k / top-p filters (0 and 1.0 switch them off)."""
        n_branch = cu_draft.numel() - 1
        _check(lib().lr_accept_sample_filtered(self.handle, _ptr(logits), logits.stride(0), _ptr(draft_ids), _ptr(cu_draft),
                                               n_branch, logits.shape[0], float(temperature), int(top_k), float(top_p),
                                               _ptr(u_accept), _ptr(u_final), _ptr(n_accept), _ptr(final_id), _ptr(p_draft),
                                               _ptr(n_kept), _ptr(scratch), _stream_ptr(stream)), "lr_accept_sample_filtered")

    def accept_sample_filtered_scratch(self, n_rows: int) -> torch.Tensor:
        n = C.c_size_t()
        _check(lib().lr_accept_sample_filtered_scratch_bytes(self.handle, n_rows, C.byref(n)),
               "lr_accept_sample_filtered_scratch_bytes")
        return torch.empty((n.value + 7) // 8, dtype=torch.int64, device=f"cuda:{self.device}")

    def accept_sample_scratch(self, n_rows: int) -> torch.Tensor:
        n = C.c_size_t()
        _check(lib().lr_accept_sample_scratch_bytes(self.handle, n_rows, C.byref(n)), "lr_accept_sample_scratch_bytes")
        return torch.empty((n.value + 7) // 8, dtype=torch.int64, device=f"cuda:{self.device}")

    @staticmethod
    def accept_scratch(n_rows: int, device) -> torch.Tensor:
        n = C.c_size_t()
        _check(lib().lr_accept_scratch_bytes(n_rows, C.byref(n)), "lr_accept_scratch_bytes")
        return torch.zeros((n.value + 7) // 8, dtype=torch.int64, device=device)


class Plan:
    """``lr_plan``: device tables and the attention work partition of one batch."""

    def __init__(self, ctx: Context, batch, stream=None):
        self.ctx = ctx
        self.host = HostBatch(batch)
        n = C.c_size_t()
        _check(lib().lr_plan_bytes(ctx.handle, C.byref(self.host.c), C.byref(n)), "lr_plan_bytes")
        self.workspace_bytes = n.value
        self.workspace = torch.empty(n.value + 256, dtype=torch.uint8, device=f"cuda:{ctx.device}")
        off = (-self.workspace.data_ptr()) % 256
        self._ws_ptr = self.workspace.data_ptr() + off
        h = C.c_void_p()
        _check(lib().lr_plan_create(ctx.handle, C.byref(self.host.c), self._ws_ptr, n.value, _stream_ptr(stream), C.byref(h)),
               "lr_plan_create")
        self.handle = h
        ctx._plans.add(self)
        self.n_req = self.host.c.n_req
        self.n_branch = self.host.c.n_branch
        self.n_page_slots = self.host.c.n_page_slots

    def close(self):
        if self.handle:
            lib().lr_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def lr_plan_set_attention_path(self, path: int) -> None:
        _check(lib().lr_plan_set_attention_path(self.handle, path), "lr_plan_set_attention_path")

    def lr_plan_debug_set_page(self, page_slot: int, new_id: int, stream=None) -> None:
        _check(lib().lr_plan_debug_set_page(self.handle, page_slot, new_id, _stream_ptr(stream)), "lr_plan_debug_set_page")

    def lr_plan_debug_set_wait_limit(self, microseconds: int) -> None:
        _check(lib().lr_plan_debug_set_wait_limit(self.handle, microseconds), "lr_plan_debug_set_wait_limit")

    def lr_plan_debug_set_phantom_bytes(self, n_bytes: int) -> None:
        _check(lib().lr_plan_debug_set_phantom_bytes(self.handle, n_bytes), "lr_plan_debug_set_phantom_bytes")

    def lr_plan_describe(self) -> dict:
        info = lr_plan_info()
        _check(lib().lr_plan_describe(self.handle, C.byref(info)), "lr_plan_describe")
        return {n: int(getattr(info, n)) for n, _ in lr_plan_info._fields_}

    def lr_verify_attention(self, q, k_pool, v_pool, out, lse=None, softmax_scale: float = 0.0, stream=None) -> None:
        _check(lib().lr_verify_attention(self.handle, _ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(out), _ptr(lse),
                                         float(softmax_scale), _stream_ptr(stream)), "lr_verify_attention")

    def lr_commit(self, verdict, n_accept, n_steps_accepted, survivor, committed_len, keep_off, keep_pages, keep_valid,
                  free_off, free_pages, stream=None) -> None:
        _check(lib().lr_commit(self.handle, _ptr(verdict), _ptr(n_accept), _ptr(n_steps_accepted), _ptr(survivor),
                               _ptr(committed_len), _ptr(keep_off), _ptr(keep_pages), _ptr(keep_valid), _ptr(free_off),
                               _ptr(free_pages), _stream_ptr(stream)), "lr_commit")

    def compact_scratch(self) -> torch.Tensor:
        n = C.c_size_t()
        _check(lib().lr_compact_scratch_bytes(self.handle, C.byref(n)), "lr_compact_scratch_bytes")
        t = torch.empty(n.value + 256, dtype=torch.uint8, device=f"cuda:{self.ctx.device}")
        off = (-t.data_ptr()) % 256
        return t[off : off + n.value]

    def lr_compact(self, keep_off, keep_pages, keep_valid, k_pool, v_pool, new_len, n_pages_kept, scratch, stream=None) -> None:
        """Moves the committed tokens (keep lists of ``lr_commit``) densely into the leading kept pages, in place."""
        _check(lib().lr_compact(self.handle, _ptr(keep_off), _ptr(keep_pages), _ptr(keep_valid), _ptr(k_pool), _ptr(v_pool),
                                _ptr(new_len), _ptr(n_pages_kept), _ptr(scratch), _stream_ptr(stream)), "lr_compact")

    def lr_poll_status(self, stream=None) -> int:
        d = C.c_int32()
        _check(lib().lr_poll_status(self.handle, _stream_ptr(stream), C.byref(d)), "lr_poll_status")
        return d.value

    def pass_staging(self) -> torch.Tensor:
        n = C.c_size_t()
        _check(lib().lr_pass_staging_bytes(self.handle, C.byref(n)), "lr_pass_staging_bytes")
        t = torch.zeros(n.value + 256, dtype=torch.uint8, device=f"cuda:{self.ctx.device}")
        return t

    def lr_verify_pass_host(self, io: lr_pass_host_io, k_pool, v_pool, staging: torch.Tensor, softmax_scale: float = 0.0,
                            stream=None) -> None:
        off = (-staging.data_ptr()) % 256
        _check(lib().lr_verify_pass_host(self.handle, C.byref(io), _ptr(k_pool), _ptr(v_pool), staging.data_ptr() + off,
                                         staging.numel() - off, float(softmax_scale), _stream_ptr(stream)),
               "lr_verify_pass_host")


# ---- host-side cycle model (no device needed) --------------------------------------------------------
def _stats(st: lr_cycle_stats) -> dict:
    return {n: int(getattr(st, n)) for n, _ in lr_cycle_stats._fields_}


def lr_cycle_simulate_sync(gamma: int, num: int, den: int, verdicts) -> dict:
    v = np.ascontiguousarray(verdicts, dtype=np.uint8)
    st = lr_cycle_stats()
    _check(lib().lr_cycle_simulate_sync(gamma, num, den, v.ctypes.data, len(v), C.byref(st)), "lr_cycle_simulate_sync")
    return _stats(st)


def lr_cycle_simulate_async(gamma: int, num: int, den: int, verdicts) -> dict:
    v = np.ascontiguousarray(verdicts, dtype=np.uint8)
    st = lr_cycle_stats()
    _check(lib().lr_cycle_simulate_async(gamma, num, den, v.ctypes.data, len(v), C.byref(st)), "lr_cycle_simulate_async")
    return _stats(st)


def lr_cycle_speedup(mode: int, k: int, alpha: float, c: float) -> float:
    return float(lib().lr_cycle_speedup(mode, k, alpha, c))


def lr_cycle_best_strategy(budget: int, alpha1: float, c1: float, alpha2: float, c2: float, asynchronous: bool = True):
    k1, k2, h = C.c_int32(), C.c_int32(), C.c_double()
    _check(lib().lr_cycle_best_strategy(budget, alpha1, c1, alpha2, c2, int(asynchronous), C.byref(k1), C.byref(k2),
                                        C.byref(h)), "lr_cycle_best_strategy")
    return k1.value, k2.value, h.value
