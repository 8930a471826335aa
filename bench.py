#!/usr/bin/env python
"""Benchmark of the verify pass: ``python bench.py --gpus N --steps K --warmup W``.

A step is one whole verify pass (nested-prefix attention -> greedy acceptance ->
commit) over one batch of seeded synthetic input.  The headline workload is the
"ragged serving sweep" configuration (the largest one that runs on one GPU)
unless ``--config`` says otherwise; the same JSON line carries, under
``per_config``, the step time, per-kernel times and roofline fraction of each of
the four full-size configurations.  Every rank owns an independent batch (requests do not interact, so
the path shards by request with no collective: weak scaling).

Cold-HBM protocol: the KV pools and the logits exist in ``--copies`` independent
copies whose total footprint is several times the L2; step i uses copy i mod
copies, so every step streams its inputs from HBM.  Every timed step is replayed
from a CUDA graph whatever ``--steps`` is, and the K-step region is repeated
until it has run for at least 0.2 s; the median region is reported.

``--impl reference`` times the CPU fp64 oracle (there is no other implementation
of this path to run) on the host cores, on the same workload and metric.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verified_tokens_per_s_per_verify_pass"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["hbm_gbs"]), float(d["bf16_tflops"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback"


def attention_work(batch):
    """Algorithmic bytes and flops of the attention step: every KV row of every span and tail once
    (K and V), Q read and O written once; 4*D flops per (query row, head, visible key)."""
    m = batch.model
    kv_bytes = batch.kv_tokens() * m.n_kv_heads * m.head_dim * 2 * 2
    qo_bytes = 2 * batch.n_q_rows * m.n_q_heads * m.head_dim * 2
    vis = 0
    for b in range(batch.n_branch):
        r = int(batch.br_req[b])
        s0 = int(batch.req_span_off[r])
        if batch.seg_parent is None:
            chain = int(batch.span_len[s0 : s0 + 1 + int(batch.br_depth[b])].sum())
        else:  # tree of draft steps: the prefix and the steps between it and the branch's node
            chain, node = int(batch.span_len[s0]), int(batch.br_depth[b])
            while node != 0:
                chain += int(batch.span_len[s0 + node])
                node = int(batch.seg_parent[s0 + node])
        q_len = int(batch.cu_q[b + 1] - batch.cu_q[b])
        own = int(batch.br_own_len[b])
        vis += sum(chain + own - q_len + i + 1 for i in range(q_len))
    flops = 4 * m.n_q_heads * m.head_dim * vis
    return kv_bytes + qo_bytes, flops


def make_workload(args, rank=None):
    """The configuration the flags name; with a rank, that rank's independent batch (seed offset by rank)."""
    from lr_workloads import make_config, make_tree

    def seeded(seed):
        if rank is None:
            return seed
        import paper_2506_19830_b200.sharding as S
        return S.rank_seed(seed, rank)

    if args.tree:
        parts = args.tree.split(",")
        W, gamma, size = int(parts[0]), int(parts[1]), (parts[2] if len(parts) > 2 else "layer")
        w = make_tree(W, gamma, seed=seeded(20250700 + 16 * W + gamma), size=size)
        return w, w.name
    w = make_config(args.config, seed=seeded(20250619 + args.config), carry_in=args.carry_in)
    return w, f"config{args.config}_{w.name}"


def accept_bytes(batch):
    return batch.n_logit_rows * batch.model.vocab * 2


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons every 100 ms while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100", "-i", str(self.gpu)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_pass_seconds(w, min_seconds, max_passes=1000):
    """Times whole oracle passes on workload w until min_seconds of CPU work are done."""
    from oracle import lr_oracle as O

    b, t = w.batch, w.tensors
    n, t0 = 0, time.perf_counter()
    while True:
        O.verify_pass(b, t.q, t.k_pool, t.v_pool, t.logits, t.draft_ids, t.verdict)
        n += 1
        el = time.perf_counter() - t0
        if el >= min_seconds or n >= max_passes:
            return el / n, n


def host_threads():
    try:
        from threadpoolctl import threadpool_info

        n = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    w, w_label = make_workload(args)
    tokens = w.batch.n_verified_tokens
    budget_end = time.perf_counter() + 150.0
    for i in range(args.warmup):
        if i >= 1 and time.perf_counter() > budget_end - 120.0:  # warm-up is bounded too: the run must end within minutes
            break
        oracle_pass_seconds(w, 0.0, 1)
    times = []
    for _ in range(args.steps):
        s, _ = oracle_pass_seconds(w, 0.0, 1)
        times.append(s)
        if time.perf_counter() > budget_end:
            break
    sec = sum(times) / len(times)
    cores = host_threads()
    val = tokens / sec
    sample = f"whole pass of {w_label}, one batch per step, {len(times)} steps"
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": len(times),
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": w_label, "seed": w.seed},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def _traffic_for(workload_label, uses_tc):
    """DRAM bytes (read + write) of one launch of the dominant attention kernel on this workload, from the ncu
    capture recorded in profiles/traffic.json -- or None when there is no capture, or when the kernel's source
    has changed since it was taken."""
    if not uses_tc:
        return None
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return None
    try:
        rec = json.load(open(path)).get(workload_label, {}).get("attn_tc_kernel")
        if rec is None:
            return None
        import hashlib

        src = os.path.join(ROOT, "paper_2506_19830_b200", "csrc", "attn_tc.cu")
        if hashlib.sha256(open(src, "rb").read()).hexdigest() != rec.get("source_sha256"):
            return None
        return int(rec["dram_bytes_read"]) + int(rec["dram_bytes_write"])
    except Exception:
        return None


class Measurement:
    """One workload on this rank's GPU: inputs resident, CUDA graphs captured, timed regions."""

    def __init__(self, args, rank, local, world, cfg=None, tree=None):
        import torch

        from paper_2506_19830_b200 import binding as B
        from paper_2506_19830_b200 import runner as R

        self.torch, self.B, self.R = torch, B, R
        self.args, self.rank, self.local, self.world = args, rank, local, world
        a = argparse.Namespace(**vars(args))
        if cfg is not None:
            a.config, a.tree = cfg, ""
        if tree is not None:
            a.tree = tree
        self.w, self.label = make_workload(a, rank)
        b, t = self.w.batch, self.w.tensors
        self.b, self.t = b, t
        dev = self.dev = f"cuda:{local}"
        self.ctx = B.Context(b.model, local)
        self.plan = B.Plan(self.ctx, b)
        self.plan.lr_plan_set_attention_path(args.path)
        self.info = self.plan.lr_plan_describe()
        self.x0 = R.DeviceInputs(b, t, dev)
        self.y = R.PassOutputs(b, dev)
        x0 = self.x0
        self.per_copy = 2 * x0.k_pool.numel() * 2 + x0.logits.numel() * 2
        copies = args.copies if args.copies > 0 else max(4, int(np.ceil(6 * 126e6 / self.per_copy)))
        copies = min(copies, max(1, int(40e9 // self.per_copy)))
        # a graph holds one step per copy; with fewer timed steps than copies only that many copies are used
        self.K = max(1, args.steps)
        self.copies = copies
        self.kc = [x0.k_pool] + [x0.k_pool.clone() for _ in range(copies - 1)]
        self.vc = [x0.v_pool] + [x0.v_pool.clone() for _ in range(copies - 1)]
        self.lc = [x0.logits] + [x0.logits.clone() for _ in range(copies - 1)]
        self.main_stream = torch.cuda.current_stream()
        self.side = torch.cuda.Stream()
        self.overlap_stream = None if args.no_overlap else torch.cuda.Stream()
        self.all_graphed = True

    def close(self):
        self.plan.close()
        self.ctx.close()
        for name in ("kc", "vc", "lc", "x0", "y"):
            setattr(self, name, None)
        self.torch.cuda.empty_cache()

    # ---- the calls --------------------------------------------------------------------------------------
    def step(self, c):
        x0, y, plan, ctx = self.x0, self.y, self.plan, self.ctx
        if self.overlap_stream is not None:  # attention || (acceptance -> commit): the two chains share no data
            self.R.run_pass_overlapped(ctx, plan, x0, y, self.overlap_stream, self.kc[c], self.vc[c], self.lc[c])
            return
        plan.lr_verify_attention(x0.q, self.kc[c], self.vc[c], y.out, None, 0.0, None)
        ctx.lr_accept_greedy(self.lc[c], x0.draft_ids, x0.cu_draft, y.n_accept, y.bonus_id, y.scratch, None, None)
        plan.lr_commit(x0.verdict, y.n_accept, y.n_steps_accepted, y.survivor, y.committed_len, y.keep_off, y.keep_pages,
                       y.keep_valid, y.free_off, y.free_pages, None)

    def attn_only(self, c):
        self.plan.lr_verify_attention(self.x0.q, self.kc[c], self.vc[c], self.y.out, None, 0.0, None)

    def accept_only(self, c):
        x0, y = self.x0, self.y
        self.ctx.lr_accept_greedy(self.lc[c], x0.draft_ids, x0.cu_draft, y.n_accept, y.bonus_id, y.scratch, None, None)

    def commit_only(self, c):
        x0, y = self.x0, self.y
        self.plan.lr_commit(x0.verdict, y.n_accept, y.n_steps_accepted, y.survivor, y.committed_len, y.keep_off, y.keep_pages,
                            y.keep_valid, y.free_off, y.free_pages, None)

    # ---- graphs and timing --------------------------------------------------------------------------------
    def make_runner(self, fn):
        """Returns run(): exactly K consecutive calls fn(i mod n) with n = min(copies, K), replayed from CUDA graphs:
        one graph of n calls, replayed K // n times, and one of K mod n calls.  --no-graph (or a failed capture)
        issues every launch from the host instead, and the line says so."""
        torch = self.torch
        K, n = self.K, min(self.copies, self.K)
        graphs = []
        if not self.args.no_graph:
            try:
                for count in (n, K % n):
                    if count == 0:
                        continue
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=self.side):  # the binding launches on torch's current stream
                        for c in range(count):
                            fn(c)
                    graphs.append((g, K // n if count == n else 1))
            except Exception as exc:  # capture not possible: plain launches
                graphs = []
                self.all_graphed = False
                if self.rank == 0:
                    print(f"bench: CUDA graph capture failed ({exc}); issuing launches from the host", file=sys.stderr)
        else:
            self.all_graphed = False

        def run():
            if graphs:
                for g, times in graphs:
                    for _ in range(times):
                        g.replay()
            else:
                for i in range(K):
                    fn(i % n)
        return run

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist

            dist.barrier()
        self.torch.cuda.synchronize()

    def timed_region(self, run):
        """Device time (ms) of one region = K steps, between events on the launching stream, barrier + sync on both sides."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        e0.record(self.main_stream)
        run()
        e1.record(self.main_stream)
        self.barrier()
        return e0.elapsed_time(e1)

    def timed_median(self, run, min_total_ms=200.0, max_regions=400):
        """Repeats the K-step region until min_total_ms of device time have been measured (at least 3 regions) and
        returns (median region ms, number of regions).  Every rank runs the same number of regions: rank 0's first
        region decides."""
        torch = self.torch
        first = self.timed_region(run)
        n = int(min(max_regions, max(3, np.ceil(min_total_ms / max(first, 1e-3)))))
        if self.world > 1:
            import torch.distributed as dist

            tn = torch.tensor([n], device=self.dev)
            dist.broadcast(tn, 0)
            n = int(tn.item())
        regions = [self.timed_region(run) for _ in range(n)]
        return float(np.median(regions)), n

    # ---- one workload: step and kernels ----------------------------------------------------------------------
    def measure(self):
        """Step time and per-kernel times of this workload, with the clocks sampled meanwhile."""
        from paper_2506_19830_b200 import sharding as S

        args, b, K = self.args, self.b, self.K
        W = max(args.warmup, 3)
        n = min(self.copies, K)
        for i in range(W):
            self.step(i % n)
        assert self.plan.lr_poll_status() == 0
        l0 = self.ctx.launch_count
        self.step(0)
        self.launches_per_step = self.ctx.launch_count - l0
        run_step = self.make_runner(self.step)
        run_attn = self.make_runner(self.attn_only)
        run_accept = self.make_runner(self.accept_only)
        run_commit = self.make_runner(self.commit_only)
        self.torch.cuda.synchronize()
        run_step()  # one untimed region as warm-up of the graphs themselves
        assert self.plan.lr_poll_status() == 0
        sampler = ClockSampler(self.local)
        if self.rank == 0:
            sampler.start()
        ms_region, n_regions = self.timed_median(run_step)
        kernel_us = {}
        for name, run in (("attention", run_attn), ("accept", run_accept), ("commit", run_commit)):
            ms, _ = self.timed_median(run, min_total_ms=100.0)
            kernel_us[name] = 1e3 * ms / K
        clocks = sampler.stop() if self.rank == 0 else None
        assert self.plan.lr_poll_status() == 0
        ms_max, tokens_total = S.reduce_measurement(ms_region, b.n_verified_tokens, self.dev)
        ms_step = ms_max / K
        self.W = W
        return {"ms_step": ms_step, "value": S.job_throughput(ms_step, tokens_total), "regions": n_regions,
                "kernel_us": kernel_us, "clocks": clocks}

    def roofline(self, kernel_us):
        hbm_peak, tc_peak, peak_kind = _peaks()
        b = self.b
        a_bytes, a_flops = attention_work(b)
        t_att = kernel_us["attention"] * 1e-6
        hbm_time, tc_time = a_bytes / (hbm_peak * 1e9), a_flops / (tc_peak * 1e12)
        if hbm_time >= tc_time:
            roof = {"bound": "hbm", "achieved": a_bytes / t_att / 1e9, "peak": hbm_peak, "unit": "GB/s"}
        else:
            roof = {"bound": "tensor", "achieved": a_flops / t_att / 1e12, "peak": tc_peak, "unit": "TFLOP/s"}
        roof["frac"] = roof["achieved"] / roof["peak"]
        uses_tc = bool(self.info["uses_tensor_core"])
        plain = self.args.path == 0 and not self.args.carry_in
        timed = "attn_generic_kernel"
        if uses_tc and self.info["path"] == 3:
            timed = "attn_pair_kernel"
        elif uses_tc:
            timed = "attn_tc_kernel" + (" + attn_tc_merge_kernel" if self.info["n_merge_targets"] > 0 and TC_MERGE_IS_A_LAUNCH else "")
        roof.update({"traffic": _traffic_for(self.label, uses_tc) if plain else None, "kernel": "lr_verify_attention",
                     "kernel_us": kernel_us["attention"], "algorithmic_bytes": a_bytes, "algorithmic_flops": a_flops,
                     "peak_source": f"of {peak_kind}", "timed": timed, "roofline_us": max(hbm_time, tc_time) * 1e6,
                     "ctas": self.info["n_cta"], "merge_targets": self.info["n_merge_targets"]})
        acc_b = accept_bytes(b)
        kernels = {
            "lr_verify_attention": {"us": kernel_us["attention"], "GB/s": a_bytes / t_att / 1e9, "TFLOP/s": a_flops / t_att / 1e12},
            "lr_accept_greedy": {"us": kernel_us["accept"], "GB/s": acc_b / (kernel_us["accept"] * 1e-6) / 1e9,
                                 "frac_of_hbm_peak": acc_b / (kernel_us["accept"] * 1e-6) / 1e9 / hbm_peak,
                                 "algorithmic_bytes": acc_b},
            "lr_commit": {"us": kernel_us["commit"]},
        }
        return roof, kernels

    def config_dict(self):
        b = self.b
        n = min(self.copies, self.K)
        return {"workload": self.label, "seed": self.w.seed, "requests_per_gpu": b.n_req, "branches_per_gpu": b.n_branch,
                "kv_tokens_per_gpu": b.kv_tokens(), "verified_tokens_per_gpu": b.n_verified_tokens,
                "l2_policy": f"rotating {n} copies of KV pools and logits ({n * self.per_copy / 1e6:.0f} MB > L2)",
                "attention_path": self.args.path, "carry_in": bool(self.args.carry_in), "cuda_graph": bool(self.all_graphed),
                "overlap": "attention || (accept -> commit) on two streams" if self.overlap_stream is not None else "none",
                "timing": "median of repeated K-step regions (>= 0.2 s in all), every step replayed from a CUDA graph",
                "per_kernel_timing": "K back-to-back launches of the kernel alone over the rotating copies, same protocol"}


# whether a split-KV merge is a kernel launch of its own (it is folded into attn_tc_kernel when False)
TC_MERGE_IS_A_LAUNCH = True


def extras(M):
    """Stochastic acceptance and compaction, timed alone on the headline workload (not part of the step)."""
    torch, B, R = M.torch, M.B, M.R
    b, t, x0, dev, ctx, plan = M.b, M.t, M.x0, M.dev, M.ctx, M.plan
    rs = np.random.default_rng(M.w.seed)
    u_acc = torch.from_numpy(rs.uniform(0, 1, max(1, len(t.draft_ids))).astype(np.float32)).to(dev)
    u_fin = torch.from_numpy(rs.uniform(0, 1, b.n_branch).astype(np.float32)).to(dev)
    samp_scratch = ctx.accept_sample_scratch(b.n_logit_rows)
    samp_n = torch.empty(b.n_branch, dtype=torch.int32, device=dev)
    samp_f = torch.empty(b.n_branch, dtype=torch.int32, device=dev)

    def sample_only(c):
        ctx.lr_accept_sample(M.lc[c], x0.draft_ids, x0.cu_draft, 0.6, u_acc, u_fin, samp_n, samp_f, samp_scratch, None, None)

    filt_scratch = ctx.accept_sample_filtered_scratch(b.n_logit_rows)

    def filtered_only(top_k, top_p):
        def f(c):
            ctx.lr_accept_sample_filtered(M.lc[c], x0.draft_ids, x0.cu_draft, 0.6, top_k, top_p, u_acc, u_fin, samp_n, samp_f,
                                          filt_scratch, None, None, None)
        return f

    # compaction moves tokens in place; every call with the same keep lists moves the same number of bytes
    cmp_k = [x0.k_pool.clone() for _ in range(2)]
    cmp_v = [x0.v_pool.clone() for _ in range(2)]
    cmp_scratch = plan.compact_scratch()
    cmp_len = torch.empty(b.n_req, dtype=torch.int32, device=dev)
    cmp_kept = torch.empty(b.n_req, dtype=torch.int32, device=dev)
    # keep lists of the commit that displaces the most: every step accepted, every draft token of the last branch kept
    yc = R.PassOutputs(b, dev, n_rows=1)
    plan.lr_commit(torch.ones_like(x0.verdict), torch.from_numpy(np.ascontiguousarray(b.br_n_draft, dtype=np.int32)).to(dev),
                   yc.n_steps_accepted, yc.survivor, yc.committed_len, yc.keep_off, yc.keep_pages, yc.keep_valid,
                   yc.free_off, yc.free_pages, None)

    def compact_only(c):
        plan.lr_compact(yc.keep_off, yc.keep_pages, yc.keep_valid, cmp_k[c % 2], cmp_v[c % 2], cmp_len, cmp_kept, cmp_scratch, None)

    out = {}
    hbm_peak, _, _ = _peaks()
    acc_b = accept_bytes(b)
    ms, _ = M.timed_median(M.make_runner(sample_only), min_total_ms=50.0)
    us = 1e3 * ms / M.K
    out["lr_accept_sample"] = {"us": us, "GB/s": acc_b / (us * 1e-6) / 1e9, "frac_of_hbm_peak": acc_b / (us * 1e-6) / 1e9 / hbm_peak,
                               "algorithmic_bytes": acc_b, "temperature": 0.6,
                               "note": "rejection-sampling acceptance; not part of the timed step"}
    for top_k, top_p in ((20, 0.95), (0, 0.95)):  # the sampling settings of the paper's two model families
        ms, _ = M.timed_median(M.make_runner(filtered_only(top_k, top_p)), min_total_ms=50.0)
        us = 1e3 * ms / M.K
        out[f"lr_accept_sample_filtered(top_k={top_k},top_p={top_p})"] = {
            "us": us, "GB/s": acc_b / (us * 1e-6) / 1e9, "frac_of_hbm_peak": acc_b / (us * 1e-6) / 1e9 / hbm_peak,
            "algorithmic_bytes": acc_b, "temperature": 0.6, "top_k": top_k, "top_p": top_p,
            "note": "top-k / top-p filters, then rejection-sampling acceptance; not part of the timed step"}
    ms, _ = M.timed_median(M.make_runner(compact_only), min_total_ms=50.0)
    us = 1e3 * ms / M.K
    # tokens lr_compact displaces: those behind the first partly filled kept page of each request
    k_off, k_val = yc.keep_off.cpu().numpy(), yc.keep_valid.cpu().numpy()
    displaced = 0
    for r in range(b.n_req):
        v = k_val[k_off[r]:k_off[r + 1]]
        partial = np.flatnonzero(v[:-1] != 16)
        if len(partial):
            displaced += int(v[partial[0] + 1:].sum())
    cmp_bytes = displaced * 2 * b.model.n_kv_heads * b.model.head_dim * 2 * 4  # K and V, read and written, twice
    out["lr_compact"] = {"us": us, "displaced_tokens": displaced, "bytes_moved": cmp_bytes,
                         "case": "all steps accepted, whole last draft kept",
                         "note": "three dependent launches, latency-bound; not part of the timed step"}
    return out


def end_to_end(M):
    """The same metric through lr_verify_pass_host: pinned host buffers in, every result out, per step."""
    torch, B = M.torch, M.B
    from paper_2506_19830_b200 import sharding as S

    b, t, plan = M.b, M.t, M.plan
    m = b.model
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()  # noqa: E731
    host = {
        "q_h": pin(t.q.view(np.int16)), "logits_h": pin(t.logits.view(np.int16)), "draft_ids_h": pin(t.draft_ids),
        "verdict_h": pin(t.verdict if len(t.verdict) else np.zeros(1, np.uint8)),
        "out_h": torch.empty((b.n_q_rows, m.n_q_heads, m.head_dim), dtype=torch.int16).pin_memory(),
    }
    for name, n in (("n_accept_h", b.n_branch), ("bonus_id_h", b.n_branch), ("n_steps_accepted_h", b.n_req),
                    ("survivor_h", b.n_req), ("committed_len_h", b.n_req), ("keep_off_h", b.n_req + 1),
                    ("free_off_h", b.n_req + 1), ("keep_pages_h", b.n_page_slots), ("keep_valid_h", b.n_page_slots),
                    ("free_pages_h", b.n_page_slots)):
        host[name] = torch.empty(n, dtype=torch.int32).pin_memory()
    io = B.lr_pass_host_io(**{k: v.data_ptr() for k, v in host.items()})
    staging = plan.pass_staging()
    ins = ("q_h", "logits_h", "draft_ids_h", "verdict_h")
    h2d = sum(host[k].numel() * host[k].element_size() for k in ins)
    d2h = sum(v.numel() * v.element_size() for k, v in host.items() if k not in ins)
    Ke = max(3, min(M.K, 50))
    n = M.copies
    for i in range(3):
        plan.lr_verify_pass_host(io, M.kc[i % n], M.vc[i % n], staging, 0.0, M.main_stream)
    M.barrier()
    t0 = time.perf_counter()
    for i in range(Ke):
        plan.lr_verify_pass_host(io, M.kc[(3 + i) % n], M.vc[(3 + i) % n], staging, 0.0, M.main_stream)
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / Ke
    e2e_ms, e2e_tokens = S.reduce_measurement(e2e_s * 1e3, b.n_verified_tokens, M.dev)
    return {"value": S.job_throughput(e2e_ms, e2e_tokens), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
            "d2h_bytes_per_step": int(d2h), "ms_per_step": e2e_ms, "steps": Ke,
            "note": "lr_verify_pass_host: pinned host Q/logits/drafts/verdicts in, all results out (one device-to-host copy), "
                    "stream sync per step; KV pools are device-resident cache state"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=5, help="headline workload (default: 5, the largest that runs on one GPU)")
    ap.add_argument("--per-config", default="auto",
                    help="configurations reported under per_config; 'auto' = 2,3,4,5 on one GPU and none on several, '' = none")
    ap.add_argument("--copies", type=int, default=0, help="independent copies of pools/logits (0 = enough for 6x L2)")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip lr_accept_sample / lr_compact / plan-creation timings")
    ap.add_argument("--carry-in", action="store_true", help="q_len = L + 1 per branch (the last accepted token is a query too)")
    ap.add_argument("--tree", default="", help="W,GAMMA[,tiny|layer|serving]: multi-branch drafting workload instead of --config")
    ap.add_argument("--no-overlap", action="store_true", help="run the three steps of a pass strictly one after another")
    ap.add_argument("--no-graph", action="store_true", help="issue every launch from Python instead of replaying CUDA graphs")
    ap.add_argument("--path", type=int, default=0, help="attention path: 0 auto, 1 CUDA cores, 2 tensor cores")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist

    from paper_2506_19830_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the verify pass has no CPU path")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    # ---- headline workload ---------------------------------------------------------------------------------------
    M = Measurement(args, rank, local, world)
    b = M.b
    plan_ms = None
    if not args.no_extras:
        # host cost of planning a batch (a serving loop plans once per cycle: the structure changes every time)
        t_plan = []
        for _ in range(5):
            t0 = time.perf_counter()
            tmp = B.Plan(M.ctx, b)
            torch.cuda.synchronize()
            t_plan.append(time.perf_counter() - t0)
            tmp.close()
        plan_ms = 1e3 * float(np.median(t_plan))
    res = M.measure()
    roof, kernels = M.roofline(res["kernel_us"])
    if not args.no_extras:
        kernels.update(extras(M))
    e2e = None if args.no_e2e else end_to_end(M)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sec, n = oracle_pass_seconds(M.w, args.cpu_seconds)
        cpu = {"value": b.n_verified_tokens / sec, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
               "sample": f"{n} whole passes of the same workload ({M.label}), {sec * 1e3:.1f} ms each",
               "ms_per_pass": sec * 1e3}
    line = {
        "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": M.K, "warmup": M.W,
        "ms_per_step": res["ms_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": M.config_dict(), "roofline": roof, "cpu_baseline": cpu, "e2e": e2e,
        "gpu_launches": int(M.launches_per_step * M.K), "clocks": res["clocks"], "kernels": kernels,
        "timed_regions": res["regions"], "plan_create_host_ms": plan_ms,
    }
    headline_cfg = None if args.tree else args.config
    head_entry = {"workload": M.label, "ms_per_step": res["ms_step"], "value": res["value"], "roofline": roof,
                  "kernels": {k: kernels[k] for k in ("lr_verify_attention", "lr_accept_greedy", "lr_commit")},
                  "clocks": res["clocks"], "cuda_graph": bool(M.all_graphed), "timed_regions": res["regions"]}
    M.close()
    del M

    # ---- the other full-size configurations, same protocol ----------------------------------------------------------
    per_config = {}
    per = args.per_config if args.per_config != "auto" else ("2,3,4,5" if world == 1 else "")
    wanted = [int(c) for c in per.split(",") if c.strip()] if (per and not args.tree and not args.carry_in) else []
    for cfg in wanted:
        if cfg == headline_cfg:
            per_config[str(cfg)] = head_entry
            continue
        Mc = Measurement(args, rank, local, world, cfg=cfg)
        r = Mc.measure()
        rf, ks = Mc.roofline(r["kernel_us"])
        per_config[str(cfg)] = {"workload": Mc.label, "ms_per_step": r["ms_step"], "value": r["value"], "roofline": rf, "kernels": ks,
                                "clocks": r["clocks"], "cuda_graph": bool(Mc.all_graphed), "timed_regions": r["regions"]}
        Mc.close()
        del Mc
    if per_config:
        line["per_config"] = per_config
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
