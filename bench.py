#!/usr/bin/env python
"""Benchmark of the MLA decode hot path (one attention layer-call over a paged latent
KV cache) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5] [--impl reference]

A step is one ``splash_mla_decode`` call (work plan, page gather, QK^T, online softmax,
P.V, epilogue, split-KV combine) over one synthetic batch.  The default workload is the
RL-rollout batch (512 requests, lognormal contexts, 128 heads, e4m3 KV with one scale per
token): the largest configuration that one GPU holds and the one in the precision of the
paper's runs.  ``--workload`` picks another configuration, and the default run also reports
the other configurations (DP-attention slice, head slice at 32K, CP ranges + LSE merge, page
migration) under ``"workloads"``, with the roofline fractions of the two target
configurations repeated under ``"targets"``.  Rank 0 prints ONE JSON line.

``--gpus N`` with N > 1 starts N ranks itself (one process per GPU under
``torch.distributed.run`` on 127.0.0.1) unless it already runs inside such a launch
(``WORLD_SIZE`` set); every rank decodes its own request slice, no collective on the data
path, and rank 0 prints the line with ``n_gpus: N``.

Timing: CUDA events on the launching stream around every step, L2 flushed between
steps by writing a 256 MiB buffer outside the timed intervals, and every workload's KV
is larger than the 126 MB L2 anyway.  ``value`` is requests decoded per second for one
layer-call with inputs resident in HBM; ``e2e`` repeats it with the step's inputs
(q, block table, lengths) copied from pinned host memory and out / lse copied back
inside the timed region (the KV pool itself is serving state that lives in HBM).

``roofline`` follows the decode kernel's own duration against the MEASURED peaks of this
pool (copy bandwidth, bf16 GEMM burst rate; for e4m3 KV the tensor peak is taken at the bf16
rate because every operand choice that meets the tolerance costs the pipe what bf16 costs).
``roofline.nominal`` repeats the arithmetic for the WHOLE CALL (plan + decode + combine)
against the nominal peaks of the part -- 8 TB/s, 2.25 PFLOP/s bf16, 4.5 PFLOP/s fp8 for the
kernels that issue 8-bit MMAs -- which is the stricter reading of the target.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_37626_b200 import sharding, workloads as W  # noqa: E402

METRIC = "mla_decode_tokens_per_s_per_gpu"
UNIT = "tokens/s"
WORKLOAD_IDS = {"c1": 1, "c2": 2, "c3": 3, "c4": 4, "c5": 5}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}
NOMINAL_PEAKS = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0, "fp8_tflops": 4500.0}
DTYPES = {0: "bf16", 1: "e4m3 KV with an fp32 scale per token, bf16 q, 8-bit MMAs in two terms, fp32 accumulate"}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return dict(FALLBACK_PEAKS)


def load_traffic():
    """Per-launch DRAM traffic of the decode kernel from committed ncu summaries."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if os.path.exists(path):
        return json.load(open(path))
    return {}


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 100 ms while running."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
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
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        # "under load": samples at or above the median of the upper half
        load = sorted(sm)[len(sm) // 2:]
        return {"sm_mhz": float(np.median(load)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


def pairs_sample(w, budget_macs: float, seed: int = 0):
    """A bounded random sample of (request, head) pairs for the oracle."""
    rng = np.random.default_rng(seed)
    heads = np.arange(w.head_begin, w.head_end)
    all_pairs = [(i, g) for i in range(w.B) for g in heads]
    order = rng.permutation(len(all_pairs))
    lens = w.seq_lens.astype(np.int64)
    picked, macs = [], 0.0
    for k in order:
        i, g = all_pairs[k]
        picked.append((i, g))
        macs += float(lens[i]) * (W.D_QK + W.D_V)
        if macs >= budget_macs:
            break
    return np.array(picked, dtype=np.int32), macs, len(all_pairs)


def time_oracle(w, seconds_target: float = 12.0):
    """Times the oracle, as it stands, on a bounded sample of the workload."""
    import oracle
    threads = oracle.num_threads()
    # probe rate with a small sample, then size the main sample
    probe, macs0, total_pairs = pairs_sample(w, 2e8 * threads, seed=1)
    t0 = time.perf_counter()
    oracle.mla_decode(w.q, w.kv_pool, w.block_table, w.seq_lens, softmax_scale=w.softmax_scale,
                      kv_scales=w.kv_scales, kv_begin=w.kv_begin, kv_end=w.kv_end, pairs=probe)
    rate = macs0 / max(time.perf_counter() - t0, 1e-6)
    sample, macs, _ = pairs_sample(w, rate * seconds_target, seed=2)
    t0 = time.perf_counter()
    oracle.mla_decode(w.q, w.kv_pool, w.block_table, w.seq_lens, softmax_scale=w.softmax_scale,
                      kv_scales=w.kv_scales, kv_begin=w.kv_begin, kv_end=w.kv_end, pairs=sample)
    dt = time.perf_counter() - t0
    total_macs = float(w.total_tokens()) * (W.D_QK + W.D_V) * (w.head_end - w.head_begin)
    full_time = dt * total_macs / macs
    return {"value": w.B / full_time, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{len(sample)} of {total_pairs} (request, head) pairs, {dt:.1f} s of CPU work, "
                      f"scaled to the whole batch by multiply-accumulates"}, dt


# --------------------------------------------------------------------------- GPU side
class GpuBench:
    def __init__(self, device):
        import torch
        from paper_2609_37626_b200 import binding
        self.torch, self.binding, self.device = torch, binding, device
        binding.load()
        self.flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=device)
        self.flush_read_buf = torch.ones(256 << 20, dtype=torch.uint8, device=device)

    def flush_l2(self):
        # Write a buffer larger than L2, then read another one: the write alone leaves 126 MB of DIRTY lines behind, and
        # the timed kernel would pay for their write-back while it streams (c3: 115.7 us against 103.4 us; the same
        # 103 us with no flush at all, the inputs being larger than L2, and 106 us under ncu, which invalidates).
        self.flush_buf.fill_(1)
        self.flush_read_buf.view(self.torch.int64).sum()

    def timed(self, fn, steps, warmup):
        torch = self.torch
        for _ in range(warmup):
            self.flush_l2(); fn()
        torch.cuda.synchronize()
        times = []
        for _ in range(steps):
            self.flush_l2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record()
            b.synchronize()
            times.append(a.elapsed_time(b))
        return np.array(times)

    def timed_round_robin(self, fns, steps, warmup):
        """Median milliseconds of each of several step functions, timed in turn within one loop."""
        torch = self.torch
        for _ in range(warmup):
            for fn in fns:
                self.flush_l2(); fn()
        torch.cuda.synchronize()
        times = [[] for _ in fns]
        for _ in range(steps):
            for k, fn in enumerate(fns):
                self.flush_l2()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); fn(); b.record()
                b.synchronize()
                times[k].append(a.elapsed_time(b))
        return [np.median(t) for t in times]

    def decode_workload(self, w, steps, warmup, peaks, traffic_table, name):
        torch, binding = self.torch, self.binding
        dw = binding.DeviceWorkload(w, self.device)
        out = torch.empty((w.B, w.H, W.D_V), dtype=torch.float32, device=self.device)
        lse = torch.empty((w.B, w.H), dtype=torch.float32, device=self.device)
        step = lambda: dw.decode(out=out, lse=lse)
        ms = self.timed(step, steps, warmup)
        launches = binding.splash_last_launch_count()
        # kernel-level durations (events recorded by the library around each kernel)
        binding.splash_set_kernel_timing(True)
        kt = []
        for _ in range(steps):
            self.flush_l2(); step()
            kt.append(binding.splash_get_kernel_timing())
        # the same with the flush's dirty lines left in L2 (write only): reported beside the main figure
        kd = []
        for _ in range(max(3, steps // 4)):
            self.flush_buf.fill_(1); step()
            kd.append(binding.splash_get_kernel_timing())
        binding.splash_set_kernel_timing(False)
        kt = np.array(kt)
        dirty_ms = float(np.array(kd)[:, 1].mean())
        ws = binding.decode_workspace(torch.device(self.device))
        rc, detail = binding.splash_workspace_status(ws)
        if rc != 0:
            raise RuntimeError(f"device status {rc} {detail}")
        dec_ms = float(kt[:, 1].mean())
        alg_bytes, alg_flops = w.algorithmic_bytes(), w.algorithmic_flops()
        t_hbm = alg_bytes / (peaks["hbm_gbs"] * 1e9)
        fp8 = w.kv_dtype == 1
        t_tensor = alg_flops / (peaks["bf16_tflops"] * 1e12)
        if t_hbm >= t_tensor:
            roof = {"bound": "hbm", "achieved": alg_bytes / (dec_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
        else:
            roof = {"bound": "tensor", "achieved": alg_flops / (dec_ms * 1e-3) / 1e12, "peak": peaks["bf16_tflops"],
                    "unit": "TFLOP/s"}
        roof["frac"] = roof["achieved"] / roof["peak"]
        roof["traffic"] = traffic_table.get(name)
        hs = w.head_end - w.head_begin
        if hs > 64:     # slices of more than 64 heads run on CTA pairs
            kernel = "decode_umma_fp8_pair_kernel" if fp8 else "decode_umma_pair_kernel"
        else:
            n = 16 if hs <= 16 else 32 if hs <= 32 else 64
            kernel = ("decode_umma_fp8_narrow_kernel<%d>" % n if n < 64 else "decode_umma_fp8_kernel") if fp8 else "decode_umma_kernel<%d>" % n
        # the stricter reading: the whole call against the nominal peaks of the part (fp8 MMA rate for e4m3 KV)
        nom_tensor = NOMINAL_PEAKS["fp8_tflops"] if fp8 else NOMINAL_PEAKS["bf16_tflops"]
        tn_hbm, tn_tensor = alg_bytes / (NOMINAL_PEAKS["hbm_gbs"] * 1e9), alg_flops / (nom_tensor * 1e12)
        tn = max(tn_hbm, tn_tensor)
        p50 = float(np.median(ms))
        roof["frac_whole_call"] = max(t_hbm, t_tensor) * 1e3 / p50
        roof["nominal"] = {"hbm_gbs": NOMINAL_PEAKS["hbm_gbs"], "tensor_tflops": nom_tensor,
                           "bound": "hbm" if tn_hbm >= tn_tensor else "tensor", "roofline_ms": tn * 1e3,
                           "frac_kernel": tn * 1e3 / dec_ms, "frac_whole_call": tn * 1e3 / p50}
        roof.update({"kernel": kernel, "kernel_ms": dec_ms, "peak_source": peaks["source"],
                     "algorithmic_bytes": alg_bytes, "algorithmic_flops": alg_flops,
                     "roofline_ms": max(t_hbm, t_tensor) * 1e3,
                     "achieved_gbs": alg_bytes / (dec_ms * 1e-3) / 1e9,
                     "achieved_tflops": alg_flops / (dec_ms * 1e-3) / 1e12,
                     "plan_ms": float(kt[:, 0].mean()), "combine_ms": float(kt[:, 2].mean()),
                     "after_write_only_flush": {"kernel_ms": dirty_ms, "frac": max(t_hbm, t_tensor) * 1e3 / dirty_ms,
                                                "what": "L2 left full of the flush's dirty lines: the kernel also pays for their write-back"},
                     "note": ("e4m3 KV: 'frac' takes the tensor peak at the bf16 rate (two 8-bit terms per operand); "
                              "'nominal' takes the fp8 rate, under which this workload is HBM-bound") if fp8 else None})
        res = {"ms_per_step": float(ms.mean()), "ms_p50": float(np.median(ms)), "ms_p95": float(np.percentile(ms, 95)),
               "tokens_per_s": w.B / (ms.mean() * 1e-3), "tokens_per_s_78_layers": w.B / (ms.mean() * 1e-3) / 78,
               "launches_per_step": launches, "roofline": roof,
               "frac_of_roofline_whole_call": max(t_hbm, t_tensor) * 1e3 / float(np.median(ms)),
               "tokens": w.total_tokens(), "requests": w.B, "heads": w.head_end - w.head_begin}
        return res, dw, out, lse

    def rows_workload(self, w, R, steps, warmup, peaks):
        """R causal query rows per request over the same cache (a multi-token decode step): whole-call time,
        roofline from the algorithmic bytes (each cache row once) and flops (every row of every head)."""
        torch, binding = self.torch, self.binding
        dw = binding.DeviceWorkload(w, self.device)
        q4 = torch.from_numpy(W.make_query_rows(1234, w.B, w.H, R).view(np.int16)).to(self.device).view(torch.bfloat16)
        out = torch.empty((w.B, w.H, R, W.D_V), dtype=torch.float32, device=self.device)
        lse = torch.empty((w.B, w.H, R), dtype=torch.float32, device=self.device)
        step = lambda: binding.splash_mla_decode(q4, dw.kv_pool, dw.block_table, dw.seq_lens, softmax_scale=w.softmax_scale,
                                                 kv_scales=dw.kv_scales, head_begin=w.head_begin, head_end=w.head_end,
                                                 out=out, lse=lse)
        ms = self.timed(step, steps, warmup)
        h = w.head_end - w.head_begin
        rows_bytes = w.B * h * (R - 1) * (W.D_QK * 2 + W.D_V * 4 + 4)        # the extra q rows read, out / lse rows written
        alg_bytes, alg_flops = w.algorithmic_bytes() + rows_bytes, w.algorithmic_flops() * R
        t_hbm, t_tensor = alg_bytes / (peaks["hbm_gbs"] * 1e9), alg_flops / (peaks["bf16_tflops"] * 1e12)
        p50 = float(np.median(ms))
        return {"q_rows": R, "ms_per_step": float(ms.mean()), "ms_p50": p50, "ms_p95": float(np.percentile(ms, 95)),
                "query_rows_per_s": w.B * R / (ms.mean() * 1e-3),
                "roofline": {"bound": "hbm" if t_hbm >= t_tensor else "tensor", "roofline_ms": max(t_hbm, t_tensor) * 1e3,
                             "frac": max(t_hbm, t_tensor) * 1e3 / p50, "of": "whole call, p50", "peak_source": peaks["source"],
                             "algorithmic_bytes": alg_bytes, "algorithmic_flops": alg_flops,
                             "launch_chains": 1, "cta_pairs_per_kv_worker": -(-h * R // 128)},
                "launches_per_step": binding.splash_last_launch_count()}

    def layer_loop(self, w, dw, out, lse, steps, warmup, layers=8):
        """One decode step of a model: the same batch through `layers` layers.  The first layer's call plans, the
        others take its partition again (SPLASH_FLAG_REUSE_PLAN); L2 flushed before every layer, as the GEMMs between
        two attention layers would leave it."""
        torch, binding = self.torch, self.binding
        def step(reuse):
            times = []
            for k in range(layers):
                self.flush_l2()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); dw.decode(out=out, lse=lse, flags=binding.SPLASH_FLAG_REUSE_PLAN if (reuse and k > 0) else 0); b.record()
                times.append((a, b))
            torch.cuda.synchronize()
            return [a.elapsed_time(b) for a, b in times]
        for _ in range(max(1, warmup // 2)):
            step(True); step(False)
        first, rest, plain = [], [], []
        for _ in range(max(2, steps // 4)):
            t = step(True); first.append(t[0]); rest.extend(t[1:])
            plain.extend(step(False))
        rc, detail = binding.splash_workspace_status(binding.decode_workspace(torch.device(self.device)))
        if rc != 0:
            raise RuntimeError(f"device status {rc} {detail}")
        per_layer = (float(np.median(first)) + (layers - 1) * float(np.median(rest))) / layers
        return {"layers": layers, "ms_first_layer": float(np.median(first)), "ms_other_layers": float(np.median(rest)),
                "ms_every_layer_planning": float(np.median(plain)), "ms_per_layer": per_layer,
                "tokens_per_s_per_layer": w.B / (per_layer * 1e-3),
                "how": "layer 0 plans, layers 1.. pass SPLASH_FLAG_REUSE_PLAN (the partition depends on lengths, ranges and shape only)"}

    def slice_workload(self, w, dw, out, lse, head_begin, head_end, steps, warmup, peaks, traffic=None):
        """A TP rank's share of workload `w`: the same cache and requests, heads [head_begin, head_end) only."""
        import copy
        torch, binding = self.torch, self.binding
        ws = copy.copy(w)
        ws.head_begin, ws.head_end = head_begin, head_end
        step = lambda: dw.decode(out=out, lse=lse, head_begin=head_begin, head_end=head_end)
        ms = self.timed(step, steps, warmup)
        launches = binding.splash_last_launch_count()
        binding.splash_set_kernel_timing(True)
        kt = []
        for _ in range(steps):
            self.flush_l2(); step()
            kt.append(binding.splash_get_kernel_timing())
        binding.splash_set_kernel_timing(False)
        kt = np.array(kt)
        rc, detail = binding.splash_workspace_status(binding.decode_workspace(torch.device(self.device)))
        if rc != 0:
            raise RuntimeError(f"device status {rc} {detail}")
        dec_ms, p50 = float(kt[:, 1].mean()), float(np.median(ms))
        alg_bytes = ws.algorithmic_bytes()
        t_hbm = alg_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3
        hs = head_end - head_begin
        n = 16 if hs <= 16 else 32 if hs <= 32 else 64
        kernel = ("decode_umma_fp8_narrow_kernel<%d>" % n if n < 64 else "decode_umma_fp8_kernel") if w.kv_dtype == 1 \
            else "decode_umma_kernel<%d>" % n
        return {"ms_per_step": float(ms.mean()), "ms_p50": p50, "ms_p95": float(np.percentile(ms, 95)),
                "tokens_per_s": w.B / (ms.mean() * 1e-3), "launches_per_step": launches, "heads": hs,
                "requests": w.B, "tokens": w.total_tokens(),
                "roofline": {"bound": "hbm", "achieved": alg_bytes / (dec_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                             "unit": "GB/s", "frac": t_hbm / dec_ms, "frac_whole_call": t_hbm / p50, "traffic": traffic,
                             "kernel": kernel, "kernel_ms": dec_ms, "plan_ms": float(kt[:, 0].mean()),
                             "combine_ms": float(kt[:, 2].mean()), "algorithmic_bytes": alg_bytes,
                             "roofline_ms": t_hbm, "peak_source": peaks["source"]}}

    def sparse_workload(self, seq_lens, H, steps, warmup, peaks, topk=2048):
        """Sparse decode: every request attends over the (at most) topk tokens of a seeded list, cache rows in the
        656-byte format.  Whole-call time; the roofline is each LISTED row once over the measured copy bandwidth."""
        torch, binding = self.torch, self.binding
        w = W.make_workload("sparse_top%d" % topk, W.BASE_SEED + 60, seq_lens, H=H, kv_dtype=2)
        sel_h, cnt_h = W.select_tokens(W.BASE_SEED + 60, w.seq_lens, topk)
        dw = binding.DeviceWorkload(w, self.device)
        sel, cnt = torch.from_numpy(sel_h).to(self.device), torch.from_numpy(cnt_h).to(self.device)
        out = torch.empty((w.B, w.H, W.D_V), dtype=torch.float32, device=self.device)
        lse = torch.empty((w.B, w.H), dtype=torch.float32, device=self.device)
        step = lambda: binding.splash_mla_decode_sparse(dw.q, dw.kv_pool, dw.block_table, dw.seq_lens, sel, cnt,
                                                        softmax_scale=w.softmax_scale, out=out, lse=lse)
        ms = self.timed(step, steps, warmup)
        launches = binding.splash_last_launch_count()
        binding.splash_set_kernel_timing(True)
        kt = []
        for _ in range(steps):
            self.flush_l2(); step()
            kt.append(binding.splash_get_kernel_timing())
        binding.splash_set_kernel_timing(False)
        kt = np.array(kt)
        rc, detail = binding.splash_workspace_status(binding.decode_workspace(torch.device(self.device)))
        if rc != 0:
            raise RuntimeError(f"device status {rc} {detail}")
        # the fused kernel (one kernel gathers, dequantises and multiplies), for comparison: not the default path
        fused = lambda: binding.splash_mla_decode_sparse(dw.q, dw.kv_pool, dw.block_table, dw.seq_lens, sel, cnt,
                                                         softmax_scale=w.softmax_scale, out=out, lse=lse,
                                                         flags=binding.SPLASH_FLAG_SPARSE_FUSED)
        ms_fused = self.timed(fused, steps, warmup)
        rc, detail = binding.splash_workspace_status(binding.decode_workspace(torch.device(self.device)))
        if rc != 0:
            raise RuntimeError(f"device status {rc} {detail} (fused sparse kernel)")
        n_sel = int(cnt_h.sum())
        alg_bytes = W.sparse_algorithmic_bytes(cnt_h, H)
        alg_flops = 2 * H * (W.D_QK + W.D_V) * n_sel
        t_hbm, t_tensor = alg_bytes / (peaks["hbm_gbs"] * 1e9), alg_flops / (peaks["bf16_tflops"] * 1e12)
        p50 = float(np.median(ms))
        return {"requests": w.B, "heads": H, "topk": topk, "listed_tokens": n_sel, "context_tokens": w.total_tokens(),
                "row_bytes": W.SPARSE_ROW_BYTES, "ms_per_step": float(ms.mean()), "ms_p50": p50,
                "ms_p95": float(np.percentile(ms, 95)), "tokens_per_s": w.B / (ms.mean() * 1e-3),
                "stages_ms": {"plan": float(kt[:, 0].mean()), "gather_and_dense_decode": float(kt[:, 1].mean()),
                              "combine": float(kt[:, 2].mean()),
                              "note": "timed with events between the kernels, which keeps them from overlapping"},
                "roofline": {"bound": "hbm" if t_hbm >= t_tensor else "tensor", "roofline_ms": max(t_hbm, t_tensor) * 1e3,
                             "frac": max(t_hbm, t_tensor) * 1e3 / p50, "of": "whole call, p50", "peak_source": peaks["source"],
                             "algorithmic_bytes": alg_bytes, "algorithmic_flops": alg_flops,
                             "bytes_moved_by_the_two_stages": n_sel * (W.SPARSE_ROW_BYTES + 2 * W.D_QK * 2)},
                "fused_kernel_variant": {"ms_p50": float(np.median(ms_fused)), "launches_per_step": binding.splash_last_launch_count(),
                                         "note": "SPLASH_FLAG_SPARSE_FUSED: every listed row crosses HBM once; not the default while slower"},
                "launches_per_step": launches}

    def dop_workload(self, steps, warmup, peaks, N=16384, T=8, h=16):
        """DOP transfer layout changes at a rank's size of a large batch: N query rows, h = H/T local heads;
        bytes read + written over the measured copy bandwidth."""
        torch, binding = self.torch, self.binding
        g = torch.Generator(device=self.device); g.manual_seed(77)
        nope = torch.randint(-2 ** 15, 2 ** 15, (N, h, 512), dtype=torch.int16, device=self.device, generator=g).view(torch.bfloat16)
        rope = torch.randint(-2 ** 15, 2 ** 15, (N, h, 64), dtype=torch.int16, device=self.device, generator=g).view(torch.bfloat16)
        send_row = torch.randperm(N, device=self.device, generator=g).to(torch.int32)
        send = torch.empty((N, h, 576), dtype=torch.bfloat16, device=self.device)
        res = {}
        def report(name, ms, nbytes):
            p50 = float(np.median(ms))
            res[name] = {"ms_p50": p50, "gbs": nbytes / (p50 * 1e-3) / 1e9, "frac_of_hbm": nbytes / (p50 * 1e-3) / 1e9 / peaks["hbm_gbs"],
                         "bytes": nbytes}
        ms = self.timed(lambda: binding.splash_dop_pack_rows(nope, rope, send_row, out=send), steps, warmup)
        report("pack_rows", ms, 2 * send.numel() * 2 + N * 4)
        recv = send.view(T, N // T, h, 576)
        swapped = torch.empty((N // T, T, h, 576), dtype=torch.bfloat16, device=self.device)
        ms = self.timed(lambda: binding.splash_dop_swap_outer(recv, out=swapped), steps, warmup)
        report("swap_outer", ms, 2 * recv.numel() * 2)
        del nope, rope, send, swapped
        o_recv = torch.empty((N, h, 512), dtype=torch.float32, device=self.device).normal_(generator=g)
        o_out = torch.empty((N, h, 512), dtype=torch.float32, device=self.device)
        ms = self.timed(lambda: binding.splash_dop_unpack_rows(o_recv, send_row, o_out), steps, warmup)
        report("unpack_rows", ms, 2 * o_recv.numel() * 4 + N * 4)
        res["shape"] = {"rows": N, "ranks": T, "local_heads": h}
        return res

    def in_kernel_clock(self, dw, out, lse):
        """SM clock seen by the decode kernel itself: cycles / nanoseconds of its main loop, per CTA, from the
        library's diagnostic trace (written by the CTA-pair kernels; None for the others), and the longest span in
        microseconds of the thread that writes the trace (the producer warp's: it ends a few tiles before its CTA)."""
        torch, binding = self.torch, self.binding
        buf = torch.zeros(64 * 8 + 512, dtype=torch.int64, device=self.device)
        self.flush_l2()
        binding.splash_debug_set_trace(buf)
        try:
            dw.decode(out=out, lse=lse)
            torch.cuda.synchronize()
        finally:
            binding.splash_debug_set_trace(None)
        t = buf.cpu().numpy()
        cyc, ns = t[512:512 + 148].astype(np.float64), t[768:768 + 148].astype(np.float64)
        ok = (cyc > 0) & (ns > 0)
        if not ok.any():
            return None, None
        return float(np.median(cyc[ok] / ns[ok]) * 1e3), float(ns[ok].max() * 1e-3)

    def e2e(self, w, dw, steps, warmup):
        """Same call with the step's inputs coming from pinned host memory and the
        results going back to it inside the timed region."""
        torch, binding = self.torch, self.binding
        hq = torch.from_numpy(w.q.view(np.int16)).pin_memory()
        ht = torch.from_numpy(w.block_table).pin_memory()
        hs = torch.from_numpy(w.seq_lens).pin_memory()
        dq = torch.empty_like(dw.q); dt_ = torch.empty_like(dw.block_table); ds = torch.empty_like(dw.seq_lens)
        out = torch.empty((w.B, w.H, W.D_V), dtype=torch.float32, device=self.device)
        lse = torch.empty((w.B, w.H), dtype=torch.float32, device=self.device)
        hb, he = w.head_begin, w.head_end
        ho = torch.empty((w.B, he - hb, W.D_V), dtype=torch.float32).pin_memory()
        hl = torch.empty((w.B, he - hb), dtype=torch.float32).pin_memory()

        def step():
            dq.view(torch.int16).copy_(hq, non_blocking=True)
            dt_.copy_(ht, non_blocking=True); ds.copy_(hs, non_blocking=True)
            binding.splash_mla_decode(dq, dw.kv_pool, dt_, ds, softmax_scale=w.softmax_scale, kv_scales=dw.kv_scales,
                                      head_begin=hb, head_end=he, kv_begin=dw.kv_begin, kv_end=dw.kv_end,
                                      out=out, lse=lse)
            ho.copy_(out[:, hb:he], non_blocking=True); hl.copy_(lse[:, hb:he], non_blocking=True)

        ms = self.timed(step, steps, warmup)
        h2d = hq.numel() * 2 + ht.numel() * 4 + hs.numel() * 4
        d2h = ho.numel() * 4 + hl.numel() * 4

        # The same steps as a serving loop would run them: two sets of buffers, the upload of step i + 1 and the
        # download of step i - 1 overlap the decode of step i (three streams; every step still uploads its inputs
        # and downloads its results).  Timed as one region over all steps; the KV read per step exceeds L2.
        s_up, s_run, s_down = (torch.cuda.Stream(device=self.device) for _ in range(3))
        bufs = []
        for _ in range(2):
            bufs.append(dict(q=torch.empty_like(dw.q), t=torch.empty_like(dw.block_table), s=torch.empty_like(dw.seq_lens),
                             out=torch.empty_like(out), lse=torch.empty_like(lse),
                             ho=torch.empty_like(ho).pin_memory(), hl=torch.empty_like(hl).pin_memory(),
                             up=None, ran=None, down=None))

        def pipelined(n):
            for i in range(n):
                b = bufs[i % 2]
                with torch.cuda.stream(s_up):
                    if b["ran"] is not None:
                        s_up.wait_event(b["ran"])            # the decode that last read these input buffers
                    b["q"].view(torch.int16).copy_(hq, non_blocking=True)
                    b["t"].copy_(ht, non_blocking=True); b["s"].copy_(hs, non_blocking=True)
                    b["up"] = torch.cuda.Event(); b["up"].record(s_up)
                with torch.cuda.stream(s_run):
                    s_run.wait_event(b["up"])
                    if b["down"] is not None:
                        s_run.wait_event(b["down"])          # the download that last read these output buffers
                    binding.splash_mla_decode(b["q"], dw.kv_pool, b["t"], b["s"], softmax_scale=w.softmax_scale,
                                              kv_scales=dw.kv_scales, head_begin=hb, head_end=he, kv_begin=dw.kv_begin,
                                              kv_end=dw.kv_end, out=b["out"], lse=b["lse"], stream=s_run)
                    b["ran"] = torch.cuda.Event(); b["ran"].record(s_run)
                with torch.cuda.stream(s_down):
                    s_down.wait_event(b["ran"])
                    b["ho"].copy_(b["out"][:, hb:he], non_blocking=True); b["hl"].copy_(b["lse"][:, hb:he], non_blocking=True)
                    b["down"] = torch.cuda.Event(); b["down"].record(s_down)

        pipelined(max(warmup, 3))
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for st in (s_up, s_run, s_down):
            st.wait_event(t0)
        pipelined(steps)
        for st in (s_up, s_run, s_down):
            torch.cuda.current_stream().wait_stream(st)
        t1.record(); t1.synchronize()
        piped_ms = t0.elapsed_time(t1) / steps
        return {"value": w.B / (piped_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                "d2h_bytes_per_step": int(d2h), "ms_per_step": float(piped_ms),
                "pipelining": "two buffer sets, upload / decode / download on three streams; %d steps timed as one region" % steps,
                "ms_per_step_one_step_at_a_time": float(ms.mean())}

    def cp_workload(self, w, steps, warmup):
        """CP: 8 contiguous KV ranges, each a partial (O, LSE) call, then splash_lse_merge."""
        torch, binding = self.torch, self.binding
        dw = binding.DeviceWorkload(w, self.device)
        ranges = [(torch.from_numpy(a).to(self.device), torch.from_numpy(b).to(self.device))
                  for a, b in W.cp_ranges(w.seq_lens, 8)]
        po = torch.empty((8, w.B, w.H, W.D_V), dtype=torch.float32, device=self.device)
        pl = torch.empty((8, w.B, w.H), dtype=torch.float32, device=self.device)
        mo = torch.empty((w.B * w.H, W.D_V), dtype=torch.float32, device=self.device)
        ml = torch.empty((w.B * w.H,), dtype=torch.float32, device=self.device)

        def step():
            for j, (a, b) in enumerate(ranges):
                dw.decode(out=po[j], lse=pl[j], kv_begin=a, kv_end=b)
            binding.splash_lse_merge(po.view(8, -1, W.D_V), pl.view(8, -1), out=mo, lse=ml)

        ms = self.timed(step, steps, warmup)
        merge = self.timed(lambda: binding.splash_lse_merge(po.view(8, -1, W.D_V), pl.view(8, -1), out=mo, lse=ml),
                           steps, warmup)
        return {"ms_8_ranges_plus_merge": float(ms.mean()), "ms_merge": float(merge.mean()),
                "launches_per_step": 8 * 3 + 1}

    def migrate_workload(self, w, dw, steps, warmup, peaks):
        torch, binding = self.torch, self.binding
        # the workload was built with a second pool of ceil(0.3 * used pages) pages appended
        total = w.num_pool_pages
        extra_pages = int(np.ceil(len(w.used_pages) * 0.3))
        n_src = total - extra_pages
        src, dst = W.migration_plan(W.BASE_SEED + 55, w.used_pages, extra_pages, 0.3)
        dsrc, ddst = torch.from_numpy(src).to(self.device), torch.from_numpy(dst).to(self.device)
        table0 = dw.block_table.clone()

        def step():
            dw.block_table.copy_(table0)
            binding.splash_kv_page_migrate(dw.kv_pool[:n_src], dw.kv_pool[n_src:], dsrc, ddst, dw.block_table,
                                           src_scales=dw.kv_scales[:n_src], dst_scales=dw.kv_scales[n_src:],
                                           src_id_base=0, dst_id_base=n_src, max_page_id=total)

        ms = self.timed(step, steps, warmup)
        page_bytes = 64 * 576 + 256
        moved = 2.0 * len(src) * page_bytes
        dw.block_table.copy_(table0)
        return {"ms_per_call": float(ms.mean()), "pages": int(len(src)), "bytes_read_plus_written": moved,
                "achieved_gbs": moved / (ms.mean() * 1e-3) / 1e9, "frac_of_hbm_peak": moved / (ms.mean() * 1e-3) / 1e9 / peaks["hbm_gbs"],
                "note": "includes the block-table restore copy issued before each call"}


    def overlap_workload(self, w, dw, steps, warmup, layers=4):
        """Layer-pipelined migration under decode (Sec. 4.1 "Handoff"): layer l's pages move on a second stream while
        layer l - 1 decodes; decode of layer l waits for its pages.  All layers use this workload's arrays (the
        migration writes the second pool and a copy of the table, so the decodes' inputs never change).  Reports the
        time the migration adds to the decode-only sequence, in units of one layer's migration."""
        torch, binding = self.torch, self.binding
        total = w.num_pool_pages
        extra_pages = int(np.ceil(len(w.used_pages) * 0.3))
        n_src = total - extra_pages
        src, dst = W.migration_plan(W.BASE_SEED + 55, w.used_pages, extra_pages, 0.3)
        dsrc, ddst = torch.from_numpy(src).to(self.device), torch.from_numpy(dst).to(self.device)
        table_next = dw.block_table.clone()
        out = torch.empty((w.B, w.H, W.D_V), dtype=torch.float32, device=self.device)
        lse = torch.empty((w.B, w.H), dtype=torch.float32, device=self.device)
        side = torch.cuda.Stream(device=self.device)
        mig_ws = torch.empty(int(binding.load().splash_kv_page_migrate_workspace_bytes(total)) + 256, dtype=torch.uint8, device=self.device)

        def migrate(stream):
            binding.splash_kv_page_migrate(dw.kv_pool[:n_src], dw.kv_pool[n_src:], dsrc, ddst, table_next,
                                           src_scales=dw.kv_scales[:n_src], dst_scales=dw.kv_scales[n_src:],
                                           src_id_base=0, dst_id_base=n_src, max_page_id=total, workspace=mig_ws, stream=stream)

        def decode_only():
            for _ in range(layers):
                dw.decode(out=out, lse=lse)

        def migrate_only():
            for _ in range(layers):
                migrate(None)

        def pipelined():
            main = torch.cuda.current_stream()
            side.wait_stream(main)
            started = None
            for l in range(layers):
                # layer l's pages move while layer l - 1 decodes
                if started is not None:
                    side.wait_event(started)
                with torch.cuda.stream(side):
                    migrate(side)
                    moved = torch.cuda.Event(); moved.record(side)
                main.wait_event(moved)
                started = torch.cuda.Event(); started.record(main)
                dw.decode(out=out, lse=lse)
            main.wait_stream(side)

        job = binding.make_migrate_job(dw.kv_pool[:n_src], dw.kv_pool[n_src:], dsrc, ddst, table_next,
                                       src_scales=dw.kv_scales[:n_src], dst_scales=dw.kv_scales[n_src:],
                                       src_id_base=0, dst_id_base=n_src, max_page_id=total, workspace=mig_ws)

        def carried():
            # the library's own overlap: layer 0's pages move on their own, then layer l's decode call carries the
            # migration of layer l + 1 in warps of the decode kernel that are otherwise idle (one stream)
            migrate(None)
            for l in range(layers):
                dw.decode(out=out, lse=lse, migrate_job=job if l + 1 < layers else None)

        def serial():
            # no overlap at all: every layer moves its pages, then decodes, on one stream
            for _ in range(layers):
                migrate(None)
                dw.decode(out=out, lse=lse)

        # the five sequences take turns inside one timing loop, so that the clock the power cap leaves (it sinks while
        # the load lasts) is the same for all of them
        t_dec, t_mig, t_ser, t_pipe, t_two = (float(x) for x in self.timed_round_robin(
            [decode_only, migrate_only, serial, carried, pipelined], steps, warmup))
        per_layer = (t_ser - t_dec) / layers           # what one layer's migration costs when nothing hides it
        return {"layers": layers, "decode_only_ms": t_dec, "migrate_only_ms": t_mig, "serial_ms": t_ser,
                "pipelined_ms": t_pipe, "exposed_ms": t_pipe - t_dec,
                "exposed_in_layer_migrations": (t_pipe - t_dec) / per_layer,
                "how": "splash_mla_decode_migrating: layer l + 1's page copy rides in layer l's decode kernel; "
                       "serial = (migrate, decode) per layer on one stream; a layer-migration = (serial - decode only) / layers",
                "two_streams_plain_calls_ms": t_two,
                "pages_per_layer": int(len(src))}


def run_reference(args, rank):
    """The oracle as the reference arm: each step is a bounded sample of the workload."""
    if rank != 0:
        return
    w = W.config(WORKLOAD_IDS[args.workload])
    per_step = max(2.0, min(20.0, 150.0 / max(args.steps + args.warmup, 1)))
    vals, cores, sample = [], None, None
    for k in range(args.warmup + args.steps):
        res, _ = time_oracle(w, seconds_target=per_step)
        if k >= args.warmup:
            vals.append(res["value"])
        cores, sample = res["cores"], res["sample"]
    v = float(np.mean(vals))
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": w.B / v * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": W.CONFIG_NAMES[WORKLOAD_IDS[args.workload] - 1], "requests": w.B,
                       "heads": w.head_end - w.head_begin, "tokens": w.total_tokens()},
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def free_port() -> int:
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def launch_ranks(n: int, argv) -> int:
    """Start n ranks of this script on this node (one process per GPU) and wait for them."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


class StubBench:
    """Stands in for the GPU side when the launcher and the rank plumbing are tested on CPU (``--stub-step``): a step
    is a short host computation, nothing here is a measurement."""

    def decode_workload(self, w, steps, warmup, *_):
        times = []
        for k in range(warmup + steps):
            t0 = time.perf_counter()
            float(np.square(w.seq_lens.astype(np.float64)).sum())
            if k >= warmup:
                times.append((time.perf_counter() - t0) * 1e3 + 1e-3)
        ms = np.array(times)
        return ({"ms_per_step": float(ms.mean()), "ms_p50": float(np.median(ms)), "ms_p95": float(np.percentile(ms, 95)),
                 "launches_per_step": 0, "roofline": None}, None, None, None)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", choices=sorted(WORKLOAD_IDS), default="c5")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--only-main", action="store_true", help="skip the other configurations")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sparse-only", action="store_true", help="print only the sparse-decode workload's numbers")
    ap.add_argument("--head-slice", default=None, metavar="BEGIN:END",
                    help="time a TP rank's share of the workload: the same cache and requests, heads [BEGIN, END) only")
    ap.add_argument("--stub-step", action="store_true",
                    help="CPU test of the launcher and the rank plumbing: gloo, a host stand-in for the step, no measurement")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    # N > 1 outside a torch.distributed launch: start the ranks here
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    stub = args.stub_step
    if stub:
        device = "cpu"
        if world > 1:
            dist.init_process_group("gloo")
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
        torch.cuda.set_device(local_rank)
        device = f"cuda:{local_rank}"
        if world > 1:
            dist.init_process_group("nccl", device_id=torch.device(device))
    peaks = load_peaks()
    traffic = load_traffic()
    gb = StubBench() if stub else GpuBench(device)

    # every rank owns its own batch (request slices are independent: weak scaling, no collective)
    idx = WORKLOAD_IDS[args.workload]
    t_gen = time.time()
    if stub:
        w = W.config(1)
    elif idx == 5:
        w = W.config(5, extra_pool_factor=0.3 if world == 1 else 0.0)      # with the second pool of the page migration
    else:
        w = W.config(idx)
    if world > 1 and not stub:
        w = W.make_workload(w.name, W.BASE_SEED + idx + 100 * rank, w.seq_lens, H=w.H, head_begin=w.head_begin,
                            head_end=w.head_end, kv_dtype=w.kv_dtype)
    gen_s = time.time() - t_gen
    traffic_key = args.workload
    if args.head_slice:
        hb, he = (int(x) for x in args.head_slice.split(":"))
        if not (0 <= hb < he <= w.H):
            raise SystemExit("--head-slice must lie inside the workload's %d heads" % w.H)
        w.head_begin, w.head_end = hb, he
        traffic_key = "%s_heads%d" % (args.workload, he - hb)

    if args.sparse_only:
        w2 = W.config(2)
        print(json.dumps({"sparse_top2048": gb.sparse_workload(w2.seq_lens, w2.H, args.steps, args.warmup, peaks)}))
        return

    sampler = ClockSampler(local_rank)
    if world > 1:
        dist.barrier()
    if not stub:
        torch.cuda.synchronize()
        sampler.start()
    main_res, dw, out, lse = gb.decode_workload(w, args.steps, args.warmup, peaks, traffic, traffic_key)
    if stub:
        if world > 1:
            dist.barrier()
        clocks = {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["stub step: no GPU"]}
        e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0, "ms_per_step": main_res["ms_per_step"]}
    else:
        torch.cuda.synchronize()
        # the timed region lasts a few milliseconds, less than one nvidia-smi sampling period: keep the same step
        # running for about a second so that the sampler sees the clocks under this load
        t_end = time.time() + 1.0
        while time.time() < t_end:
            for _ in range(20):
                gb.flush_l2(); dw.decode(out=out, lse=lse)
            torch.cuda.synchronize()
        in_kernel_mhz, longest_cta_us = gb.in_kernel_clock(dw, out, lse)
        if world > 1:
            dist.barrier()
        clocks = sampler.stop()
        clocks["sm_mhz_in_kernel"] = in_kernel_mhz
        e2e = gb.e2e(w, dw, args.steps, args.warmup)

    ms = main_res["ms_per_step"]
    e2e_ms = e2e["ms_per_step"]
    ms, e2e_ms = sharding.max_over_ranks([ms, e2e_ms], device=device)
    value = sharding.weak_scaling_value(w.B, world, ms)
    e2e_value = sharding.weak_scaling_value(w.B, world, e2e_ms)

    extra = {}
    targets = {}
    cpu = None
    if main_res["roofline"] is not None and args.workload in ("c3", "c5"):
        targets[args.workload] = main_res["roofline"]["frac"]
    if rank == 0 and world == 1 and not stub:
        if not args.no_cpu_baseline:
            cpu, _ = time_oracle(w)
        if not args.only_main:
            steps2 = max(5, args.steps // 2)
            if idx == 5:
                try:
                    extra["c5"] = {"layer_loop": gb.layer_loop(w, dw, out, lse, steps2, args.warmup),
                                   "tp8_slice": gb.slice_workload(w, dw, out, lse, 32, 48, steps2, args.warmup, peaks, traffic.get("c5_heads16")),
                                   "page_migrate": gb.migrate_workload(w, dw, steps2, args.warmup, peaks),
                                   "migrate_under_decode": gb.overlap_workload(w, dw, steps2, args.warmup)}
                except Exception as exc:  # report, do not hide
                    extra["c5"] = {"error": repr(exc)}
            del dw, out, lse
            torch.cuda.empty_cache()
            w2 = w if idx == 2 else None
            for name in ("c3", "c2", "c4", "c5"):
                if name == args.workload:
                    continue
                try:
                    wx = W.config(5, extra_pool_factor=0.3) if name == "c5" else W.config(WORKLOAD_IDS[name])
                    if name == "c2":
                        w2 = wx
                    r, dwx, ox, lx = gb.decode_workload(wx, args.steps, args.warmup, peaks, traffic, name)
                    if name in ("c3", "c5"):
                        targets[name] = r["roofline"]["frac"]
                    r["layer_loop"] = gb.layer_loop(wx, dwx, ox, lx, steps2, args.warmup)
                    if name == "c4":
                        del dwx
                        r["cp"] = gb.cp_workload(wx, steps2, args.warmup)
                    if name == "c5":
                        # a TP-8 rank's share of the same step: 16 of the 128 heads over the same e4m3 cache
                        r["tp8_slice"] = gb.slice_workload(wx, dwx, ox, lx, 32, 48, steps2, args.warmup, peaks, traffic.get("c5_heads16"))
                        r["page_migrate"] = gb.migrate_workload(wx, dwx, steps2, args.warmup, peaks)
                        r["migrate_under_decode"] = gb.overlap_workload(wx, dwx, steps2, args.warmup)
                    extra[name] = r
                    del ox, lx
                    dwx = None
                    if name != "c2":
                        del wx
                    torch.cuda.empty_cache()
                except Exception as exc:  # report, do not hide
                    extra[name] = {"error": repr(exc)}
            try:
                extra["dop_layout_changes"] = gb.dop_workload(steps2, args.warmup, peaks)
                torch.cuda.empty_cache()
            except Exception as exc:
                extra["dop_layout_changes"] = {"error": repr(exc)}
            if w2 is not None:
                # sparse decode over the DP-attention workload's context lengths, 2048 listed tokens per request
                try:
                    extra["sparse_top2048"] = gb.sparse_workload(w2.seq_lens, w2.H, steps2, args.warmup, peaks)
                    torch.cuda.empty_cache()
                except Exception as exc:
                    extra["sparse_top2048"] = {"error": repr(exc)}
                # several causal query rows per request on that workload's cache (multi-token decode steps)
                for R in (2, 4):
                    try:
                        extra["c2_rows%d" % R] = gb.rows_workload(w2, R, steps2, args.warmup, peaks)
                        torch.cuda.empty_cache()
                    except Exception as exc:
                        extra["c2_rows%d" % R] = {"error": repr(exc)}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": DTYPES[w.kv_dtype], "data": "synthetic",
            "config": {"workload": W.CONFIG_NAMES[idx - 1] if not stub else "stub", "requests_per_gpu": w.B,
                       "heads": w.head_end - w.head_begin,
                       "tokens_per_gpu": w.total_tokens(), "kv_dtype": "bf16" if w.kv_dtype == 0 else "e4m3+token scale",
                       "page_size": 64, "l2": "between steps: 256 MiB flush write, then a 256 MiB read that evicts the flush's dirty lines; KV larger than L2",
                       "parallelism": f"dp{world} (request slices, no collective)"},
            "ms_p50": main_res["ms_p50"], "ms_p95": main_res["ms_p95"],
            "tokens_per_s_78_layers": value / 78,
            "roofline": main_res["roofline"],
            "targets": targets,
            "cpu_baseline": cpu,
            "e2e": {k: (e2e_value if k == "value" else v) for k, v in e2e.items()},
            "gpu_launches": int(main_res["launches_per_step"]) * args.steps,
            "clocks": clocks,
            "input_generation_s": gen_s,
            "workloads": extra,
        }
        if stub:
            line["stub"] = True
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
