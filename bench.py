#!/usr/bin/env python
"""HiLS attention benchmark: one JSON line per run.

A "step" is one pass of the whole hot path (landmark scoring, group max, top-K selection, local
attention, per-chunk attention, fusion) over one batch of seeded synthetic input, through the C ABI.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg0|cfg1|cfg3|cfg4]
                  [--impl ours|reference] [--no-extra] [--no-e2e] [--no-cpu-baseline]

The default workload is cfg2, the largest single-GPU prefill configuration (L = 131072, K = 32); the decode half of
the metric (cfg3, cfg4) and cfg1 are measured in the same run and carried in top-level fields of the JSON line
(decode_cfg3_GBps, decode_cfg4_frac_of_measured_hbm, ...), with their per-kernel detail under "extra".

Prefill workloads report effective TFLOP/s on the gathered FLOP (what the method must do, not what
dense attention would); decode workloads report GB/s on the algorithmic bytes (landmarks scanned +
selected K/V chunks).  With N > 1 every rank runs an independent replica of the workload (the path
shards over batch / KV groups with no exchange), and `value` is the sum over ranks divided by the
slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2607_02980_b200 import workloads as wl

# dram__bytes_read.sum + dram__bytes_write.sum PER LAUNCH of each workload's dominant kernel come from the ncu
# captures recorded in profiles/ncu_dram_traffic.json (kernel, bytes, what was captured, how it was scaled, when): a
# kernel without a record there reports "traffic": null rather than a stale figure.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")


def load_traffic(path=TRAFFIC_FILE):
    """{(workload key, kernel name): record} from the committed traffic file ({} if it is missing)."""
    try:
        with open(path) as f:
            doc = json.load(f)
    except (OSError, ValueError):
        return {}
    return {(r["workload"], r["kernel"]): r for r in doc.get("records", [])}

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


# ----------------------------------------------------------------------------- algorithmic work
def prefill_flops(cfg, W=1):
    """(gathered FLOP, scoring FLOP) of one prefill call: per position, QK^T and PV over the min(K, candidates)
    selected chunks and the local window [l(i), i], l(i) = max(0, floor((i - W + 1) / S)) * S (Sec. 2.1)."""
    i = np.arange(cfg.L, dtype=np.float64)
    lo = np.maximum(0.0, np.floor((i - W + 1) / cfg.S)) * cfg.S
    ci = lo / cfg.S                                                     # candidate chunks
    gathered = 4.0 * cfg.d * (np.minimum(cfg.K, ci) * cfg.S + (i - lo) + 1)
    scoring = 2.0 * cfg.d * ci
    return float(gathered.sum()) * cfg.Hq * cfg.B, float(scoring.sum()) * cfg.Hq * cfg.B


def prefill_flops_rows(cfg, rows):
    i = np.asarray(rows, dtype=np.float64)
    ci = np.floor(i / cfg.S)
    return float((4.0 * cfg.d * (np.minimum(cfg.K, ci) * cfg.S + (i % cfg.S) + 1)).sum()) * cfg.Hq * cfg.B


def decode_bytes(cfg, seq_lens):
    """(landmark bytes scanned, gathered K/V bytes) of one decode call, bf16/fp32 element size."""
    eb = 4 if cfg.dtype == "f32" else 2
    seq = np.asarray(seq_lens, dtype=np.int64)
    ncand = (seq - 1) // cfg.S
    local = (seq - 1) % cfg.S + 1
    lm = float(ncand.sum()) * cfg.Hkv * cfg.d * eb
    kv = float((np.minimum(cfg.K, ncand) * cfg.S + local).sum()) * cfg.Hkv * cfg.d * eb * 2
    return lm, kv


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.rows, self.proc, self.thread = gpu_index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        def pump():
            for line in self.proc.stdout:
                self.rows.append([x.strip() for x in line.split(",")])
        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------- workloads
def pick_cfg(name):
    idx = {"cfg0": 0, "cfg1": 1, "cfg2": 2, "cfg3": 3, "cfg4": 4}[name]
    return wl.CONFIGS[idx]


def params_for(hils, cfg, decode, impl="auto", window=1):
    return hils.make_params(B=cfg.B, Hq=cfg.Hq, Hkv=cfg.Hkv, Hl=cfg.Hkv, L=0 if decode else cfg.L, T_max=cfg.L,
                            C=cfg.C, d=cfg.d, chunk_size=cfg.S, top_k=cfg.K, window=window,
                            dtype=0 if cfg.dtype == "f32" else 1, impl=impl)


class Workload:
    """Device-resident inputs/outputs of one configuration and the call that runs one step."""

    def __init__(self, hils, cfg, device, n_query_sets=8, window=1, with_bias=False, overlap_block=0,
                 overlap_noise=0.3, impl="auto"):
        self.hils, self.cfg, self.dev = hils, cfg, device
        self.impl = impl                         # prefill only: "packed" = the query-major kernel (Sec. 4.2)
        self.decode = cfg.mode == "decode"
        self.window = window                     # prefill only; > 1 = the paper's operator form (Sec. 2.1)
        self.bias = wl.make_bias(cfg, device) if with_bias else None
        self.p = params_for(hils, cfg, self.decode, window=window)
        self.ws = hils.alloc_workspace(self.p, self.decode, device)
        if self.decode:
            self.inp = wl.make_decode_inputs(cfg, device)
            # distinct query sets (different selected chunks) so that gathered chunks are not L2 hits
            self.queries = [self.inp["q"]] + [
                wl.make_decode_queries(cfg, self.inp["landmarks"], self.inp["seq_lens"], s)
                for s in range(1, n_query_sets)]
            self.out = torch.empty_like(self.inp["q"])
            self.lse = torch.empty((cfg.B, cfg.Hq), dtype=torch.float32, device=device)
            self.sel = torch.empty((cfg.B, cfg.Hkv, cfg.K), dtype=torch.int32, device=device)
            lm_b, kv_b = decode_bytes(cfg, self.inp["seq_lens"].cpu().numpy())
            self.work, self.work_aux = lm_b + kv_b, kv_b
            self.unit, self.metric = "GB/s", "hils_decode_algorithmic_GBps"
        else:
            self.inp = wl.make_prefill_inputs(cfg, device, overlap_block=overlap_block, overlap_noise=overlap_noise)
            self.out = torch.empty_like(self.inp["q"])
            self.lse = torch.empty((cfg.B, cfg.Hq, cfg.L), dtype=torch.float32, device=device)
            self.sel = torch.empty((cfg.B, cfg.Hkv, cfg.L, cfg.K), dtype=torch.int32, device=device)
            self.work, self.work_aux = prefill_flops(cfg, window)
            self.unit, self.metric = "TFLOP/s", "hils_prefill_effective_TFLOPs"
        # L2 flush between decode steps: write 256 MB, then read another 256 MB so that the timed kernels
        # start from an L2 full of clean lines (dirty lines would be written back under them)
        self.flush = torch.empty(64 * 1024 * 1024, dtype=torch.int32, device=device) if self.decode else None
        self.flush2 = torch.zeros(64 * 1024 * 1024, dtype=torch.int32, device=device) if self.decode else None
        self.step_no = 0

    def step(self):
        i = self.inp
        if self.decode:
            q = self.queries[self.step_no % len(self.queries)]
            self.step_no += 1
            self.hils.hils_decode(q, i["k"], i["v"], i["landmarks"], i["seq_lens"], self.cfg.S, self.cfg.K,
                                  out=self.out, lse=self.lse, sel_idx=self.sel, workspace=self.ws)
        else:
            self.hils.hils_prefill(i["q"], i["k"], i["v"], i["landmarks"], self.cfg.S, self.cfg.K, bias=self.bias,
                                   window=self.window, impl=self.impl, out=self.out, lse=self.lse, sel_idx=self.sel,
                                   workspace=self.ws)

    def between_steps(self):
        if self.flush is not None:
            self.flush.fill_(1)                  # 256 MB write: evicts the 126 MB L2
            self.sink = self.flush2.max()        # 256 MB read: the write-backs drain before the timed step

    def rate(self, seconds_per_step, n_replicas=1):
        scale = 1e12 if self.unit == "TFLOP/s" else 1e9
        return self.work * n_replicas / seconds_per_step / scale


def time_steps(w, steps, warmup, barrier):
    """K steps timed with CUDA events on the launching stream; flushes sit outside the event pairs."""
    for _ in range(warmup):
        w.between_steps()
        w.step()
    torch.cuda.synchronize()
    barrier()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    traces = []
    for s in range(steps):
        w.between_steps()
        starts[s].record()
        w.step()
        ends[s].record()
        tr = w.hils.trace_read()
        if tr:
            traces.append(tr)
    torch.cuda.synchronize()
    barrier()
    ms = [starts[s].elapsed_time(ends[s]) for s in range(steps)]
    return ms, traces


def summarise_traces(traces):
    """Mean over steps of the per-step device time of each kernel (summed over its launches)."""
    agg = {}
    for tr in traces:
        per_step = {}
        for name, ms in tr:
            per_step[name] = per_step.get(name, 0.0) + ms
        for name, ms in per_step.items():
            agg.setdefault(name, []).append(ms)
    return {k: float(np.mean(v)) for k, v in agg.items()}


def launches_per_step(traces):
    """How many launches of each traced kernel one step makes."""
    n = {}
    for name, _ in traces[0]:
        n[name] = n.get(name, 0) + 1
    return n


def kernel_times(w, steps, barrier):
    """Per-kernel CUDA-event times: the same steps run again with the library's trace events on
    (kept out of the headline timing because an event between two kernels breaks their overlap)."""
    w.hils.trace_enable(True)
    _, traces = time_steps(w, steps, 1, barrier)
    w.hils.trace_enable(False)
    w.launches = launches_per_step(traces) if traces else {}
    return summarise_traces(traces)


def roofline_for(w, kernel_ms, peaks):
    """Roofline entry of the dominant kernel of one step."""
    if not kernel_ms:
        return None
    name = max(kernel_ms, key=kernel_ms.get)
    nl = max(1, getattr(w, "launches", {}).get(name, 1))     # launches of that kernel per step
    sec = kernel_ms[name] * 1e-3 / nl                        # average duration of one launch
    src = "of measured" if peaks["_source"] == "measured" else "of fallback"
    rec = load_traffic().get((w.cfg.name.split("_")[0], name))
    common = {"kernel": name, "launches_per_step": nl, "kernel_ms_per_launch": sec * 1e3,
              "traffic": int(rec["bytes_per_launch"]) if rec else None,
              "traffic_source": ("profiles/ncu_dram_traffic.json: " + rec["capture"]) if rec else None,
              "peak_source": src}
    if w.decode:
        lm_b, kv_b = decode_bytes(w.cfg, w.inp["seq_lens"].cpu().numpy())
        algo = kv_b if "attend" in name else (lm_b if ("score" in name or "select" in name) else lm_b + kv_b)
        algo /= nl
        ach = algo / sec / 1e9
        return dict(common, bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s",
                    frac=ach / peaks["hbm_gbs"], algorithmic_bytes=algo)
    gathered, scoring = prefill_flops(w.cfg)
    algo = (scoring if ("score" in name or "select" in name) else gathered) / nl
    if w.cfg.dtype == "f32":
        # fp32 path on plain FMA units: 148 SMs x 128 lanes x 2 FLOP x max SM clock
        peak = 148 * 128 * 2 * peaks.get("sm_max_mhz", 1965.0) * 1e6 / 1e12
        bound = "alu"
    else:
        peak = peaks["bf16_tflops"]
        bound = "tensor"
    ach = algo / sec / 1e12
    return dict(common, bound=bound, achieved=ach, peak=peak, unit="TFLOP/s", frac=ach / peak,
                algorithmic_flops=algo)


def bench_paged_decode(hils, w, peaks, iters=10):
    """The decode workload again through hils_decode_paged: the same caches cut into pages of one chunk each,
    shuffled (a random block table).  Same algorithmic bytes as the contiguous run."""
    cfg, i = w.cfg, w.inp
    B, Hkv, T, d = i["k"].shape
    C, S = T // cfg.S, cfg.S
    gen = torch.Generator(device=i["k"].device).manual_seed(991)
    perm = torch.randperm(B * C, generator=gen, device=i["k"].device)
    table = perm.reshape(B, C).to(torch.int32)

    def pages(x):
        src = x.view(B, Hkv, C, S, d).permute(0, 2, 1, 3, 4).reshape(B * C, Hkv, S, d)
        out = torch.empty_like(src)
        out[perm] = src                        # page perm[b*C + c] holds chunk c of sequence b
        return out

    kp, vp = pages(i["k"]), pages(i["v"])
    ms = []
    for it in range(iters + 3):
        q = w.queries[it % len(w.queries)]
        w.between_steps()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        hils.hils_decode_paged(q, kp, vp, i["landmarks"], table, i["seq_lens"], cfg.S, cfg.K, out=w.out, lse=w.lse,
                               sel_idx=w.sel, workspace=w.ws)
        e1.record()
        torch.cuda.synchronize()
        if it >= 3:
            ms.append(e0.elapsed_time(e1))
    m = float(np.mean(ms))
    return {"metric": w.metric, "value": w.rate(m * 1e-3), "unit": w.unit, "ms_per_step": m,
            "frac_of_measured_hbm": w.rate(m * 1e-3) / peaks["hbm_gbs"], "pages": int(B * C), "page_tokens": S}


def bench_multi_token_decode(hils, w, peaks, M=4, iters=10):
    """M new tokens per sequence in one hils_decode_multi call on the decode workload's caches (the caches hold
    them already).  Bytes = M single-token decodes' algorithmic bytes (every token scans the landmarks and
    gathers its own chunks); tokens of a sequence that retrieve the same chunk find it in L2."""
    cfg, i = w.cfg, w.inp
    q = torch.stack([w.queries[m % len(w.queries)] for m in range(M)], dim=1).contiguous()     # [B, M, Hq, d]
    out = torch.empty_like(q)
    lse = torch.empty((cfg.B, M, cfg.Hq), dtype=torch.float32, device=q.device)
    sel = torch.empty((cfg.B, M, cfg.Hkv, cfg.K), dtype=torch.int32, device=q.device)
    import ctypes
    n = hils.load_library().hils_decode_multi_workspace_bytes(ctypes.byref(w.p), M)
    ws = torch.zeros(n, dtype=torch.uint8, device=q.device)

    def call():
        hils.hils_decode_multi(q, i["k"], i["v"], i["landmarks"], i["seq_lens"], cfg.S, cfg.K, out=out, lse=lse,
                               sel_idx=sel, workspace=ws)
    for _ in range(3):
        w.between_steps()
        call()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    torch.cuda.synchronize()
    for a, b in ev:
        w.between_steps()
        a.record()
        call()
        b.record()
    torch.cuda.synchronize()
    ms = float(np.mean([a.elapsed_time(b) for a, b in ev]))
    return {"metric": "hils_decode_algorithmic_GBps", "tokens_per_seq": M, "ms_per_step": ms, "ms_per_token": ms / M,
            "value": M * w.work / (ms * 1e-3) / 1e9, "unit": "GB/s",
            "frac_of_measured_hbm": M * w.work / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "l2_policy": "L2 flushed between calls; tokens of one sequence share landmark rows within a call"}


def bench_landmark_summary(hils, w, peaks, iters=10):
    """The chunk-summary kernel (Proposition 3.1) on the workload's K tensor: every chunk of every KV head once.
    HBM-bound; algorithmic bytes = K read once + the learnable queries read + the summaries written."""
    cfg = w.cfg
    k = w.inp["k"]
    lq = wl.make_landmark_queries(cfg, k.device)
    lm = torch.empty_like(lq)
    bias = torch.empty(lq.shape[:3], dtype=torch.float32, device=k.device)
    for _ in range(3):
        hils.hils_landmark_summary(lq, k, cfg.S, landmarks=lm, bias=bias)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    torch.cuda.synchronize()
    ev[0].record()
    for i in range(iters):
        hils.hils_landmark_summary(lq, k, cfg.S, landmarks=lm, bias=bias)
        ev[i + 1].record()
    torch.cuda.synchronize()
    ms = float(np.mean([ev[i].elapsed_time(ev[i + 1]) for i in range(iters)]))
    nbytes = k.numel() * k.element_size() + 2 * lq.numel() * lq.element_size() + bias.numel() * 4
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"metric": "landmark_summary_algorithmic_GBps", "value": gbs, "unit": "GB/s", "ms": ms,
            "algorithmic_bytes": nbytes, "frac_of_measured_hbm": gbs / peaks["hbm_gbs"],
            "l2_policy": "K tensor of %.0f MB > 126 MB L2, read once per call" % (k.numel() * k.element_size() / 1e6)}


class BackwardWorkload:
    """hils_prefill_backward on a prefill workload's tensors (its forward has run: out, lse, sel_idx are set)."""

    def __init__(self, w):
        self.hils, self.w = w.hils, w
        self.dout = torch.randn(w.inp["q"].shape, generator=torch.Generator(device=w.dev).manual_seed(77),
                                device=w.dev, dtype=torch.float32).to(w.inp["q"].dtype)
        self.flush = None
        # five matrix products per (row, selected key) against the forward's two
        self.work = 2.5 * w.work

    def between_steps(self):
        pass

    def step(self):
        w, i = self.w, self.w.inp
        self.grads = self.hils.hils_prefill_backward(i["q"], i["k"], i["v"], i["landmarks"], w.cfg.S, w.cfg.K, w.out,
                                                     w.lse, w.sel, self.dout, bias=w.bias, window=w.window)


def bench_backward(hils, w, peaks, steps, barrier):
    """The backward pass on the workload (gradients through `out`, selection fixed): whole-call time and the
    per-kernel split.  FLOP = 2.5 x the forward's gathered-attention FLOP (S, dO V^T, dQ, dK, dV)."""
    bw = BackwardWorkload(w)
    ms, _ = time_steps(bw, steps, 3, barrier)
    km = kernel_times(bw, 3, barrier)
    t = float(np.mean(ms))
    val = bw.work / (t * 1e-3) / 1e12
    n_launch = hils.last_launch_count()
    del bw
    return {"metric": "hils_prefill_backward_effective_TFLOPs", "value": val, "unit": "TFLOP/s", "ms_per_step": t,
            "median_ms": float(np.median(ms)), "kernel_ms": km, "launches_per_step": n_launch,
            "frac_of_measured_bf16_burst": val / peaks["bf16_tflops"],
            "inputs": "larger than L2: q, dout, out %.0f MB each; dq fp32 %.0f MB" % (
                w.inp["q"].numel() * 2 / 1e6, w.inp["q"].numel() * 4 / 1e6)}


def bench_packed(hils, dev, barrier):
    """The query-major packed kernel (tiles of 16 adjacent tokens over the union of their chunks, Sec. 4.2 and App.
    "Chunk Overlap") beside the chunk-major kernels on queries that share their chunks: one base query per 16 adjacent
    tokens plus noise.  Returns (results, launches)."""
    res, launches = {}, 0
    for name in ("cfg1", "cfg2"):
        cfg = pick_cfg(name)
        for noise in (0.3, 0.03):
            row = {}
            for impl in ("auto", "packed"):
                torch.cuda.empty_cache()
                w = Workload(hils, cfg, dev, overlap_block=16, overlap_noise=noise, impl=impl)
                ms, _ = time_steps(w, 3, 3, barrier)
                launches += hils.last_launch_count() * 6
                key = "chunk_major" if impl == "auto" else "packed"
                row[key + "_ms"] = float(np.mean(ms))
                row[key + "_TFLOPs"] = w.rate(float(np.mean(ms)) * 1e-3)
                if impl == "packed":
                    st, _ = hils.hils_chunk_overlap(w.sel, 16, cfg.C)
                    launches += 1
                    full = st[..., 0] > 0
                    row["mean_union_chunks"] = float(st[..., 1][full].float().mean().item())
                    row["slots_per_block"] = 16 * cfg.K
                del w
            res["%s_noise_%g" % (name, noise)] = row
    torch.cuda.empty_cache()
    return res, launches


def bench_chunk_overlap(hils, w, peaks, M=16, iters=10):
    """Chunk-id overlap of blocks of M adjacent queries (Sec. "Chunk Overlap", Eq. Overlap) on the selection the
    workload's last prefill wrote: the statistics, and the kernel's time against reading sel_idx once."""
    cfg, sel = w.cfg, w.sel
    stats, ov = hils.hils_chunk_overlap(sel, M, cfg.C)
    for _ in range(2):
        hils.hils_chunk_overlap(sel, M, cfg.C, stats=stats, overlap=ov)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    torch.cuda.synchronize()
    ev[0].record()
    for i in range(iters):
        hils.hils_chunk_overlap(sel, M, cfg.C, stats=stats, overlap=ov)
        ev[i + 1].record()
    torch.cuda.synchronize()
    ms = float(np.mean([ev[i].elapsed_time(ev[i + 1]) for i in range(iters)]))
    st = stats.cpu().numpy().astype(np.int64)
    o = ov.cpu().numpy()
    full = st[..., 3] == 1
    nbytes = sel.numel() * 4 + stats.numel() * 4 + ov.numel() * 4
    # the paper's left panel of Fig. chunk_overlap: what the final M queries load of the chunks they can see
    visible = max(0, (cfg.L - 1 - w.window + 1) // cfg.S) if w.window > 1 else (cfg.L - 1) // cfg.S
    last_union = float(st[..., -1, 1].mean())
    return {"block_queries": M, "top_k": cfg.K, "blocks": int(full.size), "full_blocks": int(full.sum()),
            "final_block_union_chunks": last_union, "final_block_visible_chunks": visible,
            "final_block_loaded_fraction": last_union / max(1, visible),
            "mean_overlap": float(o[full].mean()), "mean_union_chunks": float(st[..., 1][full].mean()),
            "reused_from_previous_block": float(st[..., 2][..., 1:].sum() / max(1, st[..., 1][..., 1:].sum())),
            "ms": ms, "algorithmic_bytes": nbytes, "GBps": nbytes / (ms * 1e-3) / 1e9,
            "frac_of_measured_hbm": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}


# ----------------------------------------------------------------------------- CPU oracle legs
def oracle_sample(cfg, inp_cpu, budget_rows):
    """Times the oracle, as it stands, on a bounded sample of the workload.  Returns (value, sample, secs)."""
    import oracle
    if cfg.mode == "prefill":
        rows = wl.sample_rows(cfg, budget_rows).numpy()
        t0 = time.perf_counter()
        oracle.hils_prefill(inp_cpu["q"], inp_cpu["k"], inp_cpu["v"], inp_cpu["landmarks"], None, S=cfg.S, K=cfg.K,
                            rows=rows)
        dt = time.perf_counter() - t0
        val = prefill_flops_rows(cfg, rows) / dt / 1e12
        note = "" if len(rows) >= cfg.L else " (rate on the sample; the whole workload is extrapolated from it)"
        return val, "%d seeded query positions x all %d heads of %s%s" % (len(rows), cfg.Hq, cfg.name, note), dt
    nb = min(cfg.B, budget_rows)
    sub = {k: v[:nb] for k, v in inp_cpu.items()}
    t0 = time.perf_counter()
    oracle.hils_decode(sub["q"], sub["k"], sub["v"], sub["landmarks"], None, sub["seq_lens"], S=cfg.S, K=cfg.K)
    dt = time.perf_counter() - t0
    lm_b, kv_b = decode_bytes(cfg, sub["seq_lens"].numpy())
    return (lm_b + kv_b) / dt / 1e9, "first %d of %d sequences of %s" % (nb, cfg.B, cfg.name), dt


# Query positions the oracle legs run on a prefill workload: the same seeded sample in the cpu_baseline leg of the
# GPU arm and in every step of the reference arm (a few seconds of work on the 128K-token configuration).
ORACLE_SAMPLE_ROWS = 2048


def oracle_sample_timed(cfg, inp_cpu):
    """The oracle, as it stands, on the bounded sample of the workload that both oracle legs use."""
    if cfg.mode != "prefill":
        return oracle_sample(cfg, inp_cpu, cfg.B)
    return oracle_sample(cfg, inp_cpu, ORACLE_SAMPLE_ROWS)


def reference_cfg_inputs(cfg):
    """Host inputs for the oracle legs.  Large decode caches are cut to the first sequences."""
    if cfg.mode == "decode":
        small = cfg.scaled(B=min(cfg.B, 2))
        return small, wl.make_decode_inputs(small, "cpu")
    return cfg, wl.make_prefill_inputs(cfg, "cpu")


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    cfg = pick_cfg(args.workload)
    small, inp = reference_cfg_inputs(cfg)
    budget = ORACLE_SAMPLE_ROWS if cfg.mode == "prefill" else 2
    vals, secs, sample = [], [], ""
    for s in range(args.warmup + args.steps):
        v, sample, dt = oracle_sample(small, inp, budget)
        if s >= args.warmup:
            vals.append(v); secs.append(dt)
    value = float(np.mean(vals))
    unit = "TFLOP/s" if cfg.mode == "prefill" else "GB/s"
    line = {"impl": "reference", "metric": "hils_prefill_effective_TFLOPs" if cfg.mode == "prefill"
            else "hils_decode_algorithmic_GBps", "value": value, "unit": unit, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean(secs)) * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "B": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "L_or_T": cfg.L, "d": cfg.d,
                       "chunk_size": cfg.S, "top_k": cfg.K, "window": 1,
                       "note": "each step = the CPU oracle on a bounded seeded sample of this workload: " + sample},
            "cpu_baseline": {"value": value, "unit": unit, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def aggregate_over_ranks(ms_per_step_local, work_per_replica, unit_scale, dist=None, device="cpu"):
    """Whole-job rate of N independent replicas: every rank did `work_per_replica`; the job takes as
    long as its slowest rank (MAX over ranks of the per-step time).  Returns (value, ms_per_step)."""
    world, ms = 1, float(ms_per_step_local)
    if dist is not None:
        world = dist.get_world_size()
        t = torch.tensor([ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return work_per_replica * world / (ms * 1e-3) / unit_scale, ms


# ----------------------------------------------------------------------------- ranks
def spawn_ranks(n, argv):
    """`python bench.py --gpus N` started by hand: run N copies of this script as ranks 0..N-1 of one node (one GPU
    each, rendezvous on 127.0.0.1) and relay rank 0's output.  Under torchrun (RANK already set) nothing is spawned."""
    import socket
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), HILS_BENCH_SPAWNED="1")
        env.setdefault("NCCL_DEBUG", "INFO")          # the communicator log names every rank of the job
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + list(argv), env=env,
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    rc = 0
    for pr in procs:
        rc = max(rc, abs(pr.wait()))
    return rc


def selftest_ranks(args):
    """Host-only check of the rank plumbing (used by the CPU tests): every rank joins a gloo group, reports a fake
    per-step time, and rank 0 prints the aggregated line exactly as the GPU path would."""
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    value, ms = aggregate_over_ranks(1.0 + rank, 2.0e12, 1e12, dist if world > 1 else None, "cpu")
    if rank == 0:
        print(json.dumps({"selftest": True, "n_gpus": world, "value": value, "ms_per_step": ms}))
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg2", choices=["cfg0", "cfg1", "cfg2", "cfg3", "cfg4"])
    ap.add_argument("--selftest-ranks", action="store_true", help="host-only check of the rank plumbing (gloo)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extra", action="store_true", help="skip the other single-GPU configurations")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--profile-run", action="store_true",
                    help="only run warmup+steps calls of the workload (for ncu captures); no timing extras")
    ap.add_argument("--batch", type=int, default=0, help="profile runs: override the batch size (smaller footprint)")
    ap.add_argument("--prefill-impl", choices=["auto", "packed"], default="auto",
                    help="profile runs: the prefill kernel set (packed = query-major tiles of adjacent tokens)")
    ap.add_argument("--overlap-block", type=int, default=0,
                    help="profile runs: one base query per this many adjacent tokens (0 = independent queries)")
    ap.add_argument("--overlap-noise", type=float, default=0.3, help="profile runs: noise added to the base queries")
    args = ap.parse_args()
    if args.gpus > 1 and "RANK" not in os.environ:
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    if args.selftest_ranks:
        selftest_ranks(args)
        return
    if args.profile_run:
        import paper_2607_02980_b200 as hils
        torch.cuda.set_device(0)
        cfg = pick_cfg(args.workload)
        if args.batch > 0:
            cfg = cfg.scaled(B=args.batch)
        w = Workload(hils, cfg, torch.device("cuda", 0), n_query_sets=2, overlap_block=args.overlap_block,
                     overlap_noise=args.overlap_noise, impl=args.prefill_impl)
        for _ in range(args.warmup + args.steps):
            w.between_steps()
            w.step()
        torch.cuda.synchronize()
        kpc = hils.last_launch_count()
        if args.prefill_impl != "auto":
            print(json.dumps({"profile_run": cfg.name, "B": cfg.B, "calls": args.warmup + args.steps,
                              "kernels_per_call": kpc, "prefill_impl": args.prefill_impl,
                              "overlap_block": args.overlap_block, "overlap_noise": args.overlap_noise}))
            return
        # the chunk-summary kernel over the same key tensor (two calls)
        lq = wl.make_landmark_queries(cfg, w.inp["k"].device)
        for _ in range(2):
            hils.hils_landmark_summary(lq, w.inp["k"], cfg.S)
        torch.cuda.synchronize()
        ov_calls = 0
        if not w.decode:
            # the chunk-overlap statistic of the selection just written (two calls)
            for _ in range(2):
                hils.hils_chunk_overlap(w.sel, 16, cfg.C)
            torch.cuda.synchronize()
            ov_calls = 2
        bwd_calls = 0
        if not w.decode and cfg.dtype == "bf16":
            # the backward pass over the same tensors (two calls)
            bw = BackwardWorkload(w)
            for _ in range(2):
                bw.step()
            torch.cuda.synchronize()
            bwd_calls = 2
        print(json.dumps({"profile_run": cfg.name, "B": cfg.B, "calls": args.warmup + args.steps,
                          "kernels_per_call": kpc, "landmark_summary_calls": 2, "chunk_overlap_calls": ov_calls,
                          "backward_calls": bwd_calls}))
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        run_reference(args)
        return

    import paper_2607_02980_b200 as hils
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    assert torch.cuda.device_count() > local, "rank %d has no GPU of its own (%d visible)" % (local, torch.cuda.device_count())
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x):
        if dist is None:
            return x
        t = torch.tensor([x], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    peaks = load_peaks()
    cfg = pick_cfg(args.workload)
    hils.load_library()
    w = Workload(hils, cfg, dev)
    sampler = ClockSampler(local)
    sampler.start()
    ms, traces = time_steps(w, args.steps, args.warmup, barrier)
    launches = hils.last_launch_count() * args.steps
    timed_launches = launches
    value, ms_step = aggregate_over_ranks(float(np.sum(ms)) / args.steps, w.work,
                                          1e12 if w.unit == "TFLOP/s" else 1e9, dist, dev)
    kernel_ms = kernel_times(w, max(3, min(args.steps, 10)), barrier)
    launches += hils.last_launch_count() * (max(3, min(args.steps, 10)) + 1)

    line = {"metric": w.metric, "value": value, "unit": w.unit, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": cfg.name, "B": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "L_or_T": cfg.L, "d": cfg.d,
                       "chunk_size": cfg.S, "top_k": cfg.K, "window": 1, "parallelism": "replicas x%d" % world,
                       "l2_policy": ("256 MB write + 256 MB read flush and rotating query sets between steps" if w.decode else
                                     "inputs+outputs %.0f MB > 126 MB L2" % (
                                         sum(t.numel() * t.element_size() for t in list(w.inp.values()) + [w.out]) / 1e6)),
                       "median_ms": float(np.median(ms)), "min_ms": float(np.min(ms))},
            "gpu_launches": launches, "kernel_ms": kernel_ms}
    if w.decode:
        line["decode_gathered_kv_GBps"] = None
        for name, kms in kernel_ms.items():
            if "attend" in name:
                line["decode_gathered_kv_GBps"] = w.work_aux / (kms * 1e-3) / 1e9
    else:
        line["scoring_flops"] = w.work_aux
        line["frac_of_nominal_2250_TFLOPs"] = value / world / 2250.0
        line["frac_of_measured_bf16_burst"] = value / world / peaks["bf16_tflops"]
        key = args.workload
        line["prefill_%s_TFLOPs" % key] = value / world
        line["prefill_%s_ms" % key] = ms_step
        line["prefill_%s_frac_of_measured_bf16_burst" % key] = value / world / peaks["bf16_tflops"]
    roof = roofline_for(w, kernel_ms, peaks)
    if roof:
        line["roofline"] = roof

    # ---- end to end: host buffers through the *_host entry points, copies inside the timed region
    if not args.no_e2e:
        runner = hils.HostRunner(w.p, w.decode, dev)
        host = {k: v.cpu().pin_memory() for k, v in w.inp.items()}
        h2d, d2h = runner.bytes_per_step({k: host[k] for k in host})
        def e2e_step():
            runner.run(host["q"], host["k"], host["v"], host["landmarks"], seq_lens=host.get("seq_lens"))
        for _ in range(2):
            e2e_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_e2e = max(3, min(args.steps, 10))
        e0.record()
        for _ in range(n_e2e):
            e2e_step()
        e1.record()
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1) / n_e2e)
        line["e2e"] = {"value": w.rate(e2e_ms * 1e-3, world), "unit": w.unit, "ms_per_step": e2e_ms,
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
        launches += hils.last_launch_count() * (n_e2e + 2)
        del runner, host

    clocks = sampler.stop()          # sampled over the timed steps, the per-kernel pass and the e2e steps
    line["clocks"] = clocks
    inp_cpu_primary = None

    # ---- other configurations (reported beside, never instead of, the primary workload)
    if not args.no_extra and world == 1:
        extras = {}
        if not w.decode and cfg.dtype == "bf16":
            try:
                extras[args.workload + "_backward"] = bench_backward(hils, w, peaks, max(3, args.steps), barrier)
                launches += extras[args.workload + "_backward"]["launches_per_step"] * (max(3, args.steps) + 6)
            except Exception as exc:
                extras[args.workload + "_backward"] = {"error": repr(exc)}
        try:
            if args.workload in ("cfg2", "cfg3"):
                extras["landmark_summary_" + args.workload] = bench_landmark_summary(hils, w, peaks)
                launches += 13
            if args.workload == "cfg2":
                extras["cfg2_chunk_overlap_iid_queries"] = bench_chunk_overlap(hils, w, peaks)
                launches += 13
            if args.workload == "cfg3":
                extras["cfg3_paged"] = bench_paged_decode(hils, w, peaks)
                extras["cfg3_multi_token_decode"] = bench_multi_token_decode(hils, w, peaks)
                launches += 6 * 13
        except Exception as exc:
            extras["primary_extras"] = {"error": repr(exc)}
        if rank == 0 and not args.no_cpu_baseline and not w.decode:
            inp_cpu_primary = {k: v.cpu() for k, v in w.inp.items()}
        del w
        torch.cuda.empty_cache()
        for name in ("cfg1", "cfg2", "cfg3", "cfg4", "cfg0"):
            primary = name == args.workload
            try:
                if not primary:
                    ew = Workload(hils, pick_cfg(name), dev)
                    ems, etr = time_steps(ew, max(3, args.steps), 3, barrier)
                    ek = kernel_times(ew, 3, barrier)
                    ent = {"metric": ew.metric, "value": ew.rate(float(np.mean(ems)) * 1e-3), "unit": ew.unit,
                           "ms_per_step": float(np.mean(ems)), "median_ms": float(np.median(ems)), "kernel_ms": ek,
                           "roofline": roofline_for(ew, ek, peaks)}
                    if ew.decode:
                        ent["frac_of_measured_hbm"] = ent["value"] / peaks["hbm_gbs"]
                        ent["frac_of_nominal_8000_GBps"] = ent["value"] / 8000.0
                    else:
                        ent["frac_of_measured_bf16_burst"] = ent["value"] / peaks["bf16_tflops"]
                        ent["frac_of_nominal_2250_TFLOPs"] = ent["value"] / 2250.0
                    extras[name] = ent
                    launches += hils.last_launch_count() * (max(3, args.steps) + 3)
                    # the other half of the metric and the small prefill configuration, where the driver's parser keeps them
                    if name in ("cfg3", "cfg4"):
                        line["decode_%s_GBps" % name] = ent["value"]
                        line["decode_%s_ms" % name] = ent["ms_per_step"]
                        line["decode_%s_frac_of_measured_hbm" % name] = ent["frac_of_measured_hbm"]
                        line["decode_%s_frac_of_nominal_8000_GBps" % name] = ent["frac_of_nominal_8000_GBps"]
                        for kn, kms in ek.items():
                            if "attend" in kn:
                                line["decode_%s_gathered_kv_GBps" % name] = ew.work_aux / (kms * 1e-3) / 1e9
                                line["decode_%s_gathered_kv_frac_of_measured_hbm" % name] = (
                                    ew.work_aux / (kms * 1e-3) / 1e9 / peaks["hbm_gbs"])
                    elif name in ("cfg1", "cfg2"):
                        line["prefill_%s_TFLOPs" % name] = ent["value"]
                        line["prefill_%s_ms" % name] = ent["ms_per_step"]
                        line["prefill_%s_frac_of_measured_bf16_burst" % name] = ent["frac_of_measured_bf16_burst"]
                    if name in ("cfg2", "cfg3"):
                        extras["landmark_summary_" + name] = bench_landmark_summary(hils, ew, peaks)
                        launches += 13
                    if name == "cfg3":
                        extras["cfg3_paged"] = bench_paged_decode(hils, ew, peaks)
                        launches += 3 * 13
                        extras["cfg3_multi_token_decode"] = bench_multi_token_decode(hils, ew, peaks)
                        launches += 3 * 13
                    if name == "cfg2":
                        extras["cfg2_chunk_overlap_iid_queries"] = bench_chunk_overlap(hils, ew, peaks)
                        launches += 13
                        extras["cfg2_backward"] = bench_backward(hils, ew, peaks, 3, barrier)
                        launches += extras["cfg2_backward"]["launches_per_step"] * 9
                    del ew
                if name == "cfg2":
                    # adjacent queries that retrieve mostly the same chunks, as the paper measures on a trained model
                    torch.cuda.empty_cache()
                    sw = Workload(hils, pick_cfg(name), dev, overlap_block=16)
                    sms, _ = time_steps(sw, max(3, args.steps), 3, barrier)
                    extras["cfg2_structured_overlap"] = {
                        "metric": sw.metric, "value": sw.rate(float(np.mean(sms)) * 1e-3), "unit": sw.unit,
                        "ms_per_step": float(np.mean(sms)), "kernel_ms": kernel_times(sw, 3, barrier),
                        "queries": "one base query per 16 adjacent tokens + 0.3 N(0,1)",
                        "chunk_overlap": bench_chunk_overlap(hils, sw, peaks)}
                    launches += hils.last_launch_count() * (max(3, args.steps) + 6) + 13
                    del sw
                    extras["packed_vs_chunk_major"], n_l = bench_packed(hils, dev, barrier)
                    launches += n_l
                    # the paper's operator form (Sec. 2.1 / experiments): local window W = 512 and a non-null bias
                    torch.cuda.empty_cache()
                    pw = Workload(hils, pick_cfg(name), dev, window=512, with_bias=True)
                    pms, _ = time_steps(pw, max(3, args.steps), 3, barrier)
                    pk = kernel_times(pw, 3, barrier)
                    extras["cfg2_window512_bias"] = {
                        "metric": pw.metric, "value": pw.rate(float(np.mean(pms)) * 1e-3), "unit": pw.unit,
                        "ms_per_step": float(np.mean(pms)), "kernel_ms": pk, "window": 512, "bias": True,
                        "frac_of_measured_bf16_burst": pw.rate(float(np.mean(pms)) * 1e-3) / peaks["bf16_tflops"]}
                    launches += hils.last_launch_count() * (max(3, args.steps) + 6)
                    del pw
                torch.cuda.empty_cache()
            except Exception as exc:  # keep the primary line even if an extra fails
                extras[name] = {"error": repr(exc)}
        line["extra"] = extras

    # ---- the oracle timed beside it on this machine's host cores (rank 0, N = 1 only)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        if inp_cpu_primary is not None:
            small, inp_cpu = cfg, inp_cpu_primary       # the very tensors the GPU steps ran on
        else:
            small, inp_cpu = reference_cfg_inputs(cfg)
        val, sample, secs = oracle_sample_timed(small, inp_cpu)
        line["cpu_baseline"] = {"value": val, "unit": "TFLOP/s" if cfg.mode == "prefill" else "GB/s",
                                "cores": oracle.num_threads(), "kind": "oracle", "sample": sample, "seconds": secs}
    line["gpu_launches"] = timed_launches            # kernels of this library inside the timed region
    line["gpu_launches_whole_run"] = launches        # incl. warm-up, traced, end-to-end and extra-workload passes
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
