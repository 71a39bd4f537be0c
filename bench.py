#!/usr/bin/env python
"""Decode-step throughput of the compressed-KV cache path on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--workload NAME]

One step = one fused decode launch over every layer of the workload (score update,
eviction, residual merge, compensated attention, insertion), on a cache produced by the
real prompt-compression pass.  Default workload: LLaMA2-7B shape, batch 1, 54 000-token
prompt, 5 % budget (2 700 slots per head, 1 024 units, 1.45 GB streamed per step --
far larger than L2, so no flush is needed between steps).

N > 1 (torchrun): every rank runs the same workload on its own sequence (weak scaling,
no data-path collective); value = tokens of all ranks / max-over-ranks device time.

The timed region is repeated (--repeats, default 5): `ms_per_step` is the median of the
repeats' CUDA-event times, `spread` their (max - min) / median; SM clocks are sampled every
millisecond and reported per repeat.  At N = 1 the other named workloads (c3, c4 at 10 % and
20 %, c5) are run after the headline one and reported under `configs`, each with its own
roofline and clocks (--configs none skips them).

--impl reference times the CPU oracle (the only other implementation of this path that
exists) on a bounded sample of the same workload, rank 0 only.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

FALLBACK_HBM_GBS = 6650.0


# ----------------------------------------------------------------------------- helpers
def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


KERNEL_SOURCES = ["zsm_decode.cu", "zsm_decode.cuh", "zsm_common.cuh"]


def kernel_fingerprint():
    """sha256 over the decode kernel's sources: ties a recorded ncu figure to the code it came from."""
    import hashlib
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2503_10714_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def recorded_traffic(w):
    """DRAM bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum) for this
    workload, from profiles/decode_fused_traffic.txt: lines `workload layers bytes fingerprint`
    taken on a `layers`-deep stack of the workload and scaled here by the units processed
    (traffic is proportional to units: every unit streams its own slots once).  None when no
    line matches or the kernel's sources changed since the counters were taken."""
    path = os.path.join(ROOT, "profiles", "decode_fused_traffic.txt")
    base = w.name.split("_%dlayers" % w.n_layers)[0]
    try:
        fp = kernel_fingerprint()
        with open(path) as f:
            for line in f:
                t = line.split()
                if len(t) == 4 and not line.startswith("#") and t[0] == base and t[3] == fp:
                    return int(round(float(t[2]) * w.n_layers / int(t[1])))
    except Exception:
        pass
    return None


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML every millisecond, each sample with
    its host time, so that a window of the run (one repeat of the timed region) can be
    summarised by itself."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake"}

    def __init__(self, index):
        self.samples, self.max_mhz = [], None   # (host time, MHz, reason mask)
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        while not self._stop.is_set():
            try:
                mhz = self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)
                mask = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                self.samples.append((time.perf_counter(), mhz, mask))
            except Exception:
                pass
            time.sleep(0.001)

    def __enter__(self):
        if self.nv:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self, windows=None):
        """Median SM MHz and the reasons seen, over the given (t0, t1) host-time windows (all
        samples when None); `per_repeat` lists each window's own median."""
        def inside(t):
            return windows is None or any(a <= t <= b for a, b in windows)
        sel = [(m, k) for t, m, k in self.samples if inside(t)]
        reasons = sorted({name for _, k in sel for bit, name in self.REASONS.items() if k & bit})
        out = {"sm_mhz": float(np.median([m for m, _ in sel])) if sel else None,
               "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(sel),
               "period_ms": 1}
        if windows is not None:
            per = []
            for a, b in windows:
                ms = [m for t, m, _ in self.samples if a <= t <= b]
                per.append(float(np.median(ms)) if ms else None)
            out["per_repeat_sm_mhz"] = per
        return out


NOMINAL_HBM_GBS = 8000.0   # the figure the 70 % target is stated against


def parity_counts(workload_name):
    """Near-tie / exact-tie counts of the full-size parity tests for this workload, from the
    kept record profiles/parity_counts.md (JSON lines written by tests/test_gpu_full_size.py)."""
    out = []
    try:
        with open(os.path.join(ROOT, "profiles", "parity_counts.md")) as f:
            for line in f:
                line = line.strip()
                if line.startswith("{"):
                    rec = json.loads(line)
                    if rec.get("workload") == workload_name:
                        out.append({k: rec[k] for k in ("launches", "sampled_units", "steps", "selections",
                                                         "merges", "victim_near_ties", "merge_near_ties",
                                                         "exact_tie_breaches") if k in rec})
    except Exception:
        return None
    return out or None


def algorithmic_bytes(w, bp, bc, br, n_live, n_res):
    """Bytes one decode launch must move: every live slot's K and V row once, its score read
    and written, its position read; every merged slot's fp32 K and V row and count; per unit
    q, k_new, v_new in, out, the inserted rows and the merged rows out."""
    e = 4 if w.dtype == "f32" else 2
    row = w.head_dim * e
    G = w.group
    per_unit_fixed = G * row + 2 * row + G * row + 2 * row + 2 * w.head_dim * 4 + 16
    total = 0
    for l in range(w.n_layers):
        for h in range(w.n_kv_heads):
            total += w.batch * (n_live[l, h] * (2 * row + 12) + n_res[l, h] * (2 * w.head_dim * 4 + 4)
                                + per_unit_fixed)
    return int(total)


def dist_setup(n_gpus):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl" if torch.cuda.is_available() else "gloo")
    return world, rank, local


def max_over_ranks(x: float, world: int) -> float:
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device="cuda" if torch.cuda.is_available() else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(ms_local: float, tokens_per_rank: int, world: int):
    """Tokens of all ranks divided by the slowest rank's device time (weak scaling: every rank
    processes its own `tokens_per_rank`).  Returns (tokens/s, max-over-ranks ms)."""
    ms_total = max_over_ranks(ms_local, world)
    return world * tokens_per_rank / (ms_total * 1e-3), ms_total


def rank_workload(w0, rank: int):
    """Each rank decodes its own sequence: same shape, its own seed.  No data-path collective."""
    return w0.replace(seed=w0.seed + 1000 * rank)


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


# ----------------------------------------------------------------------------- oracle leg
def oracle_sample(w, K, V, Qw, bp, bc, br, steps, layer=0):
    """Times the oracle, as it stands, on one layer's units: state from its own prompt pass
    (untimed), then `steps` decode steps over those units with OpenMP.  Returns
    (seconds per sampled step, units sampled, threads used, seconds per step on one thread)."""
    from concurrent.futures import ThreadPoolExecutor

    from oracle import zsm_oracle as zo
    zo.build()
    G = w.group
    units = []
    jobs = [(b, h) for b in range(w.batch) for h in range(w.n_kv_heads)]

    def make(job):
        b, h = job
        u = zo.Unit(w.head_dim, G, int(bp[layer, h]), int(bc[layer, h]), int(br[layer, h]),
                    lam=float(np.float32(0.98)), alpha=1.0)
        u.prefill_compress(K[b, h].double().numpy(), V[b, h].double().numpy(),
                           Qw=Qw[b, h * G:(h + 1) * G].double().numpy())
        return u
    with ThreadPoolExecutor(max_workers=os.cpu_count() or 1) as ex:
        units = list(ex.map(make, jobs))
    qs, ks, vs = [], [], []
    for step in range(steps):
        q, k, v = wl.decode_inputs(w.replace(n_layers=1), step)
        qs.append(q[0].double().numpy().reshape(len(jobs), G, w.head_dim))
        ks.append(k[0].double().numpy().reshape(len(jobs), w.head_dim))
        vs.append(v[0].double().numpy().reshape(len(jobs), w.head_dim))
    threads = 1
    t0 = time.perf_counter()
    for step in range(steps):
        _, threads = zo.decode_step_batch(units, qs[step], ks[step], vs[step])
    dt = (time.perf_counter() - t0) / steps
    # the same units one after another on one thread, a few more steps (inputs reused)
    n1 = min(steps, 4)
    t1 = time.perf_counter()
    for step in range(n1):
        for i, u in enumerate(units):
            u.decode_step(qs[step][i], ks[step][i], vs[step][i])
    dt1 = (time.perf_counter() - t1) / n1
    for u in units:
        u.close()
    return dt, len(jobs), threads, dt1


# ----------------------------------------------------------------------------- per-layer leg
def per_layer_graph(zb, cache, w, qs, ks, vs, out, first_step, steps):
    """One decode step issued as n_layers per-layer launches (what a model does between its
    GEMMs), the launches of a step captured once in a CUDA graph and replayed.  Inputs are read
    from fixed buffers that each replay refills with a device copy outside the graph."""
    dev = qs.device
    q_in, k_in, v_in = qs[first_step].clone(), ks[first_step].clone(), vs[first_step].clone()
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(3):
            for l in range(w.n_layers):
                zb.zsm_decode_step(cache, l, q_in[l], k_in[l], v_in[l], out[l], stream=side)
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for l in range(w.n_layers):
                zb.zsm_decode_step(cache, l, q_in[l], k_in[l], v_in[l], out[l],
                                   stream=torch.cuda.current_stream())
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for s in range(3):
        g.replay()
    torch.cuda.synchronize()
    ev0.record()
    for s in range(steps):
        n = first_step + (s % max(1, qs.shape[0] - first_step))
        q_in.copy_(qs[n]); k_in.copy_(ks[n]); v_in.copy_(vs[n])
        g.replay()
    ev1.record()
    ev1.synchronize()
    if zb.zsm_last_device_status(cache) != 0:
        raise RuntimeError("device status after the per-layer launches is not OK")
    ms = ev0.elapsed_time(ev1) / steps
    grid, block, smem = zb.zsm_decode_launch_info(cache, 0)
    return {"what": "%d per-layer launches per step, replayed from one CUDA graph" % w.n_layers,
            "ms_per_step": ms, "tokens_per_s": w.batch / (ms * 1e-3), "steps": steps,
            "grid_per_launch": grid, "units_per_launch": w.batch * w.n_kv_heads}


# ----------------------------------------------------------------------------- FullKV leg
def fullkv_comparator(zb, w, dev, u, stream, budget_bytes=60e9, steps=10):
    """Decode attention over the UNCOMPRESSED prompt KV of the same workload (what the paper's
    FullKV baseline does per step, cache path only), timed with CUDA events.  As many layers as
    fit in `budget_bytes` are held at once; the step time is scaled to the full stack by layers
    (layers are independent and equal)."""
    e = 2
    per_layer = 2 * w.batch * w.n_kv_heads * w.prompt_len * w.head_dim * e
    n_l = int(max(1, min(w.n_layers, budget_bytes // per_layer)))
    upl = w.batch * w.n_kv_heads
    K = torch.empty(n_l * upl, w.prompt_len, w.head_dim, dtype=w.torch_dtype, device=dev)
    V = torch.empty_like(K)
    for layer in range(n_l):
        Kp, Vp, _ = wl.prompt(w, layer, dev, u)
        K[layer * upl:(layer + 1) * upl] = Kp.reshape(upl, w.prompt_len, w.head_dim)
        V[layer * upl:(layer + 1) * upl] = Vp.reshape(upl, w.prompt_len, w.head_dim)
        del Kp, Vp
    q_all, _, _ = wl.decode_inputs(w, 0, dev, u)
    q = q_all[:n_l].reshape(n_l * upl, w.group, w.head_dim).contiguous()
    out = torch.empty_like(q)
    ws = torch.empty(zb.zsm_fullkv_workspace_bytes(n_l * upl, w.group, w.head_dim, w.prompt_len),
                     dtype=torch.uint8, device=dev)
    for _ in range(3):
        zb.zsm_fullkv_decode(K, V, q, out, ws)
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(steps):
        zb.zsm_fullkv_decode(K, V, q, out, ws)
    ev1.record(stream)
    ev1.synchronize()
    if zb.zsm_fullkv_status(ws) != 0:
        raise RuntimeError("device status after the uncompressed-cache comparator is not OK")
    ms_timed = ev0.elapsed_time(ev1) / steps
    nbytes = n_l * (per_layer + upl * 2 * w.group * w.head_dim * e)
    ms_full = ms_timed * w.n_layers / n_l
    return {"what": "decode attention over the uncompressed prompt KV, same kernels' ring and tensor-core logits",
            "context": w.prompt_len, "layers_timed": n_l, "ms_per_step": ms_full,
            "tokens_per_s": w.batch / (ms_full * 1e-3), "achieved_gbs": nbytes / (ms_timed * 1e-3) / 1e9,
            "bytes_per_step_all_layers": int(nbytes * w.n_layers / n_l)}


# ----------------------------------------------------------------------------- full-history scoring leg
def full_history_scores(zb, cache, w, dev, u, stream):
    """Prompt scores with the window taken as the whole prompt (one layer): both tensor-core
    passes, and the column-sum pass alone with the rows' log-sum-exp supplied.  Queries are
    synthetic (the prompt generator makes only the last `window` of them)."""
    T = w.prompt_len
    Kp, _, _ = wl.prompt(w, 0, dev, u)
    g = torch.Generator(device=dev)
    g.manual_seed(w.seed * 1000003 + 17)
    Q = torch.randn(w.batch, w.n_q_heads, T, w.head_dim, device=dev, generator=g).to(w.torch_dtype)
    scores = torch.empty(w.batch, w.n_kv_heads, T, dtype=torch.float32, device=dev)
    ws = torch.empty(zb.zsm_prefill_scores_full_workspace_bytes(cache, T), dtype=torch.uint8, device=dev)
    lse = ws.view(torch.float32)[: w.batch * w.n_q_heads * T]
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    for rep in range(2):  # first round warms up
        ev[0].record(stream)
        zb.zsm_prefill_scores_full(cache, Kp, Q, T, scores, ws)
        ev[1].record(stream)
        zb.zsm_prefill_scores_full(cache, Kp, Q, T, scores, None, lse)
        ev[2].record(stream)
        ev[2].synchronize()
    ms_both, ms_col = ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2])
    nres = (T + 127) // 128  # per pass: resident block rb meets 2 rb + 2 streamed tiles of 64 rows
    flop = 2.0 * w.batch * w.n_q_heads * (nres * (nres + 1)) * 128 * 64 * w.head_dim
    tf = measured_tensor_peak()
    res = {"what": "full-history prompt scores (W = T), one layer: row log-sum-exp + decayed column sums",
           "T": T, "ms_both_passes": ms_both, "ms_column_pass": ms_col,
           "tflops": 2 * flop / (ms_both * 1e-3) / 1e12, "peak_tflops": tf,
           "frac": (2 * flop / (ms_both * 1e-3) / 1e12) / tf if tf else None, "bound": "tensor"}
    # the same scores as a by-product of the prompt's causal attention (output + row statistics +
    # scores in one call): two passes over Q K^T and one over P V
    _, Vp, _ = wl.prompt(w, 0, dev, u)
    out = torch.empty_like(Q)
    lse_o = torch.empty(w.batch, w.n_q_heads, T, dtype=torch.float32, device=dev)
    for rep in range(2):
        ev[0].record(stream)
        zb.zsm_prefill_attention(cache, Kp, Vp, Q, T, out, lse_o, scores)
        ev[1].record(stream)
        zb.zsm_prefill_attention(cache, Kp, Vp, Q, T, out, lse_o)
        ev[2].record(stream)
        ev[2].synchronize()
    ms_all, ms_out = ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2])
    res["prefill_attention"] = {
        "what": "zsm_prefill_attention, one layer: attention output + log-sum-exp in one pass "
                "(two contractions), + scores (a third)",
        "ms_output_lse_scores": ms_all, "ms_output_lse": ms_out,
        "tflops": 3 * flop / (ms_all * 1e-3) / 1e12,
        "frac": (3 * flop / (ms_all * 1e-3) / 1e12) / tf if tf else None,
        "tflops_output_lse": 2 * flop / (ms_out * 1e-3) / 1e12,
        "frac_output_lse": (2 * flop / (ms_out * 1e-3) / 1e12) / tf if tf else None}
    return res


def measured_tensor_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops"])
    except Exception:
        return 1590.0


# ----------------------------------------------------------------------------- one workload
def make_budgets(zb, w):
    totals = wl.head_budgets(w)
    bp, bc, br = np.zeros_like(totals), np.zeros_like(totals), np.zeros_like(totals)
    for idx in np.ndindex(totals.shape):
        bp[idx], bc[idx], br[idx] = zb.zsm_split_budget(int(totals[idx]))
    return totals, bp, bc, br


def prompt_pass(zb, cache, w, dev, u, stream, keep_layer0):
    """Every layer's prompt through the real compression kernels, one layer after another on
    one stream (timed per layer with events).  Returns (ms total, host copy of layer 0's prompt)."""
    ws = torch.empty(zb.zsm_prefill_workspace_bytes(cache, w.prompt_len, w.window),
                     dtype=torch.uint8, device=dev)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    total, sample = 0.0, None
    for layer in range(w.n_layers):
        Kp, Vp, Qw = wl.prompt(w, layer, dev, u)
        ev0.record(stream)
        zb.zsm_prefill_compress(cache, layer, Kp, Vp, Qw, None, w.prompt_len, w.window, ws)
        ev1.record(stream)
        ev1.synchronize()
        total += ev0.elapsed_time(ev1)
        if layer == 0 and keep_layer0:
            sample = (Kp.cpu(), Vp.cpu(), Qw.cpu())
        del Kp, Vp, Qw
    del ws
    torch.cuda.empty_cache()
    if zb.zsm_last_device_status(cache) != 0:
        raise RuntimeError("device status after the prompt pass is not OK")
    return total, sample


def prompt_pass_overlapped(zb, cache, w, dev, u, n_streams=4, n_layers=8):
    """The prompt pass of `n_layers` layers issued round-robin on `n_streams` streams, each with
    its own workspace: the residual chain of one layer occupies one CTA per unit (32 of 148 SMs
    at c4), so several layers' chains run side by side.  Prompts are generated beforehand; the
    time is wall-to-wall device time over all streams, per layer."""
    per_layer_bytes = 2 * w.batch * w.n_kv_heads * w.prompt_len * w.head_dim * (4 if w.dtype == "f32" else 2)
    n_layers = int(min(n_layers, w.n_layers, max(2, 30e9 // per_layer_bytes)))
    n_streams = min(n_streams, n_layers)
    need = zb.zsm_prefill_workspace_bytes(cache, w.prompt_len, w.window)
    wss = [torch.empty(need, dtype=torch.uint8, device=dev) for _ in range(n_streams)]
    streams = [torch.cuda.Stream(device=dev) for _ in range(n_streams)]
    prompts = [wl.prompt(w, layer, dev, u) for layer in range(n_layers)]
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    main = torch.cuda.current_stream()
    ev0.record(main)
    for st in streams:
        st.wait_event(ev0)
    for layer in range(n_layers):
        st = streams[layer % n_streams]
        Kp, Vp, Qw = prompts[layer]
        zb.zsm_prefill_compress(cache, layer, Kp, Vp, Qw, None, w.prompt_len, w.window,
                                wss[layer % n_streams], stream=st)
    for st in streams:
        main.wait_stream(st)
    ev1.record(main)
    ev1.synchronize()
    if zb.zsm_last_device_status(cache) != 0:
        raise RuntimeError("device status after the overlapped prompt pass is not OK")
    ms = ev0.elapsed_time(ev1)
    del prompts, wss
    torch.cuda.empty_cache()
    return {"what": "%d layers round-robin on %d streams, one workspace per stream" % (n_layers, n_streams),
            "layers": n_layers, "streams": n_streams, "ms_per_layer": ms / n_layers,
            "ms_total_scaled": ms / n_layers * w.n_layers}


def run_workload(zb, w, args, dev, local, world, rank, headline):
    """Prompt pass, then the timed decode steps of one workload.  Returns the result dict (on
    every rank; only rank 0's is printed)."""
    stream = torch.cuda.current_stream()
    totals, bp, bc, br = make_budgets(zb, w)
    W, K, R = max(3, args.warmup), max(1, args.steps), max(1, args.repeats)
    cfg = zb.make_config(w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, bp,
                         bc, br, tune_stages=args.stages, tune_ctas_per_sm=args.ctas_per_sm,
                         tune_consumer_warps=args.consumer_warps, tune_split=args.split)
    buf = torch.empty(zb.zsm_cache_bytes(cfg), dtype=torch.uint8, device=dev)
    cache = zb.zsm_cache_create(cfg, buf)
    u = wl.directions(w, dev)
    want_cpu = headline and rank == 0 and world == 1 and not args.no_cpu_baseline
    prefill_ms, sample_prompt = prompt_pass(zb, cache, w, dev, u, stream, want_cpu)

    # ---- decode inputs for every step, resident in HBM before timing starts ----
    n_in = W + K
    qs = torch.empty(n_in, w.n_layers, w.batch, w.n_q_heads, w.head_dim, dtype=w.torch_dtype, device=dev)
    ks = torch.empty(n_in, w.n_layers, w.batch, w.n_kv_heads, w.head_dim, dtype=w.torch_dtype, device=dev)
    vs = torch.empty_like(ks)
    for s in range(n_in):
        qs[s], ks[s], vs[s] = wl.decode_inputs(w, s, dev, u)
    out = torch.empty_like(qs[0])
    for s in range(W):
        zb.zsm_decode_step(cache, -1, qs[s], ks[s], vs[s], out)
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rep_ms, windows = [], []
    with ClockSampler(local) as clocks:
        for r in range(R):
            barrier(world)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            ev0.record(stream)
            for s in range(W, W + K):   # the same K inputs each repeat; the cache keeps evolving
                zb.zsm_decode_step(cache, -1, qs[s], ks[s], vs[s], out)
            ev1.record(stream)
            ev1.synchronize()
            torch.cuda.synchronize()
            windows.append((t0, time.perf_counter()))
            barrier(world)
            rep_ms.append(max_over_ranks(ev0.elapsed_time(ev1), world))
    ms_total = float(np.median(rep_ms))
    ms_per_step = ms_total / K
    value = world * w.batch * K / (ms_total * 1e-3)
    spread = (max(rep_ms) - min(rep_ms)) / ms_total
    if zb.zsm_last_device_status(cache) != 0:
        raise RuntimeError("device status after the timed region is not OK")

    # ---- roofline of the dominant (only) kernel of the timed region ----
    n_live = np.minimum((bp + bc).astype(np.int64), w.prompt_len + W)
    n_res = br.astype(np.int64)
    abytes = algorithmic_bytes(w, bp, bc, br, n_live, n_res)
    peak, peak_kind = measured_peak()
    achieved = abytes / (ms_per_step * 1e-3) / 1e9
    grid, block, smem = zb.zsm_decode_launch_info(cache, -1)
    res = {
        "value": value, "ms_per_step": ms_per_step, "repeats": R, "spread": spread,
        "ms_per_step_repeats": [m / K for m in rep_ms],
        "config": {"workload": w.name, "layers": w.n_layers, "batch_per_gpu": w.batch,
                   "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads, "head_dim": w.head_dim,
                   "prompt_len": w.prompt_len, "slots_per_head": int(totals.mean()),
                   "launch": "one fused kernel over all layers per step",
                   "grid": grid, "block": block, "smem_bytes": smem,
                   "l2": "inputs larger than L2 (%.2f GB streamed per step)" % (abytes / 1e9)},
        "clocks": clocks.summary(windows),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": peak_kind + " copy bandwidth of this pool",
                     "frac_nominal": achieved / NOMINAL_HBM_GBS, "peak_nominal": NOMINAL_HBM_GBS,
                     "algorithmic_bytes_per_launch": abytes, "traffic": recorded_traffic(w)},
        "prompt_pass": {"ms_total": prefill_ms, "ms_per_layer": prefill_ms / w.n_layers,
                        "window": w.window, "what": "layers one after another on one stream"},
        "dtype": w.dtype,
    }
    pc = parity_counts(w.name.split("_%dlayers" % w.n_layers)[0])
    if pc is not None:
        res["parity_counts"] = pc

    # ---- the same metric through host buffers (copies inside the timed region) ----
    if headline:
        Ke = max(1, min(args.e2e_steps, K))
        q_off, k_off, v_off, in_bytes, out_bytes = zb.zsm_decode_host_layout(cache, -1)
        half = in_bytes + (out_bytes + 255) // 256 * 256
        staging = torch.empty(2 * half, dtype=torch.uint8, device=dev)
        packed = []
        for s in range(Ke):
            t = torch.zeros(in_bytes, dtype=torch.uint8)
            for off, src in ((q_off, qs[W + s]), (k_off, ks[W + s]), (v_off, vs[W + s])):
                raw = src.contiguous().view(torch.uint8).reshape(-1).cpu()
                t[off:off + raw.numel()] = raw
            packed.append(t.pin_memory())
        oh = [torch.empty(out.shape, dtype=out.dtype).pin_memory() for _ in range(2)]

        def pipelined(n):
            for s in range(n + 2):
                slot = s & 1
                if s >= 2:
                    zb.zsm_decode_step_host_wait(cache, slot)
                if s < n:
                    zb.zsm_decode_step_host_async(cache, -1, packed[s], oh[slot], staging, slot)
        pipelined(min(3, Ke))
        torch.cuda.synchronize()
        barrier(world)
        t0 = time.perf_counter()
        pipelined(Ke)
        torch.cuda.synchronize()
        e2e_s = max_over_ranks(time.perf_counter() - t0, world)
        # and one step at a time: copies in, step, copy out, wait -- nothing overlaps
        st1 = torch.empty(zb.zsm_decode_staging_bytes(cache, -1), dtype=torch.uint8, device=dev)
        qh = [qs[W + s].cpu().pin_memory() for s in range(Ke)]
        kh = [ks[W + s].cpu().pin_memory() for s in range(Ke)]
        vh = [vs[W + s].cpu().pin_memory() for s in range(Ke)]
        for s in range(min(3, Ke)):
            zb.zsm_decode_step_host(cache, -1, qh[s], kh[s], vh[s], oh[0], st1)
        torch.cuda.synchronize()
        barrier(world)
        t0 = time.perf_counter()
        for s in range(Ke):
            zb.zsm_decode_step_host(cache, -1, qh[s], kh[s], vh[s], oh[0], st1)
        torch.cuda.synchronize()
        sync_s = max_over_ranks(time.perf_counter() - t0, world)
        res["e2e"] = {"value": world * w.batch * Ke / e2e_s, "unit": "tokens/s",
                      "h2d_bytes_per_step": int(in_bytes), "d2h_bytes_per_step": int(out_bytes),
                      "steps": Ke, "ms_per_step": e2e_s / Ke * 1e3,
                      "what": "zsm_decode_step_host_async: pinned host buffers, one copy in and one "
                              "out per step, two steps in flight",
                      "one_step_at_a_time": {"value": world * w.batch * Ke / sync_s,
                                             "ms_per_step": sync_s / Ke * 1e3,
                                             "what": "zsm_decode_step_host: copies, step, copy, wait"}}
        del staging, st1, packed, qh, kh, vh

    if rank == 0 and world == 1:
        # the launch shape a model would use: one launch per layer, the L launches of a step
        # captured in a CUDA graph (reported beside the headline, not instead of it)
        if w.n_layers > 1:
            pl = per_layer_graph(zb, cache, w, qs, ks, vs, out, W, min(K, 200))
            pl["achieved_gbs"] = abytes / (pl["ms_per_step"] * 1e-3) / 1e9
            pl["frac"] = pl["achieved_gbs"] / peak
            res["per_layer_launches"] = pl
        del qs, ks, vs
        torch.cuda.empty_cache()
        if w.n_layers > 1 and not args.no_prompt_overlap:
            res["prompt_pass"]["overlapped"] = prompt_pass_overlapped(zb, cache, w, dev, u)
        if headline and not args.no_fullkv and w.dtype != "f32":
            fk = fullkv_comparator(zb, w, dev, u, stream)
            fk["compressed_speedup"] = fk["ms_per_step"] / ms_per_step
            res["fullkv"] = fk
        if headline and not args.no_full_history and w.dtype != "f32":
            res["prompt_scores_full_history"] = full_history_scores(zb, cache, w, dev, u, stream)
        if want_cpu and sample_prompt is not None:
            dt, n_sampled, threads, dt1 = oracle_sample(w, *sample_prompt, bp, bc, br, args.cpu_steps)
            n_units = w.n_layers * w.batch * w.n_kv_heads
            res["cpu_baseline"] = {
                "value": w.batch / (dt * n_units / n_sampled), "unit": "tokens/s", "cores": threads,
                "one_thread": w.batch / (dt1 * n_units / n_sampled), "kind": "oracle",
                "sample": "%d of %d units (layer 0) x %d decode steps, scaled by units" % (
                    n_sampled, n_units, args.cpu_steps)}
    zb.zsm_cache_free(cache)
    del buf
    torch.cuda.empty_cache()
    return res


# ----------------------------------------------------------------------------- main
OTHER_CONFIGS = ["c3_llama7b_b16", "c4_54k_10pct", "c4_54k_20pct", "c5_gqa_ragged"]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--repeats", type=int, default=5,
                    help="times the timed region is run; the median is reported")
    ap.add_argument("--impl", default="zsm", choices=["zsm", "reference"])
    ap.add_argument("--workload", default="c4_54k_5pct", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--configs", default="all", choices=["all", "none"],
                    help="all: also run the other named workloads (1 GPU only) and report them "
                         "under `configs`")
    ap.add_argument("--config-steps", type=int, default=100, help="timed steps of those workloads")
    ap.add_argument("--e2e-steps", type=int, default=200)
    ap.add_argument("--cpu-steps", type=int, default=64)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-fullkv", action="store_true",
                    help="skip the uncompressed-cache comparator (same box, same shapes)")
    ap.add_argument("--no-full-history", action="store_true",
                    help="skip the full-history (W = T) prompt scoring leg")
    ap.add_argument("--no-prompt-overlap", action="store_true",
                    help="skip the prompt pass with layers overlapped on several streams")
    ap.add_argument("--layers", type=int, default=0,
                    help="run a shallower stack than the workload names (profiling captures only; "
                         "the reported config says so)")
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--ctas-per-sm", type=int, default=0)
    ap.add_argument("--consumer-warps", type=int, default=0)
    ap.add_argument("--split", type=int, default=0, choices=[0, 1, 2, 4, 8],
                    help="CTAs per unit in launches with few units (0: library default, 1: never)")
    args = ap.parse_args()
    world, rank, local = dist_setup(args.gpus)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    from paper_2503_10714_b200 import binding as zb

    w = rank_workload(wl.WORKLOADS[args.workload], rank)
    if args.layers > 0:
        w = w.replace(n_layers=args.layers, name=w.name + "_%dlayers" % args.layers)
    res = run_workload(zb, w, args, dev, local, world, rank, headline=True)
    if rank != 0:
        return
    K, W = max(1, args.steps), max(3, args.warmup)
    line = {
        "metric": "decode tokens/s with ZSMerge cache update",
        "value": res["value"], "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": res["ms_per_step"], "repeats": res["repeats"], "spread": res["spread"],
        "ms_per_step_repeats": res["ms_per_step_repeats"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": res["dtype"],
        "data": "synthetic", "config": res["config"], "clocks": res["clocks"],
        "e2e": res.get("e2e"), "gpu_launches": K,
        "roofline": res["roofline"], "prompt_pass": res["prompt_pass"],
    }
    for key in ("parity_counts", "per_layer_launches", "prompt_scores_full_history", "fullkv",
                "cpu_baseline"):
        if key in res:
            line[key] = res[key]
    if world == 1 and args.configs == "all" and args.layers == 0 and args.workload == "c4_54k_5pct":
        others = {}
        sub = argparse.Namespace(**vars(args))
        sub.steps = max(1, args.config_steps)
        for name in OTHER_CONFIGS:
            try:
                r = run_workload(zb, wl.WORKLOADS[name], sub, dev, local, world, rank, headline=False)
                r["steps"] = sub.steps
                others[name] = r
            except Exception as exc:   # a workload that does not fit must not lose the headline
                others[name] = {"error": "%s: %s" % (type(exc).__name__, exc)}
        line["configs"] = others
    print(json.dumps(line))


def main_reference():
    """--impl reference: the oracle on the machine's host cores, a bounded sample per step."""
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="reference")
    ap.add_argument("--workload", default="c4_54k_5pct", choices=sorted(wl.WORKLOADS))
    args, _ = ap.parse_known_args()
    if int(os.environ.get("RANK", "0")) != 0:
        return
    w = wl.WORKLOADS[args.workload]
    from oracle import zsm_oracle as zo
    totals = wl.head_budgets(w)
    bp = np.zeros_like(totals)
    bc = np.zeros_like(totals)
    br = np.zeros_like(totals)
    for idx in np.ndindex(totals.shape):
        bp[idx], bc[idx], br[idx] = zo.split_budget(int(totals[idx]))
    Kp, Vp, Qw = wl.prompt(w, 0)
    K = max(1, min(args.steps, 256))
    W = max(3, args.warmup)
    dt, n_sampled, threads, dt1 = oracle_sample(w, Kp, Vp, Qw, bp, bc, br, W + K)
    n_units = w.n_layers * w.batch * w.n_kv_heads
    step_s = dt * n_units / n_sampled
    sample = "%d of %d units (layer 0) per step, scaled by units; %d steps" % (n_sampled, n_units, K)
    value = w.batch / step_s
    print(json.dumps({
        "impl": "reference", "metric": "decode tokens/s with ZSMerge cache update", "value": value,
        "unit": "tokens/s", "n_gpus": 1, "steps": K, "warmup": W, "ms_per_step": step_s * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": w.name, "layers": w.n_layers, "batch_per_gpu": w.batch,
                   "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads, "head_dim": w.head_dim,
                   "prompt_len": w.prompt_len, "slots_per_head": int(totals.mean())},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": threads, "kind": "oracle",
                         "one_thread": w.batch / (dt1 * n_units / n_sampled), "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


if __name__ == "__main__":
    _pre = argparse.ArgumentParser(add_help=False)
    _pre.add_argument("--impl", default="zsm")
    if _pre.parse_known_args()[0].impl == "reference":
        main_reference()
    else:
        main()
