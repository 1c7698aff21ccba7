#!/usr/bin/env python
"""Benchmark of the LiteVAR attention path (multi-diagonal window mask + CFG sharing) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference] [--no-extras]
                    [--kernel-only] [--calibration] [--kv8 [IDX ...]] [--dense] [--rho NUM DEN]

A "step" is one pass of the whole hot path over one batch: one full generation's attention,
i.e. every scale step of every layer of the chosen workload (for the single-call workloads 1 and
5: one call).  Rank 0 prints ONE JSON line.  The headline workload is the largest one: the 2K-scale
step (16384 queries against a 34240-row cache, 16 heads, batch 2) under the default window (rho = 1/4).

value            useful TFLOP/s: 256 FLOP per live map entry of every (batch row, head) the kernel
                 computes (under CFG sharing: the conditional half), inputs resident in HBM,
                 the generation's calls replayed from one CUDA graph
e2e              the same metric through the per-call API with pinned HOST buffers: every call
                 copies its Q and the new scale's K/V rows to the device and its output back
roofline         the dominant forward kernel of the workload against the roofline that binds it: the
                 tensor roofline (useful and executed FLOP per launch over the launch time measured here
                 with CUDA events, against the measured bf16 peak) on the 512px and 2K workloads, the HBM
                 roofline (compulsory bytes: Q + K/V prefix read once per computed (b, h), output written
                 for all 2B rows) on the 256px ones; `traffic` is the DRAM traffic per launch from the
                 committed ncu summary while the kernel sources are unchanged
roofline_hbm_workload2   the HBM block of the 256px VAR-d16 generation (the round-one headline), kept beside it
cpu_baseline     the CPU fp64 oracle timed on this machine's host cores on a bounded sample
all_configs      the five benchmark workloads, window and full-mask variants, one short row each
                 (unless --no-extras); per-step detail in all_configs_detail
plan_us          microseconds litevar_attn_plan takes per schedule (device planner + one synchronisation)
calibration      the window calibration kernel against the HBM roofline (also: --calibration alone)
qkv8             the 8-bit Q/K/V row quantiser against the HBM roofline, and the 256px generation
                 with Q and the appended K/V rows quantised before every call
kv8_cache        the attention reading an 8-bit K/V cache (int8 codes + scale and zero point per row) against the
                 same steps on the bf16 cache, workloads 3 and 4 (also: --kv8 alone)

With --impl reference the oracle itself is timed (rank 0 only) and printed in the same format.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2411_17178_b200 import sharding, workloads as wl  # noqa: E402

FLOP_PER_ENTRY = 4 * wl.HEAD_DIM          # QK^T and PV, multiply + add, per live (q, t)
TILE_FLOP = FLOP_PER_ENTRY * 128 * 128    # one executed 128x128 tile pair
METRIC = "multi-diag attn useful TFLOP/s (live entries only)"
UNIT = "TFLOP/s"


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm=float(d["hbm_gbs"]), bf16=float(d["bf16_tflops"]),
                    bf16_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


def kernel_source_hash():
    import hashlib
    h = hashlib.sha256()
    for f in ("litevar_fwd_tc.cu", "litevar_fwd_ws.cu", "litevar_tc_ptx.h", "litevar_fwd_small.cu", "litevar_plan.cu",
              "litevar_internal.h"):
        h.update(open(os.path.join(ROOT, "paper_2411_17178_b200", "csrc", f), "rb").read())
    return h.hexdigest()


KERNEL_NAMES = {1: "fwd_simt_kernel", 2: "fwd_tc_kernel", 3: "fwd_small_kernel", 4: "fwd_ws_kernel"}


def recorded_traffic(key):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture) recorded in
    profiles/traffic.txt under `key` (workload.variant.kernel.bytes_per_launch), or None when there is no such
    record or the kernel sources have changed since the counters were taken."""
    path = os.path.join(ROOT, "profiles", "traffic.txt")
    try:
        kv = dict(l.strip().split("=", 1) for l in open(path) if "=" in l and not l.startswith("#"))
        if kv.get("source_sha256") != kernel_source_hash():
            return None
        return int(kv[key])
    except Exception:
        return None


def config_dict(w, variant, rho, extra=None):
    """The `config` object of the JSON line; the same keys on both arms."""
    d = {"workload": f"config {w.index}: {w.name}", "variant": variant, "scales": list(w.scales),
         "steps_per_generation": len(w.steps), "layers": w.n_layers, "heads": w.n_heads,
         "batch": f"2x{w.batch_pairs}", "cfg_share": w.share_cfg,
         "window_rho": list(rho or w.rho) if variant == "window" else None}
    d["launch"] = d["l2"] = d["note"] = None
    if extra:
        d.update(extra)
    return d


# --------------------------------------------------------------------------------------- accounting
def schedule_counts(plan, w: wl.Workload):
    """Per step: live entries, executed tile pairs (from the plan), n_k, L_k."""
    out = {}
    for k in w.steps:
        st = plan.stats(k)
        out[k] = dict(live=st["live_entries"], tiles=st["live_tiles"], n_k=w.scales[k - 1] ** 2,
                      L_k=wl.cache_len(w.scales, k))
    return out


def per_layer_work(w: wl.Workload, counts, share: bool, steps=None):
    """Useful FLOP, executed FLOP and compulsory HBM bytes of one layer's calls (of the given steps)."""
    rows = 2 * w.batch_pairs
    computed = w.batch_pairs if share else rows
    useful = executed = nbytes = 0
    for k in (w.steps if steps is None else steps):
        c = counts[k]
        useful += c["live"] * FLOP_PER_ENTRY * computed * w.n_heads
        executed += c["tiles"] * TILE_FLOP * computed * w.n_heads
        row_b = wl.HEAD_DIM * 2
        nbytes += w.n_heads * (computed * (c["n_k"] + 2 * c["L_k"]) + rows * c["n_k"]) * row_b
    return useful, executed, nbytes


# --------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """nvidia-smi in a child process, one CSV line every 100 ms, for the GPU this rank uses."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.proc = None
        self.lines = []
        try:
            uuid = torch.cuda.get_device_properties(device_index).uuid
            ident = "GPU-" + str(uuid) if not str(uuid).startswith("GPU-") else str(uuid)
        except Exception:
            ident = str(device_index)
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", ident, "--query-gpu=timestamp," + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        self.lines = [l for l in out.splitlines() if l.strip()]
        self.proc = None

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
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
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        # "under load": the upper half of the samples (idle samples before the first launch drop out)
        hot = sorted(sm)[len(sm) // 2:]
        return {"sm_mhz": statistics.median(hot), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------------------- GPU arm
def device_randn_bf16(shape, seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return torch.randn(*shape, generator=g, dtype=torch.float32, device=device).to(torch.bfloat16)


class Buffers:
    """Device tensors of `n_sets` layers of one workload (seeded, generated on the device)."""

    def __init__(self, w: wl.Workload, n_sets: int, device, seed_offset: int = 0):
        rows = 2 * w.batch_pairs
        L = wl.cache_len(w.scales, max(w.steps))
        self.k, self.v, self.q, self.out = [], [], [], []
        for layer in range(n_sets):
            k = device_randn_bf16((rows, w.n_heads, L, wl.HEAD_DIM), wl.seed_for(w.index, layer, 0, 1) + seed_offset, device)
            if w.key_head_scale:
                k = (k.float() * wl.head_scales(w.n_heads).to(device).view(1, -1, 1, 1)).to(torch.bfloat16)
            self.k.append(k)
            self.v.append(device_randn_bf16((rows, w.n_heads, L, wl.HEAD_DIM), wl.seed_for(w.index, layer, 0, 2) + seed_offset,
                                            device))
            qs, outs = {}, {}
            for step in w.steps:
                n_k = w.scales[step - 1] ** 2
                qs[step] = device_randn_bf16((rows, w.n_heads, n_k, wl.HEAD_DIM),
                                             wl.seed_for(w.index, layer, step, 0) + seed_offset, device)
                outs[step] = torch.empty_like(qs[step])
            self.q.append(qs)
            self.out.append(outs)
        self.n_sets = n_sets

    def bytes(self):
        tot = 0
        for i in range(self.n_sets):
            tot += self.k[i].numel() * 2 + self.v[i].numel() * 2
            tot += sum(t.numel() * 4 for t in self.q[i].values())
        return tot


def sets_needed(w: wl.Workload, budget_bytes=3 << 30, min_bytes=400 << 20):
    """Distinct layer buffer sets: all layers when they fit the budget, else as many as the budget
    holds; at least enough that one pass over them exceeds the 126 MB L2 several times."""
    rows = 2 * w.batch_pairs
    L = wl.cache_len(w.scales, max(w.steps))
    nq = sum(w.scales[s - 1] ** 2 for s in w.steps)
    per = rows * w.n_heads * (2 * L + 2 * nq) * wl.HEAD_DIM * 2
    need = max(1, -(-min_bytes // per))
    n = max(need, min(w.n_layers, max(1, budget_bytes // per)))
    return int(n), per


def generation_calls(w: wl.Workload, n_sets: int, repeat_layers: int):
    """(step, buffer set) for every call of one generation, step-major as a model runs them."""
    return [(k, layer % n_sets) for k in w.steps for layer in range(repeat_layers)]


def run_generation(plan, w, bufs, calls, stream=None):
    for k, s in calls:
        plan.forward(k, w.batch_pairs, bufs.q[s][k], bufs.k[s], bufs.v[s], bufs.out[s][k], stream=stream)


def time_graph(plan, w, bufs, calls, steps, warmup, dist_barrier=None):
    """Capture one generation in a CUDA graph; time `steps` replays with CUDA events."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        run_generation(plan, w, bufs, calls)      # warm: function attributes, first-touch
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        run_generation(plan, w, bufs, calls)
    for _ in range(warmup):
        graph.replay()
    torch.cuda.synchronize()
    if dist_barrier:
        dist_barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    if dist_barrier:
        dist_barrier()
    return e0.elapsed_time(e1) / steps   # ms per generation


def time_eager(plan, w, bufs, calls, steps, warmup):
    for _ in range(warmup):
        run_generation(plan, w, bufs, calls)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        run_generation(plan, w, bufs, calls)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def time_e2e(plan, w: wl.Workload, steps, warmup, device):
    """Per-call API with host buffers.  Every call uploads one pinned block [Q | new K rows | new V rows] (only
    the batch rows the call computes) on an upload stream, appends the K/V rows to the device cache with one
    device copy, runs the forward (Q is read from the uploaded block) and sends the output back on a third
    stream, so that the uploads, the kernels and the downloads of neighbouring calls overlap (the link is
    full duplex).  Staging and output buffers alternate between two sets.  One layer's device cache is reused
    for every layer (the copies and the calls are the same)."""
    rows = 2 * w.batch_pairs
    share = w.share_cfg
    comp = w.batch_pairs if share else rows
    L = wl.cache_len(w.scales, max(w.steps))
    H, D = w.n_heads, wl.HEAD_DIM
    host_k, host_v = wl.make_kv(w, 0)
    off = [0]
    for s in w.scales:
        off.append(off[-1] + s * s)
    n_tok = {k: w.scales[k - 1] ** 2 for k in w.steps}
    host_in = {k: torch.stack([wl.make_q(w, 0, k)[:comp], host_k[:comp, :, off[k - 1]:off[k]],
                               host_v[:comp, :, off[k - 1]:off[k]]]).contiguous().pin_memory() for k in w.steps}
    host_out = {k: torch.empty((rows, H, n_tok[k], D), dtype=torch.bfloat16).pin_memory() for k in w.steps}
    dkv = torch.zeros((2, rows, H, L, D), dtype=torch.bfloat16, device=device)
    dk, dv = dkv[0], dkv[1]
    if min(w.steps) > 1:  # single-step workloads: the earlier scales are already cached on the device
        a = off[min(w.steps) - 1]
        dk[:, :, :a].copy_(host_k[:, :, :a])
        dv[:, :, :a].copy_(host_v[:, :, :a])
    stage = {k: [torch.empty((3, comp, H, n_tok[k], D), dtype=torch.bfloat16, device=device) for _ in range(2)]
             for k in w.steps}
    outs = {k: [torch.empty((rows, H, n_tok[k], D), dtype=torch.bfloat16, device=device) for _ in range(2)]
            for k in w.steps}
    h2d = d2h = 0
    for k in w.steps:
        h2d += w.n_layers * host_in[k].numel() * 2
        d2h += w.n_layers * host_out[k].numel() * 2
    main, back, up = torch.cuda.current_stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev = {k: [[torch.cuda.Event() for _ in range(3)] for _ in range(2)] for k in w.steps}  # uploaded, computed, downloaded

    def generation():
        used = {k: [False, False] for k in w.steps}
        for k in w.steps:
            a, b = off[k - 1], off[k]
            for layer in range(w.n_layers):
                i = layer & 1
                st, (uploaded, computed, downloaded) = stage[k][i], ev[k][i]
                if used[k][i]:
                    up.wait_event(computed)       # the staging block was read by the call two layers ago
                    main.wait_event(downloaded)   # and its output buffer has gone back to the host
                with torch.cuda.stream(up):
                    st.copy_(host_in[k], non_blocking=True)
                    uploaded.record(up)
                main.wait_event(uploaded)
                dkv[:, :comp, :, a:b].copy_(st[1:3])
                plan.forward(k, w.batch_pairs, st[0], dk, dv, outs[k][i])
                computed.record(main)
                back.wait_event(computed)
                with torch.cuda.stream(back):
                    host_out[k].copy_(outs[k][i], non_blocking=True)
                    downloaded.record(back)
                used[k][i] = True
        main.wait_stream(back)
        main.wait_stream(up)

    for _ in range(warmup):
        generation()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        generation()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps, h2d, d2h


def make_plan(w: wl.Workload, variant: str, rho=None):
    from paper_2411_17178_b200 import binding
    share = [1] * len(w.scales) if w.share_cfg else None
    if variant == "dense":
        K = len(w.scales)
        return binding.Plan(w.scales, n_heads=w.n_heads, radius=np.full((K, K), -1, np.int32), share_steps=share)
    return binding.Plan(w.scales, n_heads=w.n_heads, rho=rho or w.rho, share_steps=share)


def measure_config(w: wl.Workload, variant: str, rho, steps, warmup, device, pk, bufs=None):
    plan = make_plan(w, variant, rho)
    counts = schedule_counts(plan, w)
    useful, executed, nbytes = per_layer_work(w, counts, w.share_cfg)
    n_sets, per_set = sets_needed(w)
    if bufs is None:
        bufs = Buffers(w, n_sets, device)
    n_sets = bufs.n_sets
    repeat = max(w.n_layers, n_sets)           # single-call workloads rotate over the sets
    calls = generation_calls(w, n_sets, repeat)
    ms = time_graph(plan, w, bufs, calls, steps, warmup)
    assert plan.poll() == 0, "device-side wait timed out"
    scale = repeat / w.n_layers                # calls timed per generation's worth of calls
    us_gen = ms * 1e3 / scale
    tf = useful * w.n_layers / (us_gen * 1e-6) / 1e12
    res = dict(config=w.index, variant=variant if variant == "dense" else "rho %d/%d" % tuple(rho or w.rho),
               us_per_call=round(us_gen / (len(w.steps) * w.n_layers), 2), us_per_generation=round(us_gen, 1),
               useful_tflops=round(tf, 1),
               executed_tflops=round(executed * w.n_layers / (us_gen * 1e-6) / 1e12, 1),
               density=round(useful / executed, 3),
               useful_of_bf16_peak=round(tf / pk["bf16"], 4),
               hbm_gbs=round(nbytes * w.n_layers / (us_gen * 1e-6) / 1e9),
               hbm_frac=round(nbytes * w.n_layers / (us_gen * 1e-6) / 1e9 / pk["hbm"], 3))
    detail = dict(config=w.index, workload=w.name, variant=res["variant"],
                  calls_per_generation=len(w.steps) * w.n_layers, buffer_sets=n_sets, tiling="auto")
    if len(w.steps) > 1:
        # microseconds per call at every step: one graph of that step's calls over all layers
        per_step = {}
        for k in w.steps:
            ms_k = time_graph(plan, w, bufs, [(k, layer % n_sets) for layer in range(repeat)], max(2, steps // 2), 2)
            per_step[str(k)] = round(ms_k * 1e3 / repeat, 2)
        detail["us_per_call_by_step"] = per_step
        detail["kernel_by_step"] = {str(k): KERNEL_NAMES[plan.step_kernel(k, w.batch_pairs)] for k in w.steps}
    else:
        detail["kernel"] = KERNEL_NAMES[plan.step_kernel(w.steps[0], w.batch_pairs)]
    res = (res, detail)
    plan.close()
    return res, bufs


def measure_calibration(device, pk):
    """Window calibration (paper Section 2, steps (1)-(3)) on synthetic post-softmax maps: one pass over the
    maps, reported against the HBM roofline (bytes = the maps read once).  Not part of the timed step."""
    from paper_2411_17178_b200 import binding
    rows = []
    for name, scales, k, n_maps in (("256px step 10, 80 samples x 16 heads", wl.SCALES_256, 10, 1280),
                                    ("512px step 10, 64 maps", wl.SCALES_512, 10, 64),
                                    ("2K step 14, 1 map", wl.SCALES_2K, 14, 1)):
        n_k, L = scales[k - 1] ** 2, wl.cache_len(scales, k)
        g = torch.Generator(device=device)
        g.manual_seed(7)
        maps = torch.rand(n_maps, n_k, L, generator=g, device=device)
        maps /= maps.sum(-1, keepdim=True)
        for _ in range(3):
            rad = binding.calibrate_windows(scales, k, maps, 0.95)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(5):
            rad = binding.calibrate_windows(scales, k, maps, 0.95)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / 5
        nbytes = maps.numel() * 4
        rows.append({"workload": name, "map_bytes": nbytes, "ms_per_call": round(ms, 3),
                     "gbs": round(nbytes / ms / 1e6, 1), "hbm_frac": round(nbytes / ms / 1e6 / pk["hbm"], 4),
                     "radius_at_r0_0.95": [int(x) for x in rad]})
        del maps
        torch.cuda.empty_cache()
    return rows


def measure_qkv8(device, pk):
    """8-bit Q/K/V (paper Section 4).  (1) The row quantiser alone on a K cache of workload 3's shape against
    the HBM roofline (every row read once and written once).  (2) Workload 2's generation with the step's Q
    and appended K/V rows quantised in place before every attention call (one extra launch per call)."""
    from paper_2411_17178_b200 import binding
    w3 = wl.WORKLOADS[3]
    shape = (2 * w3.batch_pairs, w3.n_heads, wl.cache_len(w3.scales, 10), wl.HEAD_DIM)
    x = device_randn_bf16(shape, 77, device)
    y = torch.empty_like(x)
    for _ in range(3):
        binding.quantize_rows(x, 8, out=y)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(10):
        binding.quantize_rows(x, 8, out=y)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / 10
    nbytes = 2 * x.numel() * 2
    res = {"quantiser": {"tensor": list(shape), "bytes_read_plus_written": nbytes, "us_per_call": round(ms * 1e3, 2),
                         "gbs": round(nbytes / ms / 1e6, 1), "hbm_frac": round(nbytes / ms / 1e6 / pk["hbm"], 4)}}
    del x, y
    w = wl.WORKLOADS[2]
    plan = make_plan(w, "window")
    n_sets, _ = sets_needed(w)
    bufs = Buffers(w, n_sets, device)
    off = [0]
    for s_ in w.scales:
        off.append(off[-1] + s_ * s_)
    calls = generation_calls(w, n_sets, max(w.n_layers, n_sets))

    def generation():
        for k, s_ in calls:
            binding.quantize_qkv(bufs.q[s_][k], bufs.k[s_][:, :, off[k - 1]:off[k]], bufs.v[s_][:, :, off[k - 1]:off[k]])
            plan.forward(k, w.batch_pairs, bufs.q[s_][k], bufs.k[s_], bufs.v[s_], bufs.out[s_][k])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        generation()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        generation()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(20):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    res["workload2_generation_us_with_quantised_qkv"] = round(e0.elapsed_time(e1) / 20 * 1e3 * w.n_layers / max(w.n_layers, n_sets), 2)
    res["launches_per_generation"] = 2 * len(w.steps) * w.n_layers
    assert plan.poll() == 0
    plan.close()
    return res


def measure_kv8(device, pk, configs=(3, 4), reps=5, warm=3):
    """8-bit K/V cache read by the attention kernel itself (litevar_attn_forward_kv8, paper Section 4) against the
    bf16 cache, on the two workloads whose steps stream their cache from HBM (3 and 4, raster tiles): microseconds
    per generation's attention and cache bytes per layer."""
    from paper_2411_17178_b200 import binding
    out = []
    for idx in configs:
        w = wl.WORKLOADS[idx]
        n_sets = max(2, min(4, sets_needed(w)[0]))
        bufs = Buffers(w, n_sets, device)
        share = [1] * len(w.scales) if w.share_cfg else None
        plan = binding.Plan(w.scales, n_heads=w.n_heads, rho=w.rho, share_steps=share, tiling=binding.TILING_RASTER)
        k8 = [binding.quantize_rows(bufs.k[i], want_codes=True) for i in range(n_sets)]
        v8 = [binding.quantize_rows(bufs.v[i], want_codes=True) for i in range(n_sets)]
        repeat = max(w.n_layers, n_sets)
        calls = generation_calls(w, n_sets, repeat)

        def gen_bf16():
            for k, s_ in calls:
                plan.forward(k, w.batch_pairs, bufs.q[s_][k], k8[s_][0], v8[s_][0], bufs.out[s_][k])

        def gen_kv8():
            for k, s_ in calls:
                plan.forward_kv8(k, w.batch_pairs, bufs.q[s_][k], k8[s_][1], k8[s_][2], k8[s_][3], v8[s_][1], v8[s_][2],
                                 v8[s_][3], bufs.out[s_][k])
        res = {}
        for name, fn in (("bf16_cache_auto_kernels", gen_bf16), ("int8_cache", gen_kv8)):
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                fn()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                fn()
            for _ in range(warm):
                graph.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            res[name + "_us_per_generation"] = round(e0.elapsed_time(e1) / reps * 1e3 * w.n_layers / repeat, 1)
        assert plan.poll() == 0
        rows = 2 * w.batch_pairs * w.n_heads * wl.cache_len(w.scales, max(w.steps))
        res.update(config=idx, cache_bytes_per_layer_bf16=rows * 2 * 128, cache_bytes_per_layer_int8=rows * 2 * (64 + 8),
                   note="int8 path: small-step kernel on the small steps, two-threads-per-row tcgen05 kernel on the others, raster tiles; bf16 path: the kernels AUTO picks on the dequantised cache")
        out.append(res)
        plan.close()
        del bufs, k8, v8
        torch.cuda.empty_cache()
    return out


def gpu_arm(args):
    from paper_2411_17178_b200 import build as lvbuild
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the attention path has no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    barrier = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

        def barrier():
            dist.barrier()
            torch.cuda.synchronize()
    if rank == 0:
        lvbuild.build()
    if barrier:
        barrier()
    pk = peaks()
    if args.calibration:
        # the window calibration kernel alone (for profiler runs); one GPU
        if rank == 0:
            print(json.dumps({"calibration": measure_calibration(device, pk), "qkv8": measure_qkv8(device, pk),
                              "kv8_cache": measure_kv8(device, pk), "peaks": pk}), flush=True)
        if barrier:
            barrier()
            torch.distributed.destroy_process_group()
        return
    if args.kv8 is not None:
        # the 8-bit cache path against the bf16 path alone (for profiler runs); one GPU
        if rank == 0:
            print(json.dumps({"kv8_cache": measure_kv8(device, pk, tuple(args.kv8) or (3, 4), args.steps, args.warmup),
                              "peaks": pk}), flush=True)
        if barrier:
            barrier()
            torch.distributed.destroy_process_group()
        return
    w = wl.WORKLOADS[args.config]
    variant = "dense" if args.dense else "window"

    # ---- headline: K generations of the chosen workload, replicated on every rank (no collective:
    # (batch row, head) units are independent, each rank holds its own batch)
    plan = make_plan(w, variant, tuple(args.rho) if args.rho else None)
    counts = schedule_counts(plan, w)
    useful, executed, nbytes = per_layer_work(w, counts, w.share_cfg)
    n_sets, per_set = sets_needed(w)
    bufs = Buffers(w, n_sets, device, seed_offset=sharding.rank_seed(0, rank))
    repeat = max(w.n_layers, n_sets)
    calls = generation_calls(w, n_sets, repeat)
    scale = repeat / w.n_layers
    sampler = ClockSampler(local) if rank == 0 else None
    ms = time_graph(plan, w, bufs, calls, args.steps, args.warmup, barrier)
    if sampler:
        # keep the GPU in the same state a little longer so that short runs still collect samples
        t_end = time.time() + (0.0 if args.kernel_only else max(0.0, 1.0 - ms * args.steps / 1e3))
        while time.time() < t_end:
            run_generation(plan, w, bufs, calls)
            torch.cuda.synchronize()
        sampler.stop()
    status = plan.poll()
    # ---- end to end with host buffers, on every rank (the host links are shared by the ranks of a node)
    e2e_ms = h2d = d2h = None
    if not args.kernel_only:
        e2e_ms, h2d, d2h = time_e2e(plan, w, max(1, min(args.steps, 5)), 1, device)
    # the job is as slow as its slowest rank
    red = sharding.max_over_ranks([ms, e2e_ms if e2e_ms is not None else 0.0], device=device)
    ms = red[0]
    if e2e_ms is not None:
        e2e_ms = red[1]
    ms_step = ms / scale
    gen_useful = useful * w.n_layers
    value = sharding.whole_job_rate(gen_useful, world, ms_step) / 1e12
    launches_per_step = len(calls)
    if world > 1:
        import torch.distributed as dist
        barrier()
        dist.destroy_process_group()
    if rank != 0:
        return

    rho_used = tuple(args.rho) if args.rho else w.rho
    out = {
        "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_step, 5), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_dict(w, variant, rho_used, {
            "launch": "one CUDA graph replay per generation",
            "l2": f"inputs larger than L2: {bufs.bytes() / 1e6:.0f} MB over {bufs.n_sets} buffer sets visited in turn"}),
        "gpu_launches": launches_per_step * args.steps,
        "us_per_generation": round(ms_step * 1e3, 2),
        "us_per_image": round(ms_step * 1e3 / w.batch_pairs, 2),
        "cfg_effective_tflops": round(value * (2 if w.share_cfg else 1), 3),
        "executed_tflops": round(world * executed * w.n_layers / (ms_step * 1e-3) / 1e12, 3),
        "useful_frac_of_bf16_peak": round(value / world / pk["bf16"], 5),
        "device_status": status,
        "peaks": pk,
    }
    if sampler:
        out["clocks"] = sampler.summary()

    # ---- roofline of the dominant forward kernel on this workload.  AUTO may run several kernels (small steps /
    # short lists / long lists); each group of steps is replayed as its own graph and timed with CUDA events, the
    # kernel with the largest share of the generation is the one reported.
    def kernel_groups(pl, wk, bf, n_sets_, repeat_, scale_, cnts):
        groups = {}
        for k in wk.steps:
            groups.setdefault(KERNEL_NAMES[pl.step_kernel(k, wk.batch_pairs)], []).append(k)
        timed = {}
        for name, ks in groups.items():
            g_calls = [(k, layer % n_sets_) for k in ks for layer in range(repeat_)]
            g_ms = time_graph(pl, wk, bf, g_calls, max(3, args.steps // 2), 3) / scale_
            u, e, b = per_layer_work(wk, cnts, wk.share_cfg, ks)
            timed[name] = dict(steps=ks, launches=len(ks) * wk.n_layers, us=g_ms * 1e3, bytes=b * wk.n_layers,
                               useful=u * wk.n_layers, executed=e * wk.n_layers)
        return timed

    def hbm_block(timed, traffic_key):
        total_us = sum(t["us"] for t in timed.values())
        dom = max(timed, key=lambda n: timed[n]["us"])
        d = timed[dom]
        alg = d["bytes"] / d["launches"]
        sec = d["us"] * 1e-6 / d["launches"]
        return {"bound": "hbm", "achieved": round(alg / sec / 1e9, 1), "peak": pk["hbm"], "unit": "GB/s",
                "frac": round(alg / sec / 1e9 / pk["hbm"], 4),
                "traffic": recorded_traffic(f"{traffic_key}.{dom}.bytes_per_launch") if traffic_key else None,
                "kernel": dom, "peak_source": pk["source"], "steps": d["steps"],
                "launches_per_generation": d["launches"], "share_of_generation_time": round(d["us"] / total_us, 4),
                "algorithmic_bytes_per_launch": round(alg), "avg_launch_us": round(sec * 1e6, 3),
                "other_kernels": [
                    {"kernel": n, "steps": t["steps"], "launches_per_generation": t["launches"],
                     "avg_launch_us": round(t["us"] / t["launches"], 3),
                     "share_of_generation_time": round(t["us"] / total_us, 4),
                     "hbm_frac": round(t["bytes"] / (t["us"] * 1e-6) / 1e9 / pk["hbm"], 4)}
                    for n, t in timed.items() if n != dom]}

    def tensor_block(timed, traffic_key):
        total_us = sum(t["us"] for t in timed.values())
        dom = max(timed, key=lambda n: timed[n]["us"])
        d = timed[dom]
        sec = d["us"] * 1e-6 / d["launches"]
        useful_l, exec_l = d["useful"] / d["launches"], d["executed"] / d["launches"]
        return {"bound": "tensor", "achieved": round(useful_l / sec / 1e12, 2), "peak": pk["bf16"], "unit": "TFLOP/s",
                "frac": round(useful_l / sec / 1e12 / pk["bf16"], 4),
                "traffic": recorded_traffic(f"{traffic_key}.{dom}.bytes_per_launch") if traffic_key else None,
                "kernel": dom, "peak_source": pk["source"] + " (burst; a launch is timed alone)",
                "useful_flop_per_launch": round(useful_l), "executed_flop_per_launch": round(exec_l),
                "achieved_executed": round(exec_l / sec / 1e12, 2),
                "frac_executed": round(exec_l / sec / 1e12 / pk["bf16"], 4),
                "frac_of_sustained_peak": round(useful_l / sec / 1e12 / pk["bf16_sustained"], 4),
                "algorithmic_bytes_per_launch": round(d["bytes"] / d["launches"]),
                "hbm_frac_compulsory": round(d["bytes"] / d["launches"] / sec / 1e9 / pk["hbm"], 4),
                "avg_launch_us": round(sec * 1e6, 3), "steps": d["steps"],
                "launches_per_generation": d["launches"], "share_of_generation_time": round(d["us"] / total_us, 4),
                "other_kernels": [
                    {"kernel": n, "steps": t["steps"], "launches_per_generation": t["launches"],
                     "avg_launch_us": round(t["us"] / t["launches"], 3),
                     "share_of_generation_time": round(t["us"] / total_us, 4)} for n, t in timed.items() if n != dom]}

    timed = kernel_groups(plan, w, bufs, n_sets, repeat, scale, counts)
    default_run = variant == "window" and not args.rho
    tkey = f"workload{w.index}.{'dense' if variant == 'dense' else 'window'}" if (default_run or variant == "dense") else None
    out["roofline"] = tensor_block(timed, tkey) if w.index in (4, 5) else hbm_block(timed, tkey)

    if args.kernel_only:
        plan.close()
        print(json.dumps(out), flush=True)
        return

    # ---- eager per-call figure (ctypes call + tensor-map encoding per launch on the host)
    eager_ms = time_eager(plan, w, bufs, calls, max(2, min(args.steps, 10)), 1) / scale
    out["eager_us_per_generation"] = round(eager_ms * 1e3, 2)

    out["e2e"] = {"value": round(sharding.whole_job_rate(gen_useful, world, e2e_ms) / 1e12, 4), "unit": UNIT,
                  "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_ms, 4)}
    plan.close()
    del bufs
    torch.cuda.empty_cache()

    # ---- CPU oracle baseline (rank 0, N = 1 only)
    if world == 1 and not args.no_cpu:
        out["cpu_baseline"] = oracle_baseline(w, args.cpu_seconds)

    # ---- the five workloads, window and dense variants; the HBM roofline of the 256px generation; plan times
    detail = []
    if world == 1 and not args.no_extras:
        table = []
        reps, warm = 5, 3
        for idx in (1, 2, 3, 4, 5):
            wi = wl.WORKLOADS[idx]
            shared_bufs = None
            variants = [("window", r) for r in (wi.rho_sweep or (wi.rho,))] + [("dense", None)]
            for var, rho in variants:
                (row, det), shared_bufs = measure_config(wi, var, rho, reps, warm, device, pk, shared_bufs)
                table.append(row)
                detail.append(det)
            if idx == 2 and w.index != 2:
                p2 = make_plan(wi, "window")
                n2 = shared_bufs.n_sets
                rep2 = max(wi.n_layers, n2)
                out["roofline_hbm_workload2"] = hbm_block(
                    kernel_groups(p2, wi, shared_bufs, n2, rep2, rep2 / wi.n_layers, schedule_counts(p2, wi)),
                    "workload2.window")
                p2.close()
            del shared_bufs
            torch.cuda.empty_cache()
        out["all_configs"] = table
        out["plan_us"] = measure_plan_times()
        out["calibration"] = measure_calibration(device, pk)
        out["qkv8"] = measure_qkv8(device, pk)
        out["kv8_cache"] = measure_kv8(device, pk)
        out["all_configs_detail"] = detail
    # the short table goes out early in the line and the long per-step records last
    order = ["metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
             "vs_baseline", "dtype", "data", "config", "gpu_launches", "clocks", "roofline", "e2e", "cpu_baseline",
             "all_configs"]
    line = {k: out[k] for k in order if k in out}
    line.update({k: v for k, v in out.items() if k not in line})
    print(json.dumps(line), flush=True)


def measure_plan_times():
    """Microseconds per litevar_attn_plan call (window table, bounds, classification, compaction, element masks
    and launch order of every step on the device, one synchronisation at the end), best of three."""
    res = {}
    for name, scales, heads in (("256px", wl.SCALES_256, 16), ("512px", wl.SCALES_512, 36), ("2K", wl.SCALES_2K, 16)):
        from paper_2411_17178_b200 import binding
        best = None
        for _ in range(3):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            pl = binding.Plan(scales, n_heads=heads)
            t1 = time.perf_counter()
            pl.close()
            best = t1 - t0 if best is None else min(best, t1 - t0)
        res[name] = round(best * 1e6, 1)
    return res


# --------------------------------------------------------------------------------------- CPU arm
def oracle_sample(w: wl.Workload, seconds: float):
    """Run the oracle, as it stands, over layers of the workload until `seconds` have passed.
    Returns (useful FLOP done, elapsed s, description)."""
    from oracle import litevar_oracle as orc
    tab = orc.window_table(w.scales, rho=w.rho)
    rows = 2 * w.batch_pairs
    done_flop = 0.0
    t0 = time.perf_counter()
    what = []
    if w.index in (1, 2, 3, 4):
        sample_rows = min(rows, 4)           # batch 2x2 of each layer keeps one layer to about a second
        comp = sample_rows // 2 if w.share_cfg else sample_rows
        layer = 0
        while True:
            Kc, Vc = wl.make_kv(w, layer, batch_rows=sample_rows)
            t_gen = time.perf_counter()
            for k in w.steps:
                Q = wl.make_q(w, layer, k, batch_rows=sample_rows)
                orc.attention_step(w.scales, k, tab[k - 1], Q, Kc, Vc, share_cfg=w.share_cfg)
                done_flop += orc.live_count(w.scales, k, tab[k - 1]) * FLOP_PER_ENTRY * comp * w.n_heads
            layer += 1
            _ = t_gen
            if time.perf_counter() - t0 > seconds or layer >= w.n_layers:
                break
        what = f"{layer} layer(s) x all {len(w.steps)} steps, batch 2x{sample_rows // 2}, every row (input generation included)"
    else:
        k = w.steps[-1]
        Kc, Vc = wl.make_kv(w, 0)
        Q = wl.make_q(w, 0, k)
        n_k = w.scales[k - 1] ** 2
        rng = np.random.default_rng(0)
        n = 0
        m = orc.mask(w.scales, k, tab[k - 1], q_rows=range(0, n_k, 64))
        mean_live = float(m.sum(1).mean())
        while time.perf_counter() - t0 < seconds:
            smp = [(int(rng.integers(0, rows)), int(rng.integers(0, w.n_heads)), int(rng.integers(0, n_k)))
                   for _ in range(64)]
            orc.attention_sampled(w.scales, k, tab[k - 1], Q, Kc, Vc, smp)
            n += 64
        done_flop = n * mean_live * FLOP_PER_ENTRY
        what = f"{n} sampled query rows of step {k}"
    return done_flop, time.perf_counter() - t0, what


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return int(torch.get_num_threads())


def oracle_baseline(w: wl.Workload, seconds: float):
    flop, el, what = oracle_sample(w, seconds)
    return {"value": round(flop / el / 1e12, 6), "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
            "sample": what, "seconds": round(el, 2), "host_cpus": os.cpu_count()}


def reference_arm(args):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return
    w = wl.WORKLOADS[args.config]
    per_step = max(0.5, min(20.0, args.cpu_seconds / max(1, args.steps)))
    for _ in range(min(args.warmup, 1)):
        oracle_sample(w, min(per_step, 1.0))
    flop_tot, el_tot, what = 0.0, 0.0, ""
    for _ in range(args.steps):
        flop, el, what = oracle_sample(w, per_step)
        flop_tot += flop
        el_tot += el
    value = flop_tot / el_tot / 1e12
    out = {
        "impl": "reference", "metric": METRIC, "value": round(value, 6), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(el_tot / args.steps * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(w, "window", w.rho, {"note": "each step is a bounded sample of the workload run by the CPU oracle"}),
        "gpu_launches": 0,
        "cpu_baseline": {"value": round(value, 6), "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                         "sample": f"per step: {what}"},
        "e2e": {"value": round(value, 6), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=5, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--dense", action="store_true", help="full-mask variant of the same kernel")
    ap.add_argument("--no-extras", action="store_true", help="skip the five-workload table")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--kernel-only", action="store_true",
                    help="only the device-timed graph replays (for profiler runs): no eager, end-to-end, "
                         "CPU or all-workload legs")
    ap.add_argument("--calibration", action="store_true", help="only the figures of the window calibration and row quantiser kernels")
    ap.add_argument("--kv8", type=int, nargs="*", default=None, choices=[3, 4],
                    help="only the 8-bit K/V cache path against the bf16 path, on the given workloads (default 3 4)")
    ap.add_argument("--rho", type=int, nargs=2, default=None, help="window radius ratio num den (default: the workload's)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        reference_arm(args)
    else:
        gpu_arm(args)


if __name__ == "__main__":
    main()
