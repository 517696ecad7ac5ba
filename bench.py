#!/usr/bin/env python
"""Benchmark of the CateKV hot path on B200.

    python bench.py --gpus N --steps K --warmup W [--workload cfg3] [--impl reference]

A "step" is one decode step of the whole model on one batch: for every layer,
catekv_append of the token's K/V followed by catekv_decode_attn over the hybrid
per-head caches.  The caches are produced, before the timed region, by the
library's own prefill-end path (catekv_select_compact over seeded synthetic
prefill K/V, one layer at a time), which is timed and reported separately, as
is catekv_head_cv.  `value` is decode throughput in tokens/s (batch tokens per
step / step time) with everything resident in HBM; `e2e` repeats the
measurement with the step's q / k_new / v_new coming from pinned host memory
and the outputs copied back, inside the timed region.

One JSON line is printed by rank 0.  With --gpus N > 1 (under torchrun) every
rank runs an independent replica of the workload (the path has no exchange
step); the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "hybrid decode attention throughput (tokens/s = batch / (layers x layer-step time))"
UNIT = "tokens/s"
ROW_BYTES = 512  # one kept token of one KV head: 256 B of K + 256 B of V


def max_over_ranks(x: float, device=None) -> float:
    """Maximum of a per-rank time over all ranks of the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return x
    t = torch.tensor([x], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


class ClockSampler:
    """nvidia-smi sampling in the background; started before and stopped after a timed region."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file.read().splitlines():
            f = [x.strip() for x in line.split(",")]
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
        self.file.close()
        try:
            os.unlink(self.file.name)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons),
                       samples=len(sm))
        return out


# ------------------------------------------------------------------------------------------
# building the model's caches through the library's prefill-end path
# ------------------------------------------------------------------------------------------
def expected_lengths(w, mask):
    from workloads import synth  # noqa: F401
    lens = []
    for b in range(w.B):
        for h in range(w.Hkv):
            if mask[b, h]:
                T = w.budget
            else:
                T = w.n if w.eta >= 1.0 else int(math.floor(float(np.float32(w.eta)) * w.n))
            lens.append(w.n if (T >= w.n or w.sink + w.local >= w.n) else max(T, w.sink + w.local))
    return lens


PLAN_HOST_US = []  # host time of every catekv_decode_plan call of build_model


def build_model(ck, w, dev, max_new, layers=None, time_select=True):
    """Caches and plans of `layers` layers via catekv_select_compact.  Returns (layer list, select ms/layer)."""
    import torch
    from workloads import synth
    n_layers = w.layers if layers is None else layers
    num_ctas = ck.catekv_decode_num_ctas()
    out, sel_ms = [], []
    ws = torch.empty(ck.catekv_select_workspace_bytes(w.B, w.Hq, w.Hkv, w.n, w.L_obs), dtype=torch.uint8, device=dev)
    for l in range(n_layers):
        p = synth.prefill_layer(w, l, dev)
        mask = p["head_mask"]
        cache = ck.Cache(w.B, w.Hkv, expected_lengths(w, mask), max_new, dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        ck.catekv_select_compact(p["q_win"], p["k"], p["v"], p["seq_len"], mask, cache, w.budget, w.eta, w.sink,
                                 w.local, w.pool_mode, w.pool_param, ws=ws)
        e1.record()
        torch.cuda.synchronize()
        sel_ms.append(e0.elapsed_time(e1))
        if cache.struct.reserved:  # chunk mode, short last chunk: the fused append needs the exact lengths
            ck.catekv_cache_sync_lengths(cache)
        ck.catekv_workspace_status(ws)  # raises if a scoring wait ran out
        plan = ck.DecodePlan(cache, num_ctas)
        t0 = time.perf_counter()
        ck.catekv_decode_plan(cache, plan)  # host: the schedule, plus one asynchronous copy to the device
        PLAN_HOST_US.append((time.perf_counter() - t0) * 1e6)
        out.append({"cache": cache, "plan": plan, "mask": mask})
        del p
    torch.cuda.synchronize()
    return out, sel_ms


def make_step_inputs(w, n_layers, dev, n_sets=2):
    """A few sets of per-step inputs for all layers: q [L,B,Hq,d], k_new, v_new [L,B,Hkv,d]."""
    import torch
    from workloads import synth
    sets = []
    for s in range(n_sets):
        q = synth.randn_bf16((n_layers, w.B, w.Hq, w.d), dev, w.seed, "bench_q", s)
        kn = synth.randn_bf16((n_layers, w.B, w.Hkv, w.d), dev, w.seed, "bench_kn", s)
        vn = synth.randn_bf16((n_layers, w.B, w.Hkv, w.d), dev, w.seed, "bench_vn", s)
        sets.append((q, kn, vn))
    return sets


FUSED = True  # per layer: catekv_append_decode_attn (one attention launch) instead of catekv_append + catekv_decode_attn


def decode_step(ck, model, q, kn, vn, out):
    for l, m in enumerate(model):
        if FUSED:
            ck.catekv_append_decode_attn(m["cache"], kn[l], vn[l], q[l], m["plan"], out[l])
        else:
            ck.catekv_append(m["cache"], kn[l], vn[l])
            ck.catekv_decode_attn(m["cache"], q[l], m["plan"], out[l])


def capture_step(ck, model, q, kn, vn, out):
    """One decode step of the whole model as a CUDA graph.  Capturing runs the library's host code (which
    advances the host length mirrors) but not the kernels, so the graph is replayed once right away; every
    later replay is preceded by catekv_cache_advance."""
    import torch
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            decode_step(ck, model, q, kn, vn, out)
    torch.cuda.current_stream().wait_stream(s)
    g.replay()
    return g


def replay_step(ck, model, g):
    for m in model:
        ck.catekv_cache_advance(m["cache"], 1)
    g.replay()


def kept_bytes(model):
    return [int(m["cache"].seg_len.sum()) * ROW_BYTES for m in model]


def time_decode(ck, w, model, dev, steps, warmup, barrier=None, graph=True):
    """Device-resident timing: returns ms per step (CUDA events on the launching stream).  With `graph` the
    step's launches are captured once per input set and replayed."""
    import torch
    L = len(model)
    sets = make_step_inputs(w, L, dev)
    out = torch.empty((L, w.B, w.Hq, w.d), dtype=torch.bfloat16, device=dev)
    decode_step(ck, model, *sets[0], out)  # first launch of every kernel happens outside any capture
    torch.cuda.synchronize()
    graphs = [capture_step(ck, model, *st, out) for st in sets] if graph else None

    def step(i):
        if graph:
            replay_step(ck, model, graphs[i % len(graphs)])
        else:
            decode_step(ck, model, *sets[i % len(sets)], out)

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    if barrier:
        barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        step(i)
    e1.record()
    torch.cuda.synchronize()
    if barrier:
        barrier()
    return e0.elapsed_time(e1) / steps


APPEND_US = None  # mean duration of the separate append launch, set by time_kernels

# DRAM bytes per algorithmic byte of decode_partial_kernel: dram__bytes_read.sum over 512 B x kept rows, from the
# ncu capture of the two-layer configs[2] case (profiles/decode_partial_kernel_cfg2_2layers.md); traffic grows in
# proportion to the kept rows (every row crosses DRAM once), so the ratio is applied to each run's own bytes.
TRAFFIC_READ_RATIO = 1.0002
TRAFFIC_WRITE_BYTES = 4.6e6  # per launch in that capture (partials, outputs); does not grow with the rows


def _graph_of(fn):
    """Capture fn() (library calls on the current stream) into a CUDA graph."""
    import torch
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            fn()
    torch.cuda.current_stream().wait_stream(side)
    return g


def _time_graph(g, reps, before=None):
    import torch
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        if before:
            before()
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / reps  # us per replay


def time_kernels(ck, w, model, dev, steps):
    """Average duration of the attention-partials launch in the launch regime of the timed step: a CUDA graph of
    catekv_decode_partials over all layers (the same programmatic-launch chain, without the combine launches),
    replayed `steps` times, CUDA events around the replays, divided by the number of launches.  Also: the same
    for the combine launches and for the separate append launch.  Returns (partials us, combine us)."""
    import torch
    L = len(model)
    q, kn, vn = make_step_inputs(w, L, dev, n_sets=1)[0]
    out = torch.empty((L, w.B, w.Hq, w.d), dtype=torch.bfloat16, device=dev)
    g_part = _graph_of(lambda: [ck.catekv_decode_partials(m["cache"], q[l], m["plan"], out[l]) for l, m in enumerate(model)])
    part = _time_graph(g_part, steps) / L
    g_comb = _graph_of(lambda: [ck.catekv_decode_combine(m["cache"], q[l], m["plan"], out[l]) for l, m in enumerate(model)])
    comb = _time_graph(g_comb, steps) / L
    global APPEND_US
    g_app = _graph_of(lambda: [ck.catekv_append(m["cache"], kn[l], vn[l]) for l, m in enumerate(model)])
    reps = 3
    for m in model:  # the capture advanced the host mirrors by one row; the replays below add reps + 1 rows
        ck.catekv_cache_advance(m["cache"], reps)
    APPEND_US = _time_graph(g_app, reps) / L
    return part, comb


def time_e2e(ck, w, model, dev, steps, warmup, barrier=None, graph=True):
    """Same step through the public API with host buffers: H2D of q/k_new/v_new and D2H of the outputs inside
    the timed region."""
    import torch
    L = len(model)
    host_sets = []
    for q, kn, vn in make_step_inputs(w, L, "cpu"):
        host_sets.append((q.pin_memory(), kn.pin_memory(), vn.pin_memory()))
    dq = torch.empty((L, w.B, w.Hq, w.d), dtype=torch.bfloat16, device=dev)
    dk = torch.empty((L, w.B, w.Hkv, w.d), dtype=torch.bfloat16, device=dev)
    dv = torch.empty_like(dk)
    out = torch.empty_like(dq)
    hout = torch.empty((L, w.B, w.Hq, w.d), dtype=torch.bfloat16).pin_memory()

    decode_step(ck, model, dq, dk, dv, out)
    torch.cuda.synchronize()
    g = capture_step(ck, model, dq, dk, dv, out) if graph else None

    def step(i):
        q, kn, vn = host_sets[i % len(host_sets)]
        dq.copy_(q, non_blocking=True)
        dk.copy_(kn, non_blocking=True)
        dv.copy_(vn, non_blocking=True)
        if graph:
            replay_step(ck, model, g)
        else:
            decode_step(ck, model, dq, dk, dv, out)
        hout.copy_(out, non_blocking=True)
        torch.cuda.current_stream().synchronize()  # the caller needs the outputs before the next token

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    if barrier:
        barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        step(i)
    e1.record()
    torch.cuda.synchronize()
    if barrier:
        barrier()
    h2d = sum(t.numel() * t.element_size() for t in host_sets[0])
    d2h = hout.numel() * hout.element_size()
    return e0.elapsed_time(e1) / steps, h2d, d2h


def time_head_cv(ck, dev):
    """catekv_head_cv on configs[4]'s calibration shape: 8 prompts x 16K tokens, one layer (4 KV heads, G = 7)."""
    import torch
    from workloads import synth
    w = synth.WORKLOADS["cfg4"]
    n = 16384
    qs, ks = [], []
    types = np.array([1, 0, 1, 0], dtype=np.uint8)
    for pr in range(8):
        q, k = synth.calibration_prompt(w, 0, pr, n, types, dev)
        qs.append(q), ks.append(k)
    q, k = torch.cat(qs), torch.cat(ks)
    seq = [n] * 8
    ws = torch.empty(ck.catekv_head_cv_workspace_bytes(8, w.Hq, w.Hkv, n, w.L_obs, 128, 32), dtype=torch.uint8,
                     device=dev)
    for _ in range(2):
        ck.catekv_head_cv(q, k, seq, 128, 32, 0.99, 1.0, True, ws=ws)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(3):
        ck.catekv_head_cv(q, k, seq, 128, 32, 0.99, 1.0, True, ws=ws)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / 3


def select_block(w, ms, n_layers, kept_bytes, peaks):
    """catekv_select_compact per layer against what bounds it: the bytes it has to move (K twice, for the two scoring
    passes, and the kept K/V rows in and out of the gather) at the measured copy bandwidth, and its exponentials (two
    per logit) at the special-function pipe's 16 per clock per SM and the maximum SM clock."""
    import torch
    k_bytes = w.B * w.Hkv * w.n * w.d * 2
    hbm_us = (2 * k_bytes + 2 * kept_bytes) / (peaks["hbm_gbs"] * 1e3)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    exps = 2.0 * w.B * w.Hq * w.L_obs * w.n
    sfu_us = exps / (sms * 16 * 1965.0)  # 1965 MHz: clocks.max.sm
    gather_us = 2 * kept_bytes / (peaks["hbm_gbs"] * 1e3)
    bound_us = max(hbm_us, sfu_us + gather_us)
    return {"ms_per_layer": ms, "layers": n_layers, "hbm_bound_us": hbm_us, "sfu_plus_gather_bound_us": sfu_us + gather_us,
            "frac_of_bound": bound_us / (ms * 1e3)}


def time_window_attn(ck, w, dev, layer=0, reps=5):
    """catekv_window_attn on the workload's prefill shape (one layer), and catekv_select_compact with and without the
    normaliser it delivers.  Returns a dict of milliseconds and the bytes / flops the attention call has to move."""
    import torch
    from workloads import synth
    p = synth.prefill_layer(w, layer, dev)
    mask = p["head_mask"]
    ws = torch.empty(ck._lib.catekv_window_attn_workspace_bytes(w.B, w.Hq, w.Hkv, w.n, w.L_obs), dtype=torch.uint8, device=dev)
    sws = torch.empty(ck.catekv_select_workspace_bytes(w.B, w.Hq, w.Hkv, w.n, w.L_obs), dtype=torch.uint8, device=dev)
    cache = ck.Cache(w.B, w.Hkv, expected_lengths(w, mask), 8, dev)

    def timed(fn):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    res = {}
    lse_sc = [None]

    def wa():
        lse_sc[0] = ck.catekv_window_attn(p["q_win"], p["k"], p["v"], p["seq_len"], out_dtype=torch.bfloat16, ws=ws)[2]
    res["window_attn_ms"] = timed(wa)
    sel = lambda lse: ck.catekv_select_compact(p["q_win"], p["k"], p["v"], p["seq_len"], mask, cache, w.budget, w.eta, w.sink,
                                               w.local, w.pool_mode, w.pool_param, ws=sws, row_lse_scored=lse)
    res["select_ms"] = timed(lambda: sel(None))
    res["select_with_normaliser_ms"] = timed(lambda: sel(lse_sc[0]))
    kv_bytes = w.B * w.Hkv * w.n * 256
    res["k_bytes"] = kv_bytes
    res["hbm_bytes_window_attn"] = 2 * kv_bytes * ((w.G * w.L_obs + 127) // 128)  # K and V once per 128-row tile of the window
    res["flops_window_attn"] = 2.0 * w.B * w.Hq * w.L_obs * w.n * w.d * 3  # Q K^T, P_hi V, P_lo V
    return res


def time_retrieval(ck, w, dev, n_layers=4, budget=1024, cs=8, steps=8, graph=True, gather=False):
    """Decode step with query-aware retrieval on the adaptive heads (budget rows per adaptive head, chunk size 8):
    per layer catekv_append_retrieval + catekv_retrieve_select + catekv_decode_attn_indexed
    (attention in place through the index lists), replayed as a CUDA graph of the step (graph=False: host
    launches).  gather=True: catekv_retrieve_compact into a per-step cache + catekv_decode_attn instead.
    Returns (us per layer-step, attended bytes per layer-step, metadata bytes per layer-step)."""
    import torch
    from workloads import synth
    model, _ = build_model(ck, w, dev, max_new=steps + 16, layers=n_layers)
    num_ctas = ck.catekv_decode_num_ctas()
    q = synth.randn_bf16((n_layers, w.B, w.Hq, w.d), dev, w.seed, "ret_q")
    kn = synth.randn_bf16((n_layers, w.B, w.Hkv, w.d), dev, w.seed, "ret_kn")
    vn = synth.randn_bf16((n_layers, w.B, w.Hkv, w.d), dev, w.seed, "ret_vn")
    out = torch.empty((w.B, w.Hq, w.d), dtype=torch.bfloat16, device=dev)
    for l, m in enumerate(model):
        c = m["cache"]
        m["meta"] = ck.catekv_retrieval_meta(c, cs)
        ck.catekv_retrieval_build(c, cs, m["meta"])
        m["rmask"] = (m["mask"].reshape(-1) == 0).astype(np.uint8)
        m["ws"] = ck.retrieve_workspace(c)
        m["lens"] = ck.catekv_retrieve_lengths(c, cs, m["rmask"], budget, w.sink, w.local)
        if gather:
            slens = [min(int(L), budget + 2 * cs + w.local) if m["rmask"][i] else int(L) + steps + 16
                     for i, L in enumerate(c.seg_len)]
            m["step"] = ck.Cache(w.B, w.Hkv, slens, 0, dev)
            ck.catekv_retrieve_compact(c, m["meta"], cs, q[l], m["rmask"], budget, w.sink, w.local, m["step"],
                                       ws=m["ws"])
            m["splan"] = ck.DecodePlan(m["step"], num_ctas)
            ck.catekv_decode_plan(m["step"], m["splan"])
        else:
            m["idx"] = torch.zeros((w.B * w.Hkv, budget + 2 * cs + w.local), dtype=torch.int32, device=dev)
            m["sel"] = torch.zeros(w.B * w.Hkv, dtype=torch.int32, device=dev)
            m["view"] = ck.CacheView(c, m["lens"])
            m["splan"] = ck.DecodePlan(m["view"], num_ctas)
            ck.catekv_decode_plan(m["view"], m["splan"])

    def step():
        for l, m in enumerate(model):
            ck.catekv_append_retrieval(m["cache"], kn[l], vn[l], cs, m["meta"])
            if gather:
                ck.catekv_retrieve_compact(m["cache"], m["meta"], cs, q[l], m["rmask"], budget, w.sink, w.local,
                                           m["step"], ws=m["ws"])
                ck.catekv_decode_attn(m["step"], q[l], m["splan"], out)
            else:
                ck.catekv_retrieve_select(m["cache"], m["meta"], cs, q[l], m["rmask"], budget, w.sink, w.local,
                                          m["idx"], m["sel"], ws=m["ws"])
                ck.catekv_decode_attn_indexed(m["cache"], m["idx"], m["sel"], q[l], m["splan"], out)

    run = step
    if graph:
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                step()  # runs the host code (the length mirrors advance), launches nothing
        torch.cuda.current_stream().wait_stream(side)
        g.replay()

        def run():
            for m in model:
                ck.catekv_cache_advance(m["cache"], 1)
            g.replay()
    for _ in range(3):
        run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        run()
    e1.record()
    torch.cuda.synchronize()
    attended = float(np.mean([int(m["lens"].sum()) * ROW_BYTES for m in model]))
    meta_bytes = float(np.mean([int(m["cache"].seg_len[m["rmask"] == 1].sum()) // cs * 512 for m in model]))
    return e0.elapsed_time(e1) * 1e3 / (steps * n_layers), attended, meta_bytes


def time_linearity(ck, dev, B=8, Hkv=8, G=4, n=32768, budget=1024, n_layers=2, reps=6):
    """The paper's qualitative efficiency claims on this kernel: decode time grows linearly with the share of
    adaptive heads r (Section 4.4.1) and with their retained fraction eta (Section 4.4.2), and the consistent
    heads' budget hardly matters (Section 4.4.3).  Synthetic pools (random rows, no selection), CUDA-graph replay
    of the fused step.  Returns the sweeps with the R^2 of a straight-line fit."""
    import torch
    num_ctas = ck.catekv_decode_num_ctas()
    n_segs = B * Hkv
    q = torch.randn((B, Hkv * G, 128), device=dev).bfloat16()
    kn = torch.randn((B, Hkv, 128), device=dev).bfloat16()
    out = torch.empty((B, Hkv * G, 128), device=dev, dtype=torch.bfloat16)

    def measure(r, eta, b):
        n_ad = int(round(r * n_segs))
        lens = np.full(n_segs, b, dtype=np.int32)
        lens[np.linspace(0, n_segs - 1, n_ad).astype(int)] = int(eta * n)
        model = []
        for _ in range(n_layers):
            c = ck.Cache(B, Hkv, lens, reps + 8, dev)
            c.k_pool.normal_()
            c.v_pool.normal_()
            c.set_lengths(lens)
            p = ck.DecodePlan(c, num_ctas)
            ck.catekv_decode_plan(c, p)
            model.append((c, p))
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for c, p in model:
                    ck.catekv_append_decode_attn(c, kn, kn, q, p, out)
        torch.cuda.current_stream().wait_stream(side)
        g.replay()

        def rep():
            for c, _ in model:
                ck.catekv_cache_advance(c, 1)
            g.replay()
        rep()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            rep()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / (reps * n_layers)

    def fit(x, y):
        x, y = np.asarray(x, dtype=np.float64), np.asarray(y, dtype=np.float64)
        a, b0 = np.polyfit(x, y, 1)
        ss = float(((y - (a * x + b0)) ** 2).sum())
        return 1.0 - ss / float(((y - y.mean()) ** 2).sum())

    rs = [0.125, 0.25, 0.5, 0.75, 1.0]
    t_r = [measure(r, 1.0, budget) for r in rs]
    etas = [0.25, 0.5, 0.75, 1.0]
    t_e = [measure(0.5, e, budget) for e in etas]
    budgets = [512, 1024, 2048]
    t_b = [measure(0.5, 1.0, b) for b in budgets]
    return {"shape": f"B {B}, {Hkv} KV heads, G {G}, context {n}",
            "adaptive_share_r": rs, "us_per_layer_step_vs_r": t_r, "r2_vs_r": fit(rs, t_r),
            "eta": etas, "us_per_layer_step_vs_eta": t_e, "r2_vs_eta": fit(etas, t_e),
            "consistent_budget": budgets, "us_per_layer_step_vs_budget": t_b}


# ------------------------------------------------------------------------------------------
# the oracle, timed as it stands, on a bounded sample
# ------------------------------------------------------------------------------------------
def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return int(max(n)) if n else 1
    except Exception:
        return 1


def oracle_sample_rate(w, target_s=15.0, seed_rows=200_000):
    """Times oracle.decode_attention on synthetic segments; returns (rows per second, sample description,
    seconds spent).  The sample grows until about target_s seconds of CPU work have been done."""
    from oracle import catekv_oracle as orc
    from workloads import synth
    G = w.G
    rows_done, t_done = 0, 0.0
    seg_rows = min(w.n, 65536)
    i = 0
    while True:
        oc = orc.HybridCache(1, 1, w.d)
        oc.k_rows.append(synth.bits(synth.randn_bf16((seg_rows, w.d), "cpu", w.seed, "ok", i)))
        oc.v_rows.append(synth.bits(synth.randn_bf16((seg_rows, w.d), "cpu", w.seed, "ov", i)))
        q = synth.bits(synth.randn_bf16((1, G, w.d), "cpu", w.seed, "oq", i))
        t0 = time.perf_counter()
        orc.decode_attention(oc, q)
        t_done += time.perf_counter() - t0
        rows_done += seg_rows
        i += 1
        if t_done >= target_s or i >= 400:
            break
    desc = f"{i} segments of {seg_rows} rows x {G} query heads (one KV head each), oracle.decode_attention"
    return rows_done / t_done, desc, t_done


def oracle_extra_timings(w):
    """The oracle at one thread (a 3 s sample of decode_attention) and one KV head's prefill-end selection
    (oracle.select_indices on the workload's shape: window scores, pooling, top-k) at all cores."""
    from oracle import catekv_oracle as orc
    from workloads import synth
    out = {}
    try:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            rate1, _, _ = oracle_sample_rate(w, target_s=3.0)
        out["rows_per_s_1thread"] = rate1
    except Exception as e:  # threadpoolctl missing: report the reason, keep the line
        out["rows_per_s_1thread"] = None
        out["note_1thread"] = repr(e)
    n = min(w.n, 65536)
    qwin = synth.bits(synth.randn_bf16((w.G, w.L_obs, w.d), "cpu", w.seed, "osq"))
    k = synth.bits(synth.randn_bf16((n, w.d), "cpu", w.seed, "osk"))
    t0 = time.perf_counter()
    C = orc.window_scores(qwin, k, w.L_obs)
    orc.select_indices(C, n, w.sink, w.local, w.budget, w.pool_mode, w.pool_param)
    out["select_one_head_s"] = time.perf_counter() - t0
    out["select_shape"] = f"{w.G} x {w.L_obs} window queries, {n} keys, budget {w.budget}"
    return out


def workload_rows_per_layer_step(w):
    """Expected kept rows of one layer-step (mean over the seeded masks of all layers)."""
    from workloads import synth
    tot = 0
    for l in range(w.layers):
        tot += sum(expected_lengths(w, synth.head_mask(w, l)))
    return tot / w.layers


def run_reference(args):
    """--impl reference: the CPU oracle on the same metric; each step is a bounded sample, extrapolated."""
    from workloads import synth
    w = synth.WORKLOADS[args.workload]
    rows = workload_rows_per_layer_step(w)
    vals = []
    per = 4.0 if args.steps > 3 else 10.0
    for i in range(args.warmup + args.steps):
        rate, desc, spent = oracle_sample_rate(w, target_s=per if i >= args.warmup else 1.0)
        if i >= args.warmup:
            vals.append(rate)
    rate = float(np.mean(vals))
    t_layer = rows / rate
    value = w.B / (w.layers * t_layer)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": w.layers * t_layer * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "note": "CPU oracle (numpy fp64) timed on a bounded sample and extrapolated "
                   "by rows; not the target"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                         "sample": desc + f", {rate:.3e} rows/s"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def measure_workload(ck, w, dev, n_layers, steps, warmup, barrier, graph, peaks, peak_src, world, sampler):
    """Build the workload's caches, time the decode step (device-resident and end to end) and the attention kernel
    in the same launch regime; returns the pieces of a bench line.  Frees the model before returning."""
    import torch
    total_steps = 3 * (warmup + steps) + 24
    model, sel_ms = build_model(ck, w, dev, max_new=total_steps, layers=n_layers)
    plan_us = float(np.median(PLAN_HOST_US[-n_layers:]))
    if sampler:
        sampler.start()
    ms = max_over_ranks(time_decode(ck, w, model, dev, steps, warmup, barrier, graph), dev)
    clocks = sampler.stop() if sampler else None
    bytes_per_layer = float(np.mean(kept_bytes(model)))
    part_us, comb_us = time_kernels(ck, w, model, dev, max(3, min(steps, 10)))
    ms_e2e, h2d, d2h = time_e2e(ck, w, model, dev, steps, warmup, barrier, graph)
    ms_e2e = max_over_ranks(ms_e2e, dev)
    has_combine = any(ck.plan_header(m["plan"])["n_slots"] for m in model)
    del model
    torch.cuda.empty_cache()
    scale_layers = w.layers / n_layers  # only != 1 when --layers is used for profiling
    achieved = bytes_per_layer / (part_us * 1e-6) / 1e9
    return {
        "value": world * w.B / (ms * scale_layers * 1e-3),
        "ms_per_step": ms,
        "us_per_layer_step": ms * 1e3 / n_layers,
        "step_hbm_gbs": bytes_per_layer / (ms * 1e-3 / n_layers) / 1e9,
        "config": {"workload": w.name, "layers": n_layers, "batch": w.B, "context": w.n, "q_heads": w.Hq,
                   "kv_heads": w.Hkv, "head_dim": w.d, "budget_consistent": w.budget, "eta_adaptive": w.eta,
                   "window": w.L_obs, "replicas": world,
                   "l2": "no flush: per-layer working set %.0f MB x %d layers, far above the 126 MB L2"
                         % (bytes_per_layer / 1e6, n_layers),
                   "step": "one decode token of the whole model: per layer " +
                           ("catekv_append_decode_attn (append fused into the attention launch)" if FUSED
                            else "catekv_append + catekv_decode_attn"),
                   "launch": "CUDA graph replay of the step" if graph else "host launches"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"], "peak_source": peak_src,
                     "traffic": bytes_per_layer * TRAFFIC_READ_RATIO + TRAFFIC_WRITE_BYTES,
                     "traffic_source": "ncu dram__bytes_read.sum / algorithmic bytes = 1.0002 and about 4.6 MB of "
                                       "dram__bytes_write.sum per launch on the two-layer configs[2] case, scaled "
                                       "by this run's kept rows (every kept row crosses DRAM once)",
                     "kernel": "decode_partial_kernel", "bytes_per_launch": bytes_per_layer,
                     "us_per_launch": part_us,
                     "us_per_launch_how": "CUDA graph of catekv_decode_partials over all layers (the step's launch "
                                          "chain without the combine launches), CUDA events around its replays, "
                                          "divided by the launches",
                     "frac_of_8TBs": achieved / 8000.0, "combine_us": comb_us, "append_us": APPEND_US},
        "e2e": {"value": world * w.B / (ms_e2e * scale_layers * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e},
        "gpu_launches": steps * n_layers * ((1 if FUSED else 2) + (1 if has_combine else 0)),
        "clocks": clocks,
        "select_compact": select_block(w, float(np.mean(sel_ms[1:] or sel_ms)), n_layers, bytes_per_layer, peaks),
        "plan_host_us": plan_us,
    }


# ------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg3", choices=["cfg0", "cfg1", "cfg2", "cfg3", "cfg4"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling on a small case)")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel from the host instead of replaying "
                    "a captured CUDA graph of the step")
    ap.add_argument("--no-fused", action="store_true", help="catekv_append + catekv_decode_attn as two calls per layer")
    ap.add_argument("--select-only", action="store_true", help="run only the prefill-end path (catekv_select_compact) "
                    "for --layers layers and print its time; used for profiling that path on a small case")
    ap.add_argument("--retrieval-only", action="store_true", help="run only the query-aware retrieval decode step "
                    "(small case for profiling; use with --workload and --layers)")
    ap.add_argument("--head-cv-only", action="store_true", help="run only catekv_head_cv on the calibration shape "
                    "(8 prompts x 16384 tokens, 28q/4kv, window 64) and print its time; for profiling")
    ap.add_argument("--retrieval-gather", action="store_true", help="with --retrieval-only: the gather path "
                    "(catekv_retrieve_compact into a per-step cache) instead of attention in place")
    ap.add_argument("--window-attn-only", action="store_true", help="run only catekv_window_attn and the selection "
                    "with and without its normaliser on the workload's prefill shape; for profiling")
    ap.add_argument("--no-extras", action="store_true", help="skip the other configs, head_cv and the oracle timing")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            run_reference(args)
        return

    import torch
    import torch.distributed as dist
    import paper_2608_30295_b200 as pkg
    ck = pkg.binding
    from workloads import synth

    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    barrier = None
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(dev))
        barrier = lambda: dist.barrier()

    peaks, peak_src = measured_peaks()
    w = synth.WORKLOADS[args.workload]
    n_layers = args.layers or w.layers
    graph = not args.no_graph
    global FUSED
    FUSED = not args.no_fused
    if args.head_cv_only:
        ms_cv = time_head_cv(ck, dev)
        if rank == 0:
            print(json.dumps({"head_cv_ms": ms_cv, "shape": "8 prompts x 16384 tokens, 28q/4kv, window 64"}))
        return
    if args.window_attn_only:
        res = time_window_attn(ck, w, dev)
        if rank == 0:
            print(json.dumps({"workload": w.name, **res}))
        return
    if args.retrieval_only:
        ru, ra, rm = time_retrieval(ck, w, dev, n_layers=n_layers, steps=args.steps, graph=graph,
                                    gather=args.retrieval_gather)
        if rank == 0:
            print(json.dumps({"workload": w.name, "layers": n_layers, "retrieval_us_per_layer_step": ru,
                              "attended_bytes_per_layer_step": ra, "metadata_bytes_per_layer_step": rm}))
        return
    if args.select_only:
        model, sel_ms = build_model(ck, w, dev, max_new=8, layers=n_layers)
        if rank == 0:
            print(json.dumps({"workload": w.name, "layers": n_layers, "select_compact_ms_per_layer": sel_ms}))
        return

    vis = [x for x in os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",") if x]
    sampler = ClockSampler(vis[local_rank] if local_rank < len(vis) else local_rank)
    r = measure_workload(ck, w, dev, n_layers, args.steps, args.warmup, barrier, graph, peaks, peak_src, world, sampler)
    bytes_per_layer = r["roofline"]["bytes_per_launch"]
    line = {
        "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": r["config"],
        "us_per_layer_step": r["us_per_layer_step"],
        "roofline": r["roofline"],
        "e2e": r["e2e"],
        "gpu_launches": r["gpu_launches"],
        "clocks": r["clocks"],
        "select_compact": r["select_compact"],
        "plan_host_us": r["plan_host_us"],
    }
    if rank == 0 and not args.no_extras:
        # the other configurations over all their layers, each with its own roofline and end-to-end blocks
        # (configs[2] and configs[4] carry the 70 %-of-HBM target; configs[1] is reported, not gated)
        table = {}
        for name in ("cfg1", "cfg2", "cfg4"):
            if name == w.name:
                continue
            wo = synth.WORKLOADS[name]
            ro = measure_workload(ck, wo, dev, wo.layers, 10, 3, None, graph, peaks, peak_src, 1, None)
            table[name] = {"layers_timed": wo.layers, "tokens_per_s": ro["value"], "ms_per_step": ro["ms_per_step"],
                           "us_per_layer_step": ro["us_per_layer_step"], "roofline": ro["roofline"], "e2e": ro["e2e"],
                           "bytes_per_layer_step": ro["roofline"]["bytes_per_launch"],
                           # the whole replayed layer-step (attention + combine, append fused) against the same bytes
                           "step_hbm_gbs": ro["step_hbm_gbs"],
                           "step_frac_of_measured": ro["step_hbm_gbs"] / peaks["hbm_gbs"],
                           "step_frac_of_8TBs": ro["step_hbm_gbs"] / 8000.0,
                           "select_ms_per_layer": ro["select_compact"]["ms_per_layer"],
                           "select_compact": ro["select_compact"]}
        line["other_configs"] = table
        line["head_cv"] = {"ms": time_head_cv(ck, dev), "shape": "8 prompts x 16384 tokens, 28q/4kv, window 64"}
        ru, ra, rm = time_retrieval(ck, w, dev)
        line["retrieval"] = {"us_per_layer_step": ru, "attended_bytes_per_layer_step": ra,
                             "metadata_bytes_per_layer_step": rm, "budget_rows": 1024, "chunk": 8,
                             # the step's bytes (chunk metadata + attended rows) at the measured copy bandwidth
                             "hbm_bound_us": (ra + rm) / (peaks["hbm_gbs"] * 1e3),
                             "frac_of_hbm_bound": (ra + rm) / (peaks["hbm_gbs"] * 1e3) / ru,
                             "note": "query-aware retrieval on the adaptive heads of the same workload: per layer "
                                     "catekv_append_retrieval, catekv_retrieve_select, catekv_decode_attn_indexed; CUDA graph replay of the step"}
        wa = time_window_attn(ck, synth.WORKLOADS["cfg2"], dev)
        wa["tflops"] = wa["flops_window_attn"] / (wa["window_attn_ms"] * 1e-3) / 1e12
        wa["hbm_gbs"] = wa["hbm_bytes_window_attn"] / (wa["window_attn_ms"] * 1e-3) / 1e9
        wa["frac_of_bf16_peak"] = wa["tflops"] / peaks["bf16_tflops"]  # the whole call against the burst GEMM figure
        wa["frac_of_hbm_peak"] = wa["hbm_gbs"] / peaks["hbm_gbs"]
        wa["note"] = ("configs[2] prefill shape, one layer: catekv_window_attn (prefill rows of the observation window "
                      "+ their normalisers) and catekv_select_compact with / without that normaliser")
        line["window_attn"] = wa
        line["linearity"] = time_linearity(ck, dev)
        rate, desc, spent = oracle_sample_rate(w, target_s=15.0)
        rows = bytes_per_layer / ROW_BYTES
        line["cpu_baseline"] = {"value": w.B / (w.layers * rows / rate), "unit": UNIT, "cores": oracle_threads(),
                                "kind": "oracle", "sample": desc + f" ({spent:.1f} s, {rate:.3e} rows/s), "
                                "extrapolated by rows to the full step"}
        line["cpu_baseline"].update(oracle_extra_timings(w))
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
