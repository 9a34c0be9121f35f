#!/usr/bin/env python
"""Benchmark of the decode-attention step (multi-query vs multi-head) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one pass of the whole hot path over one batch: the in-place append of the new
token's key/value row, the split-m pass over the cache and the merge of the splits -- for the
multi-query variant through mqa_decode_append_step (one kernel launch at the headline size), for
the multi-head variant kv_cache_append + mha_decode_step.  The multi-query step as three separate
launches is timed beside it.  The headline
workload is the long-context configuration (b=32, h=32, k=v=128, 8192-row cache); the other
workloads (`--workload`, `--sweep`) are the parity configurations and the bandwidth sweep.
Prints ONE JSON line (rank 0).  `value` is achieved HBM GB/s of the multi-query step
(algorithmic bytes / time); the multi-head step on the same shapes is reported beside it.
`e2e` is the same step through mqa_decode_append_step_host on pinned host buffers, one call and
one stream synchronisation per token (median of five regions of K steps), and beside it the same
call captured once per cache set as a CUDA graph and replayed.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1911_02150_b200 import sharding, workloads as wl  # noqa: E402

NOMINAL_HBM_GBS = 8000.0      # the metric's stated denominator
FALLBACK_HBM_GBS = 6650.0     # earlier measurement on this machine, used only if MEASURED_PEAKS.json is absent
L2_BYTES = 126 * 2 ** 20


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def __exit__(self, *a):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.thread.join(timeout=2)

    def summary(self):
        sm, mx, reasons, power = [], [], set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(power),
                "samples": len(sm), "reasons": sorted(reasons)}


class StepState:
    """Device-resident state of one variant: rotating cache sets (to keep reads out of L2), the
    step's inputs and outputs, and the launch plan."""

    def __init__(self, mqa, variant, w, device, seed, min_rotate_bytes, host_legs=True):
        self.mqa, self.variant, self.w, self.device = mqa, variant, w, device
        b, h, m = w.b, w.h, w.m_max
        self.kvh = 1 if variant == "mqa" else h
        lens0 = wl.initial_lens(w, seed=0)
        cache_bytes = 2 * b * self.kvh * m * 128 * 2
        free, _ = torch.cuda.mem_get_info(device)
        n_sets = max(1, -(-min_rotate_bytes // cache_bytes))
        n_sets = int(min(n_sets, max(1, (free - 8 * 2 ** 30) // cache_bytes), 16))
        self.sets = []
        for i in range(n_sets):
            inp = wl.make_inputs(b, h, m, variant, seed=seed + i, device=device)
            self.sets.append(inp)
        self.lens_before = torch.from_numpy(lens0).to(device)
        self.lens_after = torch.from_numpy(lens0 + 1).to(device)
        self.sum_lens = int((lens0 + 1).sum())
        self.o = torch.empty(b, h, 128, dtype=torch.float32, device=device)
        self.ws = mqa.alloc_workspace(b, h, m, device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.n_splits, self.chunk_rows = mqa.plan_splits(variant == "mqa", b, h, m)
        self.bytes = wl.algorithmic_bytes(self.sum_lens, b, h, self.kvh)
        self.cache_bytes = cache_bytes
        self.append = mqa.kv_cache_append
        self.step_fn = mqa.mqa_decode_step if variant == "mqa" else mqa.mha_decode_step
        self.split_fn = mqa.mqa_decode_step_split if variant == "mqa" else mqa.mha_decode_step_split
        self.combine_fn = mqa.mqa_decode_step_combine if variant == "mqa" else mqa.mha_decode_step_combine
        self.launches_three = 2 + (1 if self.n_splits > 1 else 0)
        # the multi-query step is one call (append + attention + merge); multi-head is append + step
        self.launches_per_step = mqa.append_step_launches(b, h, m) if variant == "mqa" else self.launches_three
        self.host_steps = self.bound_steps = None
        if variant == "mqa":
            # the step bound once per cache set.  A decoding loop: apart from the steps themselves nothing writes lens or
            # the caches' rows, hence chained (the sets share one workspace and one o, which the promise leaves free)
            self.bound_steps = [mqa.AppendStep(s["q"], s["K"], s["V"], s["k_new"], s["v_new"], self.lens_before, self.o, self.ws,
                                               self.status, advance=False, chained=True) for s in self.sets]
        if not host_legs:
            return
        # pinned host copies of the per-step inputs / result for the end-to-end leg
        # (q, k_new, v_new packed in one pinned buffer and one device buffer: one host-to-device copy per step)
        s0 = self.sets[0]
        parts = [s0[n] for n in ("q", "k_new", "v_new")]
        sizes = [t.numel() * t.element_size() for t in parts]
        self.host_in = torch.empty(sum(sizes), dtype=torch.uint8).pin_memory()
        self.dev_in = torch.empty(sum(sizes), dtype=torch.uint8, device=device)
        self.e2e_views, self.host_views, at = [], [], 0
        for t, n in zip(parts, sizes):
            self.host_in[at : at + n].copy_(t.cpu().contiguous().view(torch.uint8).view(-1))
            self.e2e_views.append(self.dev_in[at : at + n].view(torch.bfloat16).view(t.shape))
            self.host_views.append(self.host_in[at : at + n].view(torch.bfloat16).view(t.shape))
            at += n
        self.staging = torch.empty(max(16, mqa.host_staging_bytes(b, h)), dtype=torch.uint8, device=device)
        self.host_o = torch.empty(b, h, 128, dtype=torch.float32).pin_memory()
        self.d2h_bytes = self.host_o.numel() * 4
        self.h2d_bytes = sum(sizes)
        if variant == "mqa":
            # the library's host-buffer call, bound once per cache set (what a decoding loop over fixed pinned buffers does)
            qh, kh, vh = self.host_views
            self.e2e_stream = torch.cuda.current_stream(device)
            self.host_steps = [mqa.HostStep(qh, kh, vh, self.host_o, s["K"], s["V"], self.lens_before, self.staging, self.ws,
                                            self.status, advance=False, stream=self.e2e_stream) for s in self.sets]

    def step(self, i):
        if self.bound_steps is not None:
            self.bound_steps[i % len(self.bound_steps)](torch.cuda.current_stream())   # (a capturing stream, in a graph)
        else:
            self.step_separate(i)

    def step_separate(self, i):
        """The same step as separate calls: kv_cache_append, then the decode step (pass + second pass)."""
        s = self.sets[i % len(self.sets)]
        self.append(s["K"], s["V"], s["k_new"], s["v_new"], self.lens_before, advance=False, status=self.status)
        self.step_fn(s["q"], s["K"], s["V"], self.lens_after, self.o, self.ws, self.status)

    def split_only(self, i):
        """Only the pass over the cache (the dominant kernel) of step i."""
        s = self.sets[i % len(self.sets)]
        self.split_fn(s["q"], s["K"], s["V"], self.lens_after, self.o, self.ws, self.status)

    def step_e2e(self, i):
        if self.host_steps is not None:
            # inputs in, step, o out: all enqueued by one C call on pinned host buffers (bound to the stream at set-up)
            self.host_steps[i % len(self.host_steps)]()
            self.e2e_stream.synchronize()              # the caller needs o before the next token
            return
        stream = torch.cuda.current_stream()
        s = self.sets[i % len(self.sets)]
        self.dev_in.copy_(self.host_in, non_blocking=True)
        q, k_new, v_new = self.e2e_views
        self.append(s["K"], s["V"], k_new, v_new, self.lens_before, advance=False, status=self.status)
        self.step_fn(q, s["K"], s["V"], self.lens_after, self.o, self.ws, self.status)
        self.host_o.copy_(self.o, non_blocking=True)
        stream.synchronize()

    def capture_host_steps(self):
        """The host-buffer call of every cache set captured once as a CUDA graph of its own (possible because nothing in
        it is a transfer from pageable memory: a kernel fetches the pinned inputs, the kernels store o to the host)."""
        self.host_graphs = []
        for hs in self.host_steps:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                hs(torch.cuda.current_stream())
            self.host_graphs.append(g)

    def step_e2e_graph(self, i):
        """step_e2e with the call replayed from its graph: the same work per token, one submission instead of two launches."""
        self.host_graphs[i % len(self.host_graphs)].replay()
        torch.cuda.current_stream().synchronize()


def time_region(fn, steps, device):
    """Seconds for `steps` calls of fn(i), CUDA events on the launching stream, synchronised on both sides."""
    sharding.barrier()
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        fn(i)
    e1.record()
    torch.cuda.synchronize(device)
    sharding.barrier()
    return e0.elapsed_time(e1) * 1e-3


def capture_graph(fn, steps):
    """One CUDA graph holding `steps` calls of fn(i): the launch-bound loop is replayed with one
    host call, so the device timeline has no host-side gaps between kernels."""
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(steps):
            fn(i)
    return g


def time_isolated(st: StepState, steps, device):
    """Seconds per step when the step does NOT follow a step: every timed launch comes after an unrelated kernel that
    has nothing to do with the cache (a 4 MiB fill by torch, ~2 us), has its own CUDA-event pair around it, and is
    launched from the host.  What a back-to-back loop hides -- launch latency, the set-up that programmatic dependent
    launch overlaps with the previous step, copies started early on the chained promise -- is all inside this figure,
    and so is the resolution of an event pair (about half a microsecond)."""
    spacer = torch.empty(1 << 20, dtype=torch.float32, device=device)
    n = max(steps, 20)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
    for i in range(3):
        spacer.fill_(float(i)); st.step(i)
    torch.cuda.synchronize(device)
    for i, (e0, e1) in enumerate(ev):
        spacer.fill_(float(i))
        e0.record(); st.step(i); e1.record()
    torch.cuda.synchronize(device)
    return statistics.median(e0.elapsed_time(e1) for e0, e1 in ev) * 1e-3


def quick_point(mqa, variant, w, device, steps=20, min_rotate_bytes=4 * L2_BYTES):
    """One sweep point for the default bench line: us per step (K steps as one CUDA graph, caches rotated past L2),
    GB/s, launches.  None for the fields of a point that was skipped, with the reason."""
    kvh = 1 if variant == "mqa" else w.h
    cache = 2 * w.b * kvh * w.m_max * 256
    row = {"workload": w.name, "variant": variant, "b": w.b, "h": w.h, "m": w.m_max}
    free, _ = torch.cuda.mem_get_info(device)
    if cache > 16 * 2 ** 30:
        row["skipped"] = f"a {cache >> 30} GiB cache takes longer to fill than the default run allows (bench.py --sweep runs it)"
        return row
    if cache + 6 * 2 ** 30 > free:
        row["skipped"] = f"cache of {cache >> 30} GiB does not fit"
        return row
    st = StepState(mqa, variant, w, device, 0, min_rotate_bytes=min_rotate_bytes, host_legs=False)
    for i in range(3):
        st.step(i)
    torch.cuda.synchronize(device)
    g = capture_graph(st.step, steps)
    g.replay()
    torch.cuda.synchronize(device)
    secs = statistics.median(time_region(lambda _i: g.replay(), 1, device) for _ in range(10)) / steps
    gbs = st.bytes / secs / 1e9
    row.update({"us_per_step": secs * 1e6, "gbs": gbs, "frac_of_8TBs": gbs / NOMINAL_HBM_GBS, "bytes_per_step": st.bytes,
                "launches_per_step": st.launches_per_step, "cache_sets": len(st.sets), "status": int(st.status.item())})
    del st, g
    torch.cuda.empty_cache()
    return row


# The points the >= 70 % target names (long-context configurations) and the ragged batch, for the default bench line.
LINE_SWEEP = ("sweep_b1_m32768", "sweep_b8_m32768", "sweep_b64_m32768", "sweep_b256_m32768", "sweep_b64_m4096",
              "sweep_b256_m4096", "ragged")


def run_variant(st: StepState, steps, warmup, device, sample_clocks, use_graph=True, min_warm_s=0.2):
    t0 = time.time()
    i = 0
    while i < warmup or time.time() - t0 < min_warm_s:      # at least `warmup` steps, and clocks ramped up
        st.step(i)
        i += 1
        if i % 16 == 0:
            torch.cuda.synchronize(device)
    torch.cuda.synchronize(device)
    if use_graph:
        g_step = capture_graph(st.step, steps)
        g_split = capture_graph(st.split_only, steps)
        g_step.replay(); g_split.replay()
        torch.cuda.synchronize(device)
        run_steps = lambda _i: g_step.replay()
        run_split = lambda _i: g_split.replay()
        calls = 1
    else:
        run_steps, run_split, calls = st.step, st.split_only, steps
    sampler = ClockSampler(torch.cuda.current_device()) if sample_clocks else None
    if sampler:
        sampler.__enter__()
    t0 = time.time()
    regions = []
    # every region is exactly K steps between synchronisations; regions repeat until the clock
    # monitor has seen ~0.5 s of load, and the median region is reported
    while True:
        regions.append(time_region(run_steps, calls, device))
        if not sample_clocks or time.time() - t0 > 0.5 or len(regions) >= 500:
            break
    if sampler:
        sampler.__exit__()
    secs = statistics.median(regions)
    # the same step as separate calls (append, pass over the cache, second pass)
    sep_s = None
    if st.variant == "mqa":
        if use_graph:
            g_sep = capture_graph(st.step_separate, steps)
            g_sep.replay()
            torch.cuda.synchronize(device)
            run_sep = lambda _i: g_sep.replay()
        else:
            run_sep = st.step_separate
        sep_s = statistics.median(time_region(run_sep, calls, device) for _ in range(max(3, min(20, len(regions)))))
    # per-launch duration of the pass over the cache (the dominant kernel): K back-to-back launches
    kernel_regions = [time_region(run_split, calls, device) for _ in range(max(3, min(20, len(regions))))]
    kernel_s = statistics.median(kernel_regions) / steps
    isolated_s = time_isolated(st, steps, device)
    # end to end with host buffers (eager: every step waits for its result)
    for i in range(3):
        st.step_e2e(i)
    e2e_s = statistics.median(time_region(st.step_e2e, steps, device) for _ in range(5))
    e2e_graph_s = None
    if st.host_steps is not None and use_graph:
        st.capture_host_steps()
        for i in range(3):
            st.step_e2e_graph(i)
        e2e_graph_s = statistics.median(time_region(st.step_e2e_graph, steps, device) for _ in range(5))
    status = int(st.status.item())
    return {"secs": secs, "kernel_s": kernel_s, "e2e_s": e2e_s, "e2e_graph_s": e2e_graph_s, "status": status, "separate_s": sep_s,
            "isolated_s": isolated_s,
            "clocks": sampler.summary() if sampler else None, "first_region_s": regions[0],
            "min_region_s": min(regions), "regions": len(regions), "graph": bool(use_graph)}


def layer_block(mqa, w, device, seed, steps, d_model=1024):
    """The whole incremental multi-query layer step (projections of x[b,d] to q, k_new, v_new; append + attention;
    output projection) on the same workload, d = 1024 as in the paper's models: µs per step, K steps as one CUDA graph,
    cache sets rotated past L2.  The weights (2 h d 128 + 2 d 128 bf16 elements) are read every step as well."""
    gen = torch.Generator(device=device).manual_seed(seed + 17)
    n = lambda shape, std: wl.bf16_normal(shape, std, gen, device)
    b, h, m, d = w.b, w.h, w.m_max, d_model
    W = [n((h, d, 128), (d * 128) ** -0.5), n((d, 128), d ** -0.5), n((d, 128), d ** -0.5), n((h, d, 128), (h * 128) ** -0.5)]
    nset = max(1, min(8, (8 * L2_BYTES + b * m * 512 - 1) // (b * m * 512)))
    sets = [(n((b, d), 1.0), n((b, m, 128), 1.0), n((b, m, 128), 1.0)) for _ in range(nset)]
    lens = torch.from_numpy(wl.initial_lens(w, seed)).to(device)
    y = torch.empty(b, d, dtype=torch.float32, device=device)
    ws = mqa.alloc_layer_workspace(b, h, d, m, device)
    status = torch.zeros(1, dtype=torch.int32, device=device)

    def step(i):
        x, K, V = sets[i % nset]
        mqa.mqa_layer_decode_step(x, W[0], W[1], W[2], W[3], K, V, lens, y, ws, status, advance=False)

    for i in range(3):
        step(i)
    torch.cuda.synchronize(device)
    g = capture_graph(step, steps)
    g.replay()
    torch.cuda.synchronize(device)
    secs = statistics.median(time_region(lambda _i: g.replay(), 1, device) for _ in range(20))
    weight_bytes = sum(t.numel() * 2 for t in W)
    return {"us_per_step": secs / steps * 1e6, "d_model": d, "weight_bytes": weight_bytes, "status": int(status.item()),
            "launches_per_step": 2 + mqa.append_step_launches(b, h, m), "cache_sets": nset}


def paper_loop_block(mqa, device, seed):
    """The paper's timed decoding shape (Section 4.1: 128 sequences, h = 8, 128 target positions): 128 successive steps,
    each appending one row and attending over the prefix, the cache growing from 1 to 128 rows; the loop is one CUDA
    graph, lens lives on the device and is advanced by the steps.  Multi-query: one mqa_decode_append_step per step;
    multi-head (per-head cache): kv_cache_append + mha_decode_step."""
    w = wl.WORKLOADS["paper_incremental"]
    b, h, m, steps = w.b, w.h, w.m_max, w.steps
    out = {"b": b, "h": h, "steps": steps, "cache_rows": f"1..{m}"}
    for variant in ("mqa", "mha"):
        inp = wl.make_inputs(b, h, m, variant, seed=seed, device=device)
        lens0 = torch.zeros(b, dtype=torch.int32, device=device)
        lens = lens0.clone()
        o = torch.empty(b, h, 128, dtype=torch.float32, device=device)
        ws = mqa.alloc_workspace(b, h, m, device)
        status = torch.zeros(1, dtype=torch.int32, device=device)
        if variant == "mqa":
            step = lambda i: mqa.mqa_decode_append_step(inp["q"], inp["K"], inp["V"], inp["k_new"], inp["v_new"], lens, o, ws,
                                                        status, advance=True, chained=i > 0)
            launches = mqa.append_step_launches(b, h, m)
        else:
            def step(i):
                mqa.kv_cache_append(inp["K"], inp["V"], inp["k_new"], inp["v_new"], lens, advance=True, status=status)
                mqa.mha_decode_step(inp["q"], inp["K"], inp["V"], lens, o, ws, status)
            launches = 2 + (1 if mqa.plan_splits(False, b, h, m)[0] > 1 else 0)
        for i in range(3):
            step(i)
        lens.copy_(lens0)
        torch.cuda.synchronize(device)
        g = capture_graph(step, steps)
        times = []
        for _ in range(20):
            lens.copy_(lens0)                               # every replay decodes from an empty cache
            times.append(time_region(lambda _i: g.replay(), 1, device))
        assert int(lens[0]) == steps
        secs = statistics.median(times)
        total_bytes = sum(wl.algorithmic_bytes(b * t, b, h, 1 if variant == "mqa" else h) for t in range(1, steps + 1))
        out[variant] = {"us_per_step": secs / steps * 1e6, "us_per_loop": secs * 1e6, "gbs": total_bytes / secs / 1e9,
                        "us_per_token": secs / steps / b * 1e6, "launches_per_step": launches, "status": int(status.item())}
        del inp
    out["mqa_speedup_over_mha"] = out["mha"]["us_per_step"] / out["mqa"]["us_per_step"]
    return out


def measured_tensor_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["bf16_tflops"]), float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "measured"
        except Exception:
            pass
    return 1590.0, 1400.0, "fallback"


def prefill_block(mqa, device, seed, b=32, h=32, n=4096):
    """The batched form of Section 3 under the autoregressive mask (the processing of a whole prompt: n = m positions,
    the batch and head count of the headline workload): milliseconds per call and TFLOP/s, counting the method's own
    4 k flops per (query row, visible key) pair -- not the dense n x m rectangle.  Compute-bound: set against the
    measured bf16 matmul throughput."""
    gen = torch.Generator(device=device).manual_seed(seed + 31)
    Q = wl.bf16_normal((b, h, n, 128), 128 ** -0.5, gen, device)
    K = wl.bf16_normal((b, n, 128), 1.0, gen, device)
    V = wl.bf16_normal((b, n, 128), 1.0, gen, device)
    O = torch.empty(b, h, n, 128, dtype=torch.float32, device=device)
    ws = torch.empty(max(16, mqa.prefill_workspace_bytes(b, h, n, n)), dtype=torch.uint8, device=device)
    status = torch.zeros(1, dtype=torch.int32, device=device)
    call = lambda _i: mqa.mqa_prefill_attention(Q, K, V, O, ws, None, status)
    for i in range(2):
        call(i)
    secs = statistics.median(time_region(call, 1, device) for _ in range(5))
    flops = 4 * 128 * h * b * n * (n + 1) // 2
    burst, sustained, kind = measured_tensor_peak()
    tf = flops / secs / 1e12
    return {"b": b, "h": h, "n": n, "ms": secs * 1e3, "tflops": tf, "flops": flops, "bound": "tensor", "peak": sustained,
            "peak_kind": f"bf16 matmul, sustained, of {kind}", "frac": tf / sustained, "frac_of_burst_peak": tf / burst,
            "launches": 1, "kernel": "mqa_prefill_kernel",
            "status": int(status.item())}


def many_rows_block(mqa, device, seed, w, rows=128):
    """Beam search over one shared memory (Section 4.2: beam 4): beams x heads query rows per sequence, here 4 x 32 = 128
    rows over the headline workload's caches, on the kernel with the query rows as tile rows.  us per step (attention over
    the cache, caches rotated past L2), beside the 64-row figure."""
    out = {}
    for r in (64, rows):
        w2 = wl.Workload(f"{w.name}_rows{r}", b=w.b, h=r, m_max=w.m_max, lens="full")
        row = quick_point(mqa, "mqa", w2, device, steps=10, min_rotate_bytes=4 * L2_BYTES)
        out[f"rows_{r}"] = {k: row.get(k) for k in ("us_per_step", "gbs", "frac_of_8TBs", "launches_per_step", "status", "skipped")}
        out[f"rows_{r}"]["kernel"] = mqa.plan_kernel_name(True, True, w.b, r, w.m_max)
    return out


def cpu_baseline(w, seed, budget_s=20.0):
    """The oracle, as it stands, on the host cores: one multi-query step of the same workload on
    as many whole sequences as fit the time budget."""
    import oracle
    inp = wl.make_inputs(min(w.b, 64), w.h, w.m_max, "mqa", seed=seed, device="cpu")
    lens = (wl.initial_lens(w)[: inp["b"]] + 1).astype(np.int32)
    qb, Kb, Vb = wl.bits(inp["q"]), wl.bits(inp["K"]), wl.bits(inp["V"])
    threads = oracle.num_threads()
    target_wall = budget_s / max(threads, 1)             # ~budget_s seconds of CPU work in total
    n = inp["b"]
    reps, t0 = 0, time.perf_counter()
    while True:
        oracle.mqa_decode_step(qb[:n], Kb[:n], Vb[:n], lens[:n])
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= target_wall or reps >= 1000:
            break
    by = wl.algorithmic_bytes(int(lens[:n].sum()), n, w.h, 1) * reps
    return {"value": by / dt / 1e9, "unit": "GB/s", "cores": threads, "kind": "oracle",
            "sample": f"{reps} multi-query steps over {n} of {w.b} sequences x {w.h} heads x {w.m_max} rows, fp64, "
                      f"{dt:.2f} s wall on {threads} threads", "seconds": dt}


def reference_arm(args, w):
    """--impl reference: the CPU oracle timed on this machine's host cores, a bounded sample per step."""
    rank, _, world = sharding.world_from_env()
    if rank != 0:
        return
    import oracle
    n_seq = min(w.b, 2)
    inp = wl.make_inputs(n_seq, w.h, w.m_max, "mqa", seed=0, device="cpu")
    lens = (wl.initial_lens(w)[:n_seq] + 1).astype(np.int32)
    qb, Kb, Vb = wl.bits(inp["q"]), wl.bits(inp["K"]), wl.bits(inp["V"])
    knb, vnb = wl.bits(inp["k_new"]), wl.bits(inp["v_new"])
    lens_before = (lens - 1).astype(np.int32)

    def one(_):
        lb = lens_before.copy()
        oracle.kv_cache_append(Kb, Vb, knb, vnb, lb, True)
        oracle.mqa_decode_step(qb, Kb, Vb, lb)
    for i in range(args.warmup):
        one(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        one(i)
    dt = (time.perf_counter() - t0) / args.steps
    by = wl.algorithmic_bytes(int(lens.sum()), n_seq, w.h, 1)
    val = by / dt / 1e9
    sample = f"{n_seq} of {w.b} sequences x {w.h} heads x {w.m_max} rows per step (append + multi-query step), fp64 oracle"
    print(json.dumps({
        "impl": "reference", "metric": "mqa_decode_step_hbm_gbs", "value": val, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(w), "sample": sample},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def workload_name(w):
    return (f"{w.name}: b={w.b} h={w.h} k=v=128 m_max={w.m_max} lens={w.lens}; one step = append of the new "
            f"k/v row + attention over the prefix")


def result_block(st, r, steps):
    us = r["secs"] / steps * 1e6
    gbs = st.bytes / (r["secs"] / steps) / 1e9
    return {"us_per_step": us, "gbs": gbs, "frac_of_8TBs": gbs / NOMINAL_HBM_GBS, "bytes_per_step": st.bytes,
            "n_splits": st.n_splits, "chunk_rows": st.chunk_rows, "cache_sets": len(st.sets),
            "pass_only_us": r["kernel_s"] * 1e6, "isolated_us": r["isolated_s"] * 1e6, "status": r["status"],
            "separate_calls_us_per_step": None if r.get("separate_s") is None else r["separate_s"] / steps * 1e6,
            "launches_per_step": st.launches_per_step,
            "first_region_us_per_step": r["first_region_s"] / steps * 1e6,
            "min_us_per_step": r["min_region_s"] / steps * 1e6, "regions": r["regions"], "cuda_graph": r["graph"]}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="long_context")
    ap.add_argument("--no-mha", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-layer", action="store_true", help="skip the timing of the whole layer step (projections either side)")
    ap.add_argument("--prefill-only", default=None, metavar="B,H,N",
                    help="time only the batched (prefill) form at these sizes and print its block (what the ncu capture of that kernel runs)")
    ap.add_argument("--step-only", default=None, metavar="B,H,M",
                    help="time only the multi-query append-and-attend step of this shape (full caches) and print it")
    ap.add_argument("--no-line-sweep", action="store_true", help="skip the long-context sweep points of the default line")
    ap.add_argument("--no-graph", action="store_true", help="launch every step from the host instead of replaying a CUDA graph")
    ap.add_argument("--sweep", action="store_true", help="run every workload, both variants, and write the table to --sweep-out")
    ap.add_argument("--sweep-out", default="sweep.json", help="where --sweep writes its table (JSON)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = wl.WORKLOADS[args.workload]

    if args.impl == "reference":
        reference_arm(args, w)
        return

    rank, local_rank, world = sharding.world_from_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode step has no CPU path")
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    if world > 1:
        sharding.init_process_group("nccl")
    import paper_1911_02150_b200 as mqa
    from paper_1911_02150_b200.build import build_library
    if rank == 0 or world == 1:
        build_library()
    sharding.barrier()
    mqa.lib()

    if args.sweep:
        run_sweep(mqa, args, device, rank)
        return
    if args.prefill_only:
        pb, ph, pn = (int(x) for x in args.prefill_only.split(","))
        print(json.dumps({"prefill": prefill_block(mqa, device, 0, pb, ph, pn)}))
        return
    if args.step_only:
        sb, sh, sm = (int(x) for x in args.step_only.split(","))
        w2 = wl.Workload(f"step_b{sb}_h{sh}_m{sm}", b=sb, h=sh, m_max=sm, lens="full")
        row = quick_point(mqa, "mqa", w2, device, steps=10, min_rotate_bytes=4 * L2_BYTES)
        row["kernel"] = mqa.plan_kernel_name(True, True, sb, sh, sm)
        print(json.dumps({"step": row}))
        return

    peak, peak_kind = measured_peak()
    seed = 1000 * rank                                  # every rank owns its own batch shard (weak scaling)
    st = StepState(mqa, "mqa", w, device, seed, min_rotate_bytes=8 * L2_BYTES)
    r = run_variant(st, args.steps, args.warmup, device, sample_clocks=True, use_graph=not args.no_graph)
    blk = result_block(st, r, args.steps)
    secs_max = sharding.max_over_ranks(r["secs"], device)
    e2e_max = sharding.max_over_ranks(r["e2e_s"], device)
    total_bytes = sharding.sum_over_ranks(st.bytes, device)
    value = total_bytes / (secs_max / args.steps) / 1e9
    e2e_value = total_bytes / (e2e_max / args.steps) / 1e9
    step_s = r["secs"] / args.steps
    one_launch = st.launches_per_step == 1
    # the dominant kernel: with one launch per step it IS the step, and its duration is the step's (K back-to-back
    # launches of that call, CUDA events); otherwise it is the pass over the cache, timed on its own below
    dom_s = step_s if one_launch else r["kernel_s"]
    dom_gbs = st.bytes / dom_s / 1e9
    pass_gbs = st.bytes / r["kernel_s"] / 1e9
    iso_gbs = st.bytes / r["isolated_s"] / 1e9
    step_kernel = mqa.plan_kernel_name(True, True, w.b, w.h, w.m_max)
    pass_kernel = mqa.plan_kernel_name(True, False, w.b, w.h, w.m_max)
    out = {
        "metric": "mqa_decode_step_hbm_gbs", "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": secs_max / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_name(w), "parallelism": f"batch shards x{world}, no collective",
                   "l2": f"rotating {len(st.sets)} cache sets of {st.cache_bytes >> 20} MiB (> L2) between steps",
                   "launch": "K steps replayed as one CUDA graph" if r["graph"] else "K steps launched from the host",
                   "step": "mqa_decode_append_step, MQA_STEP_CHAINED (a decoding loop: only steps write the cache)",
                   "value_is": "the back-to-back loop (each step's set-up overlaps the step before); roofline.isolated "
                               "is the same step after an unrelated kernel",
                   "n_splits": st.n_splits, "chunk_rows": st.chunk_rows},
        "us_per_step": blk["us_per_step"], "frac_of_8TBs": value / world / NOMINAL_HBM_GBS,
        "mqa": blk,
        "roofline": {"bound": "hbm", "achieved": dom_gbs, "peak": peak, "unit": "GB/s", "frac": dom_gbs / peak,
                     "frac_of_8TBs": dom_gbs / NOMINAL_HBM_GBS, "peak_kind": f"of {peak_kind}", "traffic": None,
                     "kernel": step_kernel if one_launch else pass_kernel,
                     "kernel_is": ("the step's one launch (append + pass over the cache + merge), back to back"
                                   if one_launch else "the pass over the cache, back to back (the step adds a second-pass kernel)"),
                     "kernel_us": dom_s * 1e6, "algorithmic_bytes": st.bytes,
                     "pass_only": {"kernel": pass_kernel, "kernel_us": r["kernel_s"] * 1e6, "achieved": pass_gbs,
                                   "frac": pass_gbs / peak, "frac_of_8TBs": pass_gbs / NOMINAL_HBM_GBS,
                                   "what": "mqa_decode_step_split back to back: no append, no merge"},
                     "isolated": {"kernel_us": r["isolated_s"] * 1e6, "achieved": iso_gbs, "frac": iso_gbs / peak,
                                  "frac_of_8TBs": iso_gbs / NOMINAL_HBM_GBS,
                                  "what": "the whole step launched from the host after an unrelated kernel, one CUDA-event "
                                          "pair per launch: nothing of it overlaps a step before"}},
        "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": st.h2d_bytes,
                "d2h_bytes_per_step": st.d2h_bytes, "us_per_step": e2e_max / args.steps * 1e6,
                "us_per_step_graph_replay": r["e2e_graph_s"] / args.steps * 1e6 if r.get("e2e_graph_s") else None,
                "note": ("mqa_decode_append_step_host, one call and one stream synchronisation per token: q, k_new, v_new "
                         "fetched from pinned host memory by a kernel, o stored to pinned host memory by the kernels; "
                         "us_per_step_graph_replay: the same call captured once per cache set and replayed; "
                         if st.host_steps is not None else
                         "per-step inputs q, k_new, v_new copied from pinned host memory, o copied back; ") +
                        "the KV cache is decoder state and stays resident in HBM"},
        "gpu_launches": st.launches_per_step * args.steps,
        "clocks": r["clocks"],
    }
    traffic = os.path.join(ROOT, "profiles", "traffic.txt")
    if os.path.exists(traffic):
        try:
            entry = json.load(open(traffic)).get(w.name, {})
            key = "mqa_step_dram_bytes" if one_launch else "mqa_split_dram_bytes"
            out["roofline"]["traffic"] = entry.get(key)
            out["roofline"]["traffic_source"] = entry.get(key.replace("_dram_bytes", "_source"), entry.get("source"))
        except Exception:
            pass
    del st
    torch.cuda.empty_cache()
    # (the layer step and the paper-shaped loop are latency-bound: timed before the multi-head block -- measured right
    # after its 4 GB of per-head caches streamed at 7 TB/s the same layer step reads 44-48 us instead of 40)
    if not args.no_layer:
        out["layer_step"] = layer_block(mqa, w, device, seed, max(3, min(args.steps, 20)))
        out["paper_incremental"] = paper_loop_block(mqa, device, seed)
        out["layer_step"]["projections_us"] = out["layer_step"]["us_per_step"] - blk["us_per_step"]
    # Order of the blocks: the multi-query points whose caches are below a gigabyte first, then the batched form, then the
    # points and the multi-head blocks that stream gigabytes for long: a short step timed right after one of those reads
    # 10-20 % slower (b=64 x m=4096: 28.6 us after them, 25.5 us before or alone), and so does the batched form (930 against
    # 1000 TFLOP/s).
    sweep_rows = {}
    by_size = sorted(LINE_SWEEP, key=lambda n_: wl.WORKLOADS[n_].b * wl.WORKLOADS[n_].m_max)      # smallest caches first
    small = [n_ for n_ in by_size if wl.WORKLOADS[n_].b * wl.WORKLOADS[n_].m_max * 512 <= (600 << 20)]
    if not args.no_layer and world == 1:
        out["beam4_rows"] = many_rows_block(mqa, device, seed, w)
    if not args.no_line_sweep and world == 1:
        for name in small:
            sweep_rows[(name, "mqa")] = quick_point(mqa, "mqa", wl.WORKLOADS[name], device)
    if not args.no_layer and world == 1:
        out["prefill"] = prefill_block(mqa, device, seed)
    if not args.no_line_sweep and world == 1:
        for name in by_size:
            if name not in small:
                sweep_rows[(name, "mqa")] = quick_point(mqa, "mqa", wl.WORKLOADS[name], device)
    if not args.no_mha:
        sth = StepState(mqa, "mha", w, device, seed, min_rotate_bytes=2 * L2_BYTES)
        rh = run_variant(sth, max(3, min(args.steps, 20)), 3, device, sample_clocks=False, use_graph=not args.no_graph)
        out["mha"] = result_block(sth, rh, max(3, min(args.steps, 20)))
        out["mha"]["roofline_frac"] = sth.bytes / rh["kernel_s"] / 1e9 / peak
        out["mqa_speedup_over_mha"] = out["mha"]["us_per_step"] / blk["us_per_step"]
        del sth
        torch.cuda.empty_cache()
    if not args.no_line_sweep and world == 1:
        # the other long-context points and the ragged batch: us, GB/s, fraction of 8 TB/s, launches, both variants
        for name in LINE_SWEEP:
            sweep_rows[(name, "mha")] = quick_point(mqa, "mha", wl.WORKLOADS[name], device)
        out["sweep"] = [sweep_rows[(name, variant)] for name in LINE_SWEEP for variant in ("mqa", "mha")]
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(w, seed)
    if rank == 0:
        print(json.dumps(out))


def run_sweep(mqa, args, device, rank):
    """Every workload, both variants: us per step and GB/s per point, written to args.sweep_out."""
    peak, peak_kind = measured_peak()
    rows = []
    for name, w in wl.WORKLOADS.items():
        if w.lens == "grow":
            continue
        for variant in ("mqa", "mha"):
            kvh = 1 if variant == "mqa" else w.h
            cache = 2 * w.b * kvh * w.m_max * 256
            if cache > 100 * 2 ** 30:
                rows.append({"workload": name, "variant": variant, "skipped": "cache exceeds 100 GiB"})
                continue
            free, _ = torch.cuda.mem_get_info(device)
            if cache + 6 * 2 ** 30 > free:
                rows.append({"workload": name, "variant": variant, "skipped": f"cache {cache >> 30} GiB does not fit"})
                continue
            st = StepState(mqa, variant, w, device, 0, min_rotate_bytes=4 * L2_BYTES)
            steps = 20 if cache < 8 * 2 ** 30 else 5
            r = run_variant(st, steps, 3, device, sample_clocks=False, use_graph=not args.no_graph)
            blk = result_block(st, r, steps)
            blk.update({"workload": name, "variant": variant, "b": w.b, "h": w.h, "m": w.m_max,
                        "frac_of_measured_copy": blk["gbs"] / peak})
            rows.append(blk)
            print(json.dumps(blk), file=sys.stderr)
            del st
            torch.cuda.empty_cache()
    out_dir = os.path.dirname(os.path.abspath(args.sweep_out))
    os.makedirs(out_dir, exist_ok=True)
    with open(args.sweep_out, "w") as f:
        json.dump({"peak_gbs": peak, "peak_kind": peak_kind, "rows": rows}, f, indent=1)
    if rank == 0:
        print(json.dumps({"sweep_points": len(rows), "written": args.sweep_out}))


if __name__ == "__main__":
    main()
