#!/usr/bin/env python
"""Benchmark of the StructKV prefill-time KV-compression hot path on B200.

One step = the whole hot path over one synthetic prompt: score every layer (window logits,
softmax column sums, entropy / sparsity / variance), detect the pivot, rebuild the centrality at
the pivot, select both budgets, compact K/V of every layer, gather hidden states and positions.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints one JSON line (rank 0).  With N > 1 every rank processes its own prompt (independent
problems, no collective on the data path): weak scaling.  Started without a launcher and with
--gpus N > 1, the script starts its N ranks itself.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

METRIC = "prompt tokens scored+compacted/sec at 128K ctx; % of roofline"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
SM_COUNT = 148
SFU_EXP_PER_CLK_PER_SM = 16      # special-function results per clock per SM (cc 10.0 arithmetic-throughput table)

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of the scorer launches of one layer,
# from an ncu capture of the current kernels; None = no capture of the current kernels exists.
NCU_TRAFFIC_BYTES_PER_LAYER = 549.0e6
NCU_TRAFFIC_NOTE = ("dram read + write of the two tc_score launches of one layer (llama128k shape), single-metric "
                    "ncu captures with the caches left as the previous kernel leaves them: pass 1 reads 269 MB, "
                    "pass 2 252 MB when the next layer's pass 1 ran in between (every layer but the last; 218 MB "
                    "otherwise: it starts with the tiles pass 1 asked L2 to keep), 28 + 1 MB written")


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.samples, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) == 6:
                self.samples.append(parts)

    def wait_for_samples(self, n: int, timeout_s: float = 3.0):
        t0 = time.perf_counter()
        while self.proc is not None and len(self.samples) < n and time.perf_counter() - t0 < timeout_s:
            time.sleep(0.02)

    def mark(self) -> int:
        return len(self.samples)

    def stop(self, first: int = 0):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm = self.samples[first:]
        mhz = [float(s[0]) for s in sm if s[0].replace(".", "").isdigit()]
        mx = [float(s[1]) for s in sm if s[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(s[2 + i] == "Active" for s in sm)]
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# ranks: independent prompts, no data-path collective
def rank_workload(wl, rank):
    """Each rank scores its own prompt: same recipe, rank-shifted seed."""
    import dataclasses
    return wl if rank == 0 else dataclasses.replace(wl, index=wl.index + 10 * rank)


def max_over_ranks(ms, device, world):
    """The step time of the job is the slowest rank's (device-timed) step time."""
    if world <= 1:
        return float(ms)
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_second(seq, world, ms_per_step):
    """Whole-job throughput: every rank processes one prompt of `seq` tokens per step."""
    return world * seq / (ms_per_step * 1e-3)


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def start_ranks(n, argv):
    """Started bare with --gpus N > 1: run the same command as N ranks of one node (one process per
    GPU, rendezvous on 127.0.0.1) and return the launcher's exit code."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


def plumbing_check(args):
    """The rank plumbing of the N > 1 path on host memory with gloo ranks (no scoring, nothing
    timed): per-rank prompts, the maximum over ranks, the job-level aggregation."""
    import torch.distributed as dist
    from paper_2604_06746_b200 import synth
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    wl = synth.WORKLOADS["tiny"]
    mine = rank_workload(wl, rank)
    q = synth.make_layer(mine, synth.plan(mine), 0, device="cpu", with_v=False)["q_win"]
    ms = max_over_ranks(10.0 + 5.0 * rank, "cpu", world)
    digests = [None] * world
    if world > 1:
        dist.all_gather_object(digests, (mine.index, float(q.double().sum())))
    else:
        digests = [(mine.index, float(q.double().sum()))]
    if rank == 0:
        print(json.dumps({"plumbing_check": True, "n_gpus": world, "ms_per_step": ms, "prompts": digests,
                          "value": job_tokens_per_second(wl.seq, world, ms)}))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# the step and its timing
def ev():
    return torch.cuda.Event(enable_timing=True)


class Resident:
    """A workload whose layers stay resident in HBM; one step = the whole path over them."""

    def __init__(self, wl, pl, kv_budget, dev, flags=0):
        from paper_2604_06746_b200 import pipeline, synth
        self.wl, self.kv_budget, self.st_budget = wl, kv_budget, wl.struct_budget(kv_budget)
        self.layers = [synth.make_layer(wl, pl, l, device=dev) for l in range(wl.n_layers)]
        self.hidden, self.positions = synth.make_hidden(wl, device=dev)
        # every layer's Q and K are resident and complete before any step starts (the steps are
        # bracketed by synchronisations), which is what STRUCTKV_FLAG_INPUTS_READY asks of the caller
        from paper_2604_06746_b200 import binding
        self.pf = pipeline.Prefill(wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq,
                                   kv_budget, self.st_budget, synth.torch_dtype(wl.dtype),
                                   hidden_dim=wl.hidden_dim, device=dev, flags=flags | binding.FLAG_INPUTS_READY)

    def step(self, timed):
        pf, layers = self.pf, self.layers
        e = [ev() for _ in range(4)] if timed else None
        if timed: e[0].record()
        pf.score_all(layers)                   # all layers resident: one call, passes of neighbouring layers interleaved
        pf.finish_scores(len(layers))          # Eq. 5-6 of all layers (batched): part of the scoring phase
        if timed: e[1].record()
        pf.detect_and_select(len(layers))
        if timed: e[2].record()
        pf.compact_all_kv(layers)
        pf.compact_hidden(self.hidden, self.positions)
        if timed: e[3].record()
        return e


def time_resident(res, steps, warmup, min_seconds, barrier, sampler=None):
    """W warm-up steps, then K x R steps in one timed region of at least `min_seconds`.
    Returns total ms, steps timed, R, the per-phase ms sums (CUDA events on the launching stream)
    and the index of the first clock sample that belongs to the timed region."""
    for _ in range(warmup):
        res.step(False)
    barrier()
    t0, t1 = ev(), ev()
    t0.record()
    res.step(False)
    t1.record()
    torch.cuda.synchronize()
    est_ms = max(t0.elapsed_time(t1), 1e-3)
    repeats = max(1, int(math.ceil(min_seconds * 1e3 / (steps * est_ms))))
    barrier()
    first = 0
    if sampler is not None:
        sampler.wait_for_samples(1)
        first = sampler.mark()
    start, stop = ev(), ev()
    start.record()
    events = [res.step(True) for _ in range(steps * repeats)]
    stop.record()
    barrier()
    ms = start.elapsed_time(stop)
    phase = {"score": 0.0, "pivot_select": 0.0, "compact": 0.0}
    for e in events:
        phase["score"] += e[0].elapsed_time(e[1])
        phase["pivot_select"] += e[1].elapsed_time(e[2])
        phase["compact"] += e[2].elapsed_time(e[3])
    return ms, steps * repeats, repeats, phase, first


def time_streamed(wl, pl, kv_budget, dev, sweeps=2):
    """The streamed protocol of the 256K workload: one layer's K/V resident at a time.  Every
    layer is generated outside the timed region, its scoring (and, in a second sweep, its
    compaction) is timed alone with CUDA events, and the per-layer times are summed."""
    from paper_2604_06746_b200 import pipeline, synth
    st_budget = wl.struct_budget(kv_budget)
    hidden, positions = synth.make_hidden(wl, device=dev)
    pf = pipeline.Prefill(wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, kv_budget,
                          st_budget, torch.bfloat16, hidden_dim=wl.hidden_dim, device=dev, keep_kv=False)
    tot = {"score": 0.0, "pivot_select": 0.0, "compact": 0.0}
    for sweep in range(sweeps + 1):                  # sweep 0 warms up
        acc = {"score": 0.0, "pivot_select": 0.0, "compact": 0.0}
        for l in range(wl.n_layers):
            t = synth.make_layer(wl, pl, l, device=dev, with_v=False)
            pf.score(l, t["q_win"], t["k"], t["scale"])      # untimed first touch of the fresh tensors
            torch.cuda.synchronize()
            a, b = ev(), ev()
            a.record()
            pf.score(l, t["q_win"], t["k"], t["scale"])
            b.record()
            torch.cuda.synchronize()
            acc["score"] += a.elapsed_time(b)
            del t
        a, b = ev(), ev()
        a.record()
        pf.finish_scores(wl.n_layers)
        b.record()
        torch.cuda.synchronize()
        acc["score"] += a.elapsed_time(b)
        a, b = ev(), ev()
        a.record()
        pf.detect_and_select(wl.n_layers)
        b.record()
        torch.cuda.synchronize()
        acc["pivot_select"] += a.elapsed_time(b)
        for l in range(wl.n_layers):
            t = synth.make_layer(wl, pl, l, device=dev)
            torch.cuda.synchronize()
            a, b = ev(), ev()
            a.record()
            pf.compact_kv(l, t["k"], t["v"], t["kv"])
            b.record()
            torch.cuda.synchronize()
            acc["compact"] += a.elapsed_time(b)
            del t
        a, b = ev(), ev()
        a.record()
        pf.compact_hidden(hidden, positions)
        b.record()
        torch.cuda.synchronize()
        acc["compact"] += a.elapsed_time(b)
        if sweep > 0:
            for k in tot:
                tot[k] += acc[k] / sweeps
    return pf, tot


def batch_timing(dev, reps=10):
    """One layer of Llama-3-8B-shaped scoring for a batch of four prompts of different lengths (131072
    tokens together), as ONE structkv_score_layer_batch call against four structkv_score_layer calls."""
    from paper_2604_06746_b200 import binding
    H, Hkv, d, w = 32, 8, 128, 64
    lens = (40000, 20000, 50000, 21072)
    cu = [0]
    for n in lens:
        cu.append(cu[-1] + n)
    total, B = cu[-1], len(lens)
    g = torch.Generator(device=dev)
    g.manual_seed(123)
    q = torch.randn((B, H, w, d), generator=g, device=dev).to(torch.bfloat16)
    k = torch.randn((Hkv, total, d), generator=g, device=dev).to(torch.bfloat16)
    ctx = binding.Context(H, Hkv, d, w, max(lens), torch.bfloat16, dev)
    ws = ctx.batch_workspace(B, total)
    s = torch.zeros(total, dtype=torch.float32, device=dev)
    m = torch.zeros((B, 3), dtype=torch.float32, device=dev)
    scale = 1.0 / math.sqrt(d)

    def batched():
        ctx.score_layer_batch(q, k, cu, scale, s, m, ws)

    def separate():
        for b in range(B):
            ctx.score_layer(q[b], k[:, cu[b]:cu[b + 1]], scale, s[cu[b]:cu[b + 1]], m[b])

    out = {}
    for name, fn in (("one_batched_call_us", batched), ("four_separate_calls_us", separate)):
        fn()
        torch.cuda.synchronize()
        a, b_ = ev(), ev()
        a.record()
        for _ in range(reps):
            fn()
        b_.record()
        torch.cuda.synchronize()
        out[name] = a.elapsed_time(b_) * 1e3 / reps
    out["prompt_lengths"] = list(lens)
    assert ctx.poll_device_status() == binding.OK
    ctx.close()
    return out


def scorer_roofline(wl, score_ms_per_step, peaks, sm_mhz):
    """Roofline of one structkv_score_layer call: one contraction, K read once."""
    L, R = wl.n_layers, wl.n_q_heads * wl.window
    esz = 2 if wl.dtype == "bf16" else 4
    score_s = score_ms_per_step * 1e-3 / L
    k_bytes = wl.n_kv_heads * wl.seq * wl.head_dim * esz
    flops = 2.0 * R * wl.seq * wl.head_dim
    t_hbm, t_tensor = k_bytes / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12)
    if t_hbm >= t_tensor:
        roof = {"bound": "hbm", "achieved": k_bytes / score_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        roof = {"bound": "tensor", "achieved": flops / score_s / 1e12, "peak": peaks["bf16_tflops"],
                "unit": "TFLOP/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["us_per_layer"] = score_s * 1e6
    roof["roofline_us_per_layer"] = max(t_hbm, t_tensor) * 1e6
    # the exponential unit's floor: one exponential per logit (the method's own count; the two-pass
    # kernel evaluates two), 16 per clock per SM, at the SM clock sampled during the run
    mhz = sm_mhz or 1965.0
    alu_us = R * wl.seq / (SM_COUNT * SFU_EXP_PER_CLK_PER_SM * mhz * 1e6) * 1e6
    roof["alu_ceiling"] = {"us_per_layer_one_exp_per_logit": alu_us, "us_per_layer_two_pass": 2 * alu_us,
                           "sm_mhz": mhz, "exp_per_clk_per_sm": SFU_EXP_PER_CLK_PER_SM,
                           "frac_of_one_exp_floor": alu_us / (score_s * 1e6),
                           "frac_of_two_pass_floor": 2 * alu_us / (score_s * 1e6),
                           "roofline_frac_at_two_pass_floor": roof["roofline_us_per_layer"] / (2 * alu_us)}
    return roof


def compaction_figures(wl, kv_budget, compact_ms_per_step, peaks):
    esz = 2 if wl.dtype == "bf16" else 4
    st_budget = wl.struct_budget(kv_budget)
    nbytes = wl.n_layers * 2 * 2 * wl.n_kv_heads * kv_budget * wl.head_dim * esz + 2 * st_budget * wl.hidden_dim * 2
    s = compact_ms_per_step * 1e-3
    return {"achieved": nbytes / s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": nbytes / s / 1e9 / peaks["hbm_gbs"], "bytes_per_step": nbytes}


def launches_per_step(wl, flags):
    from paper_2604_06746_b200 import binding
    # layer by layer: scorer pass 1, pass 2, column reduce + metrics (the CUDA-core scorer adds a row
    # finalisation); per step: batched head statistics (2), accumulate, 2 selections, one K/V gather
    # over all layers, hidden states, positions
    stats = 0 if (flags & binding.FLAG_NO_HEAD_STATS) else 2
    if wl.dtype == "bf16" and not (flags & (binding.FLAG_NO_HEAD_STATS | binding.FLAG_FORCE_SIMT)):
        scoring = 2 * wl.n_layers + 1          # one structkv_score_layers call: two passes per layer, one reduce over heads
    else:
        scoring = wl.n_layers * (3 if wl.dtype == "bf16" else 4)
    return scoring + stats + 1 + 2 + 1 + 2


# ------------------------------------------------------------------------------------------------
# the oracle beside it
def cpu_baseline_and_parity(wl, res, lam, weights):
    """The oracle, as it stands, over ALL layers of the workload the GPU just processed (its layers
    scored side by side in worker processes, then its own pivot / centrality / selection), timed on
    the host cores; and the parity of the timed GPU run with it."""
    from oracle import structkv_oracle as O
    from tests import oracle_pool as OP
    from tests import parity as P
    try:
        cores = len(os.sched_getaffinity(0))
    except AttributeError:
        cores = os.cpu_count()
    k64 = wl.n_kv_heads * wl.seq * wl.head_dim * 8
    workers = OP.default_workers(1.6 * k64 + 8 * wl.window * wl.seq * 8 + 3 * wl.n_q_heads * wl.seq * 8)
    host = [(l, OP.bits_of(t["q_win"]), OP.bits_of(t["k"]), t["scale"], None) for l, t in enumerate(res.layers)]
    kv0 = res.layers[0]["kv"]
    kv0_bits = kv0.view(2 * kv0.shape[1], kv0.shape[2], kv0.shape[3]).view(torch.int16).cpu().numpy()
    t0 = time.perf_counter()
    s_hist, metrics = OP.score_layers(iter(host), wl.n_layers, workers)
    t_score = time.perf_counter() - t0
    o = OP.assemble(s_hist, metrics, wl.window, (res.kv_budget,), (res.st_budget,), lam, weights)
    t_select = time.perf_counter() - t0 - t_score
    t1 = time.perf_counter()
    O.compact(kv0_bits, o["i_kv"][res.kv_budget][0])
    t_compact = (time.perf_counter() - t1) * wl.n_layers
    total = t_score + t_select + t_compact
    base = {"value": wl.seq / total, "unit": UNIT, "cores": min(cores, workers), "kind": "oracle",
            "sample": f"all {wl.n_layers} layers of {wl.name}: scoring in {workers} worker processes "
                      f"({t_score:.1f} s), pivot + centrality + both selections ({t_select:.1f} s), K/V compaction "
                      f"timed on layer 0 and scaled to all layers ({t_compact:.1f} s)"}
    pf = res.pf
    par = {"pivot_gpu": pf.pivot, "pivot_oracle": int(o["pivot"]), "pivot_match": pf.pivot == int(o["pivot"])}

    def passes(fn, *a):
        try:
            fn(*a)
            return True
        except AssertionError:
            return False
    g_s = pf.s_hist.cpu().numpy()
    par["s_hist_within_2e-3"] = all(passes(P.assert_scores_close, g_s[l], s_hist[l]) for l in range(wl.n_layers))
    par["metrics_within_2e-3"] = bool(np.all(np.abs(pf.metrics.cpu().numpy() - metrics) <= P.REL_TOL * np.abs(metrics)))
    par["c_star_within_2e-3"] = passes(P.assert_scores_close, pf.c_star.cpu().numpy(), o["C"])
    par["i_struct_match"] = passes(P.assert_selection_matches, pf.i_struct.cpu().numpy(), o["C"], res.st_budget,
                                   wl.window, o["i_struct"][res.st_budget])
    i_kv = pf.i_kv.cpu().numpy()
    par["i_kv_match_all_layers"] = all(
        passes(P.assert_selection_matches, i_kv[l], s_hist[l], res.kv_budget, wl.window,
               o["i_kv"][res.kv_budget][l]) for l in range(wl.n_layers))
    got = pf.kv_out[0].view(2 * wl.n_kv_heads, res.kv_budget, wl.head_dim).view(torch.int16).cpu().numpy()
    par["kv_layer0_bit_exact"] = bool(np.array_equal(got, O.compact(kv0_bits, i_kv[0])))
    par["rules"] = "2e-3 relative on S, C*, metrics; selection under the gap rule; gathers bit for bit"
    return base, par


def cpu_baseline_sample(wl, pl, kv_budget, n_layers_sample=1, first_layer=0):
    """The oracle on a bounded sample (single process): scoring + selection + compaction of some
    layer(s) of the workload, scaled to all layers.  Used by the reference arm."""
    from oracle import structkv_oracle as O
    from paper_2604_06746_b200 import synth
    try:
        cores = len(os.sched_getaffinity(0))
    except AttributeError:
        cores = os.cpu_count()
    t_total = 0.0
    for l in range(first_layer, first_layer + n_layers_sample):
        t = synth.make_layer(wl, pl, l % wl.n_layers, device="cpu")
        q, k, v = synth.to_f64(t["q_win"]), synth.to_f64(t["k"]), t["v"].view(torch.int16).numpy()
        kb = t["k"].view(torch.int16).numpy()
        t0 = time.perf_counter()
        out = O.score_layer(q, k, t["scale"])
        idx = O.select(out["S"], kv_budget, wl.window)
        O.compact(kb, idx)
        O.compact(v, idx)
        t_total += time.perf_counter() - t0
    per_layer = t_total / n_layers_sample
    return {"value": wl.seq / (per_layer * wl.n_layers), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n_layers_sample} of {wl.n_layers} layers of {wl.name} (score + select + compact of "
                      f"K/V), {per_layer:.2f} s per layer, scaled to all layers"}


# ------------------------------------------------------------------------------------------------
# end to end with host buffers
def measure_e2e(res, dev, steps, world):
    """The same step with HOST buffers: every step copies each layer's q / K / V, the hidden states
    and the position ids from pinned host memory to the device, runs the path through the C ABI,
    and copies the results (compacted K / V, gathered hidden states and positions, both index sets,
    the metric table) back to pinned host memory.  Copies run on their own streams: layer l + 1
    is copied in while layer l is scored, and results are copied out while the next step's inputs
    arrive; all of it is inside the timed region."""
    wl, pf, layers, hidden, positions = res.wl, res.pf, res.layers, res.hidden, res.positions
    host_layers = []
    layer_bytes = sum(layers[0][k].numel() * layers[0][k].element_size() for k in ("q_win", "kv"))
    try:
        import psutil
        host_total = psutil.virtual_memory().total
    except Exception:
        host_total = 64 << 30
    local_world = int(os.environ.get("LOCAL_WORLD_SIZE", str(world)))
    # pinned host memory is shared by the ranks of the node: stay within half of it.  With fewer
    # host buffers than layers, layer l is copied from buffer l mod k (same bytes, same copies).
    k_host = max(1, min(len(layers), int(0.5 * host_total / max(1, local_world) / layer_bytes)))
    try:
        for t in layers[:k_host]:
            host_layers.append({k: torch.empty(t[k].shape, dtype=t[k].dtype, pin_memory=True).copy_(t[k])
                                for k in ("q_win", "kv")})
        host_hidden = torch.empty(hidden.shape, dtype=hidden.dtype, pin_memory=True).copy_(hidden)
        host_pos = torch.empty(positions.shape, dtype=positions.dtype, pin_memory=True).copy_(positions)
        outs = {"kv_out": pf.kv_out, "hidden_out": pf.hidden_out, "pos_out": pf.pos_out,
                "i_kv": pf.i_kv, "i_struct": pf.i_struct, "metrics": pf.metrics}
        host_out = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True) for k, v in outs.items()}
    except RuntimeError as e:
        return {"value": None, "unit": UNIT, "unavailable": f"pinned host allocation failed: {e}"[:200]}
    h2d = layer_bytes * len(layers) \
        + host_hidden.numel() * host_hidden.element_size() + host_pos.numel() * host_pos.element_size()
    d2h = sum(v.numel() * v.element_size() for v in host_out.values())
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    arrived = [torch.cuda.Event() for _ in range(len(layers) + 1)]
    state = {"consumed": None, "copied_out": None}

    def step():
        with torch.cuda.stream(s_in):
            if state["consumed"] is not None:
                s_in.wait_event(state["consumed"])         # the previous step no longer reads the inputs
            for l, t in enumerate(layers):
                hd = host_layers[l % k_host]
                for k in ("q_win", "kv"):
                    t[k].copy_(hd[k], non_blocking=True)
                arrived[l].record(s_in)
            hidden.copy_(host_hidden, non_blocking=True)
            positions.copy_(host_pos, non_blocking=True)
            arrived[len(layers)].record(s_in)
        if state["copied_out"] is not None:
            main.wait_event(state["copied_out"])           # the previous results have left the device
        for l, t in enumerate(layers):
            main.wait_event(arrived[l])
            pf.score(l, t["q_win"], t["k"], t["scale"])
        pf.detect_and_select(len(layers))
        pf.compact_all_kv(layers)
        main.wait_event(arrived[len(layers)])
        pf.compact_hidden(hidden, positions)
        done = torch.cuda.Event()
        done.record(main)
        state["consumed"] = done
        with torch.cuda.stream(s_out):
            s_out.wait_event(done)
            for k, v in outs.items():
                host_out[k].copy_(v, non_blocking=True)
            out_ev = torch.cuda.Event()
            out_ev.record(s_out)
        state["copied_out"] = out_ev

    step()
    torch.cuda.synchronize()
    e0, e1 = ev(), ev()
    e0.record()
    for _ in range(steps):
        step()
    main.wait_event(state["copied_out"])                   # the last results are on the host
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    ms = max_over_ranks(ms, dev, world)
    return {"value": job_tokens_per_second(wl.seq, world, ms), "unit": UNIT, "ms_per_step": ms, "steps": steps,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "h2d_gb_per_s": h2d / (ms * 1e-3) / 1e9,
            "note": "inputs in pinned host memory, copied every step on a copy stream (layer l + 1 arrives "
                    "while layer l is scored); results copied back to pinned host memory on a third stream"
                    + ("" if k_host == len(layers) else f"; host buffers for {k_host} of {len(layers)} layers "
                       "(layer l is copied from buffer l mod k: half of the host memory is shared by the ranks)")}


# ------------------------------------------------------------------------------------------------
def run_reference(args):
    """The reference arm is the CPU oracle (the paper ships no code)."""
    from paper_2604_06746_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = synth.WORKLOADS[args.workload]
    pl = synth.plan(wl)
    kv_budget = args.budget or wl.budget
    for _ in range(min(args.warmup, 1)):
        cpu_baseline_sample(wl.scaled(4096, n_layers=1), synth.plan(wl.scaled(4096, n_layers=1)), 256)
    t0 = time.perf_counter()
    samples = [cpu_baseline_sample(wl, pl, kv_budget, n_layers_sample=1, first_layer=i)
               for i in range(max(1, args.steps))]
    dt = time.perf_counter() - t0
    value = len(samples) / sum(1.0 / b["value"] for b in samples)      # steps / total scaled time
    base = dict(samples[0], value=value,
                sample=f"each of the {len(samples)} steps scores, selects and compacts one layer of {wl.name} "
                       f"(layers 0..{len(samples) - 1}) and is scaled to all {wl.n_layers} layers")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * wl.seq / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(wl, kv_budget),
            "cpu_baseline": base | {"wall_s": dt},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def workload_config(wl, kv_budget):
    esz = 2 if wl.dtype == "bf16" else 4
    return {"workload": f"{wl.name}: {wl.n_layers} layers, {wl.n_q_heads} q heads / {wl.n_kv_heads} KV heads, "
                        f"head_dim {wl.head_dim}, seq {wl.seq}, window {wl.window}",
            "kv_budget": kv_budget, "struct_budget": wl.struct_budget(kv_budget),
            "lambda": 0.9, "weights": [0.2, 0.3, 0.5],
            "scoring": "all resident layers in one structkv_score_layers call (layer by layer where the "
                       "CUDA-core scorer serves the shape)",
            "l2": "inputs larger than L2 (each layer's K is %.0f MB and no layer is touched twice in a step; a "
                  "step touches %.1f GB of distinct K/V)" % (wl.n_kv_heads * wl.seq * wl.head_dim * esz / 1e6,
                                                           wl.n_layers * 2 * wl.n_kv_heads * wl.seq * wl.head_dim * esz / 1e9)}


def other_configs(dev, peaks, sm_mhz, min_seconds, skip):
    """Throughput, phases and roofline fractions of the other workloads (and of the other budgets of
    the headline workload), each timed like the headline.  The 256K workload is streamed."""
    from paper_2604_06746_b200 import synth
    out = {}
    plan = [("tiny", None), ("llama32k", None), ("llama128k", 1024), ("llama128k", 4096), ("llama128k", 16384),
            ("qwen64k", None), ("llama256k", None)]
    for name, budget in plan:
        wl = synth.WORKLOADS[name]
        kv_budget = budget or wl.budget
        key = f"{name}/B{kv_budget}"
        if key == skip:
            continue
        pl = synth.plan(wl)
        if wl.streamed:
            pf, phase = time_streamed(wl, pl, kv_budget, dev)
            ms_step, steps = sum(phase.values()), 2
            mode = "streamed: layers timed one at a time and summed"
        else:
            res = Resident(wl, pl, kv_budget, dev)
            ms, steps, _, phase_tot, _ = time_resident(res, 5, 3, min_seconds, torch.cuda.synchronize)
            ms_step = ms / steps
            phase = {k: v / steps for k, v in phase_tot.items()}
            pf = res.pf
            mode = "resident"
        entry = {"tokens_per_s": wl.seq / (ms_step * 1e-3), "ms_per_step": ms_step, "steps": steps, "mode": mode,
                 "phase_ms_per_step": phase, "pivot": pf.pivot, "dtype": wl.dtype,
                 "compaction_frac": compaction_figures(wl, kv_budget, phase["compact"], peaks)["frac"]}
        if wl.dtype == "bf16":
            r = scorer_roofline(wl, phase["score"], peaks, sm_mhz)
            entry["scorer"] = {k: r[k] for k in ("bound", "frac", "us_per_layer", "roofline_us_per_layer")}
            entry["scorer"]["frac_of_two_pass_exp_floor"] = r["alu_ceiling"]["frac_of_two_pass_floor"]
        out[key] = entry
        del pf
        if not wl.streamed:
            del res
        torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama128k")
    ap.add_argument("--budget", type=int, default=0, help="KV budget (0 = the workload's largest)")
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="the timed region repeats the K steps until it lasts at least this long")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the table of the other workloads")
    ap.add_argument("--flags", type=int, default=0)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="profile a prefix of the layers (0 = all)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--plumbing-check", action="store_true",
                    help="only exercise the multi-rank plumbing, on host memory with gloo ranks")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(start_ranks(args.gpus, sys.argv[1:]))
    if args.plumbing_check:
        return plumbing_check(args)
    if args.impl == "reference":
        return run_reference(args)

    from paper_2604_06746_b200 import binding, synth

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (no CPU fallback exists)"
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))

    wl = synth.WORKLOADS[args.workload]
    if args.layers:
        wl = wl.scaled(wl.seq, n_layers=args.layers, name=f"{wl.name}[first {args.layers} layers]",
                       budgets=wl.budgets)
    pl = synth.plan(wl)
    kv_budget = args.budget or wl.budget
    peaks = load_peaks()

    # every rank draws its own prompt (same recipe, rank-shifted seed) and keeps it resident
    res = Resident(rank_workload(wl, rank), pl, kv_budget, dev, flags=args.flags)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    warmup = max(args.warmup, 3)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
    ms, n_timed, repeats, phase_ms, first_sample = time_resident(res, args.steps, warmup, args.min_seconds,
                                                                 barrier, sampler)
    clocks = sampler.stop(first_sample) if sampler else None
    assert res.pf.ctx.poll_device_status() == binding.OK
    ms = max_over_ranks(ms, dev, world)
    pf = res.pf

    # rows beyond the core path (block-level aggregation for paged KV, attention-mass recovery)
    bs = 16
    blk = torch.zeros(((wl.seq + bs - 1) // bs,), dtype=torch.float32, device=dev)
    rec = torch.zeros((wl.n_layers,), dtype=torch.float32, device=dev)
    ex = [ev() for _ in range(3)]
    pf.ctx.block_scores(pf.c_star, bs, blk)
    pf.ctx.mass_recovery(pf.s_hist, pf.i_struct, rec)
    torch.cuda.synchronize()
    reps = 200                       # short kernels: enough launches queued that the host stays ahead
    ex[0].record()
    for it in range(reps):
        pf.ctx.block_scores(pf.c_star, bs, blk)
    ex[1].record()
    for it in range(reps):
        pf.ctx.mass_recovery(pf.s_hist, pf.i_struct, rec)
    ex[2].record()
    torch.cuda.synchronize()
    next_rows = {"block_scores_us": ex[0].elapsed_time(ex[1]) * 1e3 / reps, "block_size": bs,
                 "mass_recovery_us": ex[1].elapsed_time(ex[2]) * 1e3 / reps,
                 "note": "back-to-back launches from Python; a floor of a few us per call is host launch cost",
                 "mass_recovery_of_i_struct_min_over_layers": float(rec.min().item())}
    if wl.dtype == "bf16" and rank == 0:
        next_rows["batched_prompts_one_layer"] = batch_timing(dev)
    pivot_timed = pf.pivot
    e2e = None if args.no_e2e else measure_e2e(res, dev, args.e2e_steps, world)
    assert pf.ctx.poll_device_status() == binding.OK
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_per_step = ms / n_timed
    value = job_tokens_per_second(wl.seq, world, ms_per_step)
    sm_mhz = clocks["sm_mhz"] if clocks else None
    roof = scorer_roofline(wl, phase_ms["score"] / n_timed, peaks, sm_mhz)
    roof["traffic"] = NCU_TRAFFIC_BYTES_PER_LAYER if wl.name.startswith("llama128k") else None
    roof["traffic_note"] = NCU_TRAFFIC_NOTE
    roof["kernel"] = "structkv_score_layer (both scorer passes + reductions), per layer"
    roof["peaks"] = peaks["source"]
    if sm_mhz:
        roof["us_per_layer_x_sm_mhz"] = roof["us_per_layer"] * sm_mhz
    compaction = compaction_figures(wl, kv_budget, phase_ms["compact"] / n_timed, peaks)

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32",
            "data": "synthetic", "config": workload_config(wl, kv_budget), "pivot": pivot_timed,
            "timed_region": {"seconds": ms * 1e-3, "steps_timed": n_timed, "inner_repeats": repeats,
                             "ms_per_step_x_sm_mhz": ms_per_step * sm_mhz if sm_mhz else None},
            "phase_ms_per_step": {k: v / n_timed for k, v in phase_ms.items()},
            "roofline": roof, "compaction": compaction, "clocks": clocks,
            "gpu_launches": launches_per_step(wl, args.flags) * n_timed, "e2e": e2e, "next_rows": next_rows}
    if not args.no_cpu_baseline:
        # the oracle over the very prompt the timed steps processed, and the parity of that run
        res.step(False)
        torch.cuda.synchronize()
        line["cpu_baseline"], line["parity_of_timed_run"] = cpu_baseline_and_parity(wl, res, pf.lam, pf.weights)
    if world == 1 and not args.no_configs and not args.layers:
        del res, pf
        torch.cuda.empty_cache()
        line["configs"] = other_configs(dev, peaks, sm_mhz, min(args.min_seconds, 1.0), f"{wl.name}/B{kv_budget}")
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
