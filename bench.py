#!/usr/bin/env python
"""Benchmark of the StructKV prefill-time KV-compression hot path on B200.

One step = the whole hot path over one synthetic prompt: score every layer (window logits,
softmax column sums, entropy / sparsity / variance), detect the pivot, rebuild the centrality at
the pivot, select both budgets, compact K/V of every layer, gather hidden states and positions.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints one JSON line (rank 0).  With N > 1 (torchrun) every rank processes its own prompt
(independent problems, no collective on the data path): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
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

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant
# kernel, from the ncu capture summarised under profiles/; None until a capture exists.
NCU_TRAFFIC_BYTES_PER_LAUNCH = 557.0e6
NCU_TRAFFIC_NOTE = ("dram read+write of the two tc_score launches of one layer (llama128k shape), "
                    "profiles/tc_score_llama128k_ncu_full.md; valid for the llama128k workload only")


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

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        mhz = [float(s[0]) for s in self.samples if s[0].replace(".", "").isdigit()]
        mx = [float(s[1]) for s in self.samples if s[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(s[2 + i] == "Active" for s in self.samples)]
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(self.samples)}


def rank_workload(wl, rank):
    """Each rank scores its own prompt: same recipe, rank-shifted seed (independent problems, no
    collective on the data path)."""
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


def cpu_baseline(wl, pl, kv_budget, n_layers_sample=1, first_layer=0):
    """The oracle, as it stands, on a bounded sample: scoring + selection + compaction of the
    first layer(s) of the same workload, scaled to all layers."""
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


def measure_e2e(wl, pf, layers, hidden, positions, dev, steps, world):
    """The same step with HOST buffers: every step copies each layer's q / K / V, the hidden states
    and the position ids from pinned host memory to the device, runs the path through the C ABI,
    and copies the results (compacted K / V, gathered hidden states and positions, both index sets,
    the metric table) back to pinned host memory.  One stream, copies inside the timed region."""
    host_layers = []
    # pinned host memory is shared by the ranks of the node: stay within half of it.  With fewer
    # host buffers than layers, layer l is copied from buffer l mod k (same bytes, same copies).
    layer_bytes = sum(layers[0][k].numel() * layers[0][k].element_size() for k in ("q_win", "kv"))
    try:
        import psutil
        host_total = psutil.virtual_memory().total
    except Exception:
        host_total = 64 << 30
    local_world = int(os.environ.get("LOCAL_WORLD_SIZE", str(world)))
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

    def step():
        for l, t in enumerate(layers):
            hd = host_layers[l % k_host]
            for k in ("q_win", "kv"):
                t[k].copy_(hd[k], non_blocking=True)
            pf.score(l, t["q_win"], t["k"], t["scale"])
        hidden.copy_(host_hidden, non_blocking=True)
        positions.copy_(host_pos, non_blocking=True)
        pf.detect_and_select(len(layers))
        for l, t in enumerate(layers):
            pf.compact_kv(l, t["k"], t["v"], t.get("kv"))
        pf.compact_hidden(hidden, positions)
        for k, v in outs.items():
            host_out[k].copy_(v, non_blocking=True)

    step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    ms = max_over_ranks(ms, dev, world)
    return {"value": job_tokens_per_second(wl.seq, world, ms), "unit": UNIT, "ms_per_step": ms, "steps": steps,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "note": "inputs in pinned host memory, copied every step; results copied back to pinned host memory"
                    + ("" if k_host == len(layers) else f"; host buffers for {k_host} of {len(layers)} layers "
                       "(layer l is copied from buffer l mod k: half of the host memory is shared by the ranks)")}


def run_reference(args):
    """The reference arm of this build is the CPU oracle (the paper ships no code)."""
    from paper_2604_06746_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = synth.WORKLOADS[args.workload]
    pl = synth.plan(wl)
    kv_budget = args.budget or wl.budget
    for _ in range(min(args.warmup, 1)):
        cpu_baseline(wl.scaled(4096, n_layers=1), synth.plan(wl.scaled(4096, n_layers=1)), 256)
    t0 = time.perf_counter()
    samples = [cpu_baseline(wl, pl, kv_budget, n_layers_sample=1, first_layer=i) for i in range(max(1, args.steps))]
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
    return {"workload": f"{wl.name}: {wl.n_layers} layers, {wl.n_q_heads} q heads / {wl.n_kv_heads} KV heads, "
                        f"head_dim {wl.head_dim}, seq {wl.seq}, window {wl.window}",
            "kv_budget": kv_budget, "struct_budget": wl.struct_budget(kv_budget),
            "lambda": 0.9, "weights": [0.2, 0.3, 0.5],
            "l2": "inputs larger than L2 (each layer's K is %.0f MB, read once per step)" %
                  (wl.n_kv_heads * wl.seq * wl.head_dim * 2 / 1e6)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama128k")
    ap.add_argument("--budget", type=int, default=0, help="KV budget (0 = the workload's largest)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--flags", type=int, default=0)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="profile a prefix of the layers (0 = all)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

    from paper_2604_06746_b200 import binding, pipeline, synth

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
    st_budget = wl.struct_budget(kv_budget)
    peaks = load_peaks()

    # every rank draws its own prompt (same recipe, rank-shifted seed) and keeps it resident
    wl_rank = rank_workload(wl, rank)
    layers = [synth.make_layer(wl_rank, pl, l, device=dev) for l in range(wl.n_layers)]
    hidden, positions = synth.make_hidden(wl_rank, device=dev)
    pf = pipeline.Prefill(wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq,
                          kv_budget, st_budget, synth.torch_dtype(wl.dtype), hidden_dim=wl.hidden_dim,
                          device=dev, flags=args.flags)

    ev = lambda: torch.cuda.Event(enable_timing=True)
    phase_ms = {"score": 0.0, "pivot_select": 0.0, "compact": 0.0}

    def step(timed: bool):
        e = [ev() for _ in range(4)] if timed else None
        if timed: e[0].record()
        for l, t in enumerate(layers):
            pf.score(l, t["q_win"], t["k"], t["scale"])
        if timed: e[1].record()
        pf.detect_and_select(len(layers))
        if timed: e[2].record()
        for l, t in enumerate(layers):
            pf.compact_kv(l, t["k"], t["v"], t.get("kv"))
        pf.compact_hidden(hidden, positions)
        if timed: e[3].record()
        return e

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step(False)
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    start, stop = ev(), ev()
    start.record()
    events = [step(True) for _ in range(args.steps)]
    stop.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms = start.elapsed_time(stop)
    for e in events:
        phase_ms["score"] += e[0].elapsed_time(e[1])
        phase_ms["pivot_select"] += e[1].elapsed_time(e[2])
        phase_ms["compact"] += e[2].elapsed_time(e[3])
    assert pf.ctx.poll_device_status() == binding.OK
    ms = max_over_ranks(ms, dev, world)
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
    e2e = None if args.no_e2e else measure_e2e(wl, pf, layers, hidden, positions, dev, args.e2e_steps, world)
    assert pf.ctx.poll_device_status() == binding.OK
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_per_step = ms / args.steps
    value = job_tokens_per_second(wl.seq, world, ms_per_step)

    # roofline of the dominant kernel (the fused scorer): one contraction, K read once
    L, R = wl.n_layers, wl.n_q_heads * wl.window
    score_s = phase_ms["score"] * 1e-3 / (args.steps * L)                 # per layer (one launch group)
    k_bytes = wl.n_kv_heads * wl.seq * wl.head_dim * 2
    flops = 2.0 * R * wl.seq * wl.head_dim
    t_hbm, t_tensor = k_bytes / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12)
    if t_hbm >= t_tensor:
        roof = {"bound": "hbm", "achieved": k_bytes / score_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        roof = {"bound": "tensor", "achieved": flops / score_s / 1e12, "peak": peaks["bf16_tflops"],
                "unit": "TFLOP/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = NCU_TRAFFIC_BYTES_PER_LAUNCH if wl.name.startswith("llama128k") else None
    roof["traffic_note"] = NCU_TRAFFIC_NOTE
    roof["kernel"] = "structkv_score_layer (both scorer passes + reductions), per layer"
    roof["us_per_layer"] = score_s * 1e6
    roof["peaks"] = peaks["source"]
    # compaction against the HBM copy bandwidth
    comp_bytes = L * 2 * 2 * wl.n_kv_heads * kv_budget * wl.head_dim * 2 + 2 * st_budget * wl.hidden_dim * 2
    comp_s = phase_ms["compact"] * 1e-3 / args.steps
    compaction = {"achieved": comp_bytes / comp_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                  "frac": comp_bytes / comp_s / 1e9 / peaks["hbm_gbs"], "bytes_per_step": comp_bytes}

    n_launch = L * (5 if not (args.flags & binding.FLAG_NO_HEAD_STATS) else 4) + 1 + 2 + L + 2
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32",
            "data": "synthetic", "config": workload_config(wl, kv_budget), "pivot": pf.pivot,
            "phase_ms_per_step": {k: v / args.steps for k, v in phase_ms.items()},
            "roofline": roof, "compaction": compaction, "clocks": clocks,
            "gpu_launches": n_launch * args.steps, "e2e": e2e, "next_rows": next_rows}
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(wl, pl, kv_budget, n_layers_sample=1)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
