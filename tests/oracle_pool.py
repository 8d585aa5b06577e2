"""Runs the oracle's per-layer scoring for many layers in worker processes (test plumbing only).

The oracle is single-threaded NumPy apart from its matrix products, so the layers of a
full-size workload are scored side by side, one process per layer.  Each worker receives the
stored bits of a layer's tensors (bf16 as int16, fp32 as is), widens them exactly to float64
and calls ``oracle.structkv_oracle.score_layer`` unchanged; the parent then applies the oracle's
own ``pivot`` / ``centrality`` / ``select`` to the collected results, which is what
``oracle.structkv_oracle.prefill`` does in one process.  Nothing here computes anything itself.
"""
from __future__ import annotations

import multiprocessing as mp
import os
from typing import Dict, Iterable, List, Optional, Sequence, Tuple

import numpy as np

_THREAD_VARS = ("OMP_NUM_THREADS", "OPENBLAS_NUM_THREADS", "MKL_NUM_THREADS", "NUMEXPR_NUM_THREADS")


def bits_of(t) -> np.ndarray:
    """Stored bits of a torch tensor on the host: bf16 -> int16 view, fp32 -> float32."""
    import torch
    t = t.detach().to("cpu").contiguous()
    return t.view(torch.int16).numpy() if t.dtype == torch.bfloat16 else t.numpy()


def widen(bits: np.ndarray) -> np.ndarray:
    """Exact widening of stored bits to float64 (bf16 is the upper half of an fp32)."""
    if bits.dtype == np.int16:
        return (bits.astype(np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return bits.astype(np.float64)


def _score_one(task):
    from oracle import structkv_oracle as O
    layer, q_bits, k_bits, scale, n_keys = task
    k = widen(k_bits)
    if n_keys is not None:
        k = k[:, :n_keys]
    o = O.score_layer(widen(q_bits), k, scale)
    return layer, o["S"], (o["entropy"], o["sparsity"], o["variance"])


def default_workers(bytes_per_worker: float) -> int:
    try:
        cores = len(os.sched_getaffinity(0))
    except AttributeError:
        cores = os.cpu_count() or 1
    try:
        import psutil
        avail = psutil.virtual_memory().available
    except Exception:
        avail = 32 << 30
    return max(1, min(cores, int(0.6 * avail / max(1.0, bytes_per_worker))))


def score_layers(tasks: Iterable[Tuple[int, np.ndarray, np.ndarray, float, Optional[int]]], n_tasks: int,
                 workers: int, stack: bool = True):
    """``tasks`` yields ``(layer, q_bits, k_bits, scale, n_keys or None)``; returns the oracle's
    ``s_hist [L, N]`` and ``metrics [L, 3]`` (layers indexed by the ``layer`` field, 0 .. L-1).
    With ``stack=False`` the score vectors come back as a list (tasks of different lengths)."""
    saved = {v: os.environ.get(v) for v in _THREAD_VARS}
    for v in _THREAD_VARS:                      # one compute thread per worker: the layers run side by side
        os.environ[v] = "1"
    try:
        ctx = mp.get_context("spawn")
        s_hist: List[Optional[np.ndarray]] = [None] * n_tasks
        metrics = np.zeros((n_tasks, 3), dtype=np.float64)
        n_proc = max(1, min(workers, n_tasks))
        with ctx.Pool(processes=n_proc) as pool:
            # tasks are drawn in this thread (the caller's generator may drive the GPU); at most
            # n_proc + 1 layers are in flight, so host memory stays bounded
            pending = []

            def collect(res):
                layer, S, m = res.get()
                s_hist[layer] = S
                metrics[layer] = m

            for task in tasks:
                while len(pending) > n_proc:
                    collect(pending.pop(0))
                pending.append(pool.apply_async(_score_one, (task,)))
            for res in pending:
                collect(res)
    finally:
        for v, old in saved.items():
            if old is None:
                os.environ.pop(v, None)
            else:
                os.environ[v] = old
    return (np.stack(s_hist) if stack else s_hist), metrics


def assemble(s_hist: np.ndarray, metrics: np.ndarray, window: int, kv_budgets: Sequence[int],
             struct_budgets: Sequence[int], lam: float, weights: Sequence[float]) -> Dict[str, object]:
    """The steps of ``oracle.structkv_oracle.prefill`` after the per-layer scoring, by the oracle's
    own functions, for several budgets at once."""
    from oracle import structkv_oracle as O
    piv = O.pivot(metrics, weights)
    C = O.centrality(s_hist, lam, piv)
    return {"s_hist": s_hist, "metrics": metrics, "pivot": piv, "transition": O.transition_scores(metrics, weights),
            "C": C,
            "i_struct": {b: O.select(C, b, window) for b in struct_budgets},
            "i_kv": {b: np.stack([O.select(s_hist[l], b, window) for l in range(s_hist.shape[0])])
                     for b in kv_budgets}}
