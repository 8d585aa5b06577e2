"""Seeded synthetic inputs shaped like the paper's long-context prefill workloads.

This module only *draws tensors*.  It contains none of the method's arithmetic
(no softmax, no scoring, no selection): both the CUDA path and the CPU oracle
consume the very same bits it produces, after rounding to the storage dtype.

The tensors stand in for prompts from the paper's evaluation suites run through
Llama-3-8B / Qwen2-7B shaped models (Section 4.1): same layer / head / head_dim /
sequence-length / window / budget shapes, random values, no dataset items and no
trained weights.

Recipe (per layer ``l`` of a workload):
  * ``q_win[h, i, :]``, ``k[g, j, :]``, ``v[g, j, :]`` i.i.d. N(0, 1); the
    attention scale 1/sqrt(d) is applied by the consumer, so logits have unit
    variance at temperature 1.
  * a per-(layer, KV group) common query direction ``c[g]`` of norm sqrt(d) is
    added to every window query of the group, so "a key aligned with the window
    queries" is well defined.
  * planted hubs: ``n_hubs`` distinct prefix positions; in the layers where a hub
    is active its key gets ``+ (boost / sqrt(d)) * c[g]`` (a logit lift of
    ``boost / temperature``); elsewhere it is plain noise ("dormant").
  * optional structure: attention sink (key 0 scaled x4), low-norm delimiter
    keys (5 % of positions scaled x0.1), log-normal key norms (sigma 0.5).
  * per-layer logit temperature tau_l, exposed as ``scale = 1 / (sqrt(d) * tau_l)``.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

SEED_BASE = 0x5EED0000
HUB_BOOST = 6.0          # logit units at temperature 1
HIDDEN_DIM = 4096        # model width of the hidden states gathered past the pivot


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape and structure of one synthetic prefill workload."""
    name: str
    index: int                    # enters the seed
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    seq: int
    window: int
    budgets: Tuple[int, ...]      # KV budgets (token counts, window included)
    dtype: str                    # "fp32" | "bf16" storage of q/k/v
    n_hubs: int
    hub_span: Optional[int]       # contiguous active span length; None = use hub_layers
    hub_layers: Tuple[int, ...] = ()   # explicit active layers (used when hub_span is None)
    temperatures: Optional[Tuple[float, ...]] = None  # None = U[0.5, 2] per layer
    temperature_draw: int = 0     # which draw of the temperature vector is used (earlier ones are
                                  # discarded); fixed when a workload is designed so that no two
                                  # layer transitions are nearly tied as the sharpest one
    sink: bool = False
    delimiters: bool = False
    heavy_tail: bool = False
    hidden_dim: int = HIDDEN_DIM
    streamed: bool = False        # layers generated, consumed and dropped one at a time

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def budget(self) -> int:
        return self.budgets[-1]

    def struct_budget(self, kv_budget: Optional[int] = None) -> int:
        """Token budget of the hidden-state gather: twice the KV budget, the
        paper's default ratio of structural to KV retention (20 % : 10 %)."""
        b = self.budget if kv_budget is None else kv_budget
        return min(self.seq, 2 * b)

    def scaled(self, seq: int, n_layers: Optional[int] = None, name: Optional[str] = None,
               budgets: Optional[Sequence[int]] = None, n_hubs: Optional[int] = None) -> "Workload":
        """Same structure at a smaller size (for tests the oracle finishes in seconds)."""
        ratio = seq / self.seq
        nb = tuple(budgets) if budgets is not None else tuple(
            max(self.window + 1, min(seq, int(round(b * ratio)))) for b in self.budgets)
        nl = self.n_layers if n_layers is None else n_layers
        return dataclasses.replace(
            self, name=name or f"{self.name}@{seq}", seq=seq, n_layers=nl, budgets=nb,
            n_hubs=self.n_hubs if n_hubs is None else n_hubs,
            temperatures=None if self.temperatures is None else tuple(self.temperatures[:nl]))


WORKLOADS: Dict[str, Workload] = {
    "tiny": Workload("tiny", 0, 4, 8, 2, 64, 2048, 32, (256,), "fp32", 8, None,
                     hub_layers=(1, 2), temperatures=(0.5, 1.0, 2.0, 1.0), sink=True),
    "llama32k": Workload("llama32k", 1, 32, 32, 8, 128, 32768, 64, (2048,), "bf16", 64, 8),
    "llama128k": Workload("llama128k", 2, 32, 32, 8, 128, 131072, 64, (1024, 4096, 16384), "bf16",
                          256, 8, sink=True, delimiters=True, temperature_draw=11),
    "qwen64k": Workload("qwen64k", 3, 28, 28, 4, 128, 65536, 128, (4096,), "bf16", 128, 8,
                        heavy_tail=True),
    "llama256k": Workload("llama256k", 4, 32, 32, 8, 128, 262144, 64, (8192,), "bf16", 256, 8,
                          sink=True, streamed=True),
}


def torch_dtype(name: str) -> torch.dtype:
    return {"fp32": torch.float32, "bf16": torch.bfloat16}[name]


def layer_seed(wl: Workload, layer: int) -> int:
    return SEED_BASE + 1000 * wl.index + layer


@dataclasses.dataclass(frozen=True)
class Plan:
    """Workload-level random structure, drawn once on the host (device independent)."""
    hub_positions: np.ndarray     # [n_hubs] int64, ascending, in [1, seq - window)
    hub_active: np.ndarray        # [n_layers, n_hubs] bool
    temperatures: np.ndarray      # [n_layers] float64


def plan(wl: Workload) -> Plan:
    rng = np.random.Generator(np.random.PCG64(SEED_BASE + 1000 * wl.index + 999))
    prefix = wl.seq - wl.window
    pos = np.sort(rng.choice(np.arange(1, prefix), size=wl.n_hubs, replace=False)) \
        if wl.n_hubs > 0 else np.zeros((0,), np.int64)
    active = np.zeros((wl.n_layers, wl.n_hubs), dtype=bool)
    if wl.hub_span is None:
        for l in wl.hub_layers:
            if l < wl.n_layers:
                active[l, :] = True
    else:
        span = min(wl.hub_span, wl.n_layers)
        starts = rng.integers(0, wl.n_layers - span + 1, size=wl.n_hubs)
        for h, s in enumerate(starts):
            active[s:s + span, h] = True
    if wl.temperatures is not None:
        temps = np.asarray(wl.temperatures[:wl.n_layers], dtype=np.float64)
    else:
        for _ in range(wl.temperature_draw + 1):
            temps = rng.uniform(0.5, 2.0, size=wl.n_layers)
    return Plan(pos.astype(np.int64), active, temps)


def layer_scale(wl: Workload, pl: Plan, layer: int) -> float:
    """Logit scale of a layer: 1/sqrt(d) divided by the layer's temperature."""
    return float(1.0 / (math.sqrt(wl.head_dim) * pl.temperatures[layer]))


def make_layer(wl: Workload, pl: Plan, layer: int, device: str = "cpu",
               with_v: bool = True) -> Dict[str, torch.Tensor]:
    """Draw one layer's tensors on ``device``, already rounded to the storage dtype.

    Returns ``q_win [H, w, d]``, ``k [H_kv, N, d]``, ``v [H_kv, N, d]`` (optional)
    and the python float ``scale``.
    """
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(layer_seed(wl, layer))
    H, Hkv, d, N, w, G = wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.seq, wl.window, wl.group
    f32 = torch.float32
    common = torch.randn((Hkv, d), generator=gen, device=dev, dtype=f32)
    common = common * (math.sqrt(d) / common.norm(dim=1, keepdim=True))
    q = torch.randn((H, w, d), generator=gen, device=dev, dtype=f32)
    q = q + common.repeat_interleave(G, dim=0)[:, None, :]
    k = torch.randn((Hkv, N, d), generator=gen, device=dev, dtype=f32)
    if wl.heavy_tail:
        n = torch.randn((Hkv, N, 1), generator=gen, device=dev, dtype=f32)
        k = k * torch.exp(0.5 * n - 0.125)
    if wl.delimiters:
        k[:, 10::20, :] *= 0.1
    act = pl.hub_active[layer]
    if act.any():
        pos = torch.from_numpy(pl.hub_positions[act]).to(dev)
        k[:, pos, :] += (HUB_BOOST / math.sqrt(d)) * common[:, None, :]
    if wl.sink:
        k[:, 0, :] *= 4.0
    st = torch_dtype(wl.dtype)
    out = {"q_win": q.to(st).contiguous(), "scale": layer_scale(wl, pl, layer)}
    if with_v:
        # K and V of a layer share one allocation [2, H_kv, N, d] (a single gather then compacts both)
        kv = torch.empty((2, Hkv, N, d), device=dev, dtype=st)
        kv[0] = k.to(st)
        del q, k
        kv[1] = torch.randn((Hkv, N, d), generator=gen, device=dev, dtype=f32).to(st)
        out["kv"], out["k"], out["v"] = kv, kv[0], kv[1]
    else:
        out["k"] = k.to(st).contiguous()
    return out


def make_hidden(wl: Workload, device: str = "cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """Hidden states ``[N, hidden_dim]`` (bf16) and position ids ``[N]`` (int32)."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(SEED_BASE + 1000 * wl.index + 998)
    hid = torch.empty((wl.seq, wl.hidden_dim), device=dev, dtype=torch.bfloat16)
    step = 16384
    for s in range(0, wl.seq, step):
        e = min(wl.seq, s + step)
        hid[s:e] = torch.randn((e - s, wl.hidden_dim), generator=gen, device=dev,
                               dtype=torch.float32).to(torch.bfloat16)
    pos = torch.arange(wl.seq, device=dev, dtype=torch.int32)
    return hid, pos


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of stored bits (fp32 / bf16) to float64 on the host."""
    return t.detach().to("cpu").to(torch.float64).numpy()
