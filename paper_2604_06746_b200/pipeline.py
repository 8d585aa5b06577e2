"""Sequencing of the C-ABI calls over one prompt (the control flow of Algorithm 1
replayed over per-layer tensors): score every layer, detect the pivot, rebuild
the centrality at the pivot, select both budgets, compact K/V, hidden states
and position ids.  All arithmetic happens inside the library's kernels; this
file only owns buffers and call order.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import torch

from . import binding

PAPER_LAMBDA = 0.9
PAPER_WEIGHTS = (0.2, 0.3, 0.5)


class Prefill:
    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, window: int,
                 seq: int, kv_budget: int, struct_budget: int, dtype: torch.dtype,
                 hidden_dim: int = 0, device: str = "cuda:0", lam: float = PAPER_LAMBDA,
                 weights: Sequence[float] = PAPER_WEIGHTS, l_limit: int = -1, flags: int = 0,
                 keep_kv: bool = True, defer_head_stats: bool = True):
        self.L, self.H, self.Hkv, self.d, self.w, self.N = n_layers, n_q_heads, n_kv_heads, head_dim, window, seq
        self.kv_budget, self.struct_budget = kv_budget, struct_budget
        self.lam, self.weights, self.l_limit, self.flags = lam, tuple(weights), l_limit, flags
        self.dtype, self.device = dtype, torch.device(device)
        self.ctx = binding.Context(n_q_heads, n_kv_heads, head_dim, window, seq, dtype, device)
        dev = self.device
        f32, i32 = torch.float32, torch.int32
        self.s_hist = torch.zeros((n_layers, seq), dtype=f32, device=dev)
        self.metrics = torch.zeros((n_layers, 3), dtype=f32, device=dev)
        self.c_running = torch.zeros((seq,), dtype=f32, device=dev)
        self.c_star = torch.zeros((seq,), dtype=f32, device=dev)
        self.i_kv = torch.zeros((n_layers, kv_budget), dtype=i32, device=dev)
        self.i_struct = torch.zeros((struct_budget,), dtype=i32, device=dev)
        n_kv_out = n_layers if keep_kv else 1
        self.keep_kv = keep_kv
        # compacted K and V of a layer sit in one allocation [2, H_kv, B, d]: when the source K and V
        # are laid out the same way, one gather launch serves both
        self.kv_out = torch.empty((n_kv_out, 2, n_kv_heads, kv_budget, head_dim), dtype=dtype, device=dev)
        self.k_out = self.kv_out[:, 0]
        self.v_out = self.kv_out[:, 1]
        self.hidden_out = (torch.empty((struct_budget, hidden_dim), dtype=torch.bfloat16, device=dev)
                           if hidden_dim else None)
        self.pos_out = torch.empty((struct_budget,), dtype=i32, device=dev)
        self.pivot = -1
        self.transition: List[float] = []
        # Eq. 5-6 of all layers in one batched call before the pivot (instead of a chain of short
        # dependent launches after every layer): the pooled per-head attention of every layer is kept
        self.defer = bool(defer_head_stats) and not (flags & binding.FLAG_NO_HEAD_STATS) and n_layers <= 128
        self.head_cols = (torch.empty((n_layers, n_q_heads, seq), dtype=f32, device=dev) if self.defer else None)
        self._stats_done = 0
        self._layers_ws = None
        self._side = None
        self._kv_sources = None

    # -- Algorithm 1 lines 3-6 for one layer
    def score(self, layer: int, q_win: torch.Tensor, k: torch.Tensor, scale: float,
              head_cols_out: Optional[torch.Tensor] = None) -> None:
        if layer == 0:
            self.c_running.zero_()
            self._stats_done = 0
        if self.defer:
            self.ctx.score_layer(q_win, k, scale, self.s_hist[layer], self.metrics[layer],
                                 c_inout=self.c_running, lam=self.lam, head_cols_out=self.head_cols[layer],
                                 flags=self.flags | binding.FLAG_NO_HEAD_STATS)
            if head_cols_out is not None:
                head_cols_out.copy_(self.head_cols[layer])
            return
        self.ctx.score_layer(q_win, k, scale, self.s_hist[layer], self.metrics[layer],
                             c_inout=self.c_running, lam=self.lam, head_cols_out=head_cols_out,
                             flags=self.flags)

    def score_all(self, layers: Sequence[Dict[str, torch.Tensor]]) -> None:
        """Algorithm 1 lines 3-6 for resident layers.  Where the pooled per-head attention of every layer
        is kept anyway (head statistics in one batched call) and the layers' K tensors share one layout,
        all layers go through one structkv_score_layers call, which interleaves the scorer passes of
        neighbouring layers; otherwise layer after layer."""
        L = len(layers)
        k0 = layers[0]["k"]
        same = all(t["k"].shape == k0.shape and t["k"].stride() == k0.stride() for t in layers)
        if not (self.defer and same and L == self.L and self.flags in (0, binding.FLAG_INPUTS_READY)):
            for l, t in enumerate(layers):
                self.score(l, t["q_win"], t["k"], t["scale"])
            return
        if self._layers_ws is None:
            self._layers_ws = self.ctx.layers_workspace(self.L)
        self.c_running.zero_()
        self._stats_done = 0
        self.ctx.score_layers([t["q_win"] for t in layers], [t["k"] for t in layers],
                              [t["scale"] for t in layers], self.s_hist, self.metrics, self.head_cols,
                              self._layers_ws, c_inout=self.c_running, lam=self.lam)

    def finish_scores(self, n_scored: Optional[int] = None) -> None:
        """Sparsity and variance (Eq. 5-6) of the layers scored so far, in one batched call."""
        L = self.L if n_scored is None else n_scored
        if self.defer and self._stats_done < L:
            self.ctx.head_stats(self.head_cols[self._stats_done:L], self.metrics[self._stats_done:L])
            self._stats_done = L

    # -- Algorithm 1 lines 7-10 and 16: pivot, centrality at the pivot, both index sets
    def detect_and_select(self, n_scored: Optional[int] = None) -> int:
        L = self.L if n_scored is None else n_scored
        self.finish_scores(L)
        # The per-layer selections (Eq. 13) do not depend on the pivot: they are enqueued first, and the
        # metric table travels to the host on a side stream meanwhile, so the device is not idle while
        # the host evaluates Eq. 7-9.
        main = torch.cuda.current_stream(self.device)
        if self._side is None:
            self._side = torch.cuda.Stream(device=self.device)
        ready = torch.cuda.Event()
        ready.record(main)
        self._side.wait_event(ready)
        self.ctx.select(self.s_hist[:L], self.kv_budget, self.w, self.i_kv[:L])
        self.pivot, self.transition = self.ctx.pivot(self.metrics[:L], self.weights, self.l_limit, stream=self._side)
        self.ctx.accumulate(self.s_hist, self.pivot, self.lam, self.c_star)
        self.ctx.select(self.c_star, self.struct_budget, self.w, self.i_struct)
        return self.pivot

    # -- Algorithm 1 line 17 for one layer
    def compact_kv(self, layer: int, k: torch.Tensor, v: torch.Tensor,
                   kv: Optional[torch.Tensor] = None) -> None:
        """``kv`` (optional) is the joint storage ``[2, H_kv, N, d]`` whose halves are ``k`` and ``v``."""
        slot = layer if self.keep_kv else 0
        if kv is not None:
            self.ctx.compact(kv.view(2 * self.Hkv, kv.shape[2], self.d), self.i_kv[layer],
                             self.kv_out[slot].view(2 * self.Hkv, self.kv_budget, self.d))
            return
        self.ctx.compact(k, self.i_kv[layer], self.k_out[slot])
        self.ctx.compact(v, self.i_kv[layer], self.v_out[slot])

    def compact_all_kv(self, layers: Sequence[Dict[str, torch.Tensor]]) -> None:
        """Algorithm 1 line 17 for resident layers: one launch for all of them when every layer keeps
        K and V in one joint allocation, else one gather per layer."""
        if self.keep_kv and len(layers) <= 128 and all("kv" in t for t in layers):
            # the sources' pointers and layout are marshalled once per set of tensors, so that the launch
            # is not held up by host work after the selections
            key = tuple(t["kv"].data_ptr() for t in layers)
            if self._kv_sources is None or self._kv_sources[0] != key:
                self._kv_sources = (key, self.ctx.layer_sources(
                    [t["kv"].view(2 * self.Hkv, t["kv"].shape[2], self.d) for t in layers]))
                self._kv_dst = self.kv_out[:len(layers)].view(len(layers), 2 * self.Hkv, self.kv_budget, self.d)
            self.ctx.compact_layers(self._kv_sources[1], self.i_kv[:len(layers)], self._kv_dst)
            return
        for l, t in enumerate(layers):
            if "v" in t:
                self.compact_kv(l, t["k"], t["v"], t.get("kv"))

    # -- Algorithm 1 line 13
    def compact_hidden(self, hidden: torch.Tensor, positions: torch.Tensor) -> None:
        self.ctx.compact(hidden[None], self.i_struct, self.hidden_out[None])
        self.ctx.compact(positions[None, :, None], self.i_struct, self.pos_out[None, :, None])

    # -- Algorithm 1 past the pivot (Eq. 11-13 on the reduced sequence)
    def enable_reduced(self) -> None:
        """Buffers for layers scored after the truncation: K gathered at I_struct, the saliency of
        the reduced sequence, its selection, and that selection as original position ids."""
        dev, f32, i32 = self.device, torch.float32, torch.int32
        nr = self.struct_budget
        self.k_red = torch.empty((self.Hkv, nr, self.d), dtype=self.dtype, device=dev)
        self.s_red = torch.zeros((self.L, nr), dtype=f32, device=dev)
        self.metrics_red = torch.zeros((self.L, 3), dtype=f32, device=dev)
        self.i_red = torch.zeros((self.L, self.kv_budget), dtype=i32, device=dev)
        self.i_kv_pos = torch.zeros((self.L, self.kv_budget), dtype=i32, device=dev)
        self.recovery = torch.zeros((self.L,), dtype=f32, device=dev)

    def score_reduced(self, layer: int, q_win: torch.Tensor, k: torch.Tensor, scale: float) -> None:
        """Layer ``layer`` > L* on the keys that survived the truncation: gather K at I_struct
        (Eq. 11), score the reduced sequence (the window is its tail, so the queries are unchanged)."""
        self.ctx.compact(k, self.i_struct, self.k_red)
        self.ctx.score_layer(q_win, self.k_red, scale, self.s_red[layer], self.metrics_red[layer],
                             flags=self.flags)

    def select_reduced(self, first: int, last: int) -> None:
        """Eq. 13 on the reduced sequences of layers ``first .. last - 1`` (one batched launch), then
        each index list mapped back to original positions through the gathered position ids
        (Eq. 12; ``compact_hidden`` must have filled ``pos_out``)."""
        if last <= first:
            return
        self.ctx.select(self.s_red[first:last], self.kv_budget, self.w, self.i_red[first:last])
        for l in range(first, last):
            self.ctx.compact(self.pos_out[None, :, None], self.i_red[l], self.i_kv_pos[l][None, :, None])

    def run(self, layers: Sequence[Dict[str, torch.Tensor]], hidden: Optional[torch.Tensor] = None,
            positions: Optional[torch.Tensor] = None) -> int:
        """Whole path over resident per-layer tensors (dicts with q_win, k, v, scale)."""
        self.score_all(layers)
        self.detect_and_select(len(layers))
        self.compact_all_kv(layers)
        if hidden is not None:
            self.compact_hidden(hidden, positions)
        return self.pivot
