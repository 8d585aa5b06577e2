"""Thin ctypes binding over the C-ABI library ``libstructkv.so``.

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  PyTorch tensors supply device memory and streams.  Importing this
module raises if the library has not been built
(``python -m paper_2604_06746_b200.build``): there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libstructkv.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2604_06746_b200.build` "
        "(the StructKV hot path has no non-CUDA fallback)")

lib = ctypes.CDLL(LIB_PATH)

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)
BF16, FP32 = 0, 1
FLAG_NO_HEAD_STATS = 1
FLAG_FORCE_SIMT = 2
FLAG_INPUTS_READY = 4


class Config(ctypes.Structure):
    _fields_ = [("n_q_heads", ctypes.c_int), ("n_kv_heads", ctypes.c_int),
                ("head_dim", ctypes.c_int), ("window", ctypes.c_int),
                ("max_seq", ctypes.c_int), ("dtype", ctypes.c_int)]


_vp, _ll, _i, _f, _u = ctypes.c_void_p, ctypes.c_longlong, ctypes.c_int, ctypes.c_float, ctypes.c_uint
lib.structkv_version.restype = _i
lib.structkv_version.argtypes = []
lib.structkv_status_string.restype = ctypes.c_char_p
lib.structkv_status_string.argtypes = [_i]
lib.structkv_workspace_bytes.restype = ctypes.c_size_t
lib.structkv_workspace_bytes.argtypes = [ctypes.POINTER(Config)]
lib.structkv_create.restype = _i
lib.structkv_create.argtypes = [ctypes.POINTER(_vp), ctypes.POINTER(Config), _vp, ctypes.c_size_t]
lib.structkv_destroy.restype = None
lib.structkv_destroy.argtypes = [_vp]
lib.structkv_score_layer.restype = _i
lib.structkv_score_layer.argtypes = [_vp, _vp, _vp, _ll, _ll, _i, _f, _f, _vp, _vp, _vp, _vp, _u, _vp]
lib.structkv_score_layer_static.restype = _i
lib.structkv_score_layer_static.argtypes = [ctypes.POINTER(Config), _vp, _vp, _ll, _ll, _i, _f, _f, _vp, _vp,
                                            _vp, _vp, _u, _vp]
STATIC_SCRATCH_BYTES = 8 << 20
lib.structkv_batch_workspace_bytes.restype = ctypes.c_size_t
lib.structkv_batch_workspace_bytes.argtypes = [ctypes.POINTER(Config), _i, _ll]
lib.structkv_score_layer_batch.restype = _i
lib.structkv_score_layer_batch.argtypes = [_vp, _vp, _vp, _ll, _ll, ctypes.POINTER(_i), _i, _f, _f, _vp, _vp, _vp,
                                           _vp, _u, _vp, ctypes.c_size_t, _vp]
lib.structkv_layers_workspace_bytes.restype = ctypes.c_size_t
lib.structkv_layers_workspace_bytes.argtypes = [ctypes.POINTER(Config), _i]
lib.structkv_score_layers.restype = _i
lib.structkv_score_layers.argtypes = [_vp, _i, ctypes.POINTER(_vp), ctypes.POINTER(_vp), _ll, _ll, _i,
                                      ctypes.POINTER(_f), _f, _vp, _ll, _vp, _vp, _ll, _vp, _vp, ctypes.c_size_t, _vp]
lib.structkv_select_batch.restype = _i
lib.structkv_select_batch.argtypes = [_vp, _vp, ctypes.POINTER(_i), ctypes.POINTER(_i), _i, _i, _vp, _ll, _vp]
lib.structkv_head_stats.restype = _i
lib.structkv_head_stats.argtypes = [_vp, _vp, _ll, _ll, _i, _i, _vp, _vp]
lib.structkv_pivot.restype = _i
lib.structkv_pivot.argtypes = [_vp, _vp, _i, ctypes.POINTER(_f), _i, ctypes.POINTER(_i),
                               ctypes.POINTER(_f), _vp]
lib.structkv_accumulate.restype = _i
lib.structkv_accumulate.argtypes = [_vp, _vp, _ll, _i, _i, _f, _vp, _vp]
lib.structkv_select.restype = _i
lib.structkv_select.argtypes = [_vp, _vp, _ll, _i, _i, _i, _i, _vp, _vp]
lib.structkv_compact.restype = _i
lib.structkv_compact.argtypes = [_vp, _vp, _ll, _ll, _i, _i, _i, _vp, _i, _vp, _vp]
lib.structkv_group_saliency.restype = _i
lib.structkv_group_saliency.argtypes = [_vp, _vp, _ll, _i, _vp, _vp]
lib.structkv_compact_layers.restype = _i
lib.structkv_compact_layers.argtypes = [_vp, ctypes.POINTER(_vp), _i, _ll, _ll, _i, _i, _i, _vp, _ll, _i, _vp, _ll, _vp]
lib.structkv_compact_per_slab.restype = _i
lib.structkv_compact_per_slab.argtypes = [_vp, _vp, _ll, _ll, _i, _i, _i, _vp, _ll, _i, _vp, _vp]
lib.structkv_block_scores.restype = _i
lib.structkv_block_scores.argtypes = [_vp, _vp, _ll, _i, _i, _i, _vp, _vp]
lib.structkv_mass_recovery.restype = _i
lib.structkv_mass_recovery.argtypes = [_vp, _vp, _ll, _i, _i, _vp, _i, _vp, _vp]
lib.structkv_selftest_wait_expiry.restype = _i
lib.structkv_selftest_wait_expiry.argtypes = [_vp, ctypes.c_ulonglong, _vp]
lib.structkv_poll_device_status.restype = _i
lib.structkv_poll_device_status.argtypes = [_vp, _vp]


class StructKVError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib.structkv_status_string(status).decode()} (status {status})")


def _check(status: int, where: str) -> None:
    if status != OK:
        raise StructKVError(status, where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def version() -> int:
    return lib.structkv_version()


def workspace_bytes(cfg: Config) -> int:
    return lib.structkv_workspace_bytes(ctypes.byref(cfg))


def score_layer_static(n_q_heads: int, n_kv_heads: int, head_dim: int, window: int, max_seq: int,
                       q_window: torch.Tensor, k: torch.Tensor, scale: float, s_out: torch.Tensor,
                       metrics_out: torch.Tensor, c_inout: Optional[torch.Tensor] = None, lam: float = 0.9,
                       head_cols_out: Optional[torch.Tensor] = None, flags: int = 0,
                       stream: Optional[torch.cuda.Stream] = None) -> None:
    """structkv_score_layer_static: one layer of scoring with no context and no workspace.

    For callers that must not allocate device memory where they score (all HBM already given
    to a cache pool, or a step that cannot take the synchronisation an allocation implies): the
    scorer's scratch is a fixed array inside the library, so only configurations whose
    workspace fits ``STATIC_SCRATCH_BYTES`` are accepted, calls on one device share that array
    and must not overlap on the GPU, and the first call on a device does a one-time set-up that
    should precede any stream capture.  The current torch device must be the tensors' device.
    """
    code = {torch.bfloat16: BF16, torch.float32: FP32}[q_window.dtype]
    assert q_window.is_contiguous() and k.stride(2) == 1 and k.dtype == q_window.dtype
    cfg = Config(n_q_heads, n_kv_heads, head_dim, window, max_seq, code)
    with torch.cuda.device(q_window.device):
        _check(lib.structkv_score_layer_static(ctypes.byref(cfg), q_window.data_ptr(), k.data_ptr(),
                                               k.stride(0), k.stride(1), k.shape[1], scale, lam,
                                               s_out.data_ptr(), _ptr(c_inout), _ptr(head_cols_out),
                                               metrics_out.data_ptr(), flags, _stream(stream)),
               "structkv_score_layer_static")


class LayerSources:
    """Host-side argument block for ``Context.compact_layers`` (pointers and layout of the sources)."""

    def __init__(self, srcs: Sequence[torch.Tensor]):
        s0 = srcs[0]
        assert all(t.shape == s0.shape and t.stride() == s0.stride() and t.dtype == s0.dtype for t in srcs)
        row_elems = 1
        for sdim in s0.shape[2:]:
            row_elems *= sdim
        self.keep = list(srcs)                       # the tensors must outlive the block
        self.n_layers = len(srcs)
        self.elem_size = s0.element_size()
        self.ptrs = (_vp * self.n_layers)(*[t.data_ptr() for t in srcs])
        self.slab_stride_bytes = s0.stride(0) * self.elem_size
        self.row_stride_bytes = s0.stride(1) * self.elem_size
        self.row_bytes = row_elems * self.elem_size
        self.n_slabs, self.n_rows = s0.shape[0], s0.shape[1]


class Context:
    """Owns the library context and (through torch) its device workspace."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, window: int, max_seq: int,
                 dtype: torch.dtype, device: str = "cuda:0"):
        code = {torch.bfloat16: BF16, torch.float32: FP32}[dtype]
        self.cfg = Config(n_q_heads, n_kv_heads, head_dim, window, max_seq, code)
        self.device = torch.device(device)
        self.dtype = dtype
        self._h = _vp()
        nbytes = workspace_bytes(self.cfg)
        if nbytes == 0:
            raise StructKVError(ERR_UNSUPPORTED, "structkv_workspace_bytes")
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            _check(lib.structkv_create(ctypes.byref(self._h), ctypes.byref(self.cfg),
                                       self.workspace.data_ptr(), nbytes), "structkv_create")

    def close(self) -> None:
        if self._h:
            lib.structkv_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the four calls of the path (plus the closed-form re-accumulation) ---------------
    def score_layer(self, q_window: torch.Tensor, k: torch.Tensor, scale: float, s_out: torch.Tensor,
                    metrics_out: torch.Tensor, c_inout: Optional[torch.Tensor] = None,
                    lam: float = 0.9, head_cols_out: Optional[torch.Tensor] = None, flags: int = 0,
                    stream: Optional[torch.cuda.Stream] = None) -> None:
        """structkv_score_layer: ``k`` is ``[H_kv, N, d]`` with arbitrary head / token strides."""
        assert q_window.is_contiguous() and k.stride(2) == 1 and k.dtype == self.dtype == q_window.dtype
        _check(lib.structkv_score_layer(self._h, q_window.data_ptr(), k.data_ptr(), k.stride(0), k.stride(1),
                                        k.shape[1], scale, lam, s_out.data_ptr(), _ptr(c_inout),
                                        _ptr(head_cols_out), metrics_out.data_ptr(), flags,
                                        _stream(stream)), "structkv_score_layer")

    def score_layer_batch(self, q_window: torch.Tensor, k: torch.Tensor, cu_seqlens: Sequence[int], scale: float,
                          s_out: torch.Tensor, metrics_out: torch.Tensor, workspace: torch.Tensor,
                          c_inout: Optional[torch.Tensor] = None, lam: float = 0.9,
                          head_cols_out: Optional[torch.Tensor] = None, flags: int = 0,
                          stream: Optional[torch.cuda.Stream] = None) -> None:
        """structkv_score_layer_batch: ``q_window [B, H, w, d]``, ``k [H_kv, total, d]`` packed prompts,
        ``cu_seqlens`` host ints ``[B + 1]``."""
        B = len(cu_seqlens) - 1
        assert q_window.is_contiguous() and q_window.shape[0] == B and k.stride(2) == 1
        assert k.shape[1] == cu_seqlens[-1] and s_out.numel() == cu_seqlens[-1] and metrics_out.shape == (B, 3)
        cu = (_i * (B + 1))(*cu_seqlens)
        _check(lib.structkv_score_layer_batch(self._h, q_window.data_ptr(), k.data_ptr(), k.stride(0), k.stride(1),
                                              cu, B, scale, lam, s_out.data_ptr(), _ptr(c_inout),
                                              _ptr(head_cols_out), metrics_out.data_ptr(), flags,
                                              workspace.data_ptr(), workspace.numel(), _stream(stream)),
               "structkv_score_layer_batch")

    def score_layers(self, q_windows: Sequence[torch.Tensor], ks: Sequence[torch.Tensor], scales: Sequence[float],
                     s_out: torch.Tensor, metrics_out: torch.Tensor, head_cols_out: torch.Tensor,
                     workspace: torch.Tensor, c_inout: Optional[torch.Tensor] = None, lam: float = 0.9,
                     stream: Optional[torch.cuda.Stream] = None) -> None:
        """structkv_score_layers: layer ``l`` takes ``q_windows[l] [H, w, d]`` and ``ks[l] [H_kv, N, d]`` (all
        with the strides of ``ks[0]``); ``s_out [L, N]``, ``head_cols_out [L, H, N]``, ``metrics_out [L, 3]``."""
        L = len(q_windows)
        k0 = ks[0]
        assert len(ks) == L and len(scales) == L and L >= 1
        assert all(q.is_contiguous() for q in q_windows)
        assert all(k.shape == k0.shape and k.stride() == k0.stride() and k.stride(2) == 1 for k in ks)
        n = k0.shape[1]
        assert s_out.shape == (L, n) and s_out.stride(1) == 1 and metrics_out.is_contiguous()
        assert metrics_out.shape == (L, 3) and head_cols_out.shape[0] == L and head_cols_out[0].is_contiguous()
        qp = (_vp * L)(*[q.data_ptr() for q in q_windows])
        kp = (_vp * L)(*[k.data_ptr() for k in ks])
        sc = (_f * L)(*scales)
        _check(lib.structkv_score_layers(self._h, L, qp, kp, k0.stride(0), k0.stride(1), n, sc, lam,
                                         s_out.data_ptr(), s_out.stride(0), _ptr(c_inout), head_cols_out.data_ptr(),
                                         head_cols_out.stride(0), metrics_out.data_ptr(), workspace.data_ptr(),
                                         workspace.numel(), _stream(stream)), "structkv_score_layers")

    def layers_workspace(self, max_layers: int) -> torch.Tensor:
        n = lib.structkv_layers_workspace_bytes(ctypes.byref(self.cfg), max_layers)
        if n == 0:
            raise StructKVError(ERR_INVALID_ARG, "structkv_layers_workspace_bytes")
        return torch.empty(n, dtype=torch.uint8, device=self.device)

    def batch_workspace(self, max_batch: int, max_total_tokens: int) -> torch.Tensor:
        n = lib.structkv_batch_workspace_bytes(ctypes.byref(self.cfg), max_batch, max_total_tokens)
        if n == 0:
            raise StructKVError(ERR_INVALID_ARG, "structkv_batch_workspace_bytes")
        return torch.empty(n, dtype=torch.uint8, device=self.device)

    def select_batch(self, scores: torch.Tensor, cu_seqlens: Sequence[int], budgets: Sequence[int], window: int,
                     idx_out: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
        """structkv_select_batch: packed ``scores [total]`` -> ``idx_out [B, stride]`` int32, padded with -1."""
        B = len(budgets)
        assert scores.is_contiguous() and scores.dtype == torch.float32
        assert idx_out.dtype == torch.int32 and idx_out.is_contiguous() and idx_out.shape[0] == B
        cu = (_i * (B + 1))(*cu_seqlens)
        bu = (_i * B)(*budgets)
        _check(lib.structkv_select_batch(self._h, scores.data_ptr(), cu, bu, B, window, idx_out.data_ptr(),
                                         idx_out.stride(0), _stream(stream)), "structkv_select_batch")

    def head_stats(self, head_cols: torch.Tensor, metrics: torch.Tensor,
                   stream: Optional[torch.cuda.Stream] = None) -> None:
        """structkv_head_stats: ``head_cols [n_layers, H, n]`` -> ``metrics [n_layers, 3]`` columns 1 and 2."""
        assert head_cols.dim() == 3 and head_cols.stride(2) == 1 and head_cols.dtype == torch.float32
        assert metrics.is_contiguous() and metrics.shape == (head_cols.shape[0], 3)
        _check(lib.structkv_head_stats(self._h, head_cols.data_ptr(), head_cols.stride(0), head_cols.stride(1),
                                       head_cols.shape[0], head_cols.shape[2], metrics.data_ptr(),
                                       _stream(stream)), "structkv_head_stats")

    def pivot(self, metrics: torch.Tensor, weights: Sequence[float] = (0.2, 0.3, 0.5), l_limit: int = -1,
              stream: Optional[torch.cuda.Stream] = None) -> Tuple[int, list]:
        """structkv_pivot: ``metrics`` is the device ``[L, 3]`` fp32 table; returns ``(L*, T)``."""
        assert metrics.is_contiguous() and metrics.dtype == torch.float32
        L = metrics.shape[0]
        w = (_f * 3)(*weights)
        piv = _i(0)
        T = (_f * L)()
        _check(lib.structkv_pivot(self._h, metrics.data_ptr(), L, w, l_limit, ctypes.byref(piv), T,
                                  _stream(stream)), "structkv_pivot")
        return piv.value, list(T)

    def accumulate(self, s_hist: torch.Tensor, pivot: int, lam: float, c_out: torch.Tensor,
                   stream: Optional[torch.cuda.Stream] = None) -> None:
        _check(lib.structkv_accumulate(self._h, s_hist.data_ptr(), s_hist.stride(0), pivot, s_hist.shape[1],
                                       lam, c_out.data_ptr(), _stream(stream)), "structkv_accumulate")

    def select(self, scores: torch.Tensor, budget: int, window: int, idx_out: torch.Tensor,
               stream: Optional[torch.cuda.Stream] = None) -> None:
        """structkv_select over ``scores [batch, n]`` (or ``[n]``) into ``idx_out [batch, budget]`` int32."""
        s2 = scores if scores.dim() == 2 else scores[None]
        assert s2.stride(1) == 1 and s2.dtype == torch.float32 and idx_out.dtype == torch.int32
        assert idx_out.is_contiguous() and idx_out.numel() == s2.shape[0] * budget
        _check(lib.structkv_select(self._h, s2.data_ptr(), s2.stride(0), s2.shape[0], s2.shape[1], budget,
                                   window, idx_out.data_ptr(), _stream(stream)), "structkv_select")

    def compact(self, src: torch.Tensor, idx: torch.Tensor, dst: torch.Tensor,
                stream: Optional[torch.cuda.Stream] = None) -> None:
        """structkv_compact: ``src [n_slabs, n_rows, row...]`` (row contiguous) -> ``dst [n_slabs, n_idx, row...]``."""
        assert idx.dtype == torch.int32 and idx.is_contiguous() and dst.is_contiguous()
        row_elems = 1
        for s in src.shape[2:]:
            row_elems *= s
        es = src.element_size()
        if src.dim() > 2:
            assert src[0, 0].is_contiguous()
        _check(lib.structkv_compact(self._h, src.data_ptr(), src.stride(0) * es, src.stride(1) * es,
                                    row_elems * es, src.shape[0], src.shape[1], idx.data_ptr(),
                                    idx.numel(), dst.data_ptr(), _stream(stream)), "structkv_compact")

    @staticmethod
    def layer_sources(srcs: Sequence[torch.Tensor]) -> "LayerSources":
        """The argument block of ``compact_layers`` for a fixed list of source tensors (same shape,
        strides and dtype), checked and marshalled once: a caller that gathers from the same tensors
        many times keeps it and spares the per-call marshalling."""
        return LayerSources(srcs)

    def compact_layers(self, srcs, idx: torch.Tensor, dst: torch.Tensor,
                       stream: Optional[torch.cuda.Stream] = None) -> None:
        """structkv_compact_layers: every ``srcs[l] [n_slabs, n_rows, row...]`` (same shape and strides)
        gathered at ``idx[l]`` into ``dst[l] [n_slabs, n_idx, row...]`` by one launch.  ``srcs`` is a list of
        tensors or the ``LayerSources`` made from one."""
        ls = srcs if isinstance(srcs, LayerSources) else LayerSources(srcs)
        L = ls.n_layers
        assert idx.dtype == torch.int32 and idx.dim() == 2 and idx.shape[0] == L and idx.stride(1) == 1
        assert dst.shape[0] == L and dst[0].is_contiguous()
        _check(lib.structkv_compact_layers(self._h, ls.ptrs, L, ls.slab_stride_bytes, ls.row_stride_bytes,
                                           ls.row_bytes, ls.n_slabs, ls.n_rows, idx.data_ptr(), idx.stride(0),
                                           idx.shape[1], dst.data_ptr(), dst.stride(0) * ls.elem_size,
                                           _stream(stream)),
               "structkv_compact_layers")

    def group_saliency(self, head_cols: torch.Tensor, out: torch.Tensor,
                       stream: Optional[torch.cuda.Stream] = None) -> None:
        """structkv_group_saliency: ``head_cols [H, n]`` -> ``out [H_kv, n]`` (sum over each GQA group)."""
        assert head_cols.stride(1) == 1 and head_cols.dtype == torch.float32 and out.is_contiguous()
        assert head_cols.shape[0] == self.cfg.n_q_heads and out.shape == (self.cfg.n_kv_heads, head_cols.shape[1])
        _check(lib.structkv_group_saliency(self._h, head_cols.data_ptr(), head_cols.stride(0), head_cols.shape[1],
                                           out.data_ptr(), _stream(stream)), "structkv_group_saliency")

    def compact_per_slab(self, src: torch.Tensor, idx: torch.Tensor, dst: torch.Tensor,
                         stream: Optional[torch.cuda.Stream] = None) -> None:
        """structkv_compact_per_slab: ``src [n_slabs, n_rows, row...]``, ``idx [n_slabs, n_idx]`` int32."""
        assert idx.dtype == torch.int32 and idx.dim() == 2 and idx.stride(1) == 1 and dst.is_contiguous()
        assert idx.shape[0] == src.shape[0]
        row_elems = 1
        for sdim in src.shape[2:]:
            row_elems *= sdim
        es = src.element_size()
        _check(lib.structkv_compact_per_slab(self._h, src.data_ptr(), src.stride(0) * es, src.stride(1) * es,
                                             row_elems * es, src.shape[0], src.shape[1], idx.data_ptr(),
                                             idx.stride(0), idx.shape[1], dst.data_ptr(), _stream(stream)),
               "structkv_compact_per_slab")

    def block_scores(self, scores: torch.Tensor, block_size: int, out: torch.Tensor,
                     stream: Optional[torch.cuda.Stream] = None) -> None:
        """structkv_block_scores over ``scores [batch, n]`` (or ``[n]``) into ``out [batch, ceil(n / block_size)]``."""
        s2 = scores if scores.dim() == 2 else scores[None]
        assert s2.stride(1) == 1 and s2.dtype == torch.float32 and out.dtype == torch.float32 and out.is_contiguous()
        assert out.numel() == s2.shape[0] * ((s2.shape[1] + block_size - 1) // block_size)
        _check(lib.structkv_block_scores(self._h, s2.data_ptr(), s2.stride(0), s2.shape[0], s2.shape[1], block_size,
                                         out.data_ptr(), _stream(stream)), "structkv_block_scores")

    def mass_recovery(self, scores: torch.Tensor, idx: torch.Tensor, out: torch.Tensor,
                      stream: Optional[torch.cuda.Stream] = None) -> None:
        """structkv_mass_recovery: share of each row of ``scores [batch, n]`` that lies at ``idx``."""
        s2 = scores if scores.dim() == 2 else scores[None]
        assert s2.stride(1) == 1 and s2.dtype == torch.float32 and idx.dtype == torch.int32 and idx.is_contiguous()
        assert out.dtype == torch.float32 and out.numel() == s2.shape[0]
        _check(lib.structkv_mass_recovery(self._h, s2.data_ptr(), s2.stride(0), s2.shape[0], s2.shape[1],
                                          idx.data_ptr(), idx.numel(), out.data_ptr(), _stream(stream)),
               "structkv_mass_recovery")

    def selftest_wait_expiry(self, limit_cycles: int, stream: Optional[torch.cuda.Stream] = None) -> None:
        """structkv_selftest_wait_expiry: lets one bounded device wait run out (records TIMEOUT)."""
        _check(lib.structkv_selftest_wait_expiry(self._h, limit_cycles, _stream(stream)),
               "structkv_selftest_wait_expiry")

    def poll_device_status(self, stream: Optional[torch.cuda.Stream] = None) -> int:
        return lib.structkv_poll_device_status(self._h, _stream(stream))
