"""Float64 CPU oracle for the StructKV prefill-time KV-compression hot path.

TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct
statement of what the path computes, written from the paper's equations.  It
shares no code with the CUDA library and must never be imported by the product
package: only tests, the smoke check and the benchmark's CPU-baseline leg use it.

Every quantity here has a plain definition, and the oracle *is* that definition
written out in NumPy float64 (a library matmul / sort serves as a step; nothing
is blocked, fused or reordered).  Inputs are the stored bits of the tensors
(fp32 / bf16) widened exactly to float64.

Parity pins: every function below (the two diagnostics / paged-KV helpers included) is pinned by the CPU test-suite against
closed forms, invariants, library routines or brute force (none is unpinned).

Readings of the paper where its text is silent, ambiguous or garbled
(each is a single statement below, so an alternative is a one-line change):

  R1  Window rows: exactly ``w`` query rows, positions ``t = N-w .. N-1``
      (the printed range ``[N-w, N]`` has ``w+1`` members but is normalised by
      ``1/w`` and position ``N`` does not exist).
  R2  Softmax support: causal -- row ``t`` is normalised over keys ``j <= t``,
      window keys included (prefill of a causal LM).
  R3  Eq. 2 literally: one N-vector per layer, summed over all query heads
      (the sum over GQA groups of the within-group sums).
  R4  Entropy (Eq. 4): natural log, ``0 log 0 = 0``, mean over heads and window rows.
  R5  Sparsity (Eq. 5): the printed ``a_{t,j}`` has a dangling ``t`` while the
      index set depends on the head only; ``a^{(l,h)}`` is read as the
      window-pooled per-head vector ``abar^{(h)}_j = (1/w) sum_t a_{t,j}``
      (sums to 1) and ``k = max(1, floor(0.1 N))`` over all N positions.
  R6  Variance (Eq. 6): population variance over ``j`` of ``abar^{(h)}``.
  R7  Eq. 7: differences exist for ``l = 1 .. L-1``; min/max over those; a
      metric with zero range contributes 0.
  R8  Eq. 9: ``L*`` is the layer ``l`` whose difference ``M_l - M_{l-1}``
      maximises ``T_l`` (the printed ``+1`` turns a 0-based index into the
      difference array into that layer index; Section 4.4 calls the layer of the
      maximum gradient ``L*``).  First maximum wins; ``L_limit`` caps it.
  R9  Eq. 10 / Eq. 13: the window is always kept and does not compete; the
      budget is a token count that includes the window; ties break towards the
      lower index; the index list is returned ascending.
  R10 Eq. 3: ``C*`` sums layers ``0 .. L*`` inclusive.
"""
from __future__ import annotations

from typing import Dict, Iterator, Optional, Sequence, Tuple

import numpy as np

PAPER_WEIGHTS = (0.2, 0.3, 0.5)      # {w1, w2, w3}, Section 4.1 implementation details
PAPER_LAMBDA = 0.9                   # decay of the global centrality, same paragraph
SPARSITY_DENOMINATOR = 10            # k = 0.1 N in Eq. 5, rounded down


# --------------------------------------------------------------------------- Eq. 1
def window_attention(q_win: np.ndarray, k: np.ndarray, scale: float) -> Iterator[np.ndarray]:
    """Eq. 1: for each query head ``h`` yield the ``[w, N]`` attention weights of
    the observation-window rows (row ``i`` is position ``t = N-w+i``, R1) over
    all keys, softmax over the causal support ``j <= t`` (R2); masked entries are 0.

    ``q_win [H, w, d]``, ``k [H_kv, N, d]``; head ``h`` reads KV head ``h // G``.
    """
    q_win = np.asarray(q_win, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    H, w, d = q_win.shape
    Hkv, N, d2 = k.shape
    assert d == d2 and H % Hkv == 0 and 1 <= w <= N
    G = H // Hkv
    t = (N - w) + np.arange(w)                      # positions of the window rows
    visible = np.arange(N)[None, :] <= t[:, None]   # causal support
    for h in range(H):
        s = float(scale) * (q_win[h] @ k[h // G].T)           # [w, N] logits
        s = np.where(visible, s, -np.inf)
        m = s.max(axis=1, keepdims=True)
        e = np.exp(s - m)
        yield e / e.sum(axis=1, keepdims=True)


# ----------------------------------------------------------------- Eq. 2, 4, 5, 6
def score_layer(q_win: np.ndarray, k: np.ndarray, scale: float) -> Dict[str, np.ndarray]:
    """One layer of scoring.

    Returns
      ``S [N]``            local saliency, Eq. 2 (R3)
      ``head_cols [H, N]`` window-pooled per-head attention ``abar^{(h)}``
      ``entropy``          Eq. 4 (R4)
      ``sparsity``         Eq. 5 (R5)
      ``variance``         Eq. 6 (R6)
    """
    H, w, _ = np.shape(q_win)
    N = np.shape(k)[1]
    head_cols = np.zeros((H, N), dtype=np.float64)
    row_entropy = np.zeros((H, w), dtype=np.float64)
    for h, a in enumerate(window_attention(q_win, k, scale)):
        head_cols[h] = a.sum(axis=0) / w
        with np.errstate(divide="ignore", invalid="ignore"):
            term = np.where(a > 0.0, a * np.log(a), 0.0)
        row_entropy[h] = -term.sum(axis=1)
    S = head_cols.sum(axis=0)
    sparsity, variance = head_statistics(head_cols)
    return {
        "S": S,
        "head_cols": head_cols,
        "entropy": float(row_entropy.mean()),
        "sparsity": sparsity,
        "variance": variance,
    }


def head_statistics(head_cols: np.ndarray) -> Tuple[float, float]:
    """Eq. 5 and Eq. 6 from the window-pooled per-head attention ``head_cols [H, N]`` (R5, R6):
    the mean over heads of the mass of the ``floor(0.1 N)`` largest entries, and the mean over
    heads of the population variance over the keys."""
    head_cols = np.asarray(head_cols, dtype=np.float64)
    N = head_cols.shape[1]
    k_rho = max(1, N // SPARSITY_DENOMINATOR)
    top_mass = np.sort(head_cols, axis=1)[:, ::-1][:, :k_rho].sum(axis=1)
    return float(top_mass.mean()), float(np.var(head_cols, axis=1).mean())


# --------------------------------------------------------------------------- Eq. 3
def centrality(s_hist: np.ndarray, lam: float, pivot: int) -> np.ndarray:
    """Eq. 3: ``C_j = sum_{l=0}^{L*} lam^(L*-l) S_j^{(l)}`` (R10)."""
    s_hist = np.asarray(s_hist, dtype=np.float64)
    c = np.zeros(s_hist.shape[1], dtype=np.float64)
    for l in range(pivot + 1):
        c += (float(lam) ** (pivot - l)) * s_hist[l]
    return c


def centrality_recursive(s_hist: np.ndarray, lam: float, pivot: int) -> np.ndarray:
    """Algorithm 1 line 6: ``C <- C * lam + S^{(l)}`` for ``l = 0 .. L*``."""
    s_hist = np.asarray(s_hist, dtype=np.float64)
    c = np.zeros(s_hist.shape[1], dtype=np.float64)
    for l in range(pivot + 1):
        c = c * float(lam) + s_hist[l]
    return c


# ----------------------------------------------------------------------- Eq. 7 - 9
def normalised_gradient(metric: Sequence[float]) -> np.ndarray:
    """Eq. 7 for one metric: entries ``l = 1 .. L-1`` (index 0 unused, set to 0)."""
    m = np.asarray(metric, dtype=np.float64)
    out = np.zeros(m.shape[0], dtype=np.float64)
    if m.shape[0] < 2:
        return out
    delta = m[1:] - m[:-1]
    lo, hi = delta.min(), delta.max()
    if hi > lo:
        out[1:] = (delta - lo) / (hi - lo)
    return out


def transition_scores(metrics: np.ndarray, weights: Sequence[float] = PAPER_WEIGHTS) -> np.ndarray:
    """Eq. 8: ``T_l = w1 grad(-H)_l + w2 grad(rho)_l + w3 grad(V)_l`` for
    ``metrics [L, 3] = (entropy, sparsity, variance)``; ``T_0`` is undefined (-inf)."""
    metrics = np.asarray(metrics, dtype=np.float64)
    w1, w2, w3 = (float(x) for x in weights)
    T = (w1 * normalised_gradient(-metrics[:, 0])
         + w2 * normalised_gradient(metrics[:, 1])
         + w3 * normalised_gradient(metrics[:, 2]))
    T[0] = -np.inf
    return T


def pivot(metrics: np.ndarray, weights: Sequence[float] = PAPER_WEIGHTS,
          l_limit: Optional[int] = None) -> int:
    """Eq. 9 with Algorithm 1's ``L_limit`` (R8): the layer that maximises ``T_l``."""
    metrics = np.asarray(metrics, dtype=np.float64)
    L = metrics.shape[0]
    if L < 2:
        return 0
    T = transition_scores(metrics, weights)
    best = 1
    for l in range(2, L):
        if T[l] > T[best]:
            best = l
    if l_limit is not None and l_limit >= 0:
        best = min(best, int(l_limit))
    return best


# ------------------------------------------------------------------- Eq. 10, Eq. 13
def select(scores: np.ndarray, budget: int, window: int) -> np.ndarray:
    """Eq. 10 / Eq. 13 (R9): the ``budget - window`` best prefix tokens by
    (score descending, index ascending), sorted by position, then the window."""
    scores = np.asarray(scores)
    N = scores.shape[0]
    assert window <= budget <= N and window <= N
    prefix = N - window
    keep = budget - window
    # lexsort: last key is primary -> score descending, then index ascending
    order = np.lexsort((np.arange(prefix), -scores[:prefix]))
    top = np.sort(order[:keep].astype(np.int64))
    return np.concatenate([top, np.arange(prefix, N, dtype=np.int64)]).astype(np.int64)


# ------------------------------------------------- Algorithm 1 lines 13 and 17
def compact(src: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """``dst[g, r, ...] = src[g, idx[r], ...]`` for ``src [n_slabs, n_rows, ...]``."""
    return np.ascontiguousarray(np.asarray(src)[:, np.asarray(idx, dtype=np.int64)])


# ------------------------------------------ Section 3.2: aggregation inside a GQA group
def group_saliency(head_cols: np.ndarray, group: int) -> np.ndarray:
    """Pooled attention summed over the ``group`` query heads that share a KV head:
    ``out[g, j] = sum_{h in group g} abar^{(h)}_j``; summing over ``g`` gives Eq. 2."""
    head_cols = np.asarray(head_cols, dtype=np.float64)
    H, n = head_cols.shape
    assert H % group == 0
    out = np.zeros((H // group, n), dtype=np.float64)
    for h in range(H):
        out[h // group] += head_cols[h]
    return out


def compact_per_slab(src: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """``dst[s, r, ...] = src[s, idx[s, r], ...]``: one index list per slab (per KV head, or per
    sequence of a batch)."""
    src, idx = np.asarray(src), np.asarray(idx, dtype=np.int64)
    return np.stack([src[s][idx[s]] for s in range(src.shape[0])])


# ------------------------------------ Section 4.1 (implementation details): paged KV
def block_scores(scores: np.ndarray, block_size: int) -> np.ndarray:
    """Block-Level Aggregation: ``S_block_k = sum_{t in block_k} C[t]`` with block ``k`` =
    tokens ``[k*block_size, (k+1)*block_size)`` (the last block may be ragged)."""
    scores = np.asarray(scores, dtype=np.float64)
    n = scores.shape[0]
    n_blocks = -(-n // int(block_size))
    out = np.zeros(n_blocks, dtype=np.float64)
    for k in range(n_blocks):
        out[k] = scores[k * block_size:(k + 1) * block_size].sum()
    return out


# ------------------------------------------- Section 4.4, "Fidelity of Hidden States"
def mass_recovery(scores: np.ndarray, idx: np.ndarray) -> float:
    """Share of the attention weights covered by the retained tokens ``idx``: every window
    row of Eq. 1 sums to 1, so the share over all heads and window rows of a layer is
    ``sum_{j in idx} S_j / sum_j S_j``."""
    scores = np.asarray(scores, dtype=np.float64)
    return float(scores[np.asarray(idx, dtype=np.int64)].sum() / scores.sum())


# ------------------------------------- Eq. 11 - 13 past the pivot (Algorithm 1, l > L*)
def reduced_layer(q_win: np.ndarray, k: np.ndarray, scale: float, i_struct: np.ndarray,
                  positions: np.ndarray, kv_budget: int, window: int) -> Dict[str, np.ndarray]:
    """One layer past the pivot.  The sequence has been cut to the structural set (Eq. 11), so
    the layer only has the keys ``k[:, i_struct]``; the window is the tail of ``i_struct`` (R9),
    hence the window queries are unchanged and causality in reduced order is causality in
    original order.  Scoring (Eq. 1 - 2) and selection (Eq. 13) run on that reduced sequence;
    a selected reduced index ``r`` names the token whose original position is
    ``positions[i_struct][r]`` (Eq. 12: the position ids travel with the tokens).

    Returns ``S`` (reduced order), ``i_reduced`` (indices into the reduced sequence) and
    ``i_kv`` (the same tokens as original position ids)."""
    i_struct = np.asarray(i_struct, dtype=np.int64)
    pos_reduced = np.asarray(positions)[i_struct]                       # P' = P[I_struct]
    k_reduced = np.asarray(k, dtype=np.float64)[:, i_struct]
    out = score_layer(q_win, k_reduced, scale)
    i_reduced = select(out["S"], kv_budget, window)
    return {"S": out["S"], "entropy": out["entropy"], "i_reduced": i_reduced, "i_kv": pos_reduced[i_reduced]}


def prefill_reduced(layers: Sequence[Tuple[np.ndarray, np.ndarray, float]], positions: np.ndarray,
                    window: int, kv_budget: int, struct_budget: int, lam: float = PAPER_LAMBDA,
                    weights: Sequence[float] = PAPER_WEIGHTS, n_detect: Optional[int] = None,
                    l_limit: Optional[int] = None) -> Dict[str, object]:
    """Algorithm 1 with its truncation: the first ``n_detect`` layers (default: all) are scored on
    the full sequence and give the pivot, the centrality at the pivot and ``I_struct``; every
    layer ``l > L*`` then runs on the reduced sequence (``reduced_layer``).  ``recovery[l]`` is
    the share of layer ``l``'s full-sequence attention that the structural set covers (Section
    4.4, fidelity of hidden states), available here because the synthetic K is complete."""
    n_detect = len(layers) if n_detect is None else n_detect
    head = prefill(layers[:n_detect], window, kv_budget, struct_budget, lam, weights, l_limit)
    L_star, i_struct = head["pivot"], head["i_struct"]
    past, recovery = {}, {}
    for l in range(L_star + 1, len(layers)):
        q, k, sc = layers[l]
        past[l] = reduced_layer(q, k, sc, i_struct, positions, kv_budget, window)
        recovery[l] = mass_recovery(score_layer(q, k, sc)["S"], i_struct)
    return {"head": head, "pivot": L_star, "i_struct": i_struct, "past": past, "recovery": recovery}


# ------------------------------------------------------------------- Algorithm 1
def prefill(layers: Sequence[Tuple[np.ndarray, np.ndarray, float]], window: int,
            kv_budget: int, struct_budget: int, lam: float = PAPER_LAMBDA,
            weights: Sequence[float] = PAPER_WEIGHTS,
            l_limit: Optional[int] = None) -> Dict[str, object]:
    """The scoring / selection skeleton of Algorithm 1 over ``layers`` =
    ``[(q_win, k, scale), ...]``: per-layer saliency and metrics, pivot, global
    centrality at the pivot, the structural index set and the per-layer KV sets."""
    outs = [score_layer(q, k, sc) for (q, k, sc) in layers]
    s_hist = np.stack([o["S"] for o in outs])
    metrics = np.array([[o["entropy"], o["sparsity"], o["variance"]] for o in outs])
    L_star = pivot(metrics, weights, l_limit)
    C = centrality(s_hist, lam, L_star)
    return {
        "s_hist": s_hist,
        "metrics": metrics,
        "pivot": L_star,
        "transition": transition_scores(metrics, weights),
        "C": C,
        "i_struct": select(C, struct_budget, window),
        "i_kv": np.stack([select(s_hist[l], kv_budget, window) for l in range(len(outs))]),
    }


# --------------------------- Section 4.1 (implementation details): batches of prompts
def prefill_batch(prompts: Sequence[Sequence[Tuple[np.ndarray, np.ndarray, float]]], window: int,
                  kv_budgets: Sequence[int], struct_budgets: Sequence[int], lam: float = PAPER_LAMBDA,
                  weights: Sequence[float] = PAPER_WEIGHTS,
                  l_limit: Optional[int] = None) -> Dict[str, object]:
    """A batch of prompts of different lengths: every prompt is an independent problem with its
    own length, pivot and index sets (``prefill`` per prompt).  ``reduced_at[b, l]`` is the
    masked state transition: True where layer ``l`` of prompt ``b`` runs past that prompt's pivot,
    i.e. on its reduced sequence.  Index lists come back padded with -1 to the largest budget
    (the padded addressing of a batch); padding is never a token."""
    per = [prefill(layers, window, kb, sb, lam, weights, l_limit)
           for layers, kb, sb in zip(prompts, kv_budgets, struct_budgets)]
    L = max(len(p) for p in prompts)
    pivots = np.array([r["pivot"] for r in per], dtype=np.int64)
    reduced_at = np.arange(L)[None, :] > pivots[:, None]
    i_struct = np.full((len(per), max(struct_budgets)), -1, dtype=np.int64)
    i_kv = np.full((len(per), L, max(kv_budgets)), -1, dtype=np.int64)
    for b, r in enumerate(per):
        i_struct[b, :struct_budgets[b]] = r["i_struct"]
        i_kv[b, :len(prompts[b]), :kv_budgets[b]] = r["i_kv"]
    return {"per_prompt": per, "pivots": pivots, "reduced_at": reduced_at, "i_struct": i_struct, "i_kv": i_kv}
