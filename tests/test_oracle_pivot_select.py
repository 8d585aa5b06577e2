"""Pins for the oracle's centrality (Eq. 3), pivot (Eq. 7-9), selection
(Eq. 10 / 13) and compaction (Algorithm 1 lines 13, 17)."""
import math

import numpy as np
import pytest

from oracle import structkv_oracle as O


# ------------------------------------------------------------------ Eq. 3
def test_centrality_limits_and_mass():
    rng = np.random.default_rng(0)
    s = rng.random((6, 20))
    np.testing.assert_allclose(O.centrality(s, 1.0, 4), s[:5].sum(axis=0), rtol=1e-14)
    np.testing.assert_allclose(O.centrality(s, 1e-30, 3), s[3], rtol=1e-12)
    for lam in (0.5, 0.9, 1.0):
        for p in (0, 2, 5):
            np.testing.assert_allclose(O.centrality(s, lam, p), O.centrality_recursive(s, lam, p),
                                       rtol=1e-13)
    # rows of mass H: total centrality is the geometric series H (1 - lam^(p+1)) / (1 - lam)
    H = 7.0
    s = s / s.sum(axis=1, keepdims=True) * H
    lam, p = 0.9, 4
    assert abs(O.centrality(s, lam, p).sum() - H * (1 - lam ** (p + 1)) / (1 - lam)) < 1e-12


def test_centrality_weights_by_hand():
    s = np.array([[1.0, 0.0], [0.0, 1.0], [2.0, 2.0]])
    np.testing.assert_allclose(O.centrality(s, 0.5, 2), [0.25 + 2.0, 0.5 + 2.0], rtol=1e-15)
    np.testing.assert_allclose(O.centrality(s, 0.5, 1), [0.5, 1.0], rtol=1e-15)


# --------------------------------------------------------------- Eq. 7 - 9
def load_pivot_tables():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "pivot_tables.txt")
    cases = []
    with open(path) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            fields = dict(kv.split("=") for kv in line.split(";"))
            vec = lambda s: [float(x) for x in s.split(",")]
            cases.append((vec(fields["H"]), vec(fields["rho"]), vec(fields["V"]), vec(fields["w"]),
                          int(fields["limit"]), int(fields["pivot"]), vec(fields["T"])))
    return cases


@pytest.mark.parametrize("case", load_pivot_tables())
def test_pivot_hand_tables(case):
    H, rho, V, w, limit, expected, T = case
    metrics = np.stack([H, rho, V], axis=1)
    assert O.pivot(metrics, w, None if limit < 0 else limit) == expected
    np.testing.assert_allclose(O.transition_scores(metrics, w)[1:], T, atol=1e-12)


def test_pivot_affine_invariance_and_constant_metric():
    rng = np.random.default_rng(1)
    m = rng.random((9, 3))
    base = O.transition_scores(m)
    m2 = m * np.array([3.0, 0.25, 11.0]) + np.array([5.0, -2.0, 0.1])
    np.testing.assert_allclose(O.transition_scores(m2)[1:], base[1:], atol=1e-12)
    m3 = m.copy(); m3[:, 1] = 0.4                         # constant sparsity: its term vanishes
    t3 = O.transition_scores(m3)
    t_ref = 0.2 * O.normalised_gradient(-m[:, 0]) + 0.5 * O.normalised_gradient(m[:, 2])
    np.testing.assert_allclose(t3[1:], t_ref[1:], atol=1e-12)
    g = O.normalised_gradient(m[:, 0])
    assert g[1:].min() == 0.0 and g[1:].max() == 1.0


def test_pivot_first_maximum_and_limit():
    ent = np.array([5.0, 4.0, 3.0, 2.0])                  # equal drops: every T_l ties
    m = np.stack([ent, np.zeros(4), np.zeros(4)], axis=1)
    assert O.pivot(m, (1, 0, 0)) == 1
    ent = np.array([5.0, 5.0, 1.0, 1.0, 0.5])
    m = np.stack([ent, np.zeros(5), np.zeros(5)], axis=1)
    assert O.pivot(m, (1, 0, 0)) == 2
    assert O.pivot(m, (1, 0, 0), l_limit=1) == 1
    assert O.pivot(m, (1, 0, 0), l_limit=4) == 2


# ---------------------------------------------------------- Eq. 10 / Eq. 13
def brute_select(scores, budget, window):
    n = len(scores)
    prefix = list(range(n - window))
    prefix.sort(key=lambda j: (-scores[j], j))
    return sorted(prefix[:budget - window]) + list(range(n - window, n))


@pytest.mark.parametrize("n,window,budget", [(50, 4, 10), (50, 4, 5), (50, 4, 50), (33, 1, 2), (64, 8, 8)])
def test_select_brute_force(n, window, budget):
    rng = np.random.default_rng(n + budget)
    s = rng.random(n)
    got = O.select(s, budget, window)
    assert got.tolist() == brute_select(s.tolist(), budget, window)
    assert len(got) == budget and np.all(np.diff(got) > 0)
    assert set(range(n - window, n)) <= set(got.tolist())


def test_select_ties_go_to_lower_index():
    s = np.array([1.0, 3.0, 3.0, 3.0, 0.5, 3.0, 9.0, 9.0])   # window = last 2
    assert O.select(s, 4, 2).tolist() == [1, 2, 6, 7]
    assert O.select(s, 5, 2).tolist() == [1, 2, 3, 6, 7]
    s = np.zeros(12)
    assert O.select(s, 7, 3).tolist() == [0, 1, 2, 3, 9, 10, 11]
    # window scores never compete
    s = np.array([0.1, 0.2, 0.3, 100.0, 100.0])
    assert O.select(s, 3, 2).tolist() == [2, 3, 4]


def test_select_matches_stable_argsort():
    rng = np.random.default_rng(7)
    s = rng.integers(0, 20, size=5000).astype(np.float32)   # many ties
    w, b = 16, 700
    order = np.argsort(-s[:5000 - w], kind="stable")[:b - w]
    want = np.concatenate([np.sort(order), np.arange(5000 - w, 5000)])
    assert O.select(s, b, w).tolist() == want.tolist()


# ---------------------------------------------------------------- compaction
def test_compact_is_fancy_indexing():
    rng = np.random.default_rng(3)
    src = rng.integers(0, 255, size=(3, 40, 16), dtype=np.uint8)
    idx = np.array([0, 5, 6, 39])
    dst = O.compact(src, idx)
    assert dst.shape == (3, 4, 16) and dst.flags["C_CONTIGUOUS"]
    for g in range(3):
        for r, j in enumerate(idx):
            assert dst[g, r].tobytes() == src[g, j].tobytes()
