"""Pins for the oracle's scoring functions (Eq. 1, 2, 4, 5, 6): invariants,
closed forms, a library routine, brute force and structural properties."""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import structkv_oracle as O


def rand_case(seed, H=4, Hkv=2, w=3, d=5, N=11):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((H, w, d)), rng.standard_normal((Hkv, N, d)), 0.7


def test_rows_sum_to_one_and_causal_mask():
    q, k, sc = rand_case(1, H=4, Hkv=2, w=5, d=8, N=40)
    for a in O.window_attention(q, k, sc):
        assert a.shape == (5, 40)
        np.testing.assert_allclose(a.sum(axis=1), 1.0, atol=1e-12)
        for i in range(5):
            t = 40 - 5 + i
            assert np.all(a[i, t + 1:] == 0.0)
            assert np.all(a[i, :t + 1] > 0.0)


def test_mass_equals_number_of_heads():
    q, k, sc = rand_case(2, H=6, Hkv=3, w=4, d=8, N=64)
    out = O.score_layer(q, k, sc)
    assert abs(out["S"].sum() - 6.0) < 1e-10
    np.testing.assert_allclose(out["head_cols"].sum(axis=1), 1.0, atol=1e-12)


def uniform_closed_form(H, w, N):
    """All logits equal: row i (position t = N-w+i) is uniform over t+1 keys."""
    S = np.zeros(N)
    for j in range(N):
        m = max(0, j - (N - w))         # first window row that sees key j
        S[j] = (H / w) * math.fsum(1.0 / (N - w + i + 1) for i in range(m, w))
    ent = math.fsum(math.log(N - w + i + 1) for i in range(w)) / w
    return S, ent


@pytest.mark.parametrize("mode", ["zero_scale", "identical_keys"])
def test_uniform_closed_form(mode):
    H, Hkv, w, d, N = 4, 2, 6, 8, 50
    rng = np.random.default_rng(3)
    q = rng.standard_normal((H, w, d))
    if mode == "zero_scale":
        k, sc = rng.standard_normal((Hkv, N, d)), 0.0
    else:
        k, sc = np.repeat(rng.standard_normal((Hkv, 1, d)), N, axis=1), 0.9
    out = O.score_layer(q, k, sc)
    S, ent = uniform_closed_form(H, w, N)
    np.testing.assert_allclose(out["S"], S, rtol=1e-12)
    assert abs(out["entropy"] - ent) < 1e-12
    abar = S / H                                  # every head has the same pooled vector
    k_rho = max(1, N // 10)
    assert abs(out["sparsity"] - np.sort(abar)[::-1][:k_rho].sum()) < 1e-12
    assert abs(out["variance"] - (np.mean(abar ** 2) - (1.0 / N) ** 2)) < 1e-14


def test_single_row_reduces_to_library_softmax():
    rng = np.random.default_rng(4)
    H, d, N = 3, 16, 200
    q = rng.standard_normal((H, 1, d))
    k = rng.standard_normal((H, N, d))            # G = 1
    sc = 1.0 / math.sqrt(d)
    out = O.score_layer(q, k, sc)
    ref = np.zeros(N)
    ent = 0.0
    for h in range(H):
        p = scipy.special.softmax(sc * (k[h] @ q[h, 0]))
        ref += p
        ent += float(scipy.stats.entropy(p))
    np.testing.assert_allclose(out["S"], ref, rtol=1e-12)
    assert abs(out["entropy"] - ent / H) < 1e-12


def brute_force(q, k, sc):
    """Pure-Python loops straight from Eq. 1, 2 and 4."""
    H, w, d = q.shape
    Hkv, N, _ = k.shape
    G = H // Hkv
    S = [0.0] * N
    cols = [[0.0] * N for _ in range(H)]
    ent = 0.0
    for h in range(H):
        g = h // G
        for i in range(w):
            t = N - w + i
            logits = [sc * sum(q[h, i, c] * k[g, j, c] for c in range(d)) for j in range(t + 1)]
            z = sum(math.exp(x) for x in logits)
            for j, x in enumerate(logits):
                a = math.exp(x) / z
                cols[h][j] += a / w
                S[j] += a / w
                ent -= a * math.log(a) / (H * w)
    return np.array(S), np.array(cols), ent


@pytest.mark.parametrize("seed", [5, 6, 7])
def test_brute_force_tiny(seed):
    q, k, sc = rand_case(seed)
    out = O.score_layer(q, k, sc)
    S, cols, ent = brute_force(q, k, sc)
    np.testing.assert_allclose(out["S"], S, rtol=1e-11)
    np.testing.assert_allclose(out["head_cols"], cols, rtol=1e-11)
    assert abs(out["entropy"] - ent) < 1e-11
    k_rho = max(1, k.shape[1] // 10)
    rho = np.mean([sorted(c, reverse=True)[:k_rho] for c in cols.tolist()], axis=0).sum()
    assert abs(out["sparsity"] - rho) < 1e-12
    var = np.mean([np.mean((c - c.mean()) ** 2) for c in cols])
    assert abs(out["variance"] - var) < 1e-14


def test_prefix_permutation_equivariance():
    q, k, sc = rand_case(8, H=4, Hkv=2, w=4, d=8, N=30)
    perm = np.random.default_rng(0).permutation(30 - 4)
    full = np.concatenate([perm, np.arange(26, 30)])
    a = O.score_layer(q, k, sc)
    b = O.score_layer(q, k[:, full], sc)
    np.testing.assert_allclose(b["S"], a["S"][full], rtol=1e-12)
    assert abs(a["entropy"] - b["entropy"]) < 1e-12
    assert abs(a["sparsity"] - b["sparsity"]) < 1e-12


def test_gqa_head_to_group_mapping():
    """A key planted in KV head 1 only must show up in query heads 2 and 3 only."""
    H, Hkv, w, d, N = 4, 2, 3, 8, 40
    rng = np.random.default_rng(9)
    q = 0.01 * rng.standard_normal((H, w, d))
    q[:, :, 0] += 1.0
    k = 0.01 * rng.standard_normal((Hkv, N, d))
    k[1, 7, 0] += 12.0
    cols = O.score_layer(q, k, 1.0)["head_cols"]
    assert np.all(cols[2:, 7] > 0.99)
    assert np.all(cols[:2, 7] < 0.05)


def test_one_hot_limit():
    H, Hkv, w, d, N = 2, 1, 2, 4, 100
    q = np.zeros((H, w, d)); q[:, :, 0] = 1.0
    k = np.zeros((Hkv, N, d)); k[0, 13, 0] = 60.0
    out = O.score_layer(q, k, 1.0)
    assert 0.0 <= out["entropy"] < 1e-20
    assert abs(out["sparsity"] - 1.0) < 1e-12
    assert abs(out["variance"] - (1.0 / N) * (1.0 - 1.0 / N)) < 1e-12
    assert abs(out["S"][13] - H) < 1e-12


def test_two_level_closed_form_entropy():
    """One key with logit x among n-1 keys with logit 0 (w = 1):
    p = e^x / (e^x + n - 1),  H = -p log p - (n-1) r log r,  r = (1-p)/(n-1)."""
    n, x = 37, 2.5
    q = np.array([[[1.0]]]); k = np.zeros((1, n, 1)); k[0, 5, 0] = x
    out = O.score_layer(q, k, 1.0)
    p = math.exp(x) / (math.exp(x) + n - 1)
    r = (1 - p) / (n - 1)
    assert abs(out["entropy"] - (-p * math.log(p) - (n - 1) * r * math.log(r))) < 1e-13
    assert abs(out["S"][5] - p) < 1e-14


def test_entropy_bounds_and_scale_sign():
    q, k, _ = rand_case(10, H=4, Hkv=2, w=4, d=8, N=64)
    ents = [O.score_layer(q, k, sc)["entropy"] for sc in (0.0, 0.5, 1.0, 3.0)]
    assert all(0.0 <= e <= math.log(64) + 1e-12 for e in ents)
    assert ents[0] > ents[1] > ents[2] > ents[3]       # sharper logits, lower entropy
    # the key most aligned with a query gets the largest weight (sign of the logit)
    q1 = np.zeros((1, 1, 3)); q1[0, 0, 1] = 1.0
    k1 = np.zeros((1, 9, 3)); k1[0, 4, 1] = 3.0; k1[0, 2, 1] = -3.0
    S = O.score_layer(q1, k1, 1.0)["S"]
    assert S.argmax() == 4 and S.argmin() == 2


def test_head_statistics_closed_forms_and_brute_force():
    """Eq. 5-6 on pooled vectors given directly: uniform vectors (top mass k/N, zero variance),
    one-hot vectors (top mass 1, variance (1/N)(1 - 1/N)), a two-level vector worked by hand, and a
    pure-Python selection of the largest entries."""
    N = 50                                                       # k_rho = 5
    rho, var = O.head_statistics(np.full((3, N), 1.0 / N))
    assert rho == pytest.approx(5.0 / N, rel=1e-14) and var == pytest.approx(0.0, abs=1e-30)
    one_hot = np.zeros((2, N))
    one_hot[0, 7] = one_hot[1, 49] = 1.0
    rho, var = O.head_statistics(one_hot)
    assert rho == pytest.approx(1.0) and var == pytest.approx((1.0 / N) * (1.0 - 1.0 / N), rel=1e-13)
    # 3 entries of 0.2 and 47 of 0.4 / 47: the five largest are the three big ones and two small ones
    two = np.full((1, N), 0.4 / 47)
    two[0, [4, 20, 33]] = 0.2
    rho, var = O.head_statistics(two)
    assert rho == pytest.approx(0.6 + 2 * 0.4 / 47, rel=1e-13)
    assert var == pytest.approx((3 * 0.2 ** 2 + 47 * (0.4 / 47) ** 2) / N - (1.0 / N) ** 2, rel=1e-12)
    # heads are averaged: a uniform and a one-hot head together
    rho, var = O.head_statistics(np.stack([np.full(N, 1.0 / N), one_hot[0]]))
    assert rho == pytest.approx(0.5 * (5.0 / N + 1.0)) and var == pytest.approx(0.5 * (1.0 / N) * (1.0 - 1.0 / N))
    rng = np.random.default_rng(5)
    x = rng.random((4, 37)) ** 3
    x /= x.sum(axis=1, keepdims=True)
    want_rho = want_var = 0.0
    for row in x:
        vals = sorted(row.tolist(), reverse=True)
        want_rho += sum(vals[:3])                                # floor(0.1 * 37) = 3
        mean = sum(row.tolist()) / 37
        want_var += sum((v - mean) ** 2 for v in row.tolist()) / 37
    rho, var = O.head_statistics(x)
    assert rho == pytest.approx(want_rho / 4, rel=1e-13) and var == pytest.approx(want_var / 4, rel=1e-12)
