"""CPU pins of the oracle's post-pivot flow (Eq. 11 - 13 on the reduced sequence)."""
import numpy as np

from oracle import structkv_oracle as O


def make_layers(rng, L, H, Hkv, d, N, w):
    out = []
    for l in range(L):
        q = rng.standard_normal((H, w, d))
        k = rng.standard_normal((Hkv, N, d))
        out.append((q, k, (0.6 + 0.3 * l) / np.sqrt(d)))
    return out


def test_reduced_scores_are_the_full_attention_renormalised_over_the_kept_keys():
    """Softmax over a subset of the keys = the full softmax restricted to the subset and divided
    by the mass the subset holds in each row.  Checked from Eq. 1 directly."""
    rng = np.random.default_rng(0)
    H, Hkv, d, N, w = 4, 2, 8, 60, 5
    (q, k, sc), = make_layers(rng, 1, H, Hkv, d, N, w)
    keep = np.sort(np.concatenate([rng.choice(N - w, size=20, replace=False), np.arange(N - w, N)]))
    pos = np.arange(N) * 3 + 7
    red = O.reduced_layer(q, k, sc, keep, pos, kv_budget=12, window=w)
    expect = np.zeros(len(keep))
    for a in O.window_attention(q, k, sc):                 # [w, N] per head
        sub = a[:, keep]
        expect += (sub / sub.sum(axis=1, keepdims=True)).sum(axis=0) / w
    np.testing.assert_allclose(red["S"], expect, rtol=1e-12, atol=0)
    assert np.isclose(red["S"].sum(), H)
    # composition back to original position ids
    assert np.array_equal(red["i_kv"], pos[keep][red["i_reduced"]])
    assert np.all(np.diff(red["i_kv"]) > 0) and set(red["i_kv"]) <= set(pos[keep])
    assert np.array_equal(red["i_kv"][-w:], pos[N - w:])


def test_keeping_everything_reduces_nothing():
    rng = np.random.default_rng(1)
    H, Hkv, d, N, w, L = 4, 2, 8, 80, 4, 5
    layers = make_layers(rng, L, H, Hkv, d, N, w)
    pos = np.arange(N)
    full = O.prefill(layers, w, 20, N)
    red = O.prefill_reduced(layers, pos, w, 20, N)
    assert red["pivot"] == full["pivot"] and np.array_equal(red["i_struct"], np.arange(N))
    for l, r in red["past"].items():
        assert l > full["pivot"]
        np.testing.assert_allclose(r["S"], full["s_hist"][l], rtol=1e-12)
        assert np.array_equal(r["i_kv"], full["i_kv"][l])
        assert np.isclose(red["recovery"][l], 1.0)
    assert set(red["past"]) == set(range(full["pivot"] + 1, L))


def test_selection_past_the_pivot_stays_inside_the_structural_set():
    rng = np.random.default_rng(2)
    H, Hkv, d, N, w, L = 4, 1, 8, 120, 6, 6
    layers = make_layers(rng, L, H, Hkv, d, N, w)
    pos = np.arange(N) + 1000
    red = O.prefill_reduced(layers, pos, w, kv_budget=15, struct_budget=40, n_detect=4)
    assert red["pivot"] <= 3 and len(red["i_struct"]) == 40
    assert set(red["past"]) == set(range(red["pivot"] + 1, L))
    kept_positions = set(pos[red["i_struct"]].tolist())
    for l, r in red["past"].items():
        assert len(r["i_kv"]) == 15 and set(r["i_kv"].tolist()) <= kept_positions
        assert len(r["S"]) == 40 and np.all(r["i_reduced"] < 40)
        # a brute-force ranking of the reduced scores gives the same set
        order = sorted(range(40 - w), key=lambda j: (-r["S"][j], j))[:15 - w]
        assert sorted(order) == r["i_reduced"][:15 - w].tolist()
        assert 0.0 < red["recovery"][l] <= 1.0
        full_S = O.score_layer(*layers[l])["S"]
        assert np.isclose(red["recovery"][l], full_S[red["i_struct"]].sum() / full_S.sum())
