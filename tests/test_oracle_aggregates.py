"""Pins for the oracle's block-level aggregation (paged KV) and attention-mass recovery."""
import numpy as np
import pytest

from oracle import structkv_oracle as O


@pytest.mark.parametrize("n,bs", [(64, 16), (70, 16), (5, 8), (33, 1), (128, 128), (100, 7)])
def test_block_scores_against_a_library_segmented_sum_and_invariants(n, bs):
    rng = np.random.default_rng(n * 31 + bs)
    c = rng.random(n)
    got = O.block_scores(c, bs)
    assert got.shape == (-(-n // bs),)
    np.testing.assert_allclose(got, np.add.reduceat(c, np.arange(0, n, bs)), rtol=1e-13)   # library routine
    assert abs(got.sum() - c.sum()) < 1e-12                                                # mass is conserved
    ones = O.block_scores(np.ones(n), bs)                                                  # closed form: block sizes
    assert np.array_equal(ones[:-1], np.full(len(ones) - 1, bs)) and ones[-1] == n - bs * (len(ones) - 1)


def test_block_scores_special_cases():
    c = np.arange(10, dtype=np.float64)
    assert np.array_equal(O.block_scores(c, 1), c)                     # one token per block: identity
    assert np.array_equal(O.block_scores(c, 10), [45.0])               # one block: the total
    assert np.array_equal(O.block_scores(c, 4), [6.0, 22.0, 17.0])     # by hand: 0+1+2+3, 4+5+6+7, 8+9


def test_block_eviction_keeps_a_contiguous_anchor():
    """A run of moderately important tokens outweighs isolated spikes once scores are pooled
    per block: the block holding the run is kept, the spikes' blocks are not (Section 4.1)."""
    c = np.full(64, 0.01)
    c[16:32] = 0.3                      # a contiguous anchor (one whole block of 16)
    c[[3, 40, 59]] = 1.0                # isolated spikes in three other blocks
    blocks = O.block_scores(c, 16)
    assert int(np.argmax(blocks)) == 1
    keep_tokens = set(O.select(c, 16 + 4, 4)[:16].tolist())
    assert {3, 40, 59} <= keep_tokens   # token-wise selection starts from the spikes instead


def test_mass_recovery_closed_forms_and_brute_force():
    rng = np.random.default_rng(2)
    s = rng.random(50)
    assert O.mass_recovery(s, np.arange(50)) == pytest.approx(1.0, abs=1e-15)   # everything kept
    assert O.mass_recovery(s, np.array([], dtype=np.int64)) == 0.0              # nothing kept
    assert O.mass_recovery(np.ones(40), np.arange(10)) == pytest.approx(0.25)   # uniform: |I| / N
    idx = np.array([4, 7, 30])
    assert O.mass_recovery(s, idx) == pytest.approx(sum(s[j] for j in idx) / sum(s), rel=1e-14)
    a, b = np.array([1, 2, 3]), np.array([10, 11])                              # additive over disjoint sets
    assert O.mass_recovery(s, np.concatenate([a, b])) == pytest.approx(O.mass_recovery(s, a) + O.mass_recovery(s, b))


def test_mass_recovery_equals_the_row_wise_definition():
    """Straight from Eq. 1: the mean over heads and window rows of sum_{j in I} a_{t,j}."""
    rng = np.random.default_rng(9)
    q, k = rng.standard_normal((4, 3, 8)), rng.standard_normal((2, 30, 8))
    idx = np.array([0, 5, 6, 20, 29])
    rows = [a[:, idx].sum(axis=1) for a in O.window_attention(q, k, 0.5)]
    assert O.mass_recovery(O.score_layer(q, k, 0.5)["S"], idx) == pytest.approx(np.mean(rows), rel=1e-12)


def test_group_saliency_sums_to_eq2_and_matches_brute_force():
    rng = np.random.default_rng(21)
    q, k = rng.standard_normal((6, 4, 8)), rng.standard_normal((3, 25, 8))      # G = 2
    out = O.score_layer(q, k, 0.4)
    g = O.group_saliency(out["head_cols"], 2)
    assert g.shape == (3, 25)
    np.testing.assert_allclose(g.sum(axis=0), out["S"], rtol=1e-13)              # Eq. 2 is the sum over groups
    np.testing.assert_allclose(g.sum(axis=1), 2.0, rtol=1e-12)                   # each head's pooled row sums to 1
    for grp in range(3):                                                          # brute force over the two heads
        np.testing.assert_allclose(g[grp], out["head_cols"][2 * grp] + out["head_cols"][2 * grp + 1], rtol=1e-15)
    assert np.array_equal(O.group_saliency(out["head_cols"], 1), out["head_cols"])   # G = 1: identity
    # a head only reads its own KV group: changing the keys of group 2 leaves groups 0 and 1 alone
    k2 = k.copy(); k2[2] = rng.standard_normal((25, 8))
    g2 = O.group_saliency(O.score_layer(q, k2, 0.4)["head_cols"], 2)
    assert np.array_equal(g2[:2], g[:2]) and not np.allclose(g2[2], g[2])


def test_compact_per_slab_is_a_library_take_along_axis():
    rng = np.random.default_rng(22)
    src = rng.integers(0, 1000, size=(3, 20, 5))
    idx = np.stack([rng.choice(20, size=7, replace=False) for _ in range(3)])
    got = O.compact_per_slab(src, idx)
    assert np.array_equal(got, np.take_along_axis(src, idx[:, :, None], axis=1))
    same = np.tile(idx[:1], (3, 1))                                               # equal lists: the shared-list gather
    assert np.array_equal(O.compact_per_slab(src, same), O.compact(src, idx[0]))
