"""CPU pins of the oracle's batched prefill (prompts of different lengths, heterogeneous pivots)."""
import numpy as np

from oracle import structkv_oracle as O


def prompt(rng, L, H, Hkv, d, N, w, temps):
    return [(rng.standard_normal((H, w, d)), rng.standard_normal((Hkv, N, d)), 1.0 / (np.sqrt(d) * temps[l]))
            for l in range(L)]


def test_batch_equals_independent_prompts_and_padding_is_never_a_token():
    rng = np.random.default_rng(5)
    H, Hkv, d, w, L = 4, 2, 8, 4, 5
    lens = [50, 33, 71]
    temps = [(1.0, 2.0, 0.5, 0.6, 0.7), (1.0, 0.5, 0.55, 0.6, 2.0), (2.0, 1.9, 1.8, 0.4, 0.5)]   # pivots 2, 1, 3
    prompts = [prompt(rng, L, H, Hkv, d, n, w, t) for n, t in zip(lens, temps)]
    kvb, stb = [10, 8, 12], [20, 16, 24]
    out = O.prefill_batch(prompts, w, kvb, stb, weights=(1.0, 0.0, 0.0))
    assert out["pivots"].tolist() == [2, 1, 3]
    for b, p in enumerate(prompts):
        alone = O.prefill(p, w, kvb[b], stb[b], weights=(1.0, 0.0, 0.0))
        assert alone["pivot"] == out["pivots"][b]
        assert np.array_equal(out["i_struct"][b, :stb[b]], alone["i_struct"])
        assert np.all(out["i_struct"][b, stb[b]:] == -1)
        assert np.array_equal(out["i_kv"][b, :, :kvb[b]], alone["i_kv"])
        assert np.all(out["i_kv"][b, :, kvb[b]:] == -1)
        valid = out["i_kv"][b][out["i_kv"][b] >= 0]
        assert valid.max() < lens[b]                                  # a prompt never addresses a batch-mate's tokens
        assert np.array_equal(out["reduced_at"][b], np.arange(L) > alone["pivot"])
    # a prompt's result does not depend on its batch-mates
    again = O.prefill_batch([prompts[2], prompts[0]], w, [kvb[2], kvb[0]], [stb[2], stb[0]], weights=(1.0, 0.0, 0.0))
    assert np.array_equal(again["i_kv"][1, :, :kvb[0]], out["i_kv"][0, :, :kvb[0]])
    assert again["pivots"].tolist() == [3, 2]
    assert out["reduced_at"].sum(axis=1).tolist() == [L - 1 - 2, L - 1 - 1, L - 1 - 3]
