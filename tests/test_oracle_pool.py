"""The worker-pool plumbing around the oracle (used by the full-size GPU parity tests) returns
what the oracle returns in one process."""
import numpy as np

from oracle import structkv_oracle as O
from paper_2604_06746_b200 import synth
from tests import oracle_pool as OP


def test_pool_and_assembly_equal_the_single_process_oracle():
    wl = synth.WORKLOADS["llama32k"].scaled(700, n_layers=4, n_hubs=4, budgets=(100,))
    pl = synth.plan(wl)
    layers = [synth.make_layer(wl, pl, l, device="cpu", with_v=False) for l in range(wl.n_layers)]
    tasks = ((l, OP.bits_of(t["q_win"]), OP.bits_of(t["k"]), t["scale"], None) for l, t in enumerate(layers))
    s_hist, metrics = OP.score_layers(tasks, wl.n_layers, workers=2)
    got = OP.assemble(s_hist, metrics, wl.window, (100, 80), (200,), O.PAPER_LAMBDA, O.PAPER_WEIGHTS)
    ref = O.prefill([(synth.to_f64(t["q_win"]), synth.to_f64(t["k"]), t["scale"]) for t in layers],
                    wl.window, 100, 200)
    assert np.array_equal(got["s_hist"], ref["s_hist"]) and np.array_equal(got["metrics"], ref["metrics"])
    assert got["pivot"] == ref["pivot"] and np.array_equal(got["C"], ref["C"])
    assert np.array_equal(got["i_struct"][200], ref["i_struct"]) and np.array_equal(got["i_kv"][100], ref["i_kv"])
    assert got["i_kv"][80].shape == (4, 80)


def test_widening_is_exact_and_key_prefix_is_respected():
    import torch
    x = torch.randn(3, 50, 8).to(torch.bfloat16)
    assert np.array_equal(OP.widen(OP.bits_of(x)), synth.to_f64(x))
    y = torch.randn(2, 5, 4)
    assert np.array_equal(OP.widen(OP.bits_of(y)), synth.to_f64(y))
    wl = synth.WORKLOADS["tiny"].scaled(300, n_layers=1, n_hubs=2, budgets=(64,))
    t = synth.make_layer(wl, synth.plan(wl), 0, device="cpu", with_v=False)
    s_hist, metrics = OP.score_layers([(0, OP.bits_of(t["q_win"]), OP.bits_of(t["k"]), t["scale"], 200)], 1, 1)
    ref = O.score_layer(synth.to_f64(t["q_win"]), synth.to_f64(t["k"])[:, :200], t["scale"])
    assert np.array_equal(s_hist[0], ref["S"]) and metrics[0, 0] == ref["entropy"]
