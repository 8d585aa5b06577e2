"""GPU parity over the WHOLE depth of every full-size workload, in the launch configuration the
benchmark times: all layers of llama32k, llama128k (its three budgets), qwen64k and the streamed
llama256k go through ``pipeline.Prefill`` and are compared with the float64 oracle on the same
bits -- every S^(l) and metric triple, the pivot for both weight sets, C* and the running C,
I_struct, every I_KV^(l) under the gap rule, K/V compaction bit for bit on sampled layers, the
hidden-state and position gathers.  The oracle's layers run side by side in worker processes
(``tests/oracle_pool.py``: plumbing only)."""
import numpy as np
import pytest
import torch

from oracle import structkv_oracle as O
from paper_2604_06746_b200 import synth
from tests import oracle_pool as OP
from tests import parity as P

pytestmark = pytest.mark.gpu

PIVOT_MARGIN = 0.02          # the oracle's best and second-best transition scores must differ by this much
WEIGHT_SETS = (O.PAPER_WEIGHTS, (1.0, 0.0, 0.0))


@pytest.fixture(scope="module")
def mods(cuda_device):
    from paper_2604_06746_b200 import binding, pipeline
    return binding, pipeline


def oracle_worker_count(wl):
    k64 = wl.n_kv_heads * wl.seq * wl.head_dim * 8
    per_worker = 1.6 * k64 + 8 * wl.window * wl.seq * 8 + 3 * wl.n_q_heads * wl.seq * 8
    return OP.default_workers(per_worker)


def check_against_oracle(wl, pfs, ora, tag):
    """``pfs[(weights, kv_budget)]`` are finished Prefill objects, ``ora[weights]`` the oracle's results."""
    for (weights, kv_b), pf in pfs.items():
        o = ora[weights]
        st_b = wl.struct_budget(kv_b)
        t = f"{tag} weights={weights} budget={kv_b}"
        s_hist = pf.s_hist.cpu().numpy()
        metrics = pf.metrics.cpu().numpy()
        for l in range(wl.n_layers):
            P.assert_scores_close(s_hist[l], o["s_hist"][l], f"{t} S layer {l}")
            for c, name in enumerate(("entropy", "sparsity", "variance")):
                P.assert_metric_close(metrics[l, c], o["metrics"][l, c], f"{t} {name} layer {l}")
        T = np.sort(o["transition"][1:])[::-1]
        assert T[0] - T[1] >= PIVOT_MARGIN, f"{t}: oracle transition margin {T[0] - T[1]:.4f}"
        assert pf.pivot == o["pivot"], (t, pf.pivot, o["pivot"])
        np.testing.assert_allclose(pf.transition[1:], o["transition"][1:], atol=1e-2)
        P.assert_scores_close(pf.c_star.cpu().numpy(), o["C"], f"{t} C*")
        P.assert_scores_close(pf.c_running.cpu().numpy(),
                              O.centrality_recursive(o["s_hist"], pf.lam, wl.n_layers - 1), f"{t} C running")
        P.assert_selection_matches(pf.i_struct.cpu().numpy(), o["C"], st_b, wl.window, o["i_struct"][st_b],
                                   f"{t} I_struct")
        i_kv = pf.i_kv.cpu().numpy()
        for l in range(wl.n_layers):
            P.assert_selection_matches(i_kv[l], o["s_hist"][l], kv_b, wl.window, o["i_kv"][kv_b][l],
                                       f"{t} I_KV layer {l}")
        assert abs(float(s_hist.sum()) - wl.n_q_heads * wl.n_layers) < 1e-3 * wl.n_q_heads * wl.n_layers


def kv_bits(t):
    kv = t["kv"]
    return kv.view(2 * kv.shape[1], kv.shape[2], kv.shape[3]).view(torch.int16).cpu().numpy()


@pytest.mark.parametrize("name", ["llama32k", "llama128k", "qwen64k"])
def test_resident_workload_all_layers(mods, cuda_device, name):
    binding, pipeline = mods
    wl = synth.WORKLOADS[name]
    pl = synth.plan(wl)
    dev = cuda_device
    layers = [synth.make_layer(wl, pl, l, device=dev) for l in range(wl.n_layers)]
    width = 512
    g = torch.Generator(device=dev); g.manual_seed(11)
    hidden = torch.randn((wl.seq, width), generator=g, device=dev).to(torch.bfloat16)
    positions = torch.arange(wl.seq, device=dev, dtype=torch.int32) * 2 + 5
    pfs = {}
    for weights in WEIGHT_SETS:
        for kv_b in wl.budgets:
            pf = pipeline.Prefill(wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq,
                                  kv_b, wl.struct_budget(kv_b), torch.bfloat16, hidden_dim=width, device=dev,
                                  weights=weights)
            pf.run(layers, hidden, positions)
            torch.cuda.synchronize()
            assert pf.ctx.poll_device_status() == binding.OK
            pfs[(weights, kv_b)] = pf
    tasks = ((l, OP.bits_of(t["q_win"]), OP.bits_of(t["k"]), t["scale"], None) for l, t in enumerate(layers))
    s_hist, metrics = OP.score_layers(tasks, wl.n_layers, oracle_worker_count(wl))
    ora = {w: OP.assemble(s_hist, metrics, wl.window, wl.budgets, [wl.struct_budget(b) for b in wl.budgets],
                          O.PAPER_LAMBDA, w) for w in WEIGHT_SETS}
    check_against_oracle(wl, pfs, ora, name)
    # gathers, bit for bit against the oracle's gather on the GPU's own index sets
    hid_bits = hidden.view(torch.int16).cpu().numpy()[None]
    pos_host = positions.cpu().numpy()[None]
    sampled = sorted({0, wl.n_layers // 3, (2 * wl.n_layers) // 3, wl.n_layers - 1})
    src_bits = {l: kv_bits(layers[l]) for l in sampled}
    for (weights, kv_b), pf in pfs.items():
        idx = pf.i_struct.cpu().numpy()
        assert np.array_equal(pf.hidden_out.view(torch.int16).cpu().numpy(), O.compact(hid_bits, idx)[0])
        assert np.array_equal(pf.pos_out.cpu().numpy(), O.compact(pos_host, idx)[0])
        if weights != WEIGHT_SETS[0]:
            continue                              # the KV index sets do not depend on the pivot weights
        i_kv = pf.i_kv.cpu().numpy()
        for l in sampled:
            got = pf.kv_out[l].view(2 * wl.n_kv_heads, kv_b, wl.head_dim).view(torch.int16).cpu().numpy()
            assert np.array_equal(got, O.compact(src_bits[l], i_kv[l])), f"{name} K/V layer {l} budget {kv_b}"


def test_streamed_long_context_all_layers(mods, cuda_device):
    """llama256k the way it is meant to run: each layer generated, scored and dropped (one layer's
    K/V resident), centrality accumulated across all 32 layers; then the pivot, both index sets and
    the full-width hidden-state gather; K/V compaction on sampled layers streamed in again."""
    binding, pipeline = mods
    wl = synth.WORKLOADS["llama256k"]
    pl = synth.plan(wl)
    dev = cuda_device
    kv_b, st_b = wl.budget, wl.struct_budget()
    hidden, positions = synth.make_hidden(wl, device=dev)
    pfs = {w: pipeline.Prefill(wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, kv_b,
                               st_b, torch.bfloat16, hidden_dim=wl.hidden_dim, device=dev, weights=w,
                               keep_kv=False) for w in WEIGHT_SETS}

    def tasks():
        for l in range(wl.n_layers):
            t = synth.make_layer(wl, pl, l, device=dev, with_v=False)
            for pf in pfs.values():
                pf.score(l, t["q_win"], t["k"], t["scale"])
            yield (l, OP.bits_of(t["q_win"]), OP.bits_of(t["k"]), t["scale"], None)
            del t

    s_hist, metrics = OP.score_layers(tasks(), wl.n_layers, oracle_worker_count(wl))
    for pf in pfs.values():
        pf.detect_and_select(wl.n_layers)
        pf.compact_hidden(hidden, positions)
    torch.cuda.synchronize()
    ora = {w: OP.assemble(s_hist, metrics, wl.window, (kv_b,), (st_b,), O.PAPER_LAMBDA, w) for w in WEIGHT_SETS}
    check_against_oracle(wl, {(w, kv_b): pf for w, pf in pfs.items()}, ora, wl.name)
    pos_host = positions.cpu().numpy()[None]
    hid_bits = hidden.view(torch.int16).cpu().numpy()[None]
    for w, pf in pfs.items():
        assert pf.ctx.poll_device_status() == binding.OK
        idx = pf.i_struct.cpu().numpy()
        assert np.array_equal(pf.pos_out.cpu().numpy(), O.compact(pos_host, idx)[0])
        assert np.array_equal(pf.hidden_out.view(torch.int16).cpu().numpy(), O.compact(hid_bits, idx)[0])
    del hid_bits
    pf = pfs[WEIGHT_SETS[0]]
    i_kv = pf.i_kv.cpu().numpy()
    for l in (1, 19):                                                      # second streaming sweep
        t = synth.make_layer(wl, pl, l, device=dev)
        pf.compact_kv(l, t["k"], t["v"], t["kv"])
        torch.cuda.synchronize()
        got = pf.kv_out[0].view(2 * wl.n_kv_heads, kv_b, wl.head_dim).view(torch.int16).cpu().numpy()
        assert np.array_equal(got, O.compact(kv_bits(t), i_kv[l])), f"llama256k K/V layer {l}"
        del t
