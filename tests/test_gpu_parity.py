"""GPU parity: the CUDA path, called through the C ABI, against the float64 oracle on the
same seeded inputs -- element by element for saliency / centrality / metrics, identical pivot,
selection under the gap rule, bit-exact compaction."""
import numpy as np
import pytest
import torch

from oracle import structkv_oracle as O
from paper_2604_06746_b200 import synth
from tests import parity as P

pytestmark = pytest.mark.gpu

# The oracle's best and second-best transition scores must be this far apart for the pivot
# comparison to be meaningful (metric errors of 2e-3 move a transition score by < 1e-2).
PIVOT_MARGIN = 0.02


@pytest.fixture(scope="module")
def mods(cuda_device):
    from paper_2604_06746_b200 import binding, pipeline
    return binding, pipeline


def gpu_layers(wl, pl, device):
    """Small workloads are drawn on the host (one random stream whatever the device) and copied."""
    out = []
    for l in range(wl.n_layers):
        t = synth.make_layer(wl, pl, l, device="cpu")
        out.append({k: (v.to(device) if torch.is_tensor(v) else v) for k, v in t.items()})
    return out


def oracle_inputs(layers):
    return [(synth.to_f64(t["q_win"]), synth.to_f64(t["k"]), t["scale"]) for t in layers]


def run_and_compare(mods, wl, device, flags=0, check_hidden=True):
    binding, pipeline = mods
    pl = synth.plan(wl)
    layers = gpu_layers(wl, pl, device)
    hidden = positions = None
    if check_hidden:
        hd = 256
        g = torch.Generator(device=device); g.manual_seed(7)
        hidden = torch.randn((wl.seq, hd), generator=g, device=device).to(torch.bfloat16)
        positions = torch.arange(wl.seq, device=device, dtype=torch.int32) * 3 + 1
    kv_b, st_b = wl.budget, wl.struct_budget()
    results = {}
    for weights in (O.PAPER_WEIGHTS, (1.0, 0.0, 0.0)):
        pf = pipeline.Prefill(wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq,
                              kv_b, st_b, synth.torch_dtype(wl.dtype), hidden_dim=256 if check_hidden else 0,
                              device=device, weights=weights, flags=flags)
        pf.run(layers, hidden, positions)
        torch.cuda.synchronize()
        assert pf.ctx.poll_device_status() == binding.OK
        results[weights] = pf
    ora = {w: O.prefill(oracle_inputs(layers), wl.window, kv_b, st_b, weights=w) for w in results}

    for weights, pf in results.items():
        o = ora[weights]
        tag = f"{wl.name} weights={weights}"
        s_hist = pf.s_hist.cpu().numpy()
        metrics = pf.metrics.cpu().numpy()
        for l in range(wl.n_layers):
            P.assert_scores_close(s_hist[l], o["s_hist"][l], f"{tag} S layer {l}")
            for c, name in enumerate(("entropy", "sparsity", "variance")):
                P.assert_metric_close(metrics[l, c], o["metrics"][l, c], f"{tag} {name} layer {l}")
        # pivot: the oracle's own margin must be comfortable, then both sides must agree
        T = np.sort(o["transition"][1:])[::-1]
        assert len(T) < 2 or T[0] - T[1] >= PIVOT_MARGIN, f"{tag}: oracle transition margin {T[0] - T[1]}"
        assert pf.pivot == o["pivot"], tag
        np.testing.assert_allclose(pf.transition[1:], o["transition"][1:], atol=1e-2)
        P.assert_scores_close(pf.c_star.cpu().numpy(), o["C"], f"{tag} C*")
        # running recursion of Algorithm 1 line 6 over all layers
        P.assert_scores_close(pf.c_running.cpu().numpy(),
                              O.centrality_recursive(o["s_hist"], pf.lam, wl.n_layers - 1), f"{tag} C running")
        P.assert_selection_matches(pf.i_struct.cpu().numpy(), o["C"], st_b, wl.window, o["i_struct"],
                                   f"{tag} I_struct")
        i_kv = pf.i_kv.cpu().numpy()
        for l in range(wl.n_layers):
            P.assert_selection_matches(i_kv[l], o["s_hist"][l], kv_b, wl.window, o["i_kv"][l],
                                       f"{tag} I_KV layer {l}")
        # compaction is checked bit for bit against the oracle's gather on the GPU's own index sets
        for l, t in enumerate(layers):
            for name, out in (("k", pf.k_out), ("v", pf.v_out)):
                src = t[name].view(torch.int16 if t[name].element_size() == 2 else torch.int32).cpu().numpy()
                got = out[l].view(torch.int16 if out.element_size() == 2 else torch.int32).cpu().numpy()
                assert np.array_equal(got, O.compact(src, i_kv[l])), f"{tag} {name} layer {l}"
        if check_hidden:
            idx = pf.i_struct.cpu().numpy()
            assert np.array_equal(pf.hidden_out.view(torch.int16).cpu().numpy(),
                                  O.compact(hidden.view(torch.int16).cpu().numpy()[None], idx)[0])
            assert np.array_equal(pf.pos_out.cpu().numpy(), O.compact(positions.cpu().numpy()[None], idx)[0])
    return results, ora, pl


def test_tiny_fp32_full(mods, cuda_device):
    wl = synth.WORKLOADS["tiny"]
    results, ora, pl = run_and_compare(mods, wl, cuda_device)
    pf = results[(1.0, 0.0, 0.0)]
    assert pf.pivot == 3
    hubs = set(pl.hub_positions.tolist())
    assert hubs <= set(pf.i_struct.cpu().numpy().tolist())
    s_hist = pf.s_hist.cpu().numpy()
    np.testing.assert_allclose(s_hist.sum(axis=1), wl.n_q_heads, rtol=1e-4)


@pytest.mark.parametrize("name,seq,layers,hubs,budget", [
    ("llama32k", 4096 + 77, 6, 8, 300),       # ragged length: last key tile is partial
    ("llama128k", 3000, 5, 8, 200),           # sink + delimiters
    ("qwen64k", 2500, 5, 8, 400),             # GQA 7, window 128, heavy-tailed norms
])
@pytest.mark.parametrize("force_simt", [False, True], ids=["tensor_core", "cuda_core"])
def test_scaled_bf16_workloads(mods, cuda_device, name, seq, layers, hubs, budget, force_simt):
    binding, _ = mods
    wl = synth.WORKLOADS[name].scaled(seq, n_layers=layers, n_hubs=hubs, budgets=(budget,))
    run_and_compare(mods, wl, cuda_device, flags=binding.FLAG_FORCE_SIMT if force_simt else 0)


@pytest.mark.parametrize("H,Hkv,d,w,N,budget", [
    (4, 2, 64, 32, 700, 100),        # head_dim 64, 64 score rows per group (quarter of a row block)
    (4, 1, 128, 64, 129, 70),        # one KV head; a single full key tile plus one key
    (14, 2, 128, 128, 1500, 300),    # 896 rows per group: four row blocks, the last one half full
    (8, 8, 128, 64, 64, 64),         # N == w: every key is a window key, nothing to select
    (8, 2, 128, 64, 20000, 64),      # budget == window: only the window is kept
    (8, 2, 64, 128, 333, 333),       # budget == N: everything is kept
    (6, 2, 128, 8, 900, 50),         # the paper's default window (served by the CUDA-core scorer)
])
def test_shape_edges_bf16(mods, cuda_device, H, Hkv, d, w, N, budget):
    wl = synth.Workload(f"edge-{H}-{Hkv}-{d}-{w}-{N}", 7, 3, H, Hkv, d, N, w, (budget,), "bf16",
                        min(4, max(0, N - w - 1)), None, hub_layers=(1,), temperatures=(0.7, 1.0, 1.9),
                        sink=True)
    run_and_compare(mods, wl, cuda_device)


def test_results_are_deterministic(mods, cuda_device):
    binding, pipeline = mods
    wl = synth.WORKLOADS["tiny"]
    pl = synth.plan(wl)
    layers = gpu_layers(wl, pl, cuda_device)
    outs = []
    for _ in range(2):
        pf = pipeline.Prefill(wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq,
                              wl.budget, wl.struct_budget(), torch.float32, device=cuda_device)
        pf.run(layers)
        torch.cuda.synchronize()
        outs.append((pf.s_hist.clone(), pf.metrics.clone(), pf.i_kv.clone(), pf.i_struct.clone()))
    for a, b in zip(*outs):
        assert torch.equal(a, b)


# ---- full-size configurations, in the launch configuration the benchmark times -------------
# One or two layers of each full-size workload (the oracle needs seconds per layer at these
# sizes): saliency and metrics element by element, selection under the gap rule at every
# budget of the workload, compaction bit for bit on the selected rows.
@pytest.mark.parametrize("name,layers", [("llama32k", (0, 17)), ("llama128k", (3,)), ("qwen64k", (5,)),
                                         ("llama256k", (2,))])
def test_full_size_layers(mods, cuda_device, name, layers):
    binding, _ = mods
    wl = synth.WORKLOADS[name]
    pl = synth.plan(wl)
    dt = synth.torch_dtype(wl.dtype)
    ctx = binding.Context(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, dt, cuda_device)
    f32 = torch.float32
    for layer in layers:
        t = synth.make_layer(wl, pl, layer, device=cuda_device)
        s = torch.zeros(wl.seq, dtype=f32, device=cuda_device)
        c = torch.full((wl.seq,), 2.0, dtype=f32, device=cuda_device)
        m = torch.zeros(3, dtype=f32, device=cuda_device)
        ctx.score_layer(t["q_win"], t["k"], t["scale"], s, m, c_inout=c, lam=0.5)
        torch.cuda.synchronize()
        assert ctx.poll_device_status() == binding.OK
        o = O.score_layer(synth.to_f64(t["q_win"]), synth.to_f64(t["k"]), t["scale"])
        tag = f"{name} layer {layer}"
        P.assert_scores_close(s.cpu().numpy(), o["S"], f"{tag} S")
        P.assert_scores_close(c.cpu().numpy(), 1.0 + o["S"], f"{tag} C = 0.5 * 2 + S")
        for i, key in enumerate(("entropy", "sparsity", "variance")):
            P.assert_metric_close(m[i].item(), o[key], f"{tag} {key}")
        assert abs(s.sum().item() - wl.n_q_heads) < 1e-3 * wl.n_q_heads
        for budget in wl.budgets:
            idx = torch.zeros(budget, dtype=torch.int32, device=cuda_device)
            ctx.select(s, budget, wl.window, idx)
            torch.cuda.synchronize()
            P.assert_selection_matches(idx.cpu().numpy(), o["S"], budget, wl.window,
                                       O.select(o["S"], budget, wl.window), f"{tag} budget {budget}")
            # the selection kernel alone, on the GPU's own fp32 scores: exact, ties included
            assert np.array_equal(idx.cpu().numpy(), O.select(s.cpu().numpy(), budget, wl.window))
        out = torch.empty((2 * wl.n_kv_heads, wl.budget, wl.head_dim), dtype=dt, device=cuda_device)
        ctx.compact(t["kv"].view(2 * wl.n_kv_heads, wl.seq, wl.head_dim), idx, out)
        torch.cuda.synchronize()
        src = t["kv"].view(2 * wl.n_kv_heads, wl.seq, wl.head_dim).view(torch.int16).cpu().numpy()
        assert np.array_equal(out.view(torch.int16).cpu().numpy(), O.compact(src, idx.cpu().numpy()))
        del t
    ctx.close()


def test_hidden_state_gather_at_full_width(mods, cuda_device):
    """Hidden states of the streamed 256K workload (width 4096, bf16) at its structural budget."""
    binding, _ = mods
    wl = synth.WORKLOADS["llama256k"]
    hid, pos = synth.make_hidden(wl, device=cuda_device)
    ctx = binding.Context(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, torch.bfloat16, cuda_device)
    rng = np.random.default_rng(3)
    b = wl.struct_budget()
    idx_np = np.sort(rng.choice(wl.seq, size=b, replace=False)).astype(np.int32)
    idx = torch.from_numpy(idx_np).to(cuda_device)
    out = torch.empty((1, b, wl.hidden_dim), dtype=torch.bfloat16, device=cuda_device)
    pout = torch.empty((1, b, 1), dtype=torch.int32, device=cuda_device)
    ctx.compact(hid[None], idx, out)
    ctx.compact(pos[None, :, None], idx, pout)
    torch.cuda.synchronize()
    hid_bits = hid.view(torch.int16).cpu().numpy()[None]
    assert np.array_equal(out.view(torch.int16).cpu().numpy(), O.compact(hid_bits, idx_np))
    assert np.array_equal(pout.cpu().numpy().ravel(), idx_np)
    ctx.close()


def test_batched_head_statistics_equal_the_per_layer_ones(mods, cuda_device):
    """Eq. 5-6 computed for all layers in one structkv_head_stats call (the pipeline's default)
    give the very bits the per-layer computation inside structkv_score_layer gives."""
    binding, pipeline = mods
    wl = synth.WORKLOADS["llama32k"].scaled(5000 + 3, n_layers=5, n_hubs=8, budgets=(300,))
    pl = synth.plan(wl)
    layers = gpu_layers(wl, pl, cuda_device)
    outs = []
    for defer in (True, False):
        pf = pipeline.Prefill(wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq,
                              wl.budget, wl.struct_budget(), torch.bfloat16, device=cuda_device,
                              defer_head_stats=defer)
        assert pf.defer == defer
        pf.run(layers)
        torch.cuda.synchronize()
        assert pf.ctx.poll_device_status() == binding.OK
        outs.append((pf.metrics.clone(), pf.s_hist.clone(), pf.pivot))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1]) and outs[0][2] == outs[1][2]
    assert not torch.isnan(outs[0][0]).any()


def test_near_uniform_attention_keeps_the_variance_within_tolerance(mods, cuda_device):
    """High temperatures flatten the attention: every pooled per-head vector is close to 1/N and its
    variance (Eq. 6) is a small difference of nearly equal numbers.  The metric must still match
    the oracle's population variance (it is summed as squared deviations from 1/N)."""
    binding, _ = mods
    wl = synth.Workload("flat", 9, 3, 8, 2, 128, 6000, 64, (512,), "bf16", 0, None, hub_layers=(),
                        temperatures=(8.0, 5.0, 12.0))
    pl = synth.plan(wl)
    ctx = binding.Context(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, torch.bfloat16, cuda_device)
    for layer in range(wl.n_layers):
        t = synth.make_layer(wl, pl, layer, device="cpu", with_v=False)
        s = torch.zeros(wl.seq, dtype=torch.float32, device=cuda_device)
        m = torch.zeros(3, dtype=torch.float32, device=cuda_device)
        ctx.score_layer(t["q_win"].to(cuda_device), t["k"].to(cuda_device), t["scale"], s, m)
        torch.cuda.synchronize()
        o = O.score_layer(synth.to_f64(t["q_win"]), synth.to_f64(t["k"]), t["scale"])
        assert o["variance"] < 1e-2 / wl.seq ** 2 * 100           # the regime this test is about: tiny variance
        P.assert_scores_close(s.cpu().numpy(), o["S"], f"flat S layer {layer}")
        for i, key in enumerate(("entropy", "sparsity", "variance")):
            P.assert_metric_close(m[i].item(), o[key], f"flat {key} layer {layer}")
    assert ctx.poll_device_status() == binding.OK
    ctx.close()


def test_early_start_of_the_first_pass_changes_no_bit(mods, cuda_device):
    """With STRUCTKV_FLAG_INPUTS_READY the first scorer pass of a layer starts while the previous
    layer's column reduction is still running (its inputs are vouched for by the caller, here by a
    synchronisation); every output must equal the unflagged run bit for bit, on a chain of layers
    long enough for the passes of neighbouring layers to overlap."""
    binding, pipeline = mods
    wl = synth.WORKLOADS["llama32k"].scaled(9000 + 41, n_layers=6, n_hubs=8, budgets=(400,))
    pl = synth.plan(wl)
    layers = gpu_layers(wl, pl, cuda_device)
    torch.cuda.synchronize()
    outs = []
    for flags in (0, binding.FLAG_INPUTS_READY, binding.FLAG_INPUTS_READY):
        pf = pipeline.Prefill(wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq,
                              wl.budget, wl.struct_budget(), torch.bfloat16, device=cuda_device, flags=flags)
        torch.cuda.synchronize()
        for _ in range(3):                       # repeated sweeps: layer 0 follows layer L-1 back to back
            for l, t in enumerate(layers):
                pf.score(l, t["q_win"], t["k"], t["scale"])
        pf.detect_and_select()
        torch.cuda.synchronize()
        assert pf.ctx.poll_device_status() == binding.OK
        outs.append((pf.metrics.clone(), pf.s_hist.clone(), pf.c_running.clone(), pf.i_kv.clone(), pf.pivot))
    for o in outs[1:]:
        assert all(torch.equal(a, b) for a, b in zip(outs[0][:4], o[:4])) and o[4] == outs[0][4]
    # the batch entry point takes the flag too; any other bit is refused
    ctx = binding.Context(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, torch.bfloat16, cuda_device)
    t = layers[0]
    s1, s2 = (torch.zeros(wl.seq, device=cuda_device) for _ in range(2))
    m1, m2 = torch.zeros(3, device=cuda_device), torch.zeros((1, 3), device=cuda_device)
    ctx.score_layer(t["q_win"], t["k"], t["scale"], s1, m1, flags=binding.FLAG_INPUTS_READY)
    ctx.score_layer_batch(t["q_win"][None], t["k"], [0, wl.seq], t["scale"], s2, m2, ctx.batch_workspace(1, wl.seq),
                          flags=binding.FLAG_INPUTS_READY)
    torch.cuda.synchronize()
    assert torch.equal(s1, s2) and torch.equal(m1, m2[0])
    with pytest.raises(Exception):
        ctx.score_layer(t["q_win"], t["k"], t["scale"], s1, m1, flags=8)
    ctx.close()


def test_batched_head_statistics_on_unaligned_vectors(mods, cuda_device):
    """structkv_head_stats on enough vectors for the one-CTA-per-vector form, each longer than the
    register-resident limit and starting at every 16-byte misalignment (odd length, packed rows):
    its 16-byte memory sweeps must take the ragged ends with scalar accesses.  Eq. 5-6 against the
    oracle, vectors with ties, zeros and a few dominant entries."""
    binding, _ = mods
    L, H, N = 10, 32, 20011
    rng = np.random.default_rng(77)
    x = rng.random((L, H, N)) ** 4
    x[:, :, ::7] = 0.0                                   # exact zeros
    n_tie = min(x[:, :, 5::11].shape[2], x[:, :, 6::11].shape[2])
    x[:, :, 5:5 + 11 * n_tie:11] = x[:, :, 6:6 + 11 * n_tie:11]     # planted ties
    hot = rng.integers(0, N, size=(L, H, 6))
    for l in range(L):
        for h in range(H):
            x[l, h, hot[l, h]] += 40.0 * (1 + l)         # the top mass differs from layer to layer
    x /= x.sum(axis=2, keepdims=True)
    x32 = x.astype(np.float32)
    hc = torch.from_numpy(x32).to(cuda_device)
    m = torch.zeros((L, 3), dtype=torch.float32, device=cuda_device)
    ctx = binding.Context(H, 8, 128, 64, N, torch.bfloat16, cuda_device)
    ctx.head_stats(hc, m)
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == binding.OK
    got = m.cpu().numpy()
    for l in range(L):
        rho, var = O.head_statistics(x32[l].astype(np.float64))
        P.assert_metric_close(got[l, 1], rho, f"sparsity of layer {l}")
        P.assert_metric_close(got[l, 2], var, f"variance of layer {l}")
    ctx.close()


def test_a_captured_layer_can_be_replayed(mods, cuda_device):
    """structkv_score_layer keeps no per-launch state on the host (the second pass reads its work
    tickets modulo the number one launch draws), so a call captured into a CUDA graph gives the
    eager call's bits on every replay, also with eager calls of the same shape in between."""
    binding, _ = mods
    wl = synth.WORKLOADS["llama32k"].scaled(6000 + 19, n_layers=1, n_hubs=4, budgets=(256,))
    t = synth.make_layer(wl, synth.plan(wl), 0, device="cpu", with_v=False)
    q, k = t["q_win"].to(cuda_device), t["k"].to(cuda_device)
    ctx = binding.Context(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, torch.bfloat16, cuda_device)
    s_e, s_g = (torch.zeros(wl.seq, device=cuda_device) for _ in range(2))
    m_e, m_g = (torch.zeros(3, device=cuda_device) for _ in range(2))
    for _ in range(2):
        ctx.score_layer(q, k, t["scale"], s_e, m_e)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ctx.score_layer(q, k, t["scale"], s_g, m_g)
    for i in range(4):
        s_g.zero_(); m_g.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(s_g, s_e) and torch.equal(m_g, m_e), f"replay {i}"
        if i == 1:
            ctx.score_layer(q, k, t["scale"], s_e, m_e)       # an eager call between replays
            torch.cuda.synchronize()
    assert ctx.poll_device_status() == binding.OK
    ctx.close()


@pytest.mark.parametrize("name,seq,n_layers", [("llama32k", 9000 + 41, 7), ("qwen64k", 5000 + 3, 4), ("llama32k", 300, 1),
                                                ("llama32k", 300, 9), ("llama128k", 1200, 12)])
def test_all_layers_in_one_call_equal_the_layer_by_layer_calls(mods, cuda_device, name, seq, n_layers):
    """structkv_score_layers (first pass of layer l + 1 enqueued between the two passes of layer l, the
    second pass waiting for a completion counter, one reduce over heads for all layers at the end)
    gives, bit for bit, what structkv_score_layer gives layer after layer: S, C, pooled per-head
    attention, entropy; and the call can be repeated on the same workspace.  The short sequences give
    grids of a few CTAs, so many launches of the call are resident at once."""
    binding, _ = mods
    wl = synth.WORKLOADS[name].scaled(seq, n_layers=n_layers, n_hubs=4, budgets=(128,))
    pl = synth.plan(wl)
    layers = gpu_layers(wl, pl, cuda_device)
    H, N, dev = wl.n_q_heads, wl.seq, cuda_device
    ctx = binding.Context(H, wl.n_kv_heads, wl.head_dim, wl.window, N, torch.bfloat16, dev)
    f32 = torch.float32
    s1, s2 = (torch.zeros((n_layers, N), dtype=f32, device=dev) for _ in range(2))
    m1, m2 = (torch.zeros((n_layers, 3), dtype=f32, device=dev) for _ in range(2))
    h1, h2 = (torch.zeros((n_layers, H, N), dtype=f32, device=dev) for _ in range(2))
    c1, c2 = (torch.zeros(N, dtype=f32, device=dev) for _ in range(2))
    for l, t in enumerate(layers):
        ctx.score_layer(t["q_win"], t["k"], t["scale"], s1[l], m1[l], c_inout=c1, head_cols_out=h1[l],
                        flags=binding.FLAG_NO_HEAD_STATS)
    torch.cuda.synchronize()
    ws = ctx.layers_workspace(n_layers)
    for rep in range(3):
        c2.zero_()
        ctx.score_layers([t["q_win"] for t in layers], [t["k"] for t in layers], [t["scale"] for t in layers],
                         s2, m2, h2, ws, c_inout=c2)
        torch.cuda.synchronize()
        assert ctx.poll_device_status() == binding.OK
        assert torch.equal(s1, s2) and torch.equal(h1, h2) and torch.equal(c1, c2), f"repeat {rep}"
        assert torch.equal(m1[:, 0], m2[:, 0]) and torch.isnan(m2[:, 1:]).all()
    # a workspace that is too small is refused on the host
    small = ws[: ws.numel() - 256]
    with pytest.raises(Exception):
        ctx.score_layers([t["q_win"] for t in layers], [t["k"] for t in layers], [t["scale"] for t in layers],
                         s2, m2, h2, small, c_inout=c2)
    ctx.close()
