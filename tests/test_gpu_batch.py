"""GPU parity of batched prompts with heterogeneous pivots: prompts of different lengths are
packed along the token axis, every layer is scored for the whole batch by one launch per scorer
pass (structkv_score_layer_batch), each prompt gets its own pivot (structkv_pivot on its metric
table), its own centrality and its own index sets (structkv_select_batch, padded with -1), and its
K rows are gathered from the packed tensor.  Everything is compared with the oracle's
``prefill_batch`` (independent ``prefill`` per prompt) on the same bits."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import structkv_oracle as O
from paper_2604_06746_b200 import synth
from tests import parity as P

pytestmark = pytest.mark.gpu

# (workload, prompt lengths, layers, KV budgets): lengths include ragged tiles, a prompt barely
# longer than the window block and one that spans many key tiles
CASES = [
    ("llama32k", (3000, 777, 5123, 1500), 6, (200, 100, 300, 150)),
    ("qwen64k", (2500, 900, 4100, 1300, 600), 5, (300, 200, 400, 260, 180)),
]


@pytest.mark.parametrize("name,lens,n_layers,budgets", CASES)
def test_batched_prompts_match_independent_oracle_prompts(cuda_device, name, lens, n_layers, budgets):
    from paper_2604_06746_b200 import binding
    dev = cuda_device
    B = len(lens)
    base = synth.WORKLOADS[name]
    # every prompt is its own workload (own seed, own temperature schedule, hence its own pivot)
    wls = [dataclasses.replace(base.scaled(n, n_layers=n_layers, n_hubs=6, budgets=(budgets[b],)), index=40 + 7 * b)
           for b, n in enumerate(lens)]
    plans = [synth.plan(w) for w in wls]
    prompts = [[synth.make_layer(w, pl, l, device="cpu", with_v=False) for l in range(n_layers)]
               for w, pl in zip(wls, plans)]
    # the batch call takes ONE logit scale per layer (prompt 0's); each prompt's own temperature
    # is folded into its queries (rounded to bf16 again: those bits are the input of both sides)
    for b in range(1, len(prompts)):
        for l in range(n_layers):
            ratio = prompts[b][l]["scale"] / prompts[0][l]["scale"]
            prompts[b][l]["q_win"] = (prompts[b][l]["q_win"].float() * ratio).to(torch.bfloat16)
    w0 = wls[0]
    H, Hkv, d, win = w0.n_q_heads, w0.n_kv_heads, w0.head_dim, w0.window
    cu = [0]
    for n in lens:
        cu.append(cu[-1] + n)
    total = cu[-1]
    st_budgets = [w.struct_budget() for w in wls]
    ctx = binding.Context(H, Hkv, d, win, max(lens), torch.bfloat16, dev)
    ws = ctx.batch_workspace(B, total)
    f32, i32 = torch.float32, torch.int32
    s_hist = torch.zeros((n_layers, total), dtype=f32, device=dev)
    metrics = torch.zeros((n_layers, B, 3), dtype=f32, device=dev)
    c_run = torch.zeros(total, dtype=f32, device=dev)
    k_packed = []
    for l in range(n_layers):
        scale = prompts[0][l]["scale"]
        q = torch.stack([prompts[b][l]["q_win"] for b in range(B)]).to(dev)
        k = torch.cat([prompts[b][l]["k"] for b in range(B)], dim=1).to(dev).contiguous()
        k_packed.append(k)
        ctx.score_layer_batch(q, k, cu, scale, s_hist[l], metrics[l], ws, c_inout=c_run, lam=O.PAPER_LAMBDA)
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == binding.OK

    # the oracle: every prompt alone, at the scales the batch used
    oracle_prompts = [[(synth.to_f64(prompts[b][l]["q_win"]), synth.to_f64(prompts[b][l]["k"]), prompts[0][l]["scale"])
                       for l in range(n_layers)] for b in range(B)]
    weights = O.PAPER_WEIGHTS
    ora = O.prefill_batch(oracle_prompts, win, list(budgets), st_budgets, weights=weights)

    pivots, c_star = [], torch.zeros(total, dtype=f32, device=dev)
    m_host = metrics.cpu().numpy()
    for b in range(B):
        o = ora["per_prompt"][b]
        lo, hi = cu[b], cu[b + 1]
        for l in range(n_layers):
            P.assert_scores_close(s_hist[l, lo:hi].cpu().numpy(), o["s_hist"][l], f"prompt {b} S layer {l}")
            for c in range(3):
                P.assert_metric_close(m_host[l, b, c], o["metrics"][l, c], f"prompt {b} metric {c} layer {l}")
        T = np.sort(o["transition"][1:])[::-1]
        assert T[0] - T[1] >= 0.02, f"prompt {b}: oracle transition margin {T[0] - T[1]:.4f}"
        piv, _ = ctx.pivot(metrics[:, b, :].contiguous(), weights)
        assert piv == o["pivot"], (b, piv, o["pivot"])
        pivots.append(piv)
        # centrality at this prompt's own pivot, on its slice of the packed history
        ctx.accumulate(s_hist[:, lo:hi], piv, O.PAPER_LAMBDA, c_star[lo:hi])
        P.assert_scores_close(c_star[lo:hi].cpu().numpy(), o["C"], f"prompt {b} C*")
    assert pivots == ora["pivots"].tolist()
    assert len(set(pivots)) > 1, "the case is meant to have heterogeneous pivots"
    reduced_at = np.arange(n_layers)[None, :] > np.asarray(pivots)[:, None]
    assert np.array_equal(reduced_at, ora["reduced_at"])

    # both selections for the whole batch, padded with -1
    i_struct = torch.zeros((B, max(st_budgets)), dtype=i32, device=dev)
    ctx.select_batch(c_star, cu, st_budgets, win, i_struct)
    i_kv = torch.zeros((n_layers, B, max(budgets)), dtype=i32, device=dev)
    for l in range(n_layers):
        ctx.select_batch(s_hist[l], cu, list(budgets), win, i_kv[l])
    torch.cuda.synchronize()
    g_struct, g_kv = i_struct.cpu().numpy(), i_kv.cpu().numpy()
    for b in range(B):
        o = ora["per_prompt"][b]
        P.assert_selection_matches(g_struct[b, :st_budgets[b]], o["C"], st_budgets[b], win, o["i_struct"],
                                   f"prompt {b} I_struct")
        assert np.all(g_struct[b, st_budgets[b]:] == -1) and np.all(ora["i_struct"][b, st_budgets[b]:] == -1)
        for l in range(n_layers):
            P.assert_selection_matches(g_kv[l, b, :budgets[b]], o["s_hist"][l], budgets[b], win, o["i_kv"][l],
                                       f"prompt {b} I_KV layer {l}")
            assert np.all(g_kv[l, b, budgets[b]:] == -1)
            assert g_kv[l, b, :budgets[b]].max() < lens[b]           # never a batch-mate's token
    # gather of one layer's K rows per prompt out of the packed tensor, bit for bit
    l = n_layers - 1
    for b in range(B):
        lo, hi = cu[b], cu[b + 1]
        idx = i_kv[l, b, :budgets[b]].contiguous()
        out = torch.empty((Hkv, budgets[b], d), dtype=torch.bfloat16, device=dev)
        ctx.compact(k_packed[l][:, lo:hi], idx, out)
        torch.cuda.synchronize()
        src = k_packed[l][:, lo:hi].contiguous().view(torch.int16).cpu().numpy()
        assert np.array_equal(out.view(torch.int16).cpu().numpy(), O.compact(src, g_kv[l, b, :budgets[b]]))
    assert ctx.poll_device_status() == binding.OK
    ctx.close()


def test_a_batch_of_one_equals_the_plain_call(cuda_device):
    from paper_2604_06746_b200 import binding
    dev = cuda_device
    wl = synth.WORKLOADS["llama32k"].scaled(4096 + 77, n_layers=1, n_hubs=4, budgets=(256,))
    t = synth.make_layer(wl, synth.plan(wl), 0, device="cpu", with_v=False)
    q, k = t["q_win"].to(dev), t["k"].to(dev)
    ctx = binding.Context(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, torch.bfloat16, dev)
    s1, s2 = torch.zeros(wl.seq, device=dev), torch.zeros(wl.seq, device=dev)
    m1, m2 = torch.zeros(3, device=dev), torch.zeros((1, 3), device=dev)
    ctx.score_layer(q, k, t["scale"], s1, m1)
    ctx.score_layer_batch(q[None], k, [0, wl.seq], t["scale"], s2, m2, ctx.batch_workspace(1, wl.seq))
    torch.cuda.synchronize()
    assert torch.equal(s1, s2) and torch.equal(m1, m2[0])
    # refusals on the host
    bad = binding.lib.structkv_score_layer_batch
    cu = (binding._i * 2)(0, 10)                                      # shorter than the window
    assert bad(ctx._h, q.data_ptr(), k.data_ptr(), k.stride(0), k.stride(1), cu, 1, 1.0, 0.9, s2.data_ptr(), None,
               None, m2.data_ptr(), 0, s2.data_ptr(), 16, None) == binding.ERR_INVALID_ARG
    cu = (binding._i * 2)(0, wl.seq)
    assert bad(ctx._h, q.data_ptr(), k.data_ptr(), k.stride(0), k.stride(1), cu, 1, 1.0, 0.9, s2.data_ptr(), None,
               None, m2.data_ptr(), 0, s2.data_ptr(), 16, None) == binding.ERR_WORKSPACE
    ctx.close()


def test_batched_scoring_at_the_size_the_bench_times(cuda_device):
    """Four Llama-3-8B-shaped prompts of 40000 + 20000 + 50000 + 21072 tokens (131072 together: the
    batch bench.py times) scored by one structkv_score_layer_batch call per layer: every prompt's S,
    entropy, sparsity and variance against the oracle on that prompt alone (its layers run in worker
    processes), and the batch's outputs against four plain calls."""
    from paper_2604_06746_b200 import binding
    from tests import oracle_pool
    dev = cuda_device
    H, Hkv, d, w = 32, 8, 128, 64
    lens = (40000, 20000, 50000, 21072)
    n_layers = 2
    cu = [0]
    for n in lens:
        cu.append(cu[-1] + n)
    total, B = cu[-1], len(lens)
    base = synth.WORKLOADS["llama128k"]
    wls = [dataclasses.replace(base.scaled(n, n_layers=n_layers, n_hubs=32, budgets=(1024,)), index=60 + 3 * b)
           for b, n in enumerate(lens)]
    plans = [synth.plan(x) for x in wls]
    ctx = binding.Context(H, Hkv, d, w, max(lens), torch.bfloat16, dev)
    ws = ctx.batch_workspace(B, total)
    s_b = torch.zeros((n_layers, total), dtype=torch.float32, device=dev)
    m_b = torch.zeros((n_layers, B, 3), dtype=torch.float32, device=dev)
    s_1 = torch.zeros_like(s_b)
    m_1 = torch.zeros_like(m_b)
    tasks = []
    for l in range(n_layers):
        per = [synth.make_layer(x, pl, l, device="cpu", with_v=False) for x, pl in zip(wls, plans)]
        scale = per[0]["scale"]
        for b in range(1, B):                                # one logit scale per call: fold the others into q
            per[b]["q_win"] = (per[b]["q_win"].float() * (per[b]["scale"] / scale)).to(torch.bfloat16)
        q = torch.stack([t["q_win"] for t in per]).to(dev)
        k = torch.cat([t["k"] for t in per], dim=1).to(dev).contiguous()
        ctx.score_layer_batch(q, k, cu, scale, s_b[l], m_b[l], ws)
        for b in range(B):
            ctx.score_layer(q[b], k[:, cu[b]:cu[b + 1]], scale, s_1[l, cu[b]:cu[b + 1]], m_1[l, b])
            tasks.append((l * B + b, oracle_pool.bits_of(per[b]["q_win"]), oracle_pool.bits_of(per[b]["k"]), scale, None))
        torch.cuda.synchronize()
    assert ctx.poll_device_status() == binding.OK
    # a prompt's keys are cut into fewer segments inside a batch than alone, so the statistics are
    # summed in another order: equal to rounding, not bit for bit
    assert torch.allclose(s_b, s_1, rtol=1e-4, atol=1e-10) and torch.allclose(m_b, m_1, rtol=1e-4, atol=0.0)
    workers = oracle_pool.default_workers(8.0 * H * max(lens) * 3)
    o_s, o_m = oracle_pool.score_layers(iter(tasks), len(tasks), workers, stack=False)
    g_s, g_m = s_b.cpu().numpy(), m_b.cpu().numpy()
    for l in range(n_layers):
        for b in range(B):
            i = l * B + b
            P.assert_scores_close(g_s[l, cu[b]:cu[b + 1]], o_s[i], f"layer {l} prompt {b} S")
            for c in range(3):
                P.assert_metric_close(g_m[l, b, c], o_m[i, c], f"layer {l} prompt {b} metric {c}")
    ctx.close()
