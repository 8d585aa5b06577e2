"""GPU tests, through the C ABI, of block-level aggregation (with block-granular selection and
gathering on top of it) and of attention-mass recovery, against the oracle."""
import numpy as np
import pytest
import torch

from oracle import structkv_oracle as O
from tests import parity as P

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx(cuda_device):
    from paper_2604_06746_b200 import binding
    c = binding.Context(8, 2, 64, 32, 1 << 18, torch.float32, cuda_device)
    yield c
    c.close()


@pytest.mark.parametrize("n,bs,batch", [(131072, 16, 1), (131072, 32, 3), (5003, 16, 2), (77, 128, 1), (4096, 1, 1),
                                        (262144, 64, 1)])
def test_block_scores_match_the_oracle(ctx, n, bs, batch):
    rng = np.random.default_rng(n + bs)
    sc = (rng.random((batch, n)) ** 3).astype(np.float32)
    d = torch.from_numpy(sc).cuda()
    nb = -(-n // bs)
    out = torch.zeros((batch, nb), dtype=torch.float32, device="cuda")
    ctx.block_scores(d, bs, out)
    torch.cuda.synchronize()
    for b in range(batch):
        np.testing.assert_allclose(out[b].cpu().numpy(), O.block_scores(sc[b], bs), rtol=2e-6, atol=0)


def test_block_granular_selection_and_gather(ctx):
    """Paged layout: centrality pooled per block of 16 tokens, the best blocks kept (the block
    holding the window always), whole blocks of K gathered bit for bit."""
    rng = np.random.default_rng(7)
    n, bs, hkv, d, keep_blocks = 32768, 16, 4, 128, 300
    c = (rng.random(n) ** 4).astype(np.float32)
    c[5000:5016] += 0.5                                             # a contiguous anchor: exactly block 312
    dc = torch.from_numpy(c).cuda()
    nb = n // bs
    bsc = torch.zeros(nb, dtype=torch.float32, device="cuda")
    ctx.block_scores(dc, bs, bsc)
    idx = torch.zeros(keep_blocks, dtype=torch.int32, device="cuda")
    ctx.select(bsc, keep_blocks, 2, idx)                            # window = the last 2 blocks (32 tokens)
    torch.cuda.synchronize()
    ob = O.block_scores(c, bs)
    got = idx.cpu().numpy()
    P.assert_selection_matches(got, ob, keep_blocks, 2, O.select(ob, keep_blocks, 2), "block selection")
    assert 312 in got
    k = torch.from_numpy(rng.integers(0, 2 ** 15, size=(hkv, n, d), dtype=np.int16)).cuda()
    out = torch.zeros((hkv, keep_blocks, bs * d), dtype=torch.int16, device="cuda")
    ctx.compact(k.view(hkv, nb, bs * d), idx, out)                  # one row = one block of one KV head
    torch.cuda.synchronize()
    ref = O.compact(k.cpu().numpy().reshape(hkv, nb, bs * d), got)
    assert np.array_equal(out.cpu().numpy(), ref)


def test_mass_recovery_matches_the_oracle_and_flags_bad_indices(ctx):
    from paper_2604_06746_b200 import binding
    rng = np.random.default_rng(8)
    L, n, b = 6, 50000, 4000
    s = (rng.random((L, n)) ** 5).astype(np.float32)
    idx_np = np.sort(rng.choice(n, size=b, replace=False)).astype(np.int32)
    ds, di = torch.from_numpy(s).cuda(), torch.from_numpy(idx_np).cuda()
    out = torch.zeros(L, dtype=torch.float32, device="cuda")
    ctx.mass_recovery(ds, di, out)
    torch.cuda.synchronize()
    ref = np.array([O.mass_recovery(s[l], idx_np) for l in range(L)])
    np.testing.assert_allclose(out.cpu().numpy(), ref, rtol=1e-5)
    assert ctx.poll_device_status() == binding.OK
    bad = torch.tensor([0, n, -3, 5], dtype=torch.int32, device="cuda")
    ctx.mass_recovery(ds[0], bad, out[:1])
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == binding.ERR_INVALID_ARG
    assert out[0].item() == pytest.approx(O.mass_recovery(s[0], np.array([0, 5])), rel=1e-5)


def test_centrality_recovers_more_attention_mass_than_a_single_layer_snapshot(cuda_device):
    """The paper's fidelity argument on the tiny workload (hubs active in layers 1-2, pivot at 3):
    the set chosen from the global centrality covers more of layers 1-2's attention than the set
    chosen from the pivot layer's own saliency."""
    from paper_2604_06746_b200 import pipeline, synth
    wl = synth.WORKLOADS["tiny"]
    pl = synth.plan(wl)
    layers = [synth.make_layer(wl, pl, l, device=cuda_device) for l in range(wl.n_layers)]
    budget = 64
    pf = pipeline.Prefill(wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, budget, budget,
                          torch.float32, device=cuda_device, weights=(1.0, 0.0, 0.0))
    pf.run(layers)
    snap = torch.zeros(budget, dtype=torch.int32, device=cuda_device)
    pf.ctx.select(pf.s_hist[pf.pivot], budget, wl.window, snap)
    rec_c = torch.zeros(wl.n_layers, device=cuda_device)
    rec_s = torch.zeros(wl.n_layers, device=cuda_device)
    pf.ctx.mass_recovery(pf.s_hist, pf.i_struct, rec_c)
    pf.ctx.mass_recovery(pf.s_hist, snap, rec_s)
    torch.cuda.synchronize()
    s_hist = pf.s_hist.cpu().numpy()
    for l in range(wl.n_layers):
        assert rec_c[l].item() == pytest.approx(O.mass_recovery(s_hist[l], pf.i_struct.cpu().numpy()), rel=1e-5)
    assert rec_c[1].item() > rec_s[1].item() and rec_c[2].item() > rec_s[2].item()


def test_per_kv_head_selection_and_gather(cuda_device):
    """The per-KV-head variant of the cache selection: saliency per GQA group from the pooled
    per-head attention, one budgeted selection per KV head, one gather with a list per head."""
    from paper_2604_06746_b200 import binding, synth
    wl = synth.WORKLOADS["llama32k"].scaled(6000 + 13, n_layers=1, n_hubs=8, budgets=(500,))
    pl = synth.plan(wl)
    t = synth.make_layer(wl, pl, 0, device="cpu")
    q, k, v = t["q_win"].to(cuda_device), t["k"].to(cuda_device), t["v"].to(cuda_device)
    ctx = binding.Context(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, torch.bfloat16, cuda_device)
    f32 = torch.float32
    s = torch.zeros(wl.seq, dtype=f32, device=cuda_device)
    m = torch.zeros(3, dtype=f32, device=cuda_device)
    cols = torch.zeros((wl.n_q_heads, wl.seq), dtype=f32, device=cuda_device)
    ctx.score_layer(q, k, t["scale"], s, m, head_cols_out=cols)
    grp = torch.zeros((wl.n_kv_heads, wl.seq), dtype=f32, device=cuda_device)
    ctx.group_saliency(cols, grp)
    idx = torch.zeros((wl.n_kv_heads, wl.budget), dtype=torch.int32, device=cuda_device)
    ctx.select(grp, wl.budget, wl.window, idx)
    out_k = torch.zeros((wl.n_kv_heads, wl.budget, wl.head_dim), dtype=torch.bfloat16, device=cuda_device)
    ctx.compact_per_slab(k, idx, out_k)
    torch.cuda.synchronize()
    o = O.score_layer(synth.to_f64(t["q_win"]), synth.to_f64(t["k"]), t["scale"])
    og = O.group_saliency(o["head_cols"], wl.group)
    P.assert_scores_close(grp.cpu().numpy(), og, "group saliency")
    got = idx.cpu().numpy()
    for g in range(wl.n_kv_heads):
        P.assert_selection_matches(got[g], og[g], wl.budget, wl.window, O.select(og[g], wl.budget, wl.window),
                                   f"KV head {g}")
    assert len({tuple(r) for r in got.tolist()}) > 1                       # the heads do choose different tokens
    ref = O.compact_per_slab(t["k"].view(torch.int16).numpy(), got)
    assert np.array_equal(out_k.view(torch.int16).cpu().numpy(), ref)
    assert ctx.poll_device_status() == binding.OK
    ctx.close()


def test_per_sequence_gather_of_a_batch(ctx):
    """Masked state transition of a batch: every sequence brings its own index list (padded to a
    common length); one launch gathers all of them, bit for bit."""
    rng = np.random.default_rng(31)
    B, n, width, kmax = 5, 3000, 96, 400
    src = torch.from_numpy(rng.integers(0, 256, size=(B, n, width), dtype=np.uint8)).cuda()
    idx_np = np.stack([np.sort(rng.choice(n, size=kmax, replace=False)) for _ in range(B)]).astype(np.int32)
    pad = torch.from_numpy(np.concatenate([idx_np, np.zeros((B, 8), np.int32)], axis=1)).cuda()   # row stride 408
    dst = torch.zeros((B, kmax, width), dtype=torch.uint8, device="cuda")
    ctx.compact_per_slab(src, pad[:, :kmax], dst)
    torch.cuda.synchronize()
    assert np.array_equal(dst.cpu().numpy(), O.compact_per_slab(src.cpu().numpy(), idx_np))
