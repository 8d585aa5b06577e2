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
