"""GPU parity of the flow past the pivot (Eq. 11 - 13): layers l > L* are scored on the keys
gathered at I_struct, selected on that reduced sequence, and the selection is mapped back to
original position ids through the gathered positions; the structural set's attention-mass
recovery is reported per layer.  Everything runs through the C ABI and is compared with the
oracle's ``prefill_reduced`` on the same bits."""
import numpy as np
import pytest
import torch

from oracle import structkv_oracle as O
from paper_2604_06746_b200 import synth
from tests import parity as P

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,seq,layers,budget,n_detect", [
    ("llama32k", 6000 + 13, 6, 300, 4),      # reduced length 600: ragged last key tile
    ("qwen64k", 5000, 6, 700, 4),            # GQA 7, window 128, reduced length 1400
    ("llama128k", 20000, 9, 1024, 6),        # sink + delimiters, reduced length 2048
])
def test_post_pivot_flow_matches_the_oracle(cuda_device, name, seq, layers, budget, n_detect):
    from paper_2604_06746_b200 import binding, pipeline
    dev = cuda_device
    wl = synth.WORKLOADS[name].scaled(seq, n_layers=layers, n_hubs=8, budgets=(budget,))
    pl = synth.plan(wl)
    ts = []
    for l in range(wl.n_layers):
        t = synth.make_layer(wl, pl, l, device="cpu")
        ts.append({k: (v.to(dev) if torch.is_tensor(v) else v) for k, v in t.items()})
    st_b = wl.struct_budget()
    hidden = torch.zeros((wl.seq, 64), dtype=torch.bfloat16, device=dev)
    positions = torch.arange(wl.seq, device=dev, dtype=torch.int32) * 2 + 3
    pf = pipeline.Prefill(wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, budget, st_b,
                          torch.bfloat16, hidden_dim=64, device=dev)
    pf.enable_reduced()
    for l in range(n_detect):                                   # full-sequence layers: pivot, C*, I_struct
        pf.score(l, ts[l]["q_win"], ts[l]["k"], ts[l]["scale"])
    piv = pf.detect_and_select(n_detect)
    pf.compact_hidden(hidden, positions)                        # P' = P[I_struct]
    for l in range(piv + 1, wl.n_layers):                       # reduced-sequence layers
        pf.score_reduced(l, ts[l]["q_win"], ts[l]["k"], ts[l]["scale"])
    pf.select_reduced(piv + 1, wl.n_layers)
    # fidelity diagnostic: share of each later layer's full-sequence attention kept by I_struct
    s_full = torch.zeros((wl.n_layers, wl.seq), dtype=torch.float32, device=dev)
    m_tmp = torch.zeros(3, dtype=torch.float32, device=dev)
    for l in range(piv + 1, wl.n_layers):
        pf.ctx.score_layer(ts[l]["q_win"], ts[l]["k"], ts[l]["scale"], s_full[l], m_tmp)
    pf.ctx.mass_recovery(s_full, pf.i_struct, pf.recovery)
    torch.cuda.synchronize()
    assert pf.ctx.poll_device_status() == binding.OK

    o = O.prefill_reduced([(synth.to_f64(t["q_win"]), synth.to_f64(t["k"]), t["scale"]) for t in ts],
                          positions.cpu().numpy(), wl.window, budget, st_b, n_detect=n_detect)
    T = np.sort(o["head"]["transition"][1:])[::-1]
    assert T[0] - T[1] >= 0.02, f"oracle transition margin {T[0] - T[1]:.4f}"
    assert piv == o["pivot"] and o["pivot"] < wl.n_layers - 1
    g_struct = pf.i_struct.cpu().numpy()
    P.assert_selection_matches(g_struct, o["head"]["C"], st_b, wl.window, o["i_struct"], "I_struct")
    assert np.array_equal(g_struct, o["i_struct"]), "the reduced layers need the same structural set on both sides"
    pos_host = positions.cpu().numpy()
    for l in range(piv + 1, wl.n_layers):
        r = o["past"][l]
        P.assert_scores_close(pf.s_red[l].cpu().numpy(), r["S"], f"reduced S layer {l}")
        P.assert_metric_close(pf.metrics_red[l, 0].item(), r["entropy"], f"reduced entropy layer {l}")
        i_red = pf.i_red[l].cpu().numpy()
        P.assert_selection_matches(i_red, r["S"], budget, wl.window, r["i_reduced"], f"reduced I_KV layer {l}")
        # composition through the gathered position ids: bit exact on the GPU's own selection
        assert np.array_equal(pf.i_kv_pos[l].cpu().numpy(), pos_host[g_struct][i_red])
        if np.array_equal(i_red, r["i_reduced"]):
            assert np.array_equal(pf.i_kv_pos[l].cpu().numpy(), r["i_kv"])
        assert abs(pf.recovery[l].item() - o["recovery"][l]) <= 2e-3 * o["recovery"][l]
