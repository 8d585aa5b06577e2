"""GPU test of structkv_score_layer_static, the scoring entry point for callers that cannot
allocate device memory (a host whose HBM is already committed to a cache pool, or a step that
cannot absorb the synchronisation of cudaMalloc / cudaFree).  It scores on a fixed scratch
array inside the library instead of a caller workspace.

Checked here, through the C ABI: on two calls in a row (different layers, so the second call
meets the first call's leftovers in the shared scratch) its outputs equal those of the
ordinary context-based structkv_score_layer on the same inputs, within the parity tolerance
the other GPU tests use; and a configuration beyond the scratch size is refused on the host.
The file name sorts last so that a run stopping at the first failure has already run every
other test; the test also passes alone in a fresh process (it depends on no earlier test).
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2604_06746_b200 import synth
from tests import parity as P

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,seq", [("llama32k", 4096 + 77), ("tiny", 2048)])
def test_static_scratch_scoring_matches_context_scoring_twice(cuda_device, name, seq):
    from paper_2604_06746_b200 import binding
    wl = synth.WORKLOADS[name].scaled(seq, n_layers=2, n_hubs=8)
    pl = synth.plan(wl)
    dt = synth.torch_dtype(wl.dtype)
    ctx = binding.Context(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, dt, cuda_device)
    f32 = torch.float32
    c_ref = torch.zeros(wl.seq, dtype=f32, device=cuda_device)
    c_new = torch.zeros(wl.seq, dtype=f32, device=cuda_device)
    for layer in range(2):                      # two calls in a row on the shared scratch
        t = synth.make_layer(wl, pl, layer, device="cpu", with_v=False)
        q, k = t["q_win"].to(cuda_device), t["k"].to(cuda_device)
        s_ref = torch.zeros(wl.seq, dtype=f32, device=cuda_device)
        m_ref = torch.zeros(3, dtype=f32, device=cuda_device)
        h_ref = torch.zeros((wl.n_q_heads, wl.seq), dtype=f32, device=cuda_device)
        s_new, m_new, h_new = torch.zeros_like(s_ref), torch.zeros_like(m_ref), torch.zeros_like(h_ref)
        ctx.score_layer(q, k, t["scale"], s_ref, m_ref, c_inout=c_ref, head_cols_out=h_ref)
        binding.score_layer_static(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, q, k,
                                   t["scale"], s_new, m_new, c_inout=c_new, head_cols_out=h_new)
        torch.cuda.synchronize()
        assert ctx.poll_device_status() == binding.OK
        P.assert_scores_close(s_new.cpu().numpy(), s_ref.cpu().numpy(), f"{name} S layer {layer}")
        P.assert_scores_close(c_new.cpu().numpy(), c_ref.cpu().numpy(), f"{name} C layer {layer}")
        P.assert_scores_close(h_new.cpu().numpy(), h_ref.cpu().numpy(), f"{name} head columns layer {layer}")
        for c in range(3):
            P.assert_metric_close(m_new[c].item(), m_ref[c].item(), f"{name} metric {c} layer {layer}")
        assert np.isclose(s_new.sum().item(), wl.n_q_heads, rtol=1e-3)
    ctx.close()


def test_static_scratch_scoring_allocates_nothing_and_serves_the_pooled_columns_itself(cuda_device):
    """What the entry point exists for: after its first call on the device (which does the one-time
    set-up) further calls leave the amount of free device memory untouched.  Also the variant
    without head_cols_out, whose pooled per-head columns then live inside the fixed scratch."""
    from paper_2604_06746_b200 import binding
    wl = synth.WORKLOADS["llama32k"].scaled(4096 + 77, n_layers=1, n_hubs=8)
    t = synth.make_layer(wl, synth.plan(wl), 0, device="cpu", with_v=False)
    q, k = t["q_win"].to(cuda_device), t["k"].to(cuda_device)
    f32 = torch.float32
    ctx = binding.Context(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, torch.bfloat16, cuda_device)
    s_ref, m_ref = torch.zeros(wl.seq, dtype=f32, device=cuda_device), torch.zeros(3, dtype=f32, device=cuda_device)
    s_new, m_new = torch.zeros_like(s_ref), torch.zeros_like(m_ref)
    ctx.score_layer(q, k, t["scale"], s_ref, m_ref)
    args = (wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.seq, q, k, t["scale"], s_new, m_new)
    binding.score_layer_static(*args)                      # first call: one-time set-up happens here
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for _ in range(5):
        binding.score_layer_static(*args)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    P.assert_scores_close(s_new.cpu().numpy(), s_ref.cpu().numpy(), "S without head_cols_out")
    for c in range(3):
        P.assert_metric_close(m_new[c].item(), m_ref[c].item(), f"metric {c} without head_cols_out")
    ctx.close()


def test_static_scratch_scoring_refuses_configurations_beyond_its_scratch(cuda_device):
    from paper_2604_06746_b200 import binding
    big = binding.Config(32, 8, 128, 64, 131072, binding.BF16)
    assert binding.workspace_bytes(big) > binding.STATIC_SCRATCH_BYTES
    dummy = torch.zeros(16, device=cuda_device)
    rc = binding.lib.structkv_score_layer_static(ctypes.byref(big), dummy.data_ptr(), dummy.data_ptr(), 128, 128,
                                                 131072, 1.0, 0.9, dummy.data_ptr(), None, None,
                                                 dummy.data_ptr(), 0, None)
    assert rc == binding.ERR_WORKSPACE
    assert binding.lib.structkv_score_layer_static(None, None, None, 0, 0, 0, 1.0, 0.9, None, None, None, None,
                                                   0, None) == binding.ERR_INVALID_ARG
