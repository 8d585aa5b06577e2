"""GPU tests of selection and compaction alone, through the C ABI: exact agreement with the
oracle on fp32 scores (ties included), edge budgets, odd row sizes, strided sources."""
import numpy as np
import pytest
import torch

from oracle import structkv_oracle as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx(cuda_device):
    from paper_2604_06746_b200 import binding
    c = binding.Context(8, 2, 64, 32, 1 << 18, torch.float32, cuda_device)
    yield c
    c.close()


def gpu_select(ctx, scores, budget, window):
    s = torch.from_numpy(np.ascontiguousarray(scores, dtype=np.float32)).cuda()
    batch = 1 if s.dim() == 1 else s.shape[0]
    out = torch.full((batch, budget), -1, dtype=torch.int32, device="cuda")
    ctx.select(s, budget, window, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


@pytest.mark.parametrize("n,window,budget", [
    (1000, 32, 100), (4096, 64, 2048), (5000, 1, 2), (5000, 0, 17), (131072, 64, 16384),
    (131072 + 5, 64, 1024), (300, 32, 32), (300, 32, 300), (300, 32, 33), (262144, 64, 8192), (33, 32, 33)])
def test_select_exact_on_random_scores(ctx, n, window, budget):
    rng = np.random.default_rng(n * 7 + budget)
    scores = (rng.random(n) ** 4).astype(np.float32)
    got = gpu_select(ctx, scores, budget, window)[0]
    assert np.array_equal(got, O.select(scores, budget, window))


def test_select_exact_with_heavy_ties_and_signs(ctx):
    rng = np.random.default_rng(5)
    n, window, budget = 20000, 64, 3000
    scores = rng.integers(-3, 4, size=n).astype(np.float32)         # seven distinct values
    scores[rng.integers(0, n, 50)] = -0.0
    assert np.array_equal(gpu_select(ctx, scores, budget, window)[0], O.select(scores, budget, window))
    scores = np.zeros(n, dtype=np.float32)                           # all equal: lowest indices win
    assert np.array_equal(gpu_select(ctx, scores, budget, window)[0], O.select(scores, budget, window))
    scores = np.full(n, 1e-30, dtype=np.float32); scores[::7] = 3e-39  # denormals order correctly
    assert np.array_equal(gpu_select(ctx, scores, budget, window)[0], O.select(scores, budget, window))


def test_select_batched_with_row_stride(ctx):
    rng = np.random.default_rng(6)
    L, n, window, budget = 9, 7001, 64, 512
    big = torch.from_numpy(rng.random((L, n + 100)).astype(np.float32)).cuda()
    view = big[:, :n]                                                # row stride n + 100
    out = torch.zeros((L, budget), dtype=torch.int32, device="cuda")
    ctx.select(view, budget, window, out)
    torch.cuda.synchronize()
    ref = big.cpu().numpy()
    for l in range(L):
        assert np.array_equal(out[l].cpu().numpy(), O.select(ref[l, :n], budget, window))


def test_select_rejects_bad_arguments(ctx):
    from paper_2604_06746_b200 import binding
    s = torch.zeros(100, device="cuda")
    out = torch.zeros(200, dtype=torch.int32, device="cuda")
    lib, h = binding.lib, ctx._h
    assert lib.structkv_select(h, s.data_ptr(), 100, 1, 100, 101, 10, out.data_ptr(), None) == binding.ERR_INVALID_ARG
    assert lib.structkv_select(h, s.data_ptr(), 100, 1, 100, 5, 10, out.data_ptr(), None) == binding.ERR_INVALID_ARG
    assert lib.structkv_select(h, None, 100, 1, 100, 50, 10, out.data_ptr(), None) == binding.ERR_INVALID_ARG
    assert lib.structkv_select(h, s.data_ptr(), 10, 2, 100, 50, 10, out.data_ptr(), None) == binding.ERR_INVALID_ARG


@pytest.mark.parametrize("row_bytes,n_slabs,n_rows,n_idx", [
    (256, 8, 5000, 700), (8192, 1, 3000, 1000), (4, 1, 9000, 333), (2, 3, 500, 100), (6, 2, 500, 77),
    (128, 2, 64, 64), (48, 4, 1000, 1), (512, 8, 131072, 16384)])
def test_compact_bit_exact(ctx, row_bytes, n_slabs, n_rows, n_idx):
    rng = np.random.default_rng(row_bytes + n_idx)
    src = torch.from_numpy(rng.integers(0, 256, size=(n_slabs, n_rows, row_bytes), dtype=np.uint8)).cuda()
    idx_np = np.sort(rng.choice(n_rows, size=n_idx, replace=False)).astype(np.int32)
    idx = torch.from_numpy(idx_np).cuda()
    dst = torch.zeros((n_slabs, n_idx, row_bytes), dtype=torch.uint8, device="cuda")
    ctx.compact(src, idx, dst)
    torch.cuda.synchronize()
    assert np.array_equal(dst.cpu().numpy(), O.compact(src.cpu().numpy(), idx_np))
    assert ctx.poll_device_status() == 0


def test_compact_strided_source_and_unsorted_indices(ctx):
    rng = np.random.default_rng(11)
    # token-major storage [N, H_kv, d] viewed as [H_kv, N, d]: row stride spans all heads
    store = torch.from_numpy(rng.integers(0, 2 ** 15, size=(4000, 4, 128), dtype=np.int16)).cuda()
    src = store.permute(1, 0, 2)
    idx_np = rng.integers(0, 4000, size=900).astype(np.int32)        # unsorted, with repeats
    idx = torch.from_numpy(idx_np).cuda()
    dst = torch.zeros((4, 900, 128), dtype=torch.int16, device="cuda")
    ctx.compact(src, idx, dst)
    torch.cuda.synchronize()
    assert np.array_equal(dst.cpu().numpy(), O.compact(src.cpu().numpy(), idx_np))


def test_compact_flags_out_of_range_index_without_faulting(ctx):
    from paper_2604_06746_b200 import binding
    src = torch.arange(100 * 16, dtype=torch.uint8, device="cuda").reshape(1, 100, 16)
    idx = torch.tensor([0, 5, 100, -1, 7], dtype=torch.int32, device="cuda")
    dst = torch.full((1, 5, 16), 255, dtype=torch.uint8, device="cuda")
    ctx.compact(src, idx, dst)
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == binding.ERR_INVALID_ARG
    assert ctx.poll_device_status() == binding.OK                     # cleared by the read
    got = dst.cpu().numpy()[0]
    assert np.array_equal(got[[0, 1, 4]], src.cpu().numpy()[0][[0, 5, 7]])
    assert np.all(got[[2, 3]] == 255)                                 # skipped rows stay untouched


def test_bounded_wait_expiry_is_reported_once(cuda_device):
    """A device-side wait whose bound runs out records TIMEOUT in the status word and returns:
    the poll reports it once, the context stays usable and later polls are clean."""
    from paper_2604_06746_b200 import binding
    ctx = binding.Context(8, 2, 64, 32, 2048, torch.float32, cuda_device)
    assert ctx.poll_device_status() == binding.OK
    ctx.selftest_wait_expiry(2_000_000)                  # about a millisecond of SM cycles
    assert ctx.poll_device_status() == binding.ERR_TIMEOUT
    assert ctx.poll_device_status() == binding.OK
    scores = torch.rand(4096, device=cuda_device)
    idx = torch.zeros(64, dtype=torch.int32, device=cuda_device)
    ctx.select(scores, 64, 16, idx)                      # ordinary work still runs on the context
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == binding.OK
    assert idx[-1].item() == 4095
    ctx.close()


def test_multi_layer_gather_equals_the_oracle_per_layer(ctx):
    """structkv_compact_layers: several layers, each with its own source and index list, one launch."""
    rng = np.random.default_rng(11)
    L, slabs, n, d, b = 5, 6, 3000, 128, 257
    srcs = [torch.from_numpy(rng.integers(-2 ** 15, 2 ** 15, size=(slabs, n, d), dtype=np.int16)).cuda() for _ in range(L)]
    idx_np = np.stack([np.sort(rng.choice(n, size=b, replace=False)) for _ in range(L)]).astype(np.int32)
    idx = torch.from_numpy(idx_np).cuda()
    out = torch.zeros((L, slabs, b, d), dtype=torch.int16, device="cuda")
    ctx.compact_layers(srcs, idx, out)
    torch.cuda.synchronize()
    from paper_2604_06746_b200 import binding
    assert ctx.poll_device_status() == binding.OK
    for l in range(L):
        assert np.array_equal(out[l].cpu().numpy(), O.compact(srcs[l].cpu().numpy(), idx_np[l])), l
    # odd row size (4-byte units) and a strided source
    srcs2 = [torch.from_numpy(rng.integers(0, 255, size=(2, 500, 20), dtype=np.uint8)).cuda()[:, :, :12] for _ in range(3)]
    idx2 = torch.from_numpy(np.stack([rng.permutation(500)[:40] for _ in range(3)]).astype(np.int32)).cuda()
    out2 = torch.zeros((3, 2, 40, 12), dtype=torch.uint8, device="cuda")
    ctx.compact_layers(srcs2, idx2, out2)
    torch.cuda.synchronize()
    for l in range(3):
        assert np.array_equal(out2[l].cpu().numpy(), O.compact(srcs2[l].cpu().numpy(), idx2[l].cpu().numpy())), l
