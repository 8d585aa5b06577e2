"""Parity rules shared by the GPU tests: how CUDA results are compared with the oracle."""
import numpy as np

REL_TOL = 2e-3          # relative tolerance on centrality, saliency and the layer metrics


def assert_scores_close(gpu, ora, what=""):
    """|g - o| <= 2e-3 |o| + 1e-7 mean(o), element by element."""
    gpu = np.asarray(gpu, dtype=np.float64)
    ora = np.asarray(ora, dtype=np.float64)
    assert gpu.shape == ora.shape, (what, gpu.shape, ora.shape)
    tol = REL_TOL * np.abs(ora) + 1e-7 * np.abs(ora).mean()
    bad = np.abs(gpu - ora) > tol
    if bad.any():
        j = int(np.argmax(np.abs(gpu - ora) / np.maximum(tol, 1e-300)))
        raise AssertionError(f"{what}: {int(bad.sum())} of {bad.size} outside tolerance; worst at "
                             f"{np.unravel_index(j, gpu.shape)}: gpu {gpu.flat[j]!r} oracle {ora.flat[j]!r}")


def assert_metric_close(gpu, ora, what=""):
    assert abs(float(gpu) - float(ora)) <= REL_TOL * abs(float(ora)), (what, float(gpu), float(ora))


def assert_selection_matches(gpu_idx, oracle_scores, budget, window, oracle_idx, what=""):
    """Identical index set when the oracle's k-th and (k+1)-th prefix scores are separated by
    more than the tolerance; otherwise the sets may differ only in near-threshold tokens."""
    gpu_idx = np.asarray(gpu_idx, dtype=np.int64)
    oracle_idx = np.asarray(oracle_idx, dtype=np.int64)
    n = len(oracle_scores)
    assert gpu_idx.shape == (budget,), (what, gpu_idx.shape)
    assert np.all(np.diff(gpu_idx) > 0), what + ": not strictly ascending"
    assert np.array_equal(gpu_idx[budget - window:], np.arange(n - window, n)), what + ": window missing"
    k = budget - window
    if k == 0 or k == n - window:
        assert np.array_equal(gpu_idx, oracle_idx), what
        return
    pre = np.sort(np.asarray(oracle_scores[:n - window], dtype=np.float64))[::-1]
    th_k, th_k1 = pre[k - 1], pre[k]
    if th_k - th_k1 > REL_TOL * th_k:
        assert np.array_equal(gpu_idx, oracle_idx), what + ": index sets differ despite a clear gap"
    else:
        diff = np.setxor1d(gpu_idx, oracle_idx)
        sc = np.asarray(oracle_scores, dtype=np.float64)[diff]
        assert np.all(np.abs(sc - th_k) <= REL_TOL * th_k), what + ": differing tokens are not near the threshold"
