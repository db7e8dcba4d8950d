"""Pins for the oracle's low-rank + residual split (Sections 3.1, 3.2): closed forms on planted
spectra, library special cases, and the algebraic invariants the paper's definitions imply."""
import numpy as np
import pytest

from oracle import metrics, split
from paper_2509_00404_b200 import synth


def test_planted_noise_free_full_mode_recovers_singular_values():
    x, s = synth.planted(128, 256, 8, 200.0, 20.0, 0.0, 1001, exact=True)     # rank 8 = k + p
    sp = split.split(x, 4, 4, split.MODE_FULL, seed=3)
    assert np.allclose(sp.sigma, s[:4], rtol=1e-10)
    tail = np.linalg.svd(sp.residual, compute_uv=False)
    assert np.allclose(tail[:4], s[4:], rtol=1e-9) and tail[4] < 1e-9
    sp8 = split.split(x, 8, 0, split.MODE_FULL, seed=3)
    assert np.allclose(sp8.sigma, s, rtol=1e-10) and np.linalg.norm(sp8.residual) < 1e-9


def test_planted_noise_free_sampled_mode_k_equals_rank():
    x, s = synth.planted(2048, 256, 6, 50.0, 5.0, 0.0, 77, exact=True)
    sp = split.split(x, 6, 4, split.MODE_SAMPLED, seed=9)
    assert np.allclose(sp.sigma, s, rtol=1e-9)
    assert np.linalg.norm(sp.residual) < 1e-8 * np.linalg.norm(x)


def test_full_sketch_equals_library_svd():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((24, 40))
    sp = split.split(x, 5, 19, split.MODE_FULL, seed=1)                        # k + p = min(rows, cols)
    u, s, vt = np.linalg.svd(x, full_matrices=False)
    assert np.allclose(sp.sigma, s[:5], rtol=1e-10)
    for j in range(5):
        assert abs(abs(sp.left[:, j] @ u[:, j]) - 1) < 1e-9 and abs(abs(sp.right[:, j] @ vt[j]) - 1) < 1e-9
    best = x - (u[:, :5] * s[:5]) @ vt[:5]
    assert np.allclose(sp.residual, best, atol=1e-9)


@pytest.mark.parametrize("mode", [split.MODE_FULL, split.MODE_SAMPLED])
def test_invariants(mode):
    x, _ = synth.planted(1024, 192, 8, 300.0, 30.0, 1.0, 5)
    x = x.astype(np.float64)
    k, p = 6, 6
    sp = split.split(x, k, p, mode, seed=4)
    eye = np.eye(k)
    assert np.allclose((sp.left * sp.sigma) @ sp.right.T + sp.residual, x, atol=1e-10)
    assert np.allclose(sp.left.T @ sp.left, eye, atol=1e-10)
    assert np.allclose(sp.right.T @ sp.right, eye, atol=1e-10)
    assert np.all(np.diff(sp.sigma) <= 0) and np.all(sp.sigma > 0)
    if mode == split.MODE_FULL:
        assert np.allclose(sp.left.T @ sp.residual, 0, atol=1e-9)
    else:
        assert np.allclose(sp.residual @ sp.right, 0, atol=1e-9)
        # the residual is row-local: recompute three rows alone from the basis
        b = sp.extra["basis"]
        for i in (0, 511, 1023):
            assert np.allclose(sp.residual[i], x[i] - (x[i] @ b) @ b.T, atol=1e-12)
    # Ritz values never exceed the true singular values (Cauchy interlacing for projections)
    s_true = np.linalg.svd(x, compute_uv=False)
    assert np.all(sp.sigma <= s_true[:k] * (1 + 1e-12))
    # sign convention
    for j in range(k):
        assert sp.right[np.argmax(np.abs(sp.right[:, j])), j] > 0


def test_halko_error_bound_full_mode():
    """E||X - HH^T X||_F <= sqrt(1 + k/(p-1)) * (sum_{j>k} sigma_j^2)^(1/2) (Halko et al., Thm 10.5);
    the rank-k truncation inside the sketch adds at most the (k+1)-th singular value's share."""
    x, _ = synth.planted(256, 128, 8, 400.0, 100.0, 1.0, 8)
    x = x.astype(np.float64)
    s_true = np.linalg.svd(x, compute_uv=False)
    k, p = 8, 8
    tail = np.sqrt(np.sum(s_true[k:] ** 2))
    errs = [np.linalg.norm(split.split(x, k, p, split.MODE_FULL, seed=s).residual) for s in range(12)]
    assert min(errs) >= tail * (1 - 1e-12)                         # Eckart-Young lower bound
    assert np.mean(errs) <= 2.0 * np.sqrt(1 + k / (p - 1)) * tail


def test_sampling_rule():
    for rows, q in ((4096, 40), (16384, 40), (16384, 72), (200, 8), (128, 8)):
        n = split.default_sample_count(rows, q)
        assert n % 16 == 0 or n == rows
        assert n >= min(rows, 4 * q) and n >= min(rows, rows // 100)
        idx = split.sample_rows(rows, n, seed=13)
        g = rows // n
        assert len(idx) == n and np.all(np.diff(idx) > 0)
        assert np.all(idx // g == np.arange(n))                      # exactly one row per stratum
        assert idx.max() < rows
    assert split.default_sample_count(4096, 40) == 160 and split.default_sample_count(16384, 40) == 176
    a = split.sample_rows(4096, 160, seed=1)
    b = split.sample_rows(4096, 160, seed=2)
    assert not np.array_equal(a, b)
    offs = np.concatenate([split.sample_rows(4096, 160, seed=s) % 25 for s in range(40)])
    assert abs(offs.mean() - 12) < 1.0                               # offsets uniform over the stratum


def test_sampled_subspace_aligns_with_full_batch():
    """Section 3.1: a small row sample recovers the dominant right subspace of the whole batch."""
    x, _ = synth.llama_like(4096, 512, 1.0, 21, rank=16)
    x = x.astype(np.float64)
    sp = split.split(x, 16, 8, split.MODE_SAMPLED, seed=2)
    _, _, vt = np.linalg.svd(x, full_matrices=False)
    assert metrics.subspace_alignment(vt[:16].T, sp.right) > 0.9
    assert len(sp.extra["rows_sampled"]) == split.default_sample_count(4096, 24)


def test_rank_zero_is_identity_split():
    x = np.arange(12.0).reshape(3, 4)
    sp = split.split(x, 0, 0)
    assert np.array_equal(sp.residual, x) and sp.left.shape == (3, 0) and sp.sigma.size == 0
