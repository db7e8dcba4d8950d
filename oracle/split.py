"""Low-rank + residual split of one GEMM operand (Sections 3.1 and 3.2).

Test infrastructure: a slow restatement used to check the CUDA library; never on the product path.

T = L diag(sigma) R^T + Res, with (L, sigma, R) the top-k factors recovered by the paper's
two-step "scalable spectral decomposition":

  * random projection (randomized SVD, Halko et al.): sketch Z = T Omega with a Gaussian test
    matrix of k+p columns, thin QR Z = H R_z, small SVD of M = H^T T, keep the top k;
  * sparse random sampling: estimate the dominant right subspace from a small random subset of
    the rows and "broadcast" it to the full batch.

The paper's formula for the projected problem (eigenspaces of H^T Sigma H) does not type-check
with its own dimensions; the standard randomized SVD it cites is used.  How a subspace found on
the sampled rows yields (L, sigma) for all rows is not stated; the reading here is the
Rayleigh-Ritz step C = T B, C^T C = W Theta W^T, sigma = sqrt(Theta), L = C W / sigma, R = B W.
No power iterations.  The residual is taken against the unquantized factors.
"""
from dataclasses import dataclass, field

import numpy as np

from . import gauss, philox

MODE_FULL = 0
MODE_SAMPLED = 1


@dataclass
class Split:
    left: np.ndarray        # rows x k, orthonormal columns
    sigma: np.ndarray       # k, descending
    right: np.ndarray       # cols x k, orthonormal columns
    residual: np.ndarray    # rows x cols
    extra: dict = field(default_factory=dict)


def default_sample_count(rows, q):
    """Rows sampled: at least 4(k+p), at least 1 % of the rows, rounded up to a multiple of 16."""
    want = max(4 * q, -(-rows // 100))
    want = -(-want // 16) * 16
    return min(rows, want)


def sample_rows(rows, n_sample, seed):
    """One row per stratum of g = rows // n_sample consecutive rows (distinct, increasing)."""
    g = rows // n_sample
    j = np.arange(n_sample, dtype=np.uint64)
    w0 = philox.draw_word0(j, seed, philox.STREAM_SAMPLING)
    return (j * np.uint64(g) + w0 % np.uint64(g)).astype(np.int64)


def fix_signs(left, right):
    """Flip column pairs so the largest-magnitude entry of each right vector (lowest index on ties) is positive."""
    left, right = left.copy(), right.copy()
    for j in range(right.shape[1]):
        i = int(np.argmax(np.abs(right[:, j])))
        if right[i, j] < 0:
            right[:, j] = -right[:, j]
            left[:, j] = -left[:, j]
    return left, right


def _range_finder(x, q, seed):
    """Z = x Omega, thin QR, M = H^T x, small SVD.  Returns H, U~, s~, V~^T."""
    om = gauss.omega(x.shape[1], q, seed).astype(np.float64)
    z = x @ om
    h, _ = np.linalg.qr(z)
    m = h.T @ x
    ut, st, vtt = np.linalg.svd(m, full_matrices=False)
    return h, ut, st, vtt


def split(x, k, p, mode=MODE_FULL, seed=0, n_sample=0):
    """Split x (rows x cols, float64) into rank-k factors and a residual."""
    x = np.asarray(x, dtype=np.float64)
    rows, cols = x.shape
    if k == 0:
        return Split(np.zeros((rows, 0)), np.zeros(0), np.zeros((cols, 0)), x.copy())
    q = k + p
    if mode == MODE_FULL:
        if q > min(rows, cols):
            raise ValueError("k+p exceeds the matrix size")
        h, ut, st, vtt = _range_finder(x, q, seed)
        left = h @ ut[:, :k]
        sigma = st[:k].copy()
        right = vtt[:k, :].T
        left, right = fix_signs(left, right)
        residual = x - (left * sigma) @ right.T
        return Split(left, sigma, right, residual)
    if mode != MODE_SAMPLED:
        raise ValueError("mode")
    n_s = n_sample if n_sample else default_sample_count(rows, q)
    if q > min(n_s, cols):
        raise ValueError("k+p exceeds the sampled matrix size")
    rows_s = sample_rows(rows, n_s, seed)
    _, _, _, vtt = _range_finder(x[rows_s, :], q, seed)
    b = vtt[:k, :].T                                   # cols x k, dominant right subspace of the sample
    c = x @ b                                          # broadcast to the full batch
    theta, w = np.linalg.eigh(c.T @ c)
    order = np.argsort(theta)[::-1]
    theta, w = np.maximum(theta[order], 0.0), w[:, order]
    sigma = np.sqrt(theta)
    cw = c @ w
    left = np.divide(cw, sigma, out=np.zeros_like(cw), where=sigma > 0)
    right = b @ w
    left, right = fix_signs(left, right)
    residual = x - c @ b.T                             # row-local: r_i = x_i - (x_i B) B^T
    return Split(left, sigma, right, residual, {"rows_sampled": rows_s, "basis": b, "coeff": c})
