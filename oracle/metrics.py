"""Spectral-fidelity and subspace measures (Section 3.1 alignment; Section 4 spectral preservation figure).

Test infrastructure: a slow restatement used to check the CUDA library; never on the product path.
"""
import numpy as np


def rel_fro(a, b):
    """||a - b||_F / ||b||_F."""
    return float(np.linalg.norm(np.asarray(a, np.float64) - np.asarray(b, np.float64)) / np.linalg.norm(b))


def subspace_alignment(q1, q2):
    """Mean squared canonical correlation between two orthonormal bases (columns)."""
    s = np.linalg.svd(q1.T @ q2, compute_uv=False)
    return float(np.mean(s ** 2))


def spectral_fidelity(reference, approx):
    """Per-component relative singular-value error and |cos| between matching left singular vectors."""
    u0, s0, _ = np.linalg.svd(reference, full_matrices=False)
    u1, s1, _ = np.linalg.svd(approx, full_matrices=False)
    rel_sigma = np.abs(s1 - s0) / s0
    cos_left = np.abs(np.sum(u0 * u1, axis=0))
    return rel_sigma, cos_left
