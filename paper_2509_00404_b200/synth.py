"""Seeded synthetic inputs shared by the tests, the benchmark and the oracle's callers.

Holds none of the method's arithmetic: only planted-spectrum matrix generation and bfloat16
rounding of the generated values.  The matrices stand in for the LLaMA-3 activations, weights and
output gradients the paper analyses (a few dominant singular components on top of a Gaussian
bulk, Section 2.1); shapes follow the LLaMA-3-8B projections.

Every generator returns float32 numpy arrays whose values are exactly representable in bfloat16,
so `torch.from_numpy(a).to(torch.bfloat16)` loses nothing and both sides of a parity test see the
same numbers.
"""
import math

import numpy as np


def to_bf16_values(a):
    """Round float32 values to the nearest bfloat16 (ties to even), keep float32 storage."""
    b = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    b = (b + np.uint64(0x7FFF) + ((b >> np.uint64(16)) & np.uint64(1))) & np.uint64(0xFFFF0000)
    return b.astype(np.uint32).view(np.float32).reshape(np.shape(a))


def bf16_bits(a):
    """uint16 bit patterns of float32 values that are already bf16-representable."""
    return (np.ascontiguousarray(a, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)


def planted(rows, cols, rank, s_top, s_bot, sigma, seed, exact=False):
    """Rank-`rank` spike with orthonormal (Haar) factors and geometric singular values s_top..s_bot,
    plus an iid N(0, sigma^2) bulk.  Returns (matrix, singular values of the spike).

    exact=True skips the bfloat16 rounding (float64 result) for closed-form checks of the oracle.
    """
    rng = np.random.default_rng(seed)
    u, _ = np.linalg.qr(rng.standard_normal((rows, rank)))
    v, _ = np.linalg.qr(rng.standard_normal((cols, rank)))
    s = np.geomspace(s_top, s_bot, rank) if rank > 1 else np.array([float(s_top)])
    m = (u * s) @ v.T
    if sigma:
        m = m + sigma * rng.standard_normal((rows, cols))
    if exact:
        return m, s
    return to_bf16_values(m.astype(np.float32)), s


def llama_like(rows, cols, sigma, seed, rank=32):
    """The benchmark recipe: top singular value 100x the bulk edge sigma*(sqrt(rows)+sqrt(cols)), 10:1 span."""
    s_top = 100.0 * sigma * (math.sqrt(rows) + math.sqrt(cols))
    return planted(rows, cols, rank, s_top, s_top / 10.0, sigma, seed)


def planted_device(rows, cols, rank, sigma, seed, device="cuda"):
    """The llama_like recipe generated on the device with torch's seeded generator (benchmark-size matrices, where
    the host generator would take minutes); returns a bfloat16 tensor.  Same structure, different random stream."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    u, _ = torch.linalg.qr(torch.randn((rows, rank), generator=g, device=device))
    v, _ = torch.linalg.qr(torch.randn((cols, rank), generator=g, device=device))
    s_top = 100.0 * sigma * (math.sqrt(rows) + math.sqrt(cols))
    s = torch.logspace(math.log10(s_top), math.log10(s_top / 10.0), rank, device=device)
    m = (u * s) @ v.T
    m += sigma * torch.randn((rows, cols), generator=g, device=device)
    return m.to(torch.bfloat16)


# the small forward-only workload (128 tokens, 256 -> 256) and one LLaMA-3-8B q_proj-shaped layer
def config_small(seed=1001):
    x, sx = planted(128, 256, 8, 200.0, 20.0, 1.0, seed)
    w, sw = planted(256, 256, 8, 200.0, 20.0, 1.0, seed + 1)
    return {"x": x, "w": w, "k": 4, "p": 4, "sx": sx, "sw": sw}


def config_qproj(tokens=4096, d_in=4096, d_out=4096, seed=2000):
    x, _ = llama_like(tokens, d_in, 1.0, seed)
    w, _ = llama_like(d_out, d_in, 0.02, seed + 1)
    dy, _ = llama_like(tokens, d_out, 1e-4, seed + 2)
    return {"x": x, "w": w, "dy": dy, "k": 32, "p": 8}
