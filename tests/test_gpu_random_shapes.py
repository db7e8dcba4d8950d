"""GPU parity on seeded random shapes, ranks, oversampling, sketch modes and rounding modes: the decomposition against
the oracle (same checks as test_gpu_split: factors, residual, bit-exact bytes), and the layer's three products against
the float64 composition of the library's own quantized pieces.  Shapes are multiples of 64 up to 2048 x 1024, so the
cases cross every tile boundary of the tensor-core kernels (128-row tiles, 128-column tiles, 64-wide K chunks, 256-wide
GEMM tiles) with ragged remainders."""
import numpy as np
import pytest
import torch

from paper_2509_00404_b200 import synth

pytestmark = pytest.mark.gpu


def _split_cases(seed, count):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        rows, cols = int(rng.integers(2, 33)) * 64, int(rng.integers(1, 17)) * 64
        k, p = int(rng.integers(1, 17)) * 4, int(rng.choice([0, 4, 8]))
        full, sr = bool(rng.integers(0, 2)), bool(rng.integers(0, 2))
        q = k + p
        n_s = rows if full else min(rows, -(-max(4 * q, -(-rows // 100)) // 16) * 16)
        if q > min(n_s, cols) or q > 72 or 4 * k > min(rows, cols):   # keep a residual worth comparing (rank well below both extents)
            continue
        rank = int(rng.choice([max(k, 8), max(k // 2, 4), min(2 * k, 64)]))
        sigma = float(rng.choice([1.0, 0.02, 1e-4]))
        out.append((rows, cols, k, p, full, sr, rank, sigma, len(out)))
    return out


@pytest.mark.parametrize("case", _split_cases(7, 24), ids=lambda c: "%dx%d_k%d_p%d_%s_%s" % (c[0], c[1], c[2], c[3], "full" if c[4] else "sampled", "sr" if c[5] else "rne"))
def test_random_split_against_oracle(case):
    from paper_2509_00404_b200 import binding as B
    import test_gpu_split as T
    rows, cols, k, p, full, sr, rank, sigma, idx = case
    x, _ = synth.llama_like(rows, cols, sigma, 900 + idx, rank=rank)
    h = B.Handle(0)
    try:
        T._check_against_oracle(B, h, x, k, p, B.SKETCH_FULL if full else B.SKETCH_SAMPLED, seed=100 + idx, rounding=1 if sr else 0)
    finally:
        h.close()


def _layer_cases(seed, count):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        l, m, n = (int(rng.integers(2, 17)) * 64 for _ in range(3))
        k = int(rng.choice([0, 4, 8, 16, 24, 32]))
        p = 0 if k == 0 else int(rng.choice([0, 4, 8]))
        if k and (k + p > min(l, m, n) // 4 or 2 * k > min(m, n)):
            continue
        out.append((l, m, n, k, p, len(out)))
    return out


@pytest.mark.parametrize("case", _layer_cases(11, 12), ids=lambda c: "%dtok_%dto%d_k%d_p%d" % c[:5])
def test_random_layer_composition(case):
    from gpu_util import to_dev_bf16, rel_fro
    from paper_2509_00404_b200 import binding as B
    import test_gpu_layer as T
    l, m, n, k, p, idx = case
    x, _ = synth.llama_like(l, m, 1.0, 700 + idx, rank=max(k, 8))
    w, _ = synth.llama_like(n, m, 0.02, 800 + idx, rank=max(k, 8))
    d, _ = synth.llama_like(l, n, 1e-4, 900 + idx, rank=max(k, 8))
    h = B.Handle(0)
    try:
        xo = h.split(to_dev_bf16(x), k, p, sketch=B.SKETCH_SAMPLED, seed=1)
        wo = h.split(to_dev_bf16(w), k, p, sketch=B.SKETCH_FULL, seed=2)
        do = h.split(to_dev_bf16(d), k, p, sketch=B.SKETCH_SAMPLED, seed=3, rounding=B.ROUND_SR)
        y = h.linear_fwd(xo, wo)
        dx, dw = h.linear_bwd(do, xo, wo)
        torch.cuda.synchronize()
        assert h.device_status() == 0
        lx, rxc, rxr = T._oracle_from_gpu_operand(xo, k)
        lw, rwc, rwr = T._oracle_from_gpu_operand(wo, k)
        ld, rdc, rdr = T._oracle_from_gpu_operand(do, k)
        assert rel_fro(y.cpu().numpy(), (lx + rxc) @ (lw + rwc).T) < 2e-5
        assert rel_fro(dx.cpu().numpy(), (ld + rdc) @ (lw + rwr)) < 2e-5
        assert rel_fro(dw.cpu().numpy(), (ld + rdr).T @ (lx + rxr)) < 2e-5
    finally:
        h.close()
