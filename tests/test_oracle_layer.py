"""Pins for the oracle's layer composition (Eq. 2, Eq. 3, weight and factor gradients) and for the
paper's claim that the split preserves spectral structure better than direct NVFP4 (Section 4)."""
import numpy as np

from oracle import layer, metrics, nvfp4, split
from paper_2509_00404_b200 import synth

F32 = np.float32


def _ops(k=4, p=4, rounding=nvfp4.ROUND_RNE):
    c = synth.config_small()
    d, _ = synth.planted(128, 256, 8, 2e-2, 2e-3, 1e-4, 1003)
    xq = layer.quantize_operand(c["x"], k, p, split.MODE_FULL, 1, rounding)
    wq = layer.quantize_operand(c["w"], k, p, split.MODE_FULL, 2, rounding)
    dq = layer.quantize_operand(d, k, p, split.MODE_FULL, 3, rounding)
    return c, d, xq, wq, dq


def test_rank_zero_reduces_to_plain_nvfp4_product():
    c, d, xq, wq, dq = _ops(k=0, p=0)
    xd = nvfp4.fake_quantize(c["x"], nvfp4.AXIS_COLS)
    wd = nvfp4.fake_quantize(c["w"], nvfp4.AXIS_COLS)
    assert np.array_equal(layer.linear_fwd(xq, wq), xd @ wd.T)
    assert np.array_equal(layer.linear_dgrad(dq, wq),
                          nvfp4.fake_quantize(d, nvfp4.AXIS_COLS) @ nvfp4.fake_quantize(c["w"], nvfp4.AXIS_ROWS))
    assert np.array_equal(layer.linear_wgrad(dq, xq),
                          nvfp4.fake_quantize(d, nvfp4.AXIS_ROWS).T @ nvfp4.fake_quantize(c["x"], nvfp4.AXIS_ROWS))


def test_forward_equals_term_by_term_expansion_and_triple_loop():
    """Eq. 2 written out as its four products, and a scalar triple loop on a corner of the output."""
    _, _, xq, wq, _ = _ops()
    y = layer.linear_fwd(xq, wq)
    a, lam, b, xr = xq.left_q, np.diag(xq.sigma), xq.right_q, xq.res_by_cols
    v, s, u, wr = wq.left_q, np.diag(wq.sigma), wq.right_q, wq.res_by_cols        # W_t = V S U^T + W_Rt
    terms = (a @ lam @ b.T) @ (u @ s @ v.T) + (a @ lam @ b.T) @ wr.T + xr @ (u @ s @ v.T) + xr @ wr.T
    assert np.allclose(y, terms, rtol=1e-12, atol=1e-9)
    xd, wd = xq.dense(nvfp4.AXIS_COLS), wq.dense(nvfp4.AXIS_COLS)
    for i in range(3):
        for j in range(3):
            acc = 0.0
            for t in range(xd.shape[1]):
                acc += xd[i, t] * wd[j, t]
            assert abs(acc - y[i, j]) <= 1e-10 * max(1.0, abs(acc))


def test_dgrad_equals_the_four_terms_of_eq3_and_wgrad_its_two():
    _, _, xq, wq, dq = _ops()
    pk, t, qk, dr = dq.left_q, np.diag(dq.sigma), dq.right_q, dq.res_by_cols
    v, s, u = wq.left_q, np.diag(wq.sigma), wq.right_q
    wr_rows = wq.res_by_rows                                    # n x m, blocks along n (the contraction axis)
    # paper orientation: W = U S V^T (m x n), W_R = wr^T
    four = (pk @ t @ qk.T @ v @ s.T @ u.T + pk @ t @ qk.T @ wr_rows + dr @ v @ s.T @ u.T + dr @ wr_rows)
    assert np.allclose(layer.linear_dgrad(dq, wq), four, rtol=1e-12, atol=1e-12)
    xbar = xq.dense(nvfp4.AXIS_ROWS)
    two = xbar.T @ (pk @ t @ qk.T) + xbar.T @ dq.res_by_rows    # dL/dW_R in the paper's m x n orientation
    assert np.allclose(layer.linear_wgrad(dq, xq), two.T, rtol=1e-12, atol=1e-12)


def _representable(rng, rows, cols):
    """Values that NVFP4 with an own-amax tensor scale stores without error: E2M1 grid values times a power-of-two
    block scale, a +-6 in every block (so the block scale amax_b/(6 s_T) is that power of two exactly), and one
    element 6 * 448 so that the tensor scale amax/2688 is exactly 1."""
    grid = np.array([0, .5, 1, 1.5, 2, 3, 4, 6])
    m = rng.choice(grid, (rows, cols)) * rng.choice([-1.0, 1.0], (rows, cols))
    m[:, ::16] = 6.0 * rng.choice([-1.0, 1.0], (rows, cols // 16))
    e = rng.integers(-6, 9, (rows, cols // 16))                    # block scales 2^-6 .. 2^8: normal E4M3 numbers
    m = m * np.repeat(2.0 ** e, 16, axis=1)
    m[0, :16] = m[0, :16] / 2.0 ** e[0, 0] * 448.0                 # first block: scale 448, its 6 becomes amax = 2688
    return m.astype(F32)


def test_exactly_representable_inputs_give_the_exact_product():
    """Representable inputs, plain NVFP4 (k = 0): every piece is stored without error, so Eq. 2, Eq. 3 and the weight
    gradient of the layer must equal the exact float64 products of the inputs - not merely be close to them."""
    rng = np.random.default_rng(0)
    x, w, d = _representable(rng, 32, 64), _representable(rng, 48, 64), _representable(rng, 32, 48)
    xq = layer.quantize_operand(x, 0, 0, split.MODE_FULL, 0)
    wq = layer.quantize_operand(w, 0, 0, split.MODE_FULL, 0)
    dq = layer.quantize_operand(d, 0, 0, split.MODE_FULL, 0)
    for q, t in ((xq, x), (wq, w), (dq, d)):
        assert q.raw["res_by_cols"][2] == F32(1.0)
        assert np.array_equal(q.res_by_cols, t.astype(np.float64))
    x64, w64, d64 = (t.astype(np.float64) for t in (x, w, d))
    assert np.array_equal(layer.linear_fwd(xq, wq), x64 @ w64.T)
    # the products that contract over rows use blocks along the rows: the transpose of a representable matrix is
    # representable in that orientation
    xr, dr, wr = _representable(rng, 64, 32).T.copy(), _representable(rng, 48, 32).T.copy(), _representable(rng, 64, 48).T.copy()
    xrq = layer.quantize_operand(xr, 0, 0, split.MODE_FULL, 0)
    drq = layer.quantize_operand(dr, 0, 0, split.MODE_FULL, 0)
    wrq = layer.quantize_operand(wr, 0, 0, split.MODE_FULL, 0)
    for q, t in ((xrq, xr), (drq, dr), (wrq, wr)):
        assert np.array_equal(q.res_by_rows, t.astype(np.float64))
    assert np.array_equal(layer.linear_wgrad(drq, xrq), dr.astype(np.float64).T @ xr.astype(np.float64))
    assert np.array_equal(layer.linear_dgrad(dq, wrq), d64 @ wr.astype(np.float64))


def test_representable_low_rank_inputs_give_the_exact_product_with_a_split():
    """k > 0: a rank-2 operand whose singular vectors have entries +-1/8 (scaled Hadamard columns) is split into
    factors that NVFP4 stores without error (every block is +-1/8 throughout: code 6 under scale 448), the residual
    is zero to rounding, and the split-FP4 forward product equals the exact product to float32-scale accuracy."""
    h2 = np.array([[1.0, 1.0], [1.0, -1.0]])
    had = h2
    for _ in range(5):
        had = np.kron(had, h2)                                      # 64 x 64 Hadamard matrix
    u, v = had[:, [3, 17]] / 8.0, had[:, [5, 40]] / 8.0             # orthonormal columns with entries +-1/8
    x = ((u * np.array([8.0, 2.0])) @ v.T).astype(F32)              # entries in {+-1/8 +- 1/32}: exact in bf16
    w = ((had[:, [9, 33]] / 8.0 * np.array([4.0, 1.0])) @ (had[:, [5, 21]] / 8.0).T).astype(F32)
    xq = layer.quantize_operand(x, 2, 0, split.MODE_FULL, 3)
    wq = layer.quantize_operand(w, 2, 0, split.MODE_FULL, 4)
    assert np.allclose(xq.sigma, [8.0, 2.0], rtol=1e-12) and np.allclose(wq.sigma, [4.0, 1.0], rtol=1e-12)
    assert np.allclose(np.abs(xq.left_q), 0.125, rtol=1e-6) and np.allclose(np.abs(xq.right_q), 0.125, rtol=1e-6)
    assert np.abs(xq.res_by_cols).max() < 1e-12
    want = x.astype(np.float64) @ w.astype(np.float64).T
    got = layer.linear_fwd(xq, wq)
    assert np.linalg.norm(got - want) / np.linalg.norm(want) < 1e-6


def test_metrics_on_cases_with_known_answers():
    """subspace_alignment: identical bases 1, orthogonal bases 0, one shared direction of two 1/2.
    spectral_fidelity on diagonal matrices: singular values are the diagonal, vectors the unit vectors."""
    e = np.eye(6)
    assert np.isclose(metrics.subspace_alignment(e[:, :2], e[:, :2]), 1.0)
    assert np.isclose(metrics.subspace_alignment(e[:, :2], e[:, 2:4]), 0.0)
    assert np.isclose(metrics.subspace_alignment(e[:, :2], e[:, 1:3]), 0.5)
    rot = np.array([[np.cos(0.3), -np.sin(0.3)], [np.sin(0.3), np.cos(0.3)]])
    assert np.isclose(metrics.subspace_alignment(e[:, :2], e[:, :2] @ rot), 1.0)      # a basis change inside the span
    ref = np.diag([5.0, 3.0, 2.0, 1.0])
    rs, cos = metrics.spectral_fidelity(ref, ref)
    assert np.allclose(rs, 0.0) and np.allclose(cos, 1.0)
    rs, cos = metrics.spectral_fidelity(ref, np.diag([5.5, 2.7, 2.0, 1.0]))
    assert np.allclose(rs, [0.1, 0.1, 0.0, 0.0]) and np.allclose(cos, 1.0)
    swapped = ref[[1, 0, 2, 3]]                                      # rows 0 and 1 exchanged: left vectors e2, e1, e3, e4
    rs, cos = metrics.spectral_fidelity(ref, swapped)
    assert np.allclose(rs, 0.0) and np.allclose(cos, [0.0, 0.0, 1.0, 1.0])
    assert np.isclose(metrics.rel_fro(np.array([3.0, 4.0]), np.array([0.0, 4.0])), 0.75)


def test_residual_uses_the_source_tensor_scale_and_unquantized_factors():
    c, _, xq, _, _ = _ops()
    s_src = nvfp4.tensor_scale_from_amax(np.max(np.abs(c["x"])))
    assert xq.raw["res_by_cols"][2] == s_src and xq.raw["res_by_rows"][2] == s_src
    sp = xq.split
    assert np.allclose((sp.left * sp.sigma) @ sp.right.T + sp.residual, c["x"], atol=1e-9)
    assert xq.raw["left"][0].shape == (4, 128) and xq.raw["right"][0].shape == (4, 256)
    assert np.array_equal(xq.res_by_cols, nvfp4.dequantize(*xq.raw["res_by_cols"]))
    assert np.array_equal(xq.res_by_rows, nvfp4.dequantize(*xq.raw["res_by_rows"]).T)


def test_factor_gradients_match_finite_differences():
    """dU, dS, dV are the derivatives of <dW, U S V^T> - checked numerically."""
    _, _, xq, wq, dq = _ops()
    dw_t = layer.linear_wgrad(dq, xq)
    du, ds, dv = layer.factor_grads(dw_t, wq)
    u, v, s = wq.right_q, wq.left_q, wq.sigma
    f = lambda u_, s_, v_: np.sum(dw_t.T * ((u_ * s_) @ v_.T))
    eps = 1e-6
    rng = np.random.default_rng(1)
    for _ in range(5):
        i, j = rng.integers(u.shape[0]), rng.integers(u.shape[1])
        e = np.zeros_like(u); e[i, j] = eps
        assert np.isclose((f(u + e, s, v) - f(u - e, s, v)) / (2 * eps), du[i, j], rtol=1e-5, atol=1e-12)
        i, j = rng.integers(v.shape[0]), rng.integers(v.shape[1])
        e = np.zeros_like(v); e[i, j] = eps
        assert np.isclose((f(u, s, v + e) - f(u, s, v - e)) / (2 * eps), dv[i, j], rtol=1e-5, atol=1e-12)
    for j in range(len(s)):
        e = np.zeros_like(s); e[j] = eps * s[j]
        assert np.isclose((f(u, s + e, v) - f(u, s - e, v)) / (2 * eps * s[j]), ds[j], rtol=1e-5, atol=1e-12)


def test_split_preserves_spectrum_better_than_direct_nvfp4():
    """The paper's measurable claim (Section 4, spectral preservation figure): lower singular-value
    error and better singular-vector alignment than direct NVFP4, in particular for the small
    components that direct quantization distorts most (Section 2.3)."""
    x, _ = synth.llama_like(1024, 1024, 1.0, 31, rank=32)
    x64 = x.astype(np.float64)
    direct = nvfp4.fake_quantize(x, nvfp4.AXIS_COLS)
    xq = layer.quantize_operand(x, 32, 8, split.MODE_FULL, 5)
    ours = xq.dense(nvfp4.AXIS_COLS)
    rs_d, cos_d = metrics.spectral_fidelity(x64, direct)
    rs_o, cos_o = metrics.spectral_fidelity(x64, ours)
    assert rs_o.mean() < rs_d.mean()
    assert rs_o[32:].mean() < 0.5 * rs_d[32:].mean()
    assert cos_o[32:].mean() > cos_d[32:].mean()
    # (the 32 dominant directions are already aligned to > 0.99 either way; no claim is asserted there)
    # the residual is what the paper says it is: far narrower than the input
    assert np.abs(xq.split.residual).max() < 0.5 * np.abs(x64).max()


def test_stochastic_rounding_config_runs_and_differs_from_rne():
    _, _, xq, wq, dq = _ops(rounding=nvfp4.ROUND_SR)
    _, _, xq2, wq2, dq2 = _ops(rounding=nvfp4.ROUND_RNE)
    assert not np.array_equal(dq.res_by_cols, dq2.res_by_cols)
    ref = dq.split.residual
    assert metrics.rel_fro(dq.res_by_cols, ref) < 0.25


def test_requantizing_the_stored_pieces_of_a_split_reproduces_the_split_operand():
    """The persistent-operand route against the pinned one: the pieces that quantize_operand produced, stored in
    float32 and quantized again with the residual's original tensor scale, give the same bytes piece by piece; with
    the residual's own amax as scale (the stored-weight default) the residual changes scale but still covers every
    block, and the factors are untouched."""
    c, _, xq, _, _ = _ops()
    sp = xq.split
    s_src = nvfp4.tensor_scale_from_amax(np.max(np.abs(c["x"])))
    res32 = sp.residual.astype(F32)
    again = layer.requantize_operand(sp.left.astype(F32), sp.sigma, sp.right.astype(F32), res32, residual_scale=s_src)
    for name in ("res_by_cols", "res_by_rows", "left", "right"):
        for a, b in zip(again.raw[name], xq.raw[name]):
            assert np.array_equal(a, b), name
    assert np.array_equal(again.dense(nvfp4.AXIS_COLS), xq.dense(nvfp4.AXIS_COLS))
    own = layer.requantize_operand(sp.left.astype(F32), sp.sigma, sp.right.astype(F32), res32)
    assert own.raw["res_by_cols"][2] == nvfp4.tensor_scale_from_amax(np.max(np.abs(res32))) < s_src
    assert np.array_equal(own.raw["left"][0], xq.raw["left"][0])
    # own scale: the residual's largest element sits on code 6 of a scale-448 block and is reproduced to rounding
    i, j = np.unravel_index(np.argmax(np.abs(res32)), res32.shape)
    assert np.isclose(own.res_by_cols[i, j], res32[i, j], rtol=1e-6)
    assert metrics.rel_fro(own.res_by_cols, res32) <= metrics.rel_fro(xq.res_by_cols, res32) * 1.05


def test_conditioning_of_the_end_to_end_value_when_the_rank_cut_falls_inside_the_bulk():
    """How far the oracle's OWN split-FP4 output moves when its input is perturbed by 1e-6 relative - the size of an
    FP32 accumulation over a few thousand terms, which any FP32 pipeline carries in its sketch and projection.
    With k at most the planted rank every kept singular vector is well separated and the output moves by about 1e-3;
    with k above it the extra vectors are singular vectors of the Gaussian bulk (neighbouring singular values a
    fraction of a percent apart), they turn by ~1e-4, the NVFP4 encoder re-rounds a few blocks per thousand, and the
    output moves by more than the 2e-3 that the end-to-end comparisons allow.  This is why the GPU parity tests treat
    the cases with k above the planted rank (the rank-128 and rank-256 points of the 70B-shaped sweep) as
    conditioning-limited and check what is unique there instead."""
    def moved(k, rank, n=512, pert=1e-6):
        x, _ = synth.llama_like(n, n, 1.0, 5, rank=rank)
        w, _ = synth.llama_like(n, n, 0.02, 6, rank=rank)
        rng = np.random.default_rng(0)

        def forward(noise):
            ops = []
            for t, seed in ((x, 1), (w, 2)):
                t64 = t.astype(np.float64) * (1.0 + noise * rng.standard_normal(t.shape)) if noise else t.astype(np.float64)
                sp = split.split(t64, k, 8, split.MODE_FULL, seed)
                ops.append(layer.requantize_operand(sp.left, sp.sigma, sp.right, sp.residual,
                                                    residual_scale=nvfp4.tensor_scale_from_amax(np.max(np.abs(t)))))
            return layer.linear_fwd(*ops)
        y0, y1 = forward(0.0), forward(pert)
        return np.linalg.norm(y1 - y0) / np.linalg.norm(y0)
    assert moved(16, 16) < 2e-3 and moved(32, 32) < 2e-3
    assert moved(64, 16) > 2e-3 and moved(128, 16) > 2e-3
    assert moved(64, 16, pert=3e-6) > 1e-2                 # a few 1e-6 are enough for differences of a few per cent
