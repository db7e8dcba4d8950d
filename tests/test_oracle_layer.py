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


def test_exactly_representable_inputs_give_the_exact_product():
    rng = np.random.default_rng(0)
    grid = np.array([0, .5, 1, 1.5, 2, 3, 4, 6])
    def rep(rows, cols):
        m = rng.choice(grid, (rows, cols)) * rng.choice([-1.0, 1.0], (rows, cols))
        m[:, ::16] = 6.0                                        # every block has amax 6 -> block scale 2^e exactly
        return (m * 2.0 ** rng.integers(-2, 3, (rows, 1))).astype(F32)
    x, w = rep(32, 64), rep(48, 64)
    s_t = F32(2.0 ** -4)
    cx = nvfp4.quantize(x, tensor_scale=s_t)
    cw = nvfp4.quantize(w, tensor_scale=s_t)
    assert np.array_equal(nvfp4.dequantize(*cx), x) and np.array_equal(nvfp4.dequantize(*cw), w)
    xq = layer.quantize_operand(x, 0, 0, split.MODE_FULL, 0)
    assert np.allclose(xq.res_by_cols, x, rtol=2e-2)            # own-amax tensor scale: close, not exact


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
