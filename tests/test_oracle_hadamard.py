"""Pins of the oracle's random-Hadamard + stochastic-rounding comparison recipe (Section 4 of the paper)."""
import numpy as np
from scipy.linalg import hadamard

from oracle import hadamard as ohad, layer, metrics, nvfp4, philox, split
from paper_2509_00404_b200 import synth

F32 = np.float32


def test_butterflies_equal_the_hadamard_matrix_product():
    """Library pin: the four binary32 butterfly stages are multiplication by scipy's Sylvester matrix H16 / 4."""
    rng = np.random.default_rng(0)
    x = rng.standard_normal((7, 64)).astype(F32)
    s = ohad.signs(64, 5).astype(np.float64)
    want = ((x.astype(np.float64) * s).reshape(7, 4, 16) @ (hadamard(16) / 4.0)).reshape(7, 64)
    got = ohad.rht(x, 5)
    assert got.dtype == F32 and np.allclose(got, want, rtol=0, atol=1e-6)
    # exactly representable inputs: no rounding anywhere, equality
    xi = rng.integers(-8, 9, (3, 32)).astype(F32)
    wi = ((xi.astype(np.float64) * ohad.signs(32, 9)).reshape(3, 2, 16) @ (hadamard(16) / 4.0)).reshape(3, 32)
    assert np.array_equal(ohad.rht(xi, 9).astype(np.float64), wi)


def test_transform_is_orthogonal_and_keeps_products():
    rng = np.random.default_rng(1)
    x, w = rng.standard_normal((5, 48)).astype(F32), rng.standard_normal((6, 48)).astype(F32)
    xr, wr = ohad.rht(x, 3).astype(np.float64), ohad.rht(w, 3).astype(np.float64)
    assert np.allclose(np.linalg.norm(xr, axis=1), np.linalg.norm(x.astype(np.float64), axis=1), rtol=1e-6)
    assert np.allclose(xr @ wr.T, x.astype(np.float64) @ w.astype(np.float64).T, atol=1e-5)
    assert np.allclose(ohad.rht_inverse(xr, 3), x, atol=1e-6)


def test_signs_come_from_bit_15_of_the_draw_and_are_balanced():
    s = ohad.signs(4096, 11)
    u = philox.draw_u16(np.arange(4096, dtype=np.uint64), 11, ohad.STREAM_SIGNS)
    assert np.array_equal(s < 0, u >= 32768) and set(np.unique(s)) == {-1.0, 1.0}
    assert abs(float(s.mean())) < 0.06
    assert not np.array_equal(s, ohad.signs(4096, 12))


def test_an_outlier_is_spread_over_its_block():
    """What the rotation is for: a single large element becomes sixteen of a quarter of its size."""
    x = np.zeros((1, 32), dtype=F32)
    x[0, 5] = 64.0
    y = ohad.rht(x, 2)
    assert np.array_equal(np.abs(y[0, :16]), np.full(16, 16.0, dtype=F32)) and not y[0, 16:].any()


def test_spectral_fidelity_split_beats_the_hadamard_recipe_on_planted_anisotropy():
    """The paper's comparison (Section 4, spectral preservation figure): better alignment of singular directions and
    lower singular-value error than NVFP4 with the random-Hadamard + SR recipe - for the small components, which
    block quantization distorts most."""
    x, _ = synth.llama_like(1024, 1024, 1.0, 31, rank=32)
    x64 = x.astype(np.float64)
    recipe = ohad.fake_quantize_rht(x, nvfp4.ROUND_SR, seed=7)
    ours = layer.quantize_operand(x, 32, 8, split.MODE_FULL, 5).dense(nvfp4.AXIS_COLS)
    rs_r, cos_r = metrics.spectral_fidelity(x64, recipe)
    rs_o, cos_o = metrics.spectral_fidelity(x64, ours)
    assert rs_o[32:].mean() < 0.5 * rs_r[32:].mean()
    assert cos_o[32:].mean() > cos_r[32:].mean()
    # the recipe itself is a sane NVFP4 quantizer: relative error of the order of the format's step
    assert 0.02 < metrics.rel_fro(recipe, x64) < 0.2
