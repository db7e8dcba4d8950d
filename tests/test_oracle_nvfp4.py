"""Pins for the oracle's NVFP4 encoder (Section 2.3 block quantizer; Appendix C.1 value set).

Everything here checks the oracle against something other than itself: the value set the paper
prints, brute-force nearest-value search, closed-form counts, an independent library's casts
(ml_dtypes) and invariants of the format.
"""
import math

import ml_dtypes
import numpy as np
import pytest

from oracle import nvfp4, philox

F32 = np.float32


def _golden(name):
    """Values the paper prints (tests/golden/nvfp4_format.txt, each line with its citation)."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "nvfp4_format.txt")
    for line in open(path):
        if line.startswith(name + ":"):
            return [float(t) for t in line.split(":", 1)[1].split()]
    raise KeyError(name)


PAPER_SET = _golden("e2m1_magnitudes")             # Appendix C.1: +-{0,0.5,1,1.5,2,3,4,6}


def test_value_set_and_block_size_are_the_papers():
    assert nvfp4.E2M1_GRID.tolist() == PAPER_SET
    assert nvfp4.BLOCK == int(_golden("block_size")[0])


def test_all_16_codes_roundtrip():
    for code in range(16):
        v = (-1.0 if code & 8 else 1.0) * PAPER_SET[code & 7]
        y = np.array([v], dtype=F32)
        assert nvfp4.e2m1_encode_rne(y)[0] == code
        for u in (0, 1, 65535):
            assert nvfp4.e2m1_encode_sr(y, np.array([u]))[0] == code


def test_ties_go_to_even_code_and_neighbours_of_ties():
    mids = [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]
    expect = [0.0, 1.0, 1.0, 2.0, 2.0, 4.0, 4.0]   # value of the even-coded neighbour
    for j, (m, e) in enumerate(zip(mids, expect)):
        for sgn in (1.0, -1.0):
            c = nvfp4.e2m1_encode_rne(np.array([sgn * m], dtype=F32))[0]
            assert PAPER_SET[c & 7] == e and bool(c & 8) == (sgn < 0)
            below = np.nextafter(F32(m), F32(0))
            above = np.nextafter(F32(m), F32(10))
            assert nvfp4.e2m1_encode_rne(np.array([sgn * below], dtype=F32))[0] & 7 == j
            assert nvfp4.e2m1_encode_rne(np.array([sgn * above], dtype=F32))[0] & 7 == j + 1


def test_saturation_and_signed_zero():
    y = np.array([6.0, 6.5, 1e30, np.inf, -7.0, -0.0, 0.0, -0.1, 0.1], dtype=F32)
    c = nvfp4.e2m1_encode_rne(y)
    assert c.tolist() == [7, 7, 7, 7, 15, 8, 0, 8, 0]


def test_rne_is_nearest_value_brute_force():
    rng = np.random.default_rng(0)
    y = np.concatenate([rng.uniform(-7, 7, 200000), rng.standard_normal(100000) * 0.3]).astype(F32)
    c = nvfp4.e2m1_encode_rne(y)
    grid = np.array(PAPER_SET, dtype=np.float64)
    d = np.abs(np.abs(y.astype(np.float64))[:, None] - grid[None, :])
    best = d.min(axis=1)
    got = d[np.arange(len(y)), c & 7]
    assert np.all(got == best)                      # never farther than the nearest value
    assert np.all((c >> 3).astype(bool) == np.signbit(y))


def test_rne_matches_ml_dtypes_float4():
    rng = np.random.default_rng(1)
    y = np.concatenate([rng.uniform(-6.5, 6.5, 300000), [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0],
                        [-0.25, -0.75, -1.25, -1.75, -2.5, -3.5, -5.0]]).astype(F32)
    ref = np.clip(y, -6, 6).astype(ml_dtypes.float4_e2m1fn).astype(np.float32)
    c = nvfp4.e2m1_encode_rne(y)
    mine = np.where(c & 8, -1.0, 1.0) * np.array(PAPER_SET)[c & 7]
    assert np.array_equal(mine, ref)
    assert np.array_equal(np.signbit(mine), np.signbit(ref))


def test_e4m3_table_matches_ml_dtypes_and_layout():
    bytes_ = np.arange(127, dtype=np.uint8)
    ref = bytes_.view(ml_dtypes.float8_e4m3fn).astype(np.float32)
    assert np.array_equal(nvfp4.E4M3_POS, ref)
    assert nvfp4.E4M3_POS[0x7E] == 448 and nvfp4.E4M3_POS[1] == 2.0 ** -9 and nvfp4.E4M3_POS[0x38] == 1.0
    assert np.all(np.diff(nvfp4.E4M3_POS) > 0)
    assert math.isnan(float(np.array([0x7F], dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float32)[0]))


def test_e4m3_scale_rounds_up():
    tab = nvfp4.E4M3_POS
    assert np.array_equal(nvfp4.e4m3_ceil_code(tab), np.arange(127))          # representable: unchanged
    for c in range(126):
        a, b = tab[c], tab[c + 1]
        probes = np.array([np.nextafter(a, F32(1e9)), (a.astype(np.float64) + b) / 2, np.nextafter(b, F32(0)), b], dtype=F32)
        assert np.all(nvfp4.e4m3_ceil_code(probes) == c + 1), c
    # independent route: library round-to-nearest cast, bumped by one code when it landed below
    rng = np.random.default_rng(2)
    t = np.minimum(np.exp(rng.uniform(np.log(1e-4), np.log(448), 100000)), 448).astype(F32)
    near = t.astype(ml_dtypes.float8_e4m3fn)
    code = near.view(np.uint8).astype(np.int64)
    code = code + (near.astype(np.float32) < t)
    assert np.array_equal(nvfp4.e4m3_ceil_code(t), code)


def _random_tensor(rng, rows=48, cols=128):
    x = rng.standard_normal((rows, cols)) * np.exp(rng.uniform(-3, 3, (rows, 1)))
    x[3, 16:32] = 0.0                                 # an all-zero block
    x[5, :] *= 1e-3
    return x.astype(F32)


def test_block_quantizer_invariants():
    rng = np.random.default_rng(3)
    x = _random_tensor(rng)
    codes, sc, s_T = nvfp4.quantize(x)
    assert s_T == F32(np.max(np.abs(x)) / F32(2688.0))
    s_b = nvfp4.E4M3_POS[sc].astype(np.float64)
    deq = nvfp4.dequantize(codes, sc, s_T)
    xb = x.astype(np.float64)
    # the block scale covers the block: s_b * s_T * 6 >= amax_b (rounded *up*, Section 2.3), up to fp32 rounding of the ratio
    amax_b = np.abs(xb).reshape(48, 8, 16).max(axis=2)
    assert np.all(s_b * float(s_T) * 6 * (1 + 2 ** -22) >= amax_b)
    # and it is the smallest such E4M3 value: the next one down would not cover it
    prev = nvfp4.E4M3_POS[np.maximum(sc.astype(int) - 1, 0)].astype(np.float64)
    nz = sc > 0
    assert np.all((prev * float(s_T) * 6 * (1 - 2 ** -22))[nz] < amax_b[nz])
    # error bound: at most half the local grid step, in units of the block's scale
    y = np.abs(xb) / (np.repeat(s_b, 16, axis=1) * float(s_T) + 1e-300)
    grid = np.array(PAPER_SET)
    hi = np.searchsorted(grid, np.minimum(y, 6), side="left").clip(1, 7)
    step = grid[hi] - grid[hi - 1]
    err = np.abs(deq - xb) / (np.repeat(s_b, 16, axis=1) * float(s_T) + 1e-300)
    assert np.all(err[np.repeat(nz, 16, axis=1)] <= step[np.repeat(nz, 16, axis=1)] / 2 + 1e-6)
    # nothing saturates under the tensor's own amax scale, and a block maximum lands on 6 for normal scales
    assert np.all((codes & 7)[y > 6 + 1e-5] == 7) and np.all(y <= 6 * (1 + 2 ** -21))
    normal = sc >= 8
    top = (codes & 7).reshape(48, 8, 16).max(axis=2)
    assert np.all(top[normal] == 7)
    # zero block -> zero scale byte and zero magnitudes
    assert sc[3, 1] == 0 and np.all((codes[3, 16:32] & 7) == 0)


def test_quantizer_idempotent_on_its_own_output():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((32, 64)).astype(F32)
    c1, s1, t1 = nvfp4.quantize(x, tensor_scale=F32(2.0 ** -9))   # power of two: dequantized values exact in fp32
    d1 = nvfp4.dequantize(c1, s1, t1)
    assert np.array_equal(d1, d1.astype(F32).astype(np.float64))
    c2, s2, t2 = nvfp4.quantize(d1.astype(F32), tensor_scale=t1)
    assert np.array_equal(nvfp4.dequantize(c2, s2, t2), d1)


def test_given_tensor_scale_clamps_and_saturates():
    x = np.full((1, 16), 1.0, dtype=F32)
    x[0, 0] = 4000.0
    codes, sc, s_T = nvfp4.quantize(x, tensor_scale=F32(1.0))
    assert sc[0, 0] == 0x7E                           # t = 4000/6 > 448 -> clamped
    assert codes[0, 0] == 7                           # 4000/448 > 6 -> saturates
    assert nvfp4.dequantize(codes, sc, s_T)[0, 0] == 6 * 448


def test_axis_rows_is_axis_cols_of_the_transpose_and_pack_roundtrip():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((64, 48)).astype(F32)
    cr, sr, tr = nvfp4.quantize(x, axis=nvfp4.AXIS_ROWS)
    cc, sc, tc = nvfp4.quantize(np.ascontiguousarray(x.T), axis=nvfp4.AXIS_COLS)
    assert np.array_equal(cr, cc) and np.array_equal(sr, sc) and tr == tc
    assert cr.shape == (48, 64) and sr.shape == (48, 4)
    p = nvfp4.pack(cr)
    assert p.shape == (48, 32) and p[0, 0] == (cr[0, 0] | (cr[0, 1] << 4))
    assert np.array_equal(nvfp4.unpack(p), cr)


def test_sr_up_count_closed_form_and_unbiased():
    u = np.arange(65536)
    for y in (0.1, 0.37, 0.5 + 1 / 3, 1.9, 2.25, 3.999, 4.5, 5.999, -2.7):
        a = abs(F32(y))
        grid = np.array(PAPER_SET, dtype=np.float64)
        lo = grid[grid <= a].max()
        hi = grid[grid > a].min()
        f = (float(a) - lo) / (hi - lo)
        c = nvfp4.e2m1_encode_sr(np.full(65536, y, dtype=F32), u)
        ups = int(np.sum(grid[c & 7] == hi))
        assert ups == math.ceil(f * 65536) and ups + int(np.sum(grid[c & 7] == lo)) == 65536
        mean = np.mean(np.where(c & 8, -1.0, 1.0) * grid[c & 7])
        assert abs(mean - float(F32(y))) <= (hi - lo) * 2.0 ** -16 + 1e-12


def test_sr_keyed_by_logical_index_for_both_axes_and_unbiased_over_seeds():
    rng = np.random.default_rng(6)
    x = rng.standard_normal((32, 32)).astype(F32)
    c_c, s_c, t = nvfp4.quantize(x, nvfp4.AXIS_COLS, nvfp4.ROUND_SR, seed=11)
    again = nvfp4.quantize(x, nvfp4.AXIS_COLS, nvfp4.ROUND_SR, seed=11)[0]
    other = nvfp4.quantize(x, nvfp4.AXIS_COLS, nvfp4.ROUND_SR, seed=12)[0]
    assert np.array_equal(c_c, again) and not np.array_equal(c_c, other)
    # the draw used for element (i, j) is draw_u16(i*cols + j): recompute one element by hand
    i, j = 7, 21
    u = philox.draw_u16(np.array([i * 32 + j]), 11, philox.STREAM_RESIDUAL)
    s_b = nvfp4.E4M3_POS[s_c[i, j // 16]]
    y = F32(x[i, j] * (F32(1.0) / (s_b * t)))
    assert nvfp4.e2m1_encode_sr(np.array([y]), u)[0] == c_c[i, j]
    c_r = nvfp4.quantize(x, nvfp4.AXIS_ROWS, nvfp4.ROUND_SR, seed=11)[0]
    assert c_r.shape == (32, 32)
    acc = np.zeros_like(x, dtype=np.float64)
    n = 400
    for seed in range(n):
        acc += nvfp4.fake_quantize(x, nvfp4.AXIS_COLS, rounding=nvfp4.ROUND_SR, seed=seed)
    step = np.repeat(nvfp4.E4M3_POS[s_c].astype(np.float64), 16, axis=1) * float(t) * 2.0
    assert np.all(np.abs(acc / n - x) <= 4 * step / 2 / math.sqrt(n) + 1e-9)


def test_hand_worked_block():
    """One block worked by hand from the definition: amax 12 with tensor scale 1 -> t = 2 -> scale 2.0 (byte 0x40)."""
    x = np.array([[12, -6, 5, 4.9, 3.1, 1, 0.4, -0.6, 0, 2, 7, -12, 9, 10, 11, 0.5]], dtype=F32)
    codes, sc, s_T = nvfp4.quantize(x, tensor_scale=F32(1.0))
    assert sc[0, 0] == 0x40
    # x/2 = 6, -3, 2.5 (tie -> 2), 2.45 -> 2, 1.55 -> 1.5, 0.5, 0.2 -> 0, -0.3 -> -0.5, 0, 1, 3.5 (tie -> 4), -6,
    #       4.5 -> 4, 5 (tie -> 4), 5.5 -> 6, 0.25 (tie -> 0)
    want = [6, -3, 2, 2, 1.5, 0.5, 0, -0.5, 0, 1, 4, -6, 4, 4, 6, 0]
    got = nvfp4.dequantize(codes, sc, s_T)[0] / 2
    assert got.tolist() == want


def test_index_override_reproduces_slices_of_the_full_tensor():
    """Quantizing rows (or columns) of a tensor on their own, keyed by their indices in the full tensor and with the
    full tensor's scale, gives the same codes and scales as slicing the full result - for both roundings."""
    rng = np.random.default_rng(7)
    x = (rng.standard_normal((64, 96)) * 3).astype(np.float32)
    rows, cols = np.array([3, 17, 40, 63]), np.array([0, 5, 95])
    s_T = nvfp4.tensor_scale_from_amax(np.max(np.abs(x)))
    for rounding in (nvfp4.ROUND_RNE, nvfp4.ROUND_SR):
        fc = nvfp4.quantize(x, nvfp4.AXIS_COLS, rounding, seed=9, tensor_scale=s_T)
        idx = rows[:, None].astype(np.uint64) * np.uint64(96) + np.arange(96, dtype=np.uint64)[None, :]
        pc = nvfp4.quantize(x[rows], nvfp4.AXIS_COLS, rounding, seed=9, tensor_scale=s_T, index=idx)
        assert np.array_equal(pc[0], fc[0][rows]) and np.array_equal(pc[1], fc[1][rows])
        fr = nvfp4.quantize(x, nvfp4.AXIS_ROWS, rounding, seed=9, tensor_scale=s_T)
        idx = np.arange(64, dtype=np.uint64)[:, None] * np.uint64(96) + cols[None, :].astype(np.uint64)
        pr = nvfp4.quantize(x[:, cols], nvfp4.AXIS_ROWS, rounding, seed=9, tensor_scale=s_T, index=idx)
        assert np.array_equal(pr[0], fr[0][cols]) and np.array_equal(pr[1], fr[1][cols])
    # and the draws do depend on the keys
    a = nvfp4.quantize(x[rows], nvfp4.AXIS_COLS, nvfp4.ROUND_SR, seed=9, tensor_scale=s_T)
    assert not np.array_equal(a[0], fc[0][rows])
