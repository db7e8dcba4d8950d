"""Pins for the oracle's random sources: Philox4x32-10 and the quantile-table Gaussian test matrix."""
import os
import shutil
import statistics
import subprocess

import ml_dtypes
import numpy as np
import pytest

from oracle import gauss, philox

HERE = os.path.dirname(os.path.abspath(__file__))


def test_philox_matches_curand_header_on_host(tmp_path):
    """The vendor's header implements the same published generator; run its block function on the host."""
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        pytest.skip("nvcc not available")
    exe = str(tmp_path / "philox_curand_host")
    subprocess.run([nvcc, "-O1", "-o", exe, os.path.join(HERE, "philox_curand_host.cu")], check=True)
    rng = np.random.default_rng(0)
    cases = rng.integers(0, 2 ** 32, size=(64, 6), dtype=np.uint64)
    cases[0] = 0
    cases[1] = 0xFFFFFFFF
    cases[2] = [1, 0, 0, 0, 0, 0]
    cases[3] = [0, 0, 0, 0, 1, 0]
    text = "\n".join(" ".join("%x" % v for v in row) for row in cases) + "\n"
    out = subprocess.run([exe], input=text, capture_output=True, text=True, check=True).stdout.split()
    ref = np.array([int(t, 16) for t in out], dtype=np.uint64).reshape(64, 4)
    mine = np.stack(philox.philox4x32_10(cases[:, 0], cases[:, 1], cases[:, 2], cases[:, 3], 0, 0), axis=1)
    for i, row in enumerate(cases):          # keys are scalars in the oracle: one call per case
        o = philox.philox4x32_10(row[0], row[1], row[2], row[3], int(row[4]), int(row[5]))
        assert [int(v) for v in o] == [int(v) for v in ref[i]], i
    assert mine.shape == (64, 4)


def test_draw_rule_eight_elements_share_one_counter():
    seed = 0x123456789ABCDEF
    e = np.arange(80, 96, dtype=np.uint64)
    u = philox.draw_u16(e, seed, 0x10)
    for blk in (10, 11):
        w = philox.philox4x32_10(blk, 0, 0x10, 0, seed & 0xFFFFFFFF, seed >> 32)
        halves = []
        for word in w:
            halves += [int(word) & 0xFFFF, int(word) >> 16]
        assert u[(blk - 10) * 8:(blk - 10) * 8 + 8].tolist() == halves
    big = np.array([(1 << 35) + 5], dtype=np.uint64)     # index above 2**32 * 8 reaches the second counter word
    w = philox.philox4x32_10(0, 1, 0x10, 0, seed & 0xFFFFFFFF, seed >> 32)
    assert int(philox.draw_u16(big, seed, 0x10)[0]) == (int(w[2]) >> 16)


def test_draws_are_uniform_and_stream_separated():
    u = philox.draw_u16(np.arange(1 << 18), 42, 0x10).astype(np.float64)
    assert abs(u.mean() - 32767.5) < 4 * 65536 / np.sqrt(12 * len(u))
    counts = np.bincount((u // 4096).astype(int), minlength=16)
    chi2 = np.sum((counts - len(u) / 16) ** 2 / (len(u) / 16))
    assert chi2 < 50
    v = philox.draw_u16(np.arange(1 << 18), 42, 0x11)
    assert np.mean(u == v) < 1e-3
    assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 0.01


def test_quantile_table_against_stdlib_inverse_cdf_and_symmetry():
    levels = gauss.quantile_level(np.arange(65536))
    nd = statistics.NormalDist()
    ref = np.array([nd.inv_cdf((u + 0.5) / 65536.0) for u in range(65536)])
    ref_bf16 = ref.astype(np.float32).astype(ml_dtypes.bfloat16).astype(np.float32)
    assert np.array_equal(levels, ref_bf16)
    assert np.array_equal(levels, -levels[::-1])
    assert np.all(np.diff(levels) >= 0)
    assert abs(levels[0] + 4.3125) < 0.02 and levels[32768] > 0 and levels[32767] < 0
    # no exact quantile sits close enough to a bfloat16 rounding boundary for a 1e-9 error to flip it
    b = ref.astype(np.float32).view(np.uint32)
    lo = (b & np.uint32(0xFFFF0000)).view(np.float32).astype(np.float64)
    hi = ((b & np.uint32(0xFFFF0000)) + np.uint32(0x10000)).view(np.float32).astype(np.float64)
    mid = (lo + hi) / 2
    assert np.min(np.abs(ref - mid) / np.abs(ref)) > 1e-9


def test_omega_moments_and_indexing():
    om = gauss.omega(4096, 40, seed=5)
    assert om.shape == (4096, 40) and om.dtype == np.float32
    assert abs(om.mean()) < 4 / np.sqrt(om.size) and abs(om.var() - 1) < 0.02
    assert abs(np.mean(om ** 4) - 3) < 0.15
    u = philox.draw_u16(np.array([17 * 40 + 3]), 5, philox.STREAM_OMEGA)
    assert om[17, 3] == gauss.quantile_level(u)[0]
    assert not np.array_equal(om, gauss.omega(4096, 40, seed=6))
    assert np.array_equal(gauss.round_to_bf16(om), om)


def test_round_to_bf16_matches_ml_dtypes():
    rng = np.random.default_rng(7)
    x = np.concatenate([rng.standard_normal(100000) * 10, [1.00390625, 1.01171875, -1.00390625]]).astype(np.float32)
    assert np.array_equal(gauss.round_to_bf16(x), x.astype(ml_dtypes.bfloat16).astype(np.float32))
