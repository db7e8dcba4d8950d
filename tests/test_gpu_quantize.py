"""GPU parity: NVFP4 quantizer (metis_quantize_nvfp4) against the oracle, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import gauss, nvfp4 as onv
from paper_2509_00404_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2509_00404_b200 import binding as B
    h = B.Handle(0)
    yield B, h
    h.close()


def _adversarial(rng, rows, cols):
    """Heavy-tailed rows, exact ties, zero blocks, signed zeros, block maxima on E4M3 boundaries."""
    x = rng.standard_normal((rows, cols)) * np.exp(rng.uniform(-4, 4, (rows, 1)))
    x[1, :16] = 0.0
    x[2, 16:32] = -0.0
    x[3, :16] = np.array([6, 5, 3.5, 2.5, 1.75, 1.25, 0.75, 0.25, -6, -5, -3.5, -2.5, -1.75, -1.25, -0.75, -0.25])
    x[4, :16] = 448.0 * 6 / 7
    x[5, 32:48] = 1e-30
    x = synth.to_bf16_values(x.astype(np.float32))
    return x


def _compare(B, h, x, xd, axes, rounding, layout, seed=1234, tensor_scale=None):
    from gpu_util import nv_to_numpy
    bc, br = h.quantize_nvfp4(xd, axes, rounding, seed=seed, layout=layout, tensor_scale=tensor_scale)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    for t, axis in ((bc, onv.AXIS_COLS), (br, onv.AXIS_ROWS)):
        if t is None:
            continue
        c, s, ts = nv_to_numpy(t)
        oc, os_, ots = onv.quantize(x, axis, rounding, seed=seed, tensor_scale=tensor_scale)
        assert ts == ots
        assert np.array_equal(s, os_)
        assert np.array_equal(c, oc)


@pytest.mark.parametrize("rounding", [0, 1])
@pytest.mark.parametrize("layout", [0, 1])
def test_quantizer_bit_exact_both_axes(ctx, rounding, layout):
    from gpu_util import to_dev_bf16
    B, h = ctx
    rng = np.random.default_rng(10 + rounding)
    x = _adversarial(rng, 320, 448)                  # spans several 128-tiles with a ragged tail in both directions
    _compare(B, h, x, to_dev_bf16(x), B.BLOCKS_BOTH, rounding, layout)


@pytest.mark.parametrize("rounding", [0, 1])
def test_quantizer_strided_views_and_unaligned_scale_rows(ctx, rounding):
    """The paths beside the fast one: a BF16 operand that is a column slice of a wider tensor (leading dimension larger
    than the width, rows starting 16 bytes off a 32-byte boundary: no 32-byte loads), and a linear scale layout whose
    rows are not a multiple of four blocks (scale bytes written one by one)."""
    from gpu_util import to_dev_bf16
    B, h = ctx
    rng = np.random.default_rng(40 + rounding)
    x = _adversarial(rng, 336, 400)                              # 25 and 21 blocks per stored row
    wide = torch.zeros((336, 400 + 24), dtype=torch.bfloat16, device="cuda")
    wide[:, 8:408] = to_dev_bf16(x)
    view = wide[:, 8:408]
    assert view.data_ptr() % 32 == 16 and view.stride(0) == 424
    _compare(B, h, x, view, B.BLOCKS_BOTH, rounding, B.SF_LINEAR)
    _compare(B, h, np.ascontiguousarray(x[:320, :384]), wide[:320, 8:392], B.BLOCKS_BOTH, rounding, B.SF_TILED)   # tiled scales want multiples of 64
    _compare(B, h, x, to_dev_bf16(x), B.BLOCKS_BOTH, rounding, B.SF_LINEAR)


def test_quantizer_fp32_input_given_scale_and_single_axis(ctx):
    B, h = ctx
    rng = np.random.default_rng(3)
    x = (rng.standard_normal((64, 128)) * 3).astype(np.float32)
    xd = torch.from_numpy(x).cuda()
    _compare(B, h, x, xd, B.BLOCKS_ALONG_COLS, B.ROUND_RNE, B.SF_LINEAR, tensor_scale=np.float32(0.01))
    _compare(B, h, x, xd, B.BLOCKS_ALONG_ROWS, B.ROUND_SR, B.SF_TILED, tensor_scale=np.float32(0.004))  # saturates some blocks
    _compare(B, h, x, xd, B.BLOCKS_ALONG_COLS, B.ROUND_SR, B.SF_LINEAR)


def test_quantizer_all_zero_and_tiny_shapes(ctx):
    B, h = ctx
    x = np.zeros((16, 64), dtype=np.float32)
    _compare(B, h, x, torch.from_numpy(x).cuda(), B.BLOCKS_BOTH, B.ROUND_RNE, B.SF_LINEAR)
    x = np.full((16, 16), -2.5, dtype=np.float32)
    _compare(B, h, x, torch.from_numpy(x).cuda(), B.BLOCKS_BOTH, B.ROUND_SR, B.SF_LINEAR)


def test_every_fp32_tie_and_neighbour_rounds_like_the_oracle(ctx):
    """All seven E2M1 midpoints, +-1 ulp, both signs, placed in blocks whose scale is exactly 1."""
    B, h = ctx
    mids = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], dtype=np.float32)
    vals = np.concatenate([mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(9))])
    vals = np.concatenate([vals, -vals]).astype(np.float32)           # 42 values
    x = np.zeros((16, 64), dtype=np.float32)
    x[:, 0] = 6.0
    x[:, 16] = 6.0
    x[:, 32] = 6.0
    x[:, 48] = 6.0
    flat = x.reshape(-1)
    slots = [i for i in range(flat.size) if i % 16 != 0][: vals.size]
    flat[slots] = vals
    _compare(B, h, x, torch.from_numpy(x).cuda(), B.BLOCKS_ALONG_COLS, B.ROUND_RNE, B.SF_LINEAR, tensor_scale=np.float32(1.0))


def test_rejects_bad_arguments(ctx):
    B, h = ctx
    x = torch.zeros((16, 24), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.MetisError):
        h.quantize_nvfp4(x, B.BLOCKS_ALONG_COLS, layout=B.SF_LINEAR)            # cols not a multiple of 16
    x = torch.zeros((16, 48), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.MetisError):
        h.quantize_nvfp4(x, B.BLOCKS_ALONG_COLS, layout=B.SF_TILED)             # tiled scales need a multiple of 64


def test_quantile_table_matches_oracle(ctx):
    B, h = ctx
    ref = gauss.quantile_level(np.arange(65536))
    assert np.array_equal(h.quantile_table(), (ref.view(np.uint32) >> 16).astype(np.uint16))


@pytest.mark.parametrize("case", [(128, 256, 1, "bf16"), (200, 192, 0, "fp32"), (1024, 4096, 1, "bf16")], ids=lambda c: "%dx%d_%s_%s" % (c[0], c[1], "sr" if c[2] else "rne", c[3]))
def test_random_hadamard_recipe_matches_the_oracle_byte_for_byte(case):
    """The comparison recipe of Section 4 (random Hadamard transform of every 16-block, then NVFP4 with stochastic
    rounding): codes, scale bytes and tensor scale against the oracle, and the product-preserving property on the
    GPU's own bytes."""
    from oracle import hadamard as ohad
    from gpu_util import nv_to_numpy
    from paper_2509_00404_b200 import binding as B, synth
    rows, cols, rounding, dt = case
    x, _ = synth.llama_like(rows, cols, 1.0, 900 + rows, rank=8)
    if dt == "fp32":
        x = (x * np.float32(1.2345)).astype(np.float32)
    xd = torch.from_numpy(x).cuda() if dt == "fp32" else torch.from_numpy(x).to(torch.bfloat16).cuda()
    h = B.Handle(0)
    try:
        layout = B.SF_TILED if cols % 64 == 0 else B.SF_LINEAR
        t = h.quantize_rht_nvfp4(xd, rounding=rounding, seed=17, layout=layout)
        torch.cuda.synchronize()
        assert h.device_status() == 0
        c, s, ts = nv_to_numpy(t)
        oc, os_, ots = ohad.quantize_rht(x, rounding, seed=17)
        assert ts == ots and np.array_equal(s, os_) and np.array_equal(c, oc)
        back = ohad.rht_inverse(onv.dequantize(c, s, ts), 17)
        assert np.linalg.norm(back - x) / np.linalg.norm(x) < 0.2
    finally:
        h.close()
