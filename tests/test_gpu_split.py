"""GPU parity: metis_split (sketch, orthonormalisation, top-k projection, residual, quantization)."""
import numpy as np
import pytest
import torch

from oracle import nvfp4 as onv, split as osp, metrics
from paper_2509_00404_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2509_00404_b200 import binding as B
    h = B.Handle(0)
    yield B, h
    h.close()


def _run(B, h, x, k, p, mode, seed, rounding=0):
    from gpu_util import to_dev_bf16
    op, dense = h.split(to_dev_bf16(x), k, p, sketch=mode, seed=seed, rounding=rounding, want_residual=True)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    return op, dense.cpu().numpy()


def _check_against_oracle(B, h, x, k, p, mode, seed, rounding=0):
    from gpu_util import nv_to_numpy, rel_fro
    op, dense = _run(B, h, x, k, p, mode, seed, rounding)
    sp = osp.split(x.astype(np.float64), k, p, mode, seed=seed)
    sig = op.sigma.cpu().numpy()
    assert np.max(np.abs(sig - sp.sigma) / sp.sigma) < 1e-3                 # top-k singular values
    # residual before quantization: the factors are FP32 and the low-rank part is an FP32 sum of k terms, so it
    # carries ~sqrt(k) 2^-24 relative noise, which shows up in the residual magnified by ||X|| / ||R||
    # (4 sqrt(k) = 32 at k = 64, and that figure is kept for every smaller rank)
    growth = 4.0 * np.sqrt(max(k, 64))
    tol_r = max(1e-6, growth * 2.0 ** -24 * np.linalg.norm(x) / np.linalg.norm(sp.residual))
    err_r = rel_fro(dense, sp.residual)
    print("split %dx%d k=%d p=%d mode=%d: sigma %.2e residual %.2e (tolerance %.2e)" % (x.shape[0], x.shape[1], k, p, mode,
          np.max(np.abs(sig - sp.sigma) / sp.sigma), err_r, tol_r))
    assert tol_r < 1e-4 * growth / 32 and err_r < tol_r
    left, right = op.left.cpu().numpy().T.astype(np.float64), op.right.cpu().numpy().T.astype(np.float64)
    assert rel_fro(left, sp.left) < 1e-3 and rel_fro(right, sp.right) < 1e-3
    # invariants that hold whatever the oracle says
    assert np.allclose(left.T @ left, np.eye(k), atol=1e-4) and np.allclose(right.T @ right, np.eye(k), atol=1e-4)
    assert rel_fro((left * sig) @ right.T + dense, x) < 1e-5 * max(1.0, 0.1 * np.linalg.norm(x) / np.linalg.norm(sp.residual))
    # the fused quantizer saw `dense`: the oracle's encoder on the same values must give the same bytes
    s_src = onv.tensor_scale_from_amax(np.max(np.abs(x)))
    for t, axis in ((op.res_by_cols, onv.AXIS_COLS), (op.res_by_rows, onv.AXIS_ROWS)):
        c, s, ts = nv_to_numpy(t)
        oc, os_, _ = onv.quantize(dense, axis, rounding, seed=seed, tensor_scale=s_src)
        assert ts == s_src and np.array_equal(s, os_) and np.array_equal(c, oc)
    # factors: quantized from the FP32 factors the library kept
    for t, f, stream in ((op.left_q, op.left, 0x11), (op.right_q, op.right, 0x12)):
        c, s, ts = nv_to_numpy(t)
        oc, os_, ots = onv.quantize(f.cpu().numpy()[:k], onv.AXIS_COLS, rounding, seed=seed, stream=stream)
        assert ts == ots and np.array_equal(s[:k], os_) and np.array_equal(c[:k], oc)
    return op, sp


def test_full_mode_small_config(ctx):
    B, h = ctx
    c = synth.config_small()
    _check_against_oracle(B, h, c["x"], 4, 4, B.SKETCH_FULL, seed=11)
    _check_against_oracle(B, h, c["w"], 4, 4, B.SKETCH_FULL, seed=12)


def test_sampled_mode_and_stochastic_rounding(ctx):
    B, h = ctx
    x, _ = synth.llama_like(2048, 512, 1.0, 41, rank=16)
    _check_against_oracle(B, h, x, 16, 8, B.SKETCH_SAMPLED, seed=21)
    d, _ = synth.llama_like(1024, 384, 1e-4, 42, rank=8)
    _check_against_oracle(B, h, d, 8, 8, B.SKETCH_SAMPLED, seed=22, rounding=1)


def test_full_mode_tall_operand_uses_the_row_split_tensor_core_path(ctx):
    """More than 1024 rows: the sketch spans several row tiles and the projection runs on its tensor-core kernel."""
    B, h = ctx
    x, _ = synth.llama_like(1536, 320, 0.02, 43, rank=8)
    _check_against_oracle(B, h, x, 8, 8, B.SKETCH_FULL, seed=31)


@pytest.mark.parametrize("shape_kp", [((1088, 448), 8, 8), ((2112, 192), 24, 8), ((1024, 1088), 40, 8)])
def test_full_mode_ragged_shapes_on_the_tensor_core_sketch_and_projection(ctx, shape_kp):
    """Full sketches of operands whose rows are not a multiple of 128 and whose columns are not a multiple of 128:
    clipped TMA boxes in both roles of x (K-major for the sketch, MN-major for the projection), every width of the
    projection's accumulator (k + p = 16, 32, 48), rows split over several slices."""
    B, h = ctx
    (rows, cols), k, p = shape_kp
    x, _ = synth.llama_like(rows, cols, 0.5, 47, rank=max(k, 8))
    _check_against_oracle(B, h, x, k, p, B.SKETCH_FULL, seed=33)


@pytest.mark.parametrize("case", [(1024, 512, 80, 8, 80), (2048, 1024, 128, 8, 128), (2048, 1024, 128, 8, 64), (1024, 1024, 100, 4, 100),
                                  (2048, 2048, 256, 8, 256), (2048, 2048, 256, 8, 64), (2304, 1088, 136, 0, 136)],
                         ids=lambda c: "%dx%d_k%d_p%d_rank%d" % c)
@pytest.mark.parametrize("mode_name", ["full", "sampled"])
def test_wide_ranks_on_the_cluster_solver(ctx, case, mode_name):
    """Ranks above 64 (k + p up to 264): the sketch no longer fits one CTA, so the orthonormalisation and both
    eigen-decompositions run on the tiled FP64 kernels and the eight-CTA cluster Jacobi solver, and the tensor-core
    passes run in groups of sketch columns.  Same checks as every other rank; planted rank equal to k and planted
    rank 64 (the cut then falls inside the bulk, as at the rank-256 point of the 70B-shaped sweep)."""
    B, h = ctx
    rows, cols, k, p, rank = case
    x, _ = synth.llama_like(rows, cols, 1.0, 40 + k, rank=rank)
    mode = B.SKETCH_FULL if mode_name == "full" else B.SKETCH_SAMPLED
    _check_against_oracle(B, h, x, k, p, mode, seed=5, rounding=1 if rank == 64 else 0)


def test_planted_noise_free_spectrum_is_recovered(ctx):
    """Closed form: with no bulk and rank <= k+p the sketch captures the whole matrix and Lambda is the planted
    spectrum.  The library only takes bfloat16 input, whose rounding adds a full-rank perturbation of relative size
    2^-9 per element, so the planted values are met to 1e-3 and the oracle on the same bf16 input to 1e-5."""
    B, h = ctx
    x, s = synth.planted(128, 256, 8, 200.0, 20.0, 0.0, 1001)
    op, dense = _run(B, h, x, 4, 4, B.SKETCH_FULL, seed=3)
    sig = op.sigma.cpu().numpy()
    assert np.max(np.abs(sig - s[:4]) / s[:4]) < 1e-3
    sp = osp.split(x.astype(np.float64), 4, 4, osp.MODE_FULL, seed=3)
    assert np.max(np.abs(sig - sp.sigma) / sp.sigma) < 1e-5
    x2, s2 = synth.planted(2048, 256, 8, 50.0, 5.0, 0.0, 77)
    op2, dense2 = _run(B, h, x2, 8, 4, B.SKETCH_SAMPLED, seed=9)           # k = planted rank, k + p > rank
    sig2 = op2.sigma.cpu().numpy()
    assert np.max(np.abs(sig2 - s2) / s2) < 1e-3
    sp2 = osp.split(x2.astype(np.float64), 8, 4, osp.MODE_SAMPLED, seed=9)
    assert np.max(np.abs(sig2 - sp2.sigma) / sp2.sigma) < 1e-5
    assert np.linalg.norm(dense2) < 2e-2 * np.linalg.norm(x2)               # only bf16 rounding noise is left


@pytest.mark.parametrize("shape", [(320, 448), (192, 320), (448, 192)])
def test_ragged_tiles_sampled_and_full(ctx, shape):
    """Rows and columns that are multiples of 64 (the tiled scale layout) but not of the 128-wide tiles: partial TMA boxes, partial
    accumulator tiles, half-valid 32-row slabs and 32-column steps in the fused residual quantizer."""
    B, h = ctx
    rows, cols = shape
    x, _ = synth.llama_like(rows, cols, 1.0, 500 + rows, rank=8)
    _check_against_oracle(B, h, x, 8, 4, B.SKETCH_SAMPLED, seed=31)
    _check_against_oracle(B, h, x, 8, 4, B.SKETCH_SAMPLED, seed=32, rounding=1)
    _check_against_oracle(B, h, x, 8, 4, B.SKETCH_FULL, seed=33)


def test_all_zero_operand_is_degenerate_but_clean(ctx):
    """x = 0: every pivot of the orthonormalisation is dependent, every eigenvalue zero.  The library must return
    zero factors, a zero residual (signs kept, scale bytes 0) and status OK - no NaN anywhere."""
    from gpu_util import nv_to_numpy
    B, h = ctx
    x = torch.zeros((256, 320), dtype=torch.bfloat16, device="cuda")
    for mode in (B.SKETCH_SAMPLED, B.SKETCH_FULL):
        op, dense = h.split(x, 8, 4, sketch=mode, seed=5, want_residual=True)
        torch.cuda.synchronize()
        assert h.device_status() == 0
        assert torch.count_nonzero(dense) == 0
        for t in (op.left, op.right, op.sigma):
            assert torch.isfinite(t).all() and torch.count_nonzero(t[:8]) == 0
        for t in (op.res_by_cols, op.res_by_rows, op.left_q, op.right_q):
            c, s, ts = nv_to_numpy(t)
            assert np.count_nonzero(c & 7) == 0 and np.count_nonzero(s) == 0 and np.isfinite(ts)


@pytest.mark.parametrize("mode_name", ["sampled", "full"])
def test_rank_deficient_operand(ctx, mode_name):
    """An operand of exact rank 3 (small integers: no BF16 rounding) split with k = 8: the sketch has dependent columns
    and five of the eight singular values are zero.  What is unique must match - the three non-zero singular values
    (against a library SVD and the oracle), the projector onto their right singular vectors, a residual that is
    zero - and the rest must be clean: finite everywhere, zero factors for the zero values, status OK."""
    from gpu_util import to_dev_bf16
    B, h = ctx
    mode = B.SKETCH_SAMPLED if mode_name == "sampled" else B.SKETCH_FULL
    rng = np.random.default_rng(77)
    rows, cols, r, k, p = 640, 384, 3, 8, 4
    u = rng.integers(-2, 3, size=(rows, r)).astype(np.float64)
    v = rng.integers(-2, 3, size=(cols, r)).astype(np.float64)
    x = u @ v.T                                                   # integers of magnitude <= 12: exact in BF16
    op, dense = h.split(to_dev_bf16(x), k, p, sketch=mode, seed=9, want_residual=True)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    sig = op.sigma.cpu().numpy().astype(np.float64)
    left, right = op.left.cpu().numpy().astype(np.float64), op.right.cpu().numpy().astype(np.float64)
    dense = dense.cpu().numpy().astype(np.float64)
    assert np.isfinite(sig).all() and np.isfinite(left).all() and np.isfinite(right).all() and np.isfinite(dense).all()
    s_true = np.linalg.svd(x, compute_uv=False)[:r]
    assert np.max(np.abs(sig[:r] - s_true) / s_true) < 1e-4
    sp = osp.split(x, k, p, osp.MODE_SAMPLED if mode_name == "sampled" else osp.MODE_FULL, seed=9)
    assert np.max(np.abs(sp.sigma[:r] - s_true) / s_true) < 1e-8
    assert np.max(np.abs(sig[r:k])) < 1e-3 * s_true[0]
    # projector onto the top right singular vectors (unique although the vectors of equal values are not)
    vt = np.linalg.svd(x, full_matrices=False)[2][:r]
    pr = right[:r].T @ right[:r]
    assert np.linalg.norm(pr - vt.T @ vt) < 1e-4
    # everything is in the low-rank part: reconstruction from the first three factors, residual at rounding level
    recon = (left[:r].T * sig[:r]) @ right[:r]
    assert np.linalg.norm(recon - x) < 1e-5 * np.linalg.norm(x)
    assert np.linalg.norm(dense) < 1e-5 * np.linalg.norm(x)
    assert np.linalg.norm((left[:k].T * sig[:k]) @ right[:k] + dense - x) < 1e-5 * np.linalg.norm(x)


@pytest.mark.parametrize("mode_name", ["sampled", "full"])
def test_repeated_singular_values_inside_the_top_k(ctx, mode_name):
    """Four equal singular values, then distinct ones, over a Gaussian bulk, k = 8: the singular vectors of the equal
    values are any basis of their 4-dimensional space, so only that space is compared (projector), together with the
    singular values, the projector of the whole rank-8 part and the residual, which do not depend on the choice."""
    from gpu_util import rel_fro
    B, h = ctx
    mode, omode = (B.SKETCH_SAMPLED, osp.MODE_SAMPLED) if mode_name == "sampled" else (B.SKETCH_FULL, osp.MODE_FULL)
    rng = np.random.default_rng(31)
    rows, cols, k, p = 1024, 512, 8, 8
    u, _ = np.linalg.qr(rng.standard_normal((rows, k)))
    v, _ = np.linalg.qr(rng.standard_normal((cols, k)))
    sv = np.array([400.0, 400.0, 400.0, 400.0, 300.0, 250.0, 200.0, 150.0])
    x = synth.to_bf16_values((u * sv) @ v.T + 0.05 * rng.standard_normal((rows, cols))).astype(np.float64)
    op, dense = _run(B, h, x, k, p, mode, seed=4)
    sp = osp.split(x, k, p, omode, seed=4)
    sig = op.sigma.cpu().numpy().astype(np.float64)
    assert np.max(np.abs(sig - sp.sigma) / sp.sigma) < 1e-3
    right = op.right.cpu().numpy().astype(np.float64)[:k].T
    left = op.left.cpu().numpy().astype(np.float64)[:k].T
    for cols_ in (slice(0, 4), slice(0, k)):
        assert np.linalg.norm(right[:, cols_] @ right[:, cols_].T - sp.right[:, cols_] @ sp.right[:, cols_].T) < 2e-3
        assert np.linalg.norm(left[:, cols_] @ left[:, cols_].T - sp.left[:, cols_] @ sp.left[:, cols_].T) < 2e-3
    assert np.allclose(right.T @ right, np.eye(k), atol=1e-4) and np.allclose(left.T @ left, np.eye(k), atol=1e-4)
    tol_r = max(1e-6, 32 * 2.0 ** -24 * np.linalg.norm(x) / np.linalg.norm(sp.residual))
    assert rel_fro(dense, sp.residual) < tol_r
    assert rel_fro((left * sig) @ right.T + dense, x) < 1e-5


@pytest.mark.parametrize("mode_name", ["sampled", "full"])
def test_ill_conditioned_sketch_needs_the_second_orthonormalisation_pass(ctx, mode_name):
    """Block-diagonal operand of exact small-integer entries: a rank-4 block with singular values near 500 and a
    full-rank block scaled by 2^-16 (singular values near 7e-4).  The sketch columns beyond the fourth differ from
    combinations of the first four only at the 1e-6 level, so the Gram matrix has pivots near 1e-10 of its largest
    (1.1e-10 ... 4.6e-10, computed from the oracle's sketch for this seed): neither dependent (below 1e-13) nor
    well-conditioned (above 1e-8), the case the second CholeskyQR pass exists for.  Checked against a
    library SVD and the oracle: top singular values, their right projector, orthonormal factors, exact split."""
    from gpu_util import to_dev_bf16
    B, h = ctx
    mode, omode = (B.SKETCH_SAMPLED, osp.MODE_SAMPLED) if mode_name == "sampled" else (B.SKETCH_FULL, osp.MODE_FULL)
    rng = np.random.default_rng(123)
    rows, cols, r, k, p = 640, 384, 4, 4, 4
    x = np.zeros((rows, cols))
    x[: rows // 2, : cols // 2] = rng.integers(-2, 3, size=(rows // 2, r)) @ rng.integers(-2, 3, size=(r, cols // 2))
    x[rows // 2 :, cols // 2 :] = rng.integers(-2, 3, size=(rows // 2, cols // 2)) * 2.0 ** -16
    assert np.array_equal(synth.to_bf16_values(x), x)
    op, dense = h.split(to_dev_bf16(x), k, p, sketch=mode, seed=6, want_residual=True)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    sig = op.sigma.cpu().numpy().astype(np.float64)[:k]
    left = op.left.cpu().numpy().astype(np.float64)[:k].T
    right = op.right.cpu().numpy().astype(np.float64)[:k].T
    dense = dense.cpu().numpy().astype(np.float64)
    uu, ss, vt = np.linalg.svd(x, full_matrices=False)
    assert ss[3] / ss[4] > 1e4
    assert np.max(np.abs(sig - ss[:k]) / ss[:k]) < 1e-5
    sp = osp.split(x, k, p, omode, seed=6)
    assert np.max(np.abs(sp.sigma - ss[:k]) / ss[:k]) < 1e-7
    # the orthonormal basis is stored in FP32: entries of the small block's rows, exactly zero in the true vectors,
    # come out at the 1e-5 level (FP32 rounding of columns that are 1e6 times smaller than the first ones)
    assert np.linalg.norm(right @ right.T - vt[:k].T @ vt[:k]) < 1e-3
    assert np.linalg.norm(left @ left.T - uu[:, :k] @ uu[:, :k].T) < 1e-3
    assert np.allclose(left.T @ left, np.eye(k), atol=1e-4) and np.allclose(right.T @ right, np.eye(k), atol=1e-4)
    assert np.linalg.norm((left * sig) @ right.T + dense - x) < 1e-6 * np.linalg.norm(x)
    # the residual is the small block (plus FP32 rounding of the large one)
    assert np.linalg.norm(dense - sp.residual) < 1e-6 * np.linalg.norm(x)


def test_rank_zero_is_plain_quantization(ctx):
    from gpu_util import to_dev_bf16, nv_to_numpy
    B, h = ctx
    c = synth.config_small()
    op = h.split(to_dev_bf16(c["x"]), 0, 0, seed=5)
    torch.cuda.synchronize()
    for t, axis in ((op.res_by_cols, onv.AXIS_COLS), (op.res_by_rows, onv.AXIS_ROWS)):
        cg, sg, ts = nv_to_numpy(t)
        oc, os_, ots = onv.quantize(c["x"], axis)
        assert ts == ots and np.array_equal(sg, os_) and np.array_equal(cg, oc)


@pytest.mark.parametrize("k", [0, 8])
def test_supplied_source_amax_gives_the_same_bytes(ctx, k):
    """metis_split with the producer's amax|x| handed in (no reduction pass of its own for k = 0) against the default."""
    from gpu_util import to_dev_bf16, nv_to_numpy
    B, h = ctx
    x, _ = synth.llama_like(384, 512, 1.0, 71, rank=8)
    xd = to_dev_bf16(x)
    a = h.split(xd, k, 8 if k else 0, seed=5)
    amax = xd.float().abs().max().reshape(1)
    b = h.split(xd, k, 8 if k else 0, seed=5, src_amax=amax)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    for name in ("res_by_cols", "res_by_rows"):
        ca, sa, ta = nv_to_numpy(getattr(a, name))
        cb, sb, tb = nv_to_numpy(getattr(b, name))
        assert ta == tb and np.array_equal(ca, cb) and np.array_equal(sa, sb)


def _same_operand(a, b):
    from gpu_util import nv_to_numpy
    for name in ("left_q", "right_q", "res_by_cols", "res_by_rows"):
        ca, sa, ta = nv_to_numpy(getattr(a, name))
        cb, sb, tb = nv_to_numpy(getattr(b, name))
        assert ta == tb and np.array_equal(ca, cb) and np.array_equal(sa, sb), name
    for name in ("left", "sigma", "right"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name


@pytest.mark.parametrize("k", [0, 8, 80])
def test_strided_and_fp32_operands_give_the_bytes_of_the_contiguous_bf16_operand(ctx, k):
    """metis_split takes a leading dimension and FP32 input: the operand is gathered / rounded to BF16 once and the
    decomposition is that of the contiguous BF16 tensor, byte for byte (k = 0 quantizes the FP32 values themselves)."""
    from gpu_util import to_dev_bf16, nv_to_numpy
    B, h = ctx
    rows, cols, p = 512, 768, (8 if k else 0)
    x, _ = synth.llama_like(rows, cols, 1.0, 73, rank=16)
    xd = to_dev_bf16(x)
    ref = h.split(xd, k, p, seed=5)
    wide = torch.zeros((rows, cols + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, 24:24 + cols] = xd
    view = wide[:, 24:24 + cols]
    assert view.stride(0) == cols + 64 and view.data_ptr() % 16 == 0
    _same_operand(ref, h.split(view, k, p, seed=5))
    _same_operand(ref, h.split(xd.float(), k, p, seed=5))                      # BF16 values held in FP32
    noisy = xd.float() * (1.0 + 1e-3 * torch.randn((rows, cols), device="cuda"))   # not representable in BF16
    got = h.split(noisy, k, p, seed=5)
    if k:
        _same_operand(h.split(noisy.bfloat16(), k, p, seed=5), got)
    else:
        qc, qr = h.quantize_nvfp4(noisy, B.BLOCKS_BOTH, B.ROUND_RNE, seed=5)
        for mine, theirs in ((got.res_by_cols, qc), (got.res_by_rows, qr)):
            ca, sa, ta = nv_to_numpy(mine)
            cb, sb, tb = nv_to_numpy(theirs)
            assert ta == tb and np.array_equal(ca, cb) and np.array_equal(sa, sb)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    with pytest.raises(B.MetisError):
        h.split(wide[:, 4:4 + cols], k, p, seed=5)                             # rows not 16-byte aligned


def test_workspace_and_shape_errors(ctx):
    B, h = ctx
    x = torch.zeros((128, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.MetisError):
        h.split(x[:64], 68, 8)                 # k + p = 76 sketch columns on a 64-row operand
    big = torch.zeros((2048, 2048), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.MetisError) as e:
        h.split(big, 260, 8)                   # beyond the largest rank (256)
    assert e.value.code == 2                   # METIS_ERR_SHAPE
    with pytest.raises(B.MetisError) as e:
        h.split(big, 256, 24)                  # k + p above 272
    assert e.value.code == 2
    with pytest.raises(B.MetisError):
        h.split(x, 6, 2)                       # k not a multiple of 4


@pytest.mark.parametrize("bad", [float("nan"), float("inf"), -float("inf")])
def test_non_finite_operand_is_reported_in_the_device_status(bad):
    """A NaN or an infinity anywhere in the operand sets METIS_DEV_NONFINITE (sampled and full sketch, plain
    quantization, the amax-scaled stand-alone quantizer); a clean operand on the same handle leaves the word alone."""
    from paper_2509_00404_b200 import binding as B
    x, _ = synth.llama_like(256, 512, 1.0, 77, rank=8)
    xd = torch.from_numpy(x).to(torch.bfloat16).cuda()
    dirty = xd.clone()
    dirty[131, 257] = bad
    for kind in ("sampled", "full", "plain", "quantize"):
        h = B.Handle(0)
        try:
            run = {"sampled": lambda t: h.split(t, 8, 8, sketch=B.SKETCH_SAMPLED, seed=5),
                   "full": lambda t: h.split(t, 8, 8, sketch=B.SKETCH_FULL, seed=5),
                   "plain": lambda t: h.split(t, 0, 0, seed=5),
                   "quantize": lambda t: h.quantize_nvfp4(t, B.BLOCKS_BOTH, B.ROUND_RNE)}[kind]
            run(xd)
            torch.cuda.synchronize()
            assert h.device_status() == 0, kind
            run(dirty)
            torch.cuda.synchronize()
            assert h.device_status() & B.DEV_NONFINITE, kind
            assert not (h.device_status() & B.DEV_TIMEOUT), kind
        finally:
            h.close()
