"""GPU parity: block-scaled FP4 GEMM on identical codes against the exact float64 product."""
import numpy as np
import pytest
import torch

from oracle import nvfp4 as onv

pytestmark = pytest.mark.gpu

TOL = 1e-5        # relative Frobenius error on identical codes (FP32 accumulation of exactly representable products)


@pytest.fixture(scope="module")
def ctx():
    from paper_2509_00404_b200 import binding as B
    h = B.Handle(0)
    yield B, h
    h.close()


def _case(B, h, M, N, K, seed, impl, out_dtype=torch.float32, scale=1.0):
    from gpu_util import nv_from_numpy, rel_fro
    rng = np.random.default_rng(seed)
    a = (rng.standard_normal((M, K)) * np.exp(rng.uniform(-2, 2, (M, 1))) * scale).astype(np.float32)
    b = (rng.standard_normal((N, K)) * np.exp(rng.uniform(-2, 2, (N, 1)))).astype(np.float32)
    ca, cb = onv.quantize(a), onv.quantize(b)
    ref = onv.dequantize(*ca) @ onv.dequantize(*cb).T
    d = h.gemm_nvfp4(nv_from_numpy(B, *ca), nv_from_numpy(B, *cb), out_dtype=out_dtype, impl=impl)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    return rel_fro(d.float().cpu().numpy(), ref)


@pytest.mark.parametrize("shape", [(128, 128, 64), (128, 128, 256), (256, 256, 1024), (384, 640, 2048),
                                   (200, 72, 320), (136, 4, 256), (4, 136, 192), (128, 256, 4096)])
def test_tensor_core_gemm_matches_exact_product(ctx, shape):
    B, h = ctx
    assert _case(B, h, *shape, seed=sum(shape), impl=0) < TOL


@pytest.mark.parametrize("shape", [(64, 64, 64), (200, 72, 320), (128, 256, 1024)])
def test_check_kernel_matches_exact_product(ctx, shape):
    B, h = ctx
    assert _case(B, h, *shape, seed=1 + sum(shape), impl=1) < TOL


@pytest.mark.parametrize("shape", [(256, 256, 14336), (256, 256, 16384), (128, 256, 16384)])
def test_longest_contractions_of_the_workloads(ctx, shape):
    """K = 14336 (FFN down-projection) and K = 16384 (weight gradient at 16384 tokens): the longest FP32 accumulations
    in tensor memory that the workload list contains, through the two-CTA kernel and the one-CTA kernel."""
    B, h = ctx
    err = _case(B, h, *shape, seed=sum(shape), impl=0)
    print("GEMM on identical codes %dx%dx%d: relative Frobenius error %.3e" % (*shape, err))
    assert err < TOL


def test_bf16_output_and_many_tiles(ctx):
    B, h = ctx
    # more tiles than SMs: exercises the persistent loop, both accumulator buffers and the barrier phase wrap
    assert _case(B, h, 2048, 1536, 512, seed=5, impl=0, out_dtype=torch.bfloat16) < 3e-3
    assert _case(B, h, 2048, 1536, 512, seed=5, impl=0) < TOL


def test_last_partial_wave_is_cut_into_half_tiles(ctx):
    B, h = ctx
    # 9 x 9 tiles of 256 x 256 on 74 CTA pairs: one whole wave, then 7 tiles as 14 half-tile items; the last
    # column of tiles is ragged (192 wide), so one right half lies partly outside the matrix
    assert _case(B, h, 2304, 2240, 512, seed=6, impl=0) < TOL
    assert _case(B, h, 2200, 2304, 320, seed=7, impl=0, out_dtype=torch.bfloat16) < 3e-3


def test_tensor_scales_multiply_the_result(ctx):
    B, h = ctx
    assert _case(B, h, 128, 128, 128, seed=9, impl=0, scale=1e-4) < TOL


def test_rejects_bad_shapes(ctx):
    B, h = ctx
    a, b = B.NvFp4(128, 128), B.NvFp4(128, 192)
    with pytest.raises(B.MetisError):
        h.gemm_nvfp4(a, b)
    a, b = B.NvFp4(128, 48, B.SF_LINEAR), B.NvFp4(128, 48, B.SF_LINEAR)
    with pytest.raises(B.MetisError):
        h.gemm_nvfp4(a, b, impl=0)
