// Scalar check kernel for the block-scaled FP4 product: decodes every code and scale and accumulates
// in FP32 with plain FMAs.  Slow by design; used for tiny or skinny shapes and to cross-check the
// tensor-core kernel on identical codes.
#include "common.cuh"

namespace {

constexpr int BM = 64, BN = 64, BK = 64;   // one 64-element K slab = 4 scale blocks per row

__global__ void __launch_bounds__(256)
gemm_check_kernel(const uint8_t* __restrict__ a_codes, const uint8_t* __restrict__ a_sf, const float* a_ts, int a_layout,
                  const uint8_t* __restrict__ b_codes, const uint8_t* __restrict__ b_sf, const float* b_ts, int b_layout,
                  int64_t M, int64_t N, int64_t K, void* __restrict__ d, int d_dtype, int64_t ldd) {
  __shared__ float As[BK][BM + 1];
  __shared__ float Bs[BK][BN + 1];
  const int tid = threadIdx.x;
  const int64_t m0 = (int64_t)blockIdx.y * BM, n0 = (int64_t)blockIdx.x * BN;
  const int tx = tid & 15, ty = tid >> 4;          // 16 x 16 threads, 4 x 4 outputs each
  float acc[4][4] = {};
  const int64_t bpr = K / 16;
  for (int64_t k0 = 0; k0 < K; k0 += BK) {
    // decode: each thread handles one (row, 16-element block) of A and of B
    {
      const int r = tid >> 2, b = tid & 3;         // 64 rows x 4 blocks
      const int64_t gk = k0 + b * 16;
      {
        const int64_t gr = m0 + r;
        const bool ok = gr < M && gk < K;
        const float sf = ok ? metis_e4m3_value(a_sf[metis_sf_offset(gr, gk / 16, bpr, a_layout)]) : 0.0f;
        uint2 q = make_uint2(0u, 0u);
        if (ok) q = *reinterpret_cast<const uint2*>(a_codes + gr * (K / 2) + gk / 2);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const uint32_t c = ((i < 8 ? q.x : q.y) >> (4 * (i & 7))) & 15u;
          As[b * 16 + i][r] = metis_e2m1_value(c) * sf;
        }
      }
      {
        const int64_t gr = n0 + r;
        const bool ok = gr < N && gk < K;
        const float sf = ok ? metis_e4m3_value(b_sf[metis_sf_offset(gr, gk / 16, bpr, b_layout)]) : 0.0f;
        uint2 q = make_uint2(0u, 0u);
        if (ok) q = *reinterpret_cast<const uint2*>(b_codes + gr * (K / 2) + gk / 2);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const uint32_t c = ((i < 8 ? q.x : q.y) >> (4 * (i & 7))) & 15u;
          Bs[b * 16 + i][r] = metis_e2m1_value(c) * sf;
        }
      }
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < BK; ++kk) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
  const float alpha = (*a_ts) * (*b_ts);
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t gr = m0 + ty * 4 + i, gc = n0 + tx * 4 + j;
      if (gr < M && gc < N) {
        const float v = acc[i][j] * alpha;
        if (d_dtype == METIS_BF16) reinterpret_cast<__nv_bfloat16*>(d)[gr * ldd + gc] = __float2bfloat16_rn(v);
        else reinterpret_cast<float*>(d)[gr * ldd + gc] = v;
      }
    }
}

}  // namespace

metis_status_t metis_launch_gemm_check(const metis_nvfp4_t* a, const metis_nvfp4_t* b, void* d, int d_dtype,
                                       int64_t ldd, cudaStream_t s) {
  const int64_t M = a->rows, N = b->rows, K = a->k_len;
  if (M == 0 || N == 0) return METIS_OK;
  dim3 grid((unsigned)metis_ceil_div(N, BN), (unsigned)metis_ceil_div(M, BM));
  gemm_check_kernel<<<grid, 256, 0, s>>>(a->codes, a->scales, a->tensor_scale, a->sf_layout, b->codes, b->scales,
                                         b->tensor_scale, b->sf_layout, M, N, K, d, d_dtype, ldd); METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  return METIS_OK;
}
