// Tensor amax and the stand-alone NVFP4 quantizer (Section 2.3; value set of Appendix C.1).
#include "quant_tile.cuh"

namespace {

__global__ void amax_kernel(const void* __restrict__ x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                            float* __restrict__ out) {
  float m = 0.0f;
  const int64_t n8 = cols / 8;
  if (dtype == METIS_BF16 && (cols & 7) == 0 && (ld & 7) == 0) {
    const int64_t total = rows * n8;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
      const int64_t r = i / n8, g = i - r * n8;
      const uint4 q = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(x) + r * ld + g * 8);
      const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        m = fmaxf(m, fabsf(__uint_as_float(w[j] << 16)));
        m = fmaxf(m, fabsf(__uint_as_float(w[j] & 0xFFFF0000u)));
      }
    }
  } else {
    const int64_t total = rows * cols;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
      const int64_t r = i / cols, c = i - r * cols;
      m = fmaxf(m, fabsf(metis_ld_as_float(x, dtype, r * ld + c)));
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  __shared__ float wmax[32];
  if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x < 32) {
    m = threadIdx.x < (blockDim.x >> 5) ? wmax[threadIdx.x] : 0.0f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    // non-negative floats order like their bit patterns
    if (threadIdx.x == 0) atomicMax(reinterpret_cast<unsigned int*>(out), __float_as_uint(m));
  }
}

__global__ void __launch_bounds__(metis_qt::THREADS)
quantize_kernel(const void* __restrict__ x, int dtype, int64_t ld, metis_qt::QuantParams p,
                const float* __restrict__ tscale_src, int tscale_is_amax, float* ts_out0, float* ts_out1) {
  using namespace metis_qt;
  extern __shared__ __align__(16) unsigned char smem[];
  float* tile = reinterpret_cast<float*>(smem);
  Stage* stage = reinterpret_cast<Stage*>(smem + sizeof(float) * TILE * PITCH);
  uint16_t* rnd = reinterpret_cast<uint16_t*>(smem + sizeof(float) * TILE * PITCH + sizeof(Stage));

  const int64_t row0 = (int64_t)blockIdx.y * TILE, col0 = (int64_t)blockIdx.x * TILE;
  const float s_T = tscale_is_amax ? metis_tensor_scale(*tscale_src) : *tscale_src;
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
    if (ts_out0 != nullptr && ts_out0 != tscale_src) *ts_out0 = s_T;
    if (ts_out1 != nullptr && ts_out1 != tscale_src) *ts_out1 = s_T;
  }
  const int tid = threadIdx.x;
  // load the tile (zero fill outside the matrix), 8 elements per step
  for (int i = tid; i < TILE * (TILE / 8); i += THREADS) {
    const int r = i >> 4, g = i & 15;
    const int64_t gr = row0 + r, gc = col0 + g * 8;
    float v[8];
    if (gr < p.rows && gc + 8 <= p.cols && dtype == METIS_BF16 && (ld & 7) == 0) {
      const uint4 q = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(x) + gr * ld + gc);
      const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        v[2 * j] = __uint_as_float(w[j] << 16);
        v[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
      }
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = (gr < p.rows && gc + j < p.cols) ? metis_ld_as_float(x, dtype, gr * ld + gc + j) : 0.0f;
    }
    *reinterpret_cast<float4*>(tile + r * PITCH + g * 8) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(tile + r * PITCH + g * 8 + 4) = make_float4(v[4], v[5], v[6], v[7]);
  }
  if (p.rounding == METIS_ROUND_SR) fill_draws(rnd, p, row0, col0);
  __syncthreads();
  quantize_tile(tile, rnd, stage, p, row0, col0, s_T);
}

}  // namespace

metis_status_t metis_launch_amax(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, float* amax_out,
                                 cudaStream_t s) {
  METIS_CUDA_TRY(cudaMemsetAsync(amax_out, 0, sizeof(float), s));
  if (rows * cols == 0) return METIS_OK;
  const int64_t work = metis_ceil_div(rows * cols, 8 * 256);
  const int grid = (int)(work < 148 * 8 ? (work < 1 ? 1 : work) : 148 * 8);
  amax_kernel<<<grid, 256, 0, s>>>(x, dtype, rows, cols, ld, amax_out); METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  return METIS_OK;
}

metis_status_t metis_launch_quantize(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, int rounding,
                                     uint64_t seed, uint32_t stream_id, int64_t e_stride_r, int64_t e_stride_c,
                                     const float* tscale_src, int tscale_is_amax, const metis_nvfp4_t* by_cols,
                                     const metis_nvfp4_t* by_rows, cudaStream_t s) {
  using namespace metis_qt;
  if (rows == 0 || cols == 0) return METIS_OK;
  QuantParams p{};
  p.rows = rows; p.cols = cols; p.rounding = rounding; p.seed = seed; p.stream_id = stream_id;
  p.e_stride_r = e_stride_r; p.e_stride_c = e_stride_c;
  if (by_cols) { p.c_codes = by_cols->codes; p.c_scales = by_cols->scales; p.c_layout = by_cols->sf_layout; }
  if (by_rows) { p.r_codes = by_rows->codes; p.r_scales = by_rows->scales; p.r_layout = by_rows->sf_layout; }
  const bool sr = rounding == METIS_ROUND_SR;
  const size_t smem = smem_bytes(sr);
  static bool attr_set[2] = {false, false};
  if (!attr_set[sr]) {
    METIS_CUDA_TRY(cudaFuncSetAttribute(quantize_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes(true)));
    attr_set[0] = attr_set[1] = true;
  }
  dim3 grid((unsigned)metis_ceil_div(cols, TILE), (unsigned)metis_ceil_div(rows, TILE));
  quantize_kernel<<<grid, THREADS, smem, s>>>(x, dtype, ld, p, tscale_src, tscale_is_amax,
                                              by_cols ? by_cols->tensor_scale : nullptr,
                                              by_rows ? by_rows->tensor_scale : nullptr); METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  return METIS_OK;
}
