// Context life cycle, host-side argument checks and the C entry points that do not live with their kernels.
#include <cuda.h>
#include <math.h>
#include <stdlib.h>

#include <atomic>

#include "tc_ptx.cuh"

size_t metis_split_ws_bytes(int64_t rows, int64_t cols, int k, int p);
size_t metis_linear_ws_bytes(int64_t M, int64_t N, int k);

static std::atomic<unsigned long long> g_metis_launch_count{0};
void metis_count_launch() { g_metis_launch_count.fetch_add(1, std::memory_order_relaxed); }

namespace {

// Standard normal quantile for 0 < p <= 0.5 by Newton iteration on the complementary error function,
// started from the classical rational approximation (Abramowitz & Stegun 26.2.23).
double inv_norm_cdf_lower(double p) {
  const double t = sqrt(-2.0 * log(p));
  double x = -(t - (2.515517 + 0.802853 * t + 0.010328 * t * t) / (1.0 + 1.432788 * t + 0.189269 * t * t + 0.001308 * t * t * t));
  for (int it = 0; it < 8; ++it) {
    const double f = 0.5 * erfc(-x * 0.70710678118654752440) - p;
    const double df = 0.39894228040143267794 * exp(-0.5 * x * x);
    const double step = f / df;
    x -= step / (1.0 + 0.5 * x * step);             // Halley correction
  }
  return x;
}

}  // namespace

extern "C" {

metis_status_t metis_create(metis_handle_t* out, int device) {
  if (!out) return METIS_ERR_INVALID_ARG;
  *out = nullptr;
  METIS_CUDA_TRY(cudaSetDevice(device));
  cudaDeviceProp prop;
  METIS_CUDA_TRY(cudaGetDeviceProperties(&prop, device));
  if (prop.major != 10) return METIS_ERR_ARCH;
  metis_context* ctx = static_cast<metis_context*>(calloc(1, sizeof(metis_context)));
  if (!ctx) return METIS_ERR_INVALID_ARG;
  ctx->device = device;
  ctx->sm_count = prop.multiProcessorCount;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ctx->encode_tiled, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !ctx->encode_tiled) {
    free(ctx);
    return METIS_ERR_CUDA;
  }
  __nv_bfloat16* host = static_cast<__nv_bfloat16*>(malloc(65536 * sizeof(__nv_bfloat16)));
  if (!host) { free(ctx); return METIS_ERR_INVALID_ARG; }
  for (int u = 0; u < 32768; ++u) {
    const double v = inv_norm_cdf_lower((u + 0.5) / 65536.0);
    host[u] = __float2bfloat16_rn((float)v);
    host[65535 - u] = __float2bfloat16_rn((float)(-v));
  }
  cudaError_t e = cudaMalloc(&ctx->quantile_lut, 65536 * sizeof(__nv_bfloat16));
  if (e == cudaSuccess) e = cudaMalloc(&ctx->dev_status, 256);
  if (e == cudaSuccess) e = cudaMemcpy(ctx->quantile_lut, host, 65536 * sizeof(__nv_bfloat16), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemset(ctx->dev_status, 0, 256);
  free(host);
  int prio_least = 0, prio_greatest = 0;
  if (e == cudaSuccess) e = cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest);
  for (int i = 0; i < METIS_N_SIDE && e == cudaSuccess; ++i) {
    // highest priority: the side streams carry the short latency-critical chains, which must not queue up
    // behind the thousands of blocks of a big pass running on the caller's stream
    e = cudaStreamCreateWithPriority(&ctx->side[i], cudaStreamNonBlocking, prio_greatest);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_join[i], cudaEventDisableTiming);
  }
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming);
  metis_status_t st = e == cudaSuccess ? METIS_OK : METIS_ERR_CUDA;
  // kernel attributes of this device (the device is current here)
  if (st == METIS_OK) st = metis_quantize_set_attrs();
  if (st == METIS_OK) st = metis_gemm_set_attrs(ctx);
  if (st == METIS_OK) st = metis_split_set_attrs();
  if (st == METIS_OK) st = metis_coeff_set_attrs();
  if (st == METIS_OK) st = metis_residual_set_attrs();
  if (st == METIS_OK) st = metis_linear_set_attrs();
  if (st != METIS_OK) {
    metis_destroy(ctx);                                // releases whatever was created so far
    return st;
  }
  *out = ctx;
  return METIS_OK;
}

metis_status_t metis_destroy(metis_handle_t h) {
  if (!h) return METIS_OK;
  for (int i = 0; i < METIS_N_SIDE; ++i) {
    if (h->side[i]) { cudaStreamSynchronize(h->side[i]); cudaStreamDestroy(h->side[i]); }
    if (h->ev_join[i]) cudaEventDestroy(h->ev_join[i]);
  }
  if (h->ev_fork) cudaEventDestroy(h->ev_fork);
  cudaFree(h->quantile_lut);
  cudaFree(h->dev_status);
  free(h);
  return METIS_OK;
}

metis_status_t metis_last_device_status(metis_handle_t h, uint32_t* out, metis_stream_t stream) {
  if (!h || !out) return METIS_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  METIS_CUDA_TRY(cudaMemcpyAsync(out, h->dev_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
  METIS_CUDA_TRY(cudaMemsetAsync(h->dev_status, 0, sizeof(uint32_t), s));
  METIS_CUDA_TRY(cudaStreamSynchronize(s));
  return METIS_OK;
}

metis_status_t metis_debug_quantile_table(metis_handle_t h, uint16_t* host_out) {
  if (!h || !host_out) return METIS_ERR_INVALID_ARG;
  METIS_CUDA_TRY(cudaMemcpy(host_out, h->quantile_lut, 65536 * sizeof(uint16_t), cudaMemcpyDeviceToHost));
  return METIS_OK;
}

namespace {
__global__ void index_check_kernel(uint32_t* status, int64_t off, int64_t n, int64_t extent) {
  (void)metis_dbg_ok(status, off, n, extent);
}
}  // namespace

int32_t metis_debug_build(void) {
#ifdef METIS_DEBUG_BUILD
  return 1;
#else
  return 0;
#endif
}

metis_status_t metis_debug_index_check(metis_handle_t h, int64_t offset, int64_t nbytes, int64_t extent, metis_stream_t stream) {
  if (!h || nbytes <= 0 || extent < 0) return METIS_ERR_INVALID_ARG;
  index_check_kernel<<<1, 1, 0, reinterpret_cast<cudaStream_t>(stream)>>>(h->dev_status, offset, nbytes, extent); METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  return METIS_OK;
}

uint64_t metis_debug_launch_count(void) { return g_metis_launch_count.load(std::memory_order_relaxed); }

size_t metis_sf_bytes(int64_t rows, int64_t k_len, int32_t sf_layout) {
  if (rows <= 0 || k_len <= 0) return 0;
  if (sf_layout == METIS_SF_TILED) return (size_t)(metis_ceil_div(rows, 128) * metis_ceil_div(k_len, 64) * 512);
  return (size_t)(rows * metis_ceil_div(k_len, 16));
}

metis_status_t metis_workspace_bytes(int32_t op, int64_t rows, int64_t cols, int32_t k, int32_t p, size_t* bytes) {
  if (!bytes || rows <= 0 || cols <= 0 || k < 0 || p < 0) return METIS_ERR_INVALID_ARG;
  switch (op) {
    case 0: *bytes = 256; return METIS_OK;
    case 1: *bytes = metis_split_ws_bytes(rows, cols, k, p); return METIS_OK;
    case 2: *bytes = metis_linear_ws_bytes(rows, cols, k); return METIS_OK;
    case 3: *bytes = 2 * metis_linear_ws_bytes(rows, cols, k); return METIS_OK;    // two products' intermediates side by side
    case 4: *bytes = ((metis_split_ws_bytes(rows, cols, k, p) + 255) & ~(size_t)255) +      // split of an FP32 or strided operand:
                     (((size_t)rows * (size_t)cols * 2 + 255) & ~(size_t)255); return METIS_OK;   // plus its contiguous BF16 copy
    default: return METIS_ERR_INVALID_ARG;
  }
}

namespace {
__global__ void timestamp_kernel(unsigned long long* slot) {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  *slot = t;
}
}  // namespace

namespace {
// Failure-detection hook: the producer / consumer skeleton of the tensor-core kernels with nothing in flight.
// Warp 0 waits (bounded) on a "data landed" barrier that nobody will ever arrive at; warp 1 waits on a second one
// and must notice the shared `dead` flag; everybody then meets at the CTA barrier and returns.  No TMA, no MMA, no
// tensor memory: the only thing exercised is the give-up path of the bounded wait and the status word.
__global__ void __launch_bounds__(64) wait_timeout_kernel(uint32_t* dev_status, uint32_t polls, uint32_t* seen) {
  __shared__ __align__(8) uint64_t bars[2];
  __shared__ int dead;
  using namespace metis_tc;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) { mbar_init(smem_u32(&bars[0]), 1); mbar_init(smem_u32(&bars[1]), 1); dead = 0; fence_barrier_init(); }
  __syncthreads();
  bool ok = true;
  if (lane == 0) ok = mbar_wait_n(smem_u32(&bars[warp]), 0, dev_status, &dead, warp == 0 ? polls : 16u * polls + 4096u);
  __syncwarp();
  __syncthreads();
  if (lane == 0) seen[warp] = (ok ? 0u : 1u) | (dead ? 2u : 0u);
}
}  // namespace

metis_status_t metis_debug_wait_timeout(metis_handle_t h, uint32_t polls, uint32_t* device_seen, metis_stream_t stream) {
  if (!h || !device_seen || polls == 0 || polls > (1u << 20)) return METIS_ERR_INVALID_ARG;
  wait_timeout_kernel<<<1, 64, 0, reinterpret_cast<cudaStream_t>(stream)>>>(h->dev_status, polls, device_seen);
  METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  return METIS_OK;
}

metis_status_t metis_debug_timestamp(metis_handle_t h, uint64_t* device_slot, metis_stream_t stream) {
  if (!h || !device_slot) return METIS_ERR_INVALID_ARG;
  timestamp_kernel<<<1, 1, 0, reinterpret_cast<cudaStream_t>(stream)>>>(reinterpret_cast<unsigned long long*>(device_slot));
  METIS_CUDA_TRY(cudaGetLastError());
  return METIS_OK;
}

metis_status_t metis_quantize_nvfp4(metis_handle_t h, const void* x, int32_t dtype, int64_t rows, int64_t cols,
                                    int64_t ld, int32_t rounding, uint64_t seed, uint32_t stream_id, int32_t tscale,
                                    metis_nvfp4_t* out_by_cols, metis_nvfp4_t* out_by_rows, void* ws, size_t ws_bytes,
                                    metis_stream_t stream) {
  METIS_NVTX("metis_quantize_nvfp4");
  if (!h || !x || (!out_by_cols && !out_by_rows)) return METIS_ERR_INVALID_ARG;
  if (dtype != METIS_BF16 && dtype != METIS_FP32) return METIS_ERR_INVALID_ARG;
  if (rounding != METIS_ROUND_RNE && rounding != METIS_ROUND_SR) return METIS_ERR_INVALID_ARG;
  if (tscale != METIS_TSCALE_AMAX_SELF && tscale != METIS_TSCALE_GIVEN) return METIS_ERR_INVALID_ARG;
  if (rows <= 0 || cols <= 0 || ld < cols) return METIS_ERR_SHAPE;
  if (!metis_aligned16(x)) return METIS_ERR_ALIGNMENT;
  metis_nvfp4_t* outs[2] = {out_by_cols, out_by_rows};
  for (int i = 0; i < 2; ++i) {
    metis_nvfp4_t* o = outs[i];
    if (!o) continue;
    if (!o->codes || !o->scales || !o->tensor_scale) return METIS_ERR_INVALID_ARG;
    if (!metis_aligned16(o->codes) || !metis_aligned16(o->scales)) return METIS_ERR_ALIGNMENT;
    const int64_t klen = i == 0 ? cols : rows;
    if (klen % 16) return METIS_ERR_SHAPE;
    if (o->sf_layout == METIS_SF_TILED && klen % 64) return METIS_ERR_SHAPE;
    if (o->sf_layout != METIS_SF_TILED && o->sf_layout != METIS_SF_LINEAR) return METIS_ERR_INVALID_ARG;
    o->rows = i == 0 ? rows : cols;
    o->k_len = klen;
  }
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const float* ts_src;
  int is_amax = 0;
  if (tscale == METIS_TSCALE_AMAX_SELF) {
    if (!ws || ws_bytes < 256) return METIS_ERR_WORKSPACE;
    float* amax = static_cast<float*>(ws);
    METIS_TRY(metis_launch_amax(x, dtype, rows, cols, ld, amax, s));
    METIS_TRY(metis_launch_amax_check(h, amax, s));
    ts_src = amax;
    is_amax = 1;
  } else {
    ts_src = out_by_cols ? out_by_cols->tensor_scale : out_by_rows->tensor_scale;
  }
  return metis_launch_quantize(x, dtype, rows, cols, ld, rounding, seed, stream_id, cols, 1, ts_src, is_amax,
                               out_by_cols, out_by_rows, s, h->dev_status);
}

metis_status_t metis_quantize_rht_nvfp4(metis_handle_t h, const void* x, int32_t dtype, int64_t rows, int64_t cols, int64_t ld,
                                        int32_t rounding, uint64_t seed, uint32_t stream_id, metis_nvfp4_t* out, void* ws,
                                        size_t ws_bytes, metis_stream_t stream) {
  METIS_NVTX("metis_quantize_rht_nvfp4");
  if (!h || !x || !out || !out->codes || !out->scales || !out->tensor_scale) return METIS_ERR_INVALID_ARG;
  if (dtype != METIS_BF16 && dtype != METIS_FP32) return METIS_ERR_INVALID_ARG;
  if (rounding != METIS_ROUND_RNE && rounding != METIS_ROUND_SR) return METIS_ERR_INVALID_ARG;
  if (out->sf_layout != METIS_SF_TILED && out->sf_layout != METIS_SF_LINEAR) return METIS_ERR_INVALID_ARG;
  if (rows <= 0 || cols <= 0 || ld < cols || cols % 16 || (out->sf_layout == METIS_SF_TILED && cols % 64)) return METIS_ERR_SHAPE;
  if (!metis_aligned16(out->codes)) return METIS_ERR_ALIGNMENT;
  if (!ws || ws_bytes < 256) return METIS_ERR_WORKSPACE;
  out->rows = rows; out->k_len = cols;
  return metis_launch_quantize_rht(h, x, dtype, rows, cols, ld, rounding, seed, stream_id, out, static_cast<float*>(ws),
                                   reinterpret_cast<cudaStream_t>(stream));
}

metis_status_t metis_requantize_operand(metis_handle_t h, const void* residual, int32_t res_dtype, int64_t ld_res,
                                        int32_t rounding, uint64_t seed, int32_t residual_axes, int32_t res_tscale,
                                        metis_operand_t* op, void* ws, size_t ws_bytes, metis_stream_t stream) {
  METIS_NVTX("metis_requantize_operand");
  if (!h || !residual || !op) return METIS_ERR_INVALID_ARG;
  if (res_dtype != METIS_BF16 && res_dtype != METIS_FP32) return METIS_ERR_INVALID_ARG;
  if (rounding != METIS_ROUND_RNE && rounding != METIS_ROUND_SR) return METIS_ERR_INVALID_ARG;
  if (res_tscale != METIS_TSCALE_AMAX_SELF && res_tscale != METIS_TSCALE_GIVEN) return METIS_ERR_INVALID_ARG;
  const int64_t rows = op->rows, cols = op->cols;
  const int k = op->k;
  if (rows <= 0 || cols <= 0 || rows % 16 || cols % 16 || k < 0 || k > 256 || ld_res < cols) return METIS_ERR_SHAPE;
  if (!metis_aligned16(residual)) return METIS_ERR_ALIGNMENT;
  const bool want_c = (residual_axes & METIS_BLOCKS_ALONG_COLS) != 0, want_r = (residual_axes & METIS_BLOCKS_ALONG_ROWS) != 0;
  if (!want_c && !want_r) return METIS_ERR_INVALID_ARG;
  metis_nvfp4_t rc = op->res_by_cols, rr = op->res_by_rows;
  rc.rows = rows; rc.k_len = cols; rr.rows = cols; rr.k_len = rows;
  if (want_c && (!rc.codes || !rc.scales || !rc.tensor_scale || (rc.sf_layout == METIS_SF_TILED && cols % 64))) return METIS_ERR_INVALID_ARG;
  if (want_r && (!rr.codes || !rr.scales || !rr.tensor_scale || (rr.sf_layout == METIS_SF_TILED && rows % 64))) return METIS_ERR_INVALID_ARG;
  metis_nvfp4_t lq = op->left_q, rq = op->right_q;
  if (k > 0) {
    if (!op->left || !op->right || !op->sigma || !lq.codes || !lq.scales || !lq.tensor_scale || !rq.codes || !rq.scales || !rq.tensor_scale)
      return METIS_ERR_INVALID_ARG;
    if ((lq.sf_layout == METIS_SF_TILED && rows % 64) || (rq.sf_layout == METIS_SF_TILED && cols % 64)) return METIS_ERR_SHAPE;
    lq.rows = k; lq.k_len = rows; rq.rows = k; rq.k_len = cols;
  }
  if (!ws || ws_bytes < 256 || !metis_aligned16(ws)) return METIS_ERR_WORKSPACE;
  float* amax = static_cast<float*>(ws);                 // [0] residual, [1] left, [2] right
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const float* ts_src;
  int is_amax = 0;
  if (res_tscale == METIS_TSCALE_AMAX_SELF) {
    METIS_TRY(metis_launch_amax(residual, res_dtype, rows, cols, ld_res, amax, s));
    METIS_TRY(metis_launch_amax_check(h, amax, s));
    ts_src = amax; is_amax = 1;
  } else {
    ts_src = want_c ? rc.tensor_scale : rr.tensor_scale;
  }
  METIS_TRY(metis_launch_quantize(residual, res_dtype, rows, cols, ld_res, rounding, seed, METIS_STREAM_RESIDUAL, cols, 1, ts_src, is_amax,
                                  want_c ? &rc : nullptr, want_r ? &rr : nullptr, s, h->dev_status));
  if (k > 0) {
    METIS_TRY(metis_launch_amax(op->left, METIS_FP32, k, rows, rows, amax + 1, s));
    METIS_TRY(metis_launch_amax(op->right, METIS_FP32, k, cols, cols, amax + 2, s));
    METIS_TRY(metis_launch_quantize_factors(op->left, rows, op->right, cols, k, rounding, seed, amax + 1, amax + 2, &lq, &rq, s));
  }
  return METIS_OK;
}

metis_status_t metis_gemm_nvfp4(metis_handle_t h, const metis_nvfp4_t* a, const metis_nvfp4_t* b, void* d,
                                int32_t d_dtype, int64_t ldd, int32_t impl, metis_stream_t stream) {
  METIS_NVTX("metis_gemm_nvfp4");
  if (!h || !a || !b || !d) return METIS_ERR_INVALID_ARG;
  if (!a->codes || !b->codes || !a->scales || !b->scales || !a->tensor_scale || !b->tensor_scale) return METIS_ERR_INVALID_ARG;
  if (a->k_len != b->k_len || a->k_len % 16) return METIS_ERR_SHAPE;
  if (ldd < b->rows) return METIS_ERR_SHAPE;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (impl == 1) return metis_launch_gemm_check(a, b, d, d_dtype, ldd, s);
  if (impl != 0) return METIS_ERR_INVALID_ARG;
  return metis_launch_gemm_tc(h, a, b, d, d_dtype, ldd, s);
}

}  // extern "C"
