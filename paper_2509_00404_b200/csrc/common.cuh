// Shared device/host helpers of the Metis B200 library: context, error plumbing, Philox, NVFP4 scalar math.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <nvtx3/nvToolsExt.h>

#include "../../include/metis.h"

// One NVTX range per entry point of the C ABI (visible in a timeline tool; a no-op when no tool is attached).
struct metis_nvtx_range {
  explicit metis_nvtx_range(const char* name) { nvtxRangePushA(name); }
  ~metis_nvtx_range() { nvtxRangePop(); }
};
#define METIS_NVTX(name) metis_nvtx_range nvtx_range_(name)

constexpr int METIS_N_SIDE = 5;                        // side streams per handle (the backward pass uses all five)
struct metis_context {
  int device;
  int sm_count;
  __nv_bfloat16* quantile_lut;   // 65536 bf16 standard-normal quantiles (Section 3.1 Gaussian test matrix)
  uint32_t* dev_status;          // device status word (METIS_DEV_* bits)
  void* encode_tiled;            // cuTensorMapEncodeTiled entry point, resolved at create
  // Internal fork/join: independent sub-chains of one call run on these side streams and are joined back into
  // the caller's stream with events before the call's last kernels (everything stays asynchronous).
  cudaStream_t side[METIS_N_SIDE];
  cudaEvent_t ev_fork, ev_join[METIS_N_SIDE];
  int max_pairs;                 // two-CTA clusters of the large GEMM that this device keeps resident at once
};

// Per-device kernel attributes (dynamic shared memory above 48 KiB).  Function attributes belong to the device
// that is current when they are set, so metis_create sets them for the handle's device, once per handle; no
// launch helper keeps a process-wide "already set" flag.
metis_status_t metis_quantize_set_attrs();
metis_status_t metis_gemm_set_attrs(metis_context* ctx);
metis_status_t metis_split_set_attrs();
metis_status_t metis_coeff_set_attrs();
metis_status_t metis_residual_set_attrs();
metis_status_t metis_linear_set_attrs();

// fork: side stream i starts after everything enqueued so far on `main`
static inline metis_status_t metis_fork(metis_context* ctx, cudaStream_t main, int n_side) {
  if (cudaEventRecord(ctx->ev_fork, main) != cudaSuccess) return METIS_ERR_CUDA;
  for (int i = 0; i < n_side; ++i)
    if (cudaStreamWaitEvent(ctx->side[i], ctx->ev_fork, 0) != cudaSuccess) return METIS_ERR_CUDA;
  return METIS_OK;
}
// join: `main` continues after everything enqueued so far on side stream i
static inline metis_status_t metis_join(metis_context* ctx, cudaStream_t main, int i) {
  if (cudaEventRecord(ctx->ev_join[i], ctx->side[i]) != cudaSuccess) return METIS_ERR_CUDA;
  if (cudaStreamWaitEvent(main, ctx->ev_join[i], 0) != cudaSuccess) return METIS_ERR_CUDA;
  return METIS_OK;
}

// Programmatic dependent launch: a kernel launched with this helper may be scheduled while the kernel before it
// in the stream is still draining; it must call metis_pdl_wait() before it touches global memory (the wait
// returns when the preceding kernel has completed and its writes are visible).  Saves the launch gap between
// the many short dependent kernels of a decomposition.
__device__ __forceinline__ void metis_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel of the stream (if it was launched with the helper below) be scheduled as soon as SMs have
// room, before this kernel has finished; it still waits for this kernel's completion in its own metis_pdl_wait().
__device__ __forceinline__ void metis_pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline cudaError_t metis_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

#define METIS_CUDA_TRY(expr)                         \
  do {                                               \
    cudaError_t e__ = (expr);                        \
    if (e__ != cudaSuccess) return METIS_ERR_CUDA;   \
  } while (0)

#define METIS_TRY(expr)                              \
  do {                                               \
    metis_status_t s__ = (expr);                     \
    if (s__ != METIS_OK) return s__;                 \
  } while (0)

// Number of kernels the library has launched in this process (read through metis_debug_launch_count).
// Process-wide and atomic: handles on several devices or threads may launch at the same time.
void metis_count_launch();
#define METIS_COUNT_LAUNCH() metis_count_launch()

static inline bool metis_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline int64_t metis_ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al. 2011).  One call yields 128 bits = eight 16-bit draws.
// Draw rule: element index e -> counter (lo32(e>>3), hi32(e>>3), stream, 0), key (lo32 seed, hi32 seed),
// 16-bit half number e&7 of the four output words (low half first).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 metis_philox(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ uint4 metis_philox_block(uint64_t block_index, uint64_t seed, uint32_t stream) {
  return metis_philox((uint32_t)block_index, (uint32_t)(block_index >> 32), stream, 0u, (uint32_t)seed,
                      (uint32_t)(seed >> 32));
}

__device__ __forceinline__ uint32_t metis_u16_of(const uint4& w, uint32_t h) {
  const uint32_t word = (h >> 1) == 0 ? w.x : (h >> 1) == 1 ? w.y : (h >> 1) == 2 ? w.z : w.w;
  return (word >> (16u * (h & 1u))) & 0xFFFFu;
}

__device__ __forceinline__ uint32_t metis_draw_u16(uint64_t e, uint64_t seed, uint32_t stream) {
  return metis_u16_of(metis_philox_block(e >> 3, seed, stream), (uint32_t)(e & 7u));
}

// ---------------------------------------------------------------------------------------------
// NVFP4 scalar arithmetic (Section 2.3).  Every step is a single IEEE binary32 operation with
// round-to-nearest-even and no contraction; this order defines the format's rounding decisions.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float metis_tensor_scale(float amax) { return amax == 0.0f ? 1.0f : __fdiv_rn(amax, 2688.0f); }

// smallest non-negative finite E4M3 value >= t (0 <= t <= 448); returns the byte and the value
__device__ __forceinline__ uint32_t metis_e4m3_ceil(float t, float* value) {
  if (!(t > 0.0f)) { *value = 0.0f; return 0u; }
  if (t <= 0.015625f) {                       // subnormal range: multiples of 2^-9 up to 2^-6
    const int f = (int)ceilf(__fmul_rn(t, 512.0f));
    *value = __fmul_rn((float)f, 0.001953125f);
    return (uint32_t)f;                       // f == 8 is the first normal number (byte 0x08)
  }
  uint32_t b = __float_as_uint(t);
  b = (b + 0xFFFFFu) & 0xFFF00000u;           // keep 3 mantissa bits, round up (carry moves the exponent)
  *value = __uint_as_float(b);
  const uint32_t e = (b >> 23) - 127u + 7u;
  return (e << 3) | ((b >> 20) & 7u);
}

__device__ __forceinline__ float metis_e4m3_value(uint32_t byte) {
  const uint32_t e = (byte >> 3) & 15u, f = byte & 7u;
  return e == 0 ? __fmul_rn((float)f, 0.001953125f) : __uint_as_float(((e + 120u) << 23) | (f << 20));
}

__device__ __forceinline__ float metis_e2m1_value(uint32_t code) {
  const uint32_t m = code & 7u;
  const float mag = m < 4 ? 0.5f * (float)m : (m == 4 ? 2.0f : m == 5 ? 3.0f : m == 6 ? 4.0f : 6.0f);
  return (code & 8u) ? -mag : mag;
}

// two round-to-nearest-even E2M1 codes in one byte: lo in bits 0-3, hi in bits 4-7
__device__ __forceinline__ uint32_t metis_e2m1x2_rne(float lo, float hi) {
  uint32_t out;
  asm("{ .reg .b8 t8; cvt.rn.satfinite.e2m1x2.f32 t8, %1, %2; cvt.u32.u8 %0, t8; }" : "=r"(out) : "f"(hi), "f"(lo));
  return out;
}

// stochastic rounding of y to E2M1 with a 16-bit draw: up iff frac * 65536 > u, frac = (a - lo)/(hi - lo), a = min(|y|, 6).
// E2M1 is a tiny float format: one mantissa bit per binade from 1 upwards, and below 1 the grid {0, 0.5, 1} has the
// spacing of the binade [1, 2).  So for a >= 1 the lower neighbour is the top mantissa bit of a and frac is the other
// 22 bits, and a < 1 is mapped onto [1, 2] by adding 1 (rounded UP, so that bits lost in the addition still count as
// "frac > 0"; a carry into the next grid point is the round-up it stands for).  Then
//   frac * 65536 > u  <=>  (mantissa & 0x3FFFFF) > 64 u,
// an exact integer comparison, and the code is  offset + 2 * exponent + top bit + up.  No branches.
__device__ __forceinline__ uint32_t metis_e2m1_sr(float y, uint32_t u16) {
  const float a = fminf(fabsf(y), 6.0f);
  const uint32_t sign = (__float_as_uint(y) >> 28) & 8u;
  const bool small = a < 1.0f;
  const uint32_t bits = __float_as_uint(small ? __fadd_ru(a, 1.0f) : a);
  const uint32_t g = ((bits >> 22) & 0x1FFu) - 254u;               // 2 * exponent + top mantissa bit (0 at 1.0)
  const uint32_t up = (bits & 0x3FFFFFu) > (u16 << 6) ? 1u : 0u;
  return sign | ((small ? 0u : 2u) + g + up);
}

// byte offset of scale (row r, block b) in the 128x4-tiled layout; blocks_per_row = k_len/16
__host__ __device__ __forceinline__ int64_t metis_sf_offset_tiled(int64_t r, int64_t b, int64_t blocks_per_row) {
  return ((r >> 7) * (blocks_per_row >> 2) + (b >> 2)) * 512 + (r & 31) * 16 + ((r & 127) >> 5) * 4 + (b & 3);
}
__host__ __device__ __forceinline__ int64_t metis_sf_offset(int64_t r, int64_t b, int64_t blocks_per_row, int layout) {
  return layout == METIS_SF_TILED ? metis_sf_offset_tiled(r, b, blocks_per_row) : r * blocks_per_row + b;
}

__device__ __forceinline__ float metis_ld_as_float(const void* p, int dtype, int64_t idx) {
  return dtype == METIS_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[idx])
                             : reinterpret_cast<const float*>(p)[idx];
}

// splits of eight consecutive FP32 values into BF16 hi / lo / lo2, packed two per word
__device__ __forceinline__ void metis_split3x8(const float (&v)[8], uint4& h, uint4& l, uint4& l2) {
  uint32_t hh[4], ll[4], mm[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float x = v[2 * i], y = v[2 * i + 1];
    const __nv_bfloat16 xh = __float2bfloat16_rn(x), yh = __float2bfloat16_rn(y);
    const float xr = x - __bfloat162float(xh), yr = y - __bfloat162float(yh);
    const __nv_bfloat16 xl = __float2bfloat16_rn(xr), yl = __float2bfloat16_rn(yr);
    const __nv_bfloat16 xm = __float2bfloat16_rn(xr - __bfloat162float(xl)), ym = __float2bfloat16_rn(yr - __bfloat162float(yl));
    hh[i] = (uint32_t)__bfloat16_as_ushort(xh) | ((uint32_t)__bfloat16_as_ushort(yh) << 16);
    ll[i] = (uint32_t)__bfloat16_as_ushort(xl) | ((uint32_t)__bfloat16_as_ushort(yl) << 16);
    mm[i] = (uint32_t)__bfloat16_as_ushort(xm) | ((uint32_t)__bfloat16_as_ushort(ym) << 16);
  }
  h = make_uint4(hh[0], hh[1], hh[2], hh[3]); l = make_uint4(ll[0], ll[1], ll[2], ll[3]); l2 = make_uint4(mm[0], mm[1], mm[2], mm[3]);
}


// ---- debug-build index checks ----------------------------------------------------------------
// metis_dbg_ok: is a store of n bytes at byte offset off inside a buffer of extent bytes?  If not, the status word gets
// METIS_DEV_INDEX and the caller skips the store.  METIS_DBG_GUARD(...) stmt;  compiles to the bare statement in a
// release build.
__device__ __forceinline__ bool metis_dbg_ok(uint32_t* status, int64_t off, int64_t n, int64_t extent) {
  if (off >= 0 && off + n <= extent) return true;
  if (status != nullptr) atomicOr(status, METIS_DEV_INDEX);
  return false;
}
#ifdef METIS_DEBUG_BUILD
#define METIS_DBG_GUARD(status, off, n, extent) if (!metis_dbg_ok((status), (int64_t)(off), (int64_t)(n), (int64_t)(extent))) {} else
#else
#define METIS_DBG_GUARD(status, off, n, extent)
#endif

// ---- internal entry points shared between translation units --------------------------------
metis_status_t metis_launch_amax(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, float* amax_out,
                                 cudaStream_t s);
metis_status_t metis_launch_quantize(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, int rounding,
                                     uint64_t seed, uint32_t stream_id, int64_t e_stride_r, int64_t e_stride_c,
                                     const float* tscale_src, int tscale_is_amax, const metis_nvfp4_t* by_cols,
                                     const metis_nvfp4_t* by_rows, cudaStream_t s, uint32_t* dbg_status = nullptr);
int metis_coeff_slices(int64_t rows, int64_t cols, int* chunks_per_slice);
bool metis_coeff_tc_usable(const void* x, const void* bs, int64_t cols, int kp);
metis_status_t metis_launch_coeff_tc(metis_context* ctx, const void* x, int64_t rows, int64_t cols, const void* bs, int kp,
                                     float* part, float* amax, int raw, cudaStream_t s);
metis_status_t metis_launch_quantize_factors(const float* left, int64_t rows, const float* right, int64_t cols, int k, int rounding,
                                             uint64_t seed, const float* amax_left, const float* amax_right,
                                             const metis_nvfp4_t* lq, const metis_nvfp4_t* rq, cudaStream_t s);
metis_status_t metis_launch_amax_check(metis_context* ctx, const float* amax, cudaStream_t s);
metis_status_t metis_launch_quantize_rht(metis_context* ctx, const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, int rounding, uint64_t seed,
                                         uint32_t stream_id, const metis_nvfp4_t* out, float* amax_ws, cudaStream_t s);
bool metis_project_tc_usable(const void* x, const void* hsp, int64_t cols, int jp);
int metis_project_slices(int64_t rows, int64_t cols);
metis_status_t metis_launch_project_tc(metis_context* ctx, const void* x, int64_t rows, int64_t cols, const void* hsp, int jp,
                                       int64_t ldh, float* part, cudaStream_t s);
int metis_residual_kx(int kp);
bool metis_residual_tc_usable(const void* x, int64_t cols);
metis_status_t metis_launch_gemm_check(const metis_nvfp4_t* a, const metis_nvfp4_t* b, void* d, int d_dtype,
                                       int64_t ldd, cudaStream_t s);
metis_status_t metis_launch_gemm_tc(metis_context* ctx, const metis_nvfp4_t* a, const metis_nvfp4_t* b, void* d,
                                    int d_dtype, int64_t ldd, cudaStream_t s);
