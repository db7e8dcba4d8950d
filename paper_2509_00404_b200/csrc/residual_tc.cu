// Fused residual + NVFP4 quantizer of the split (Section 3.2: the residual is taken against the unquantized
// factors and quantized on its own):
//
//   R = x - C B^T          on 128 x 128 tiles, never written to HBM in high precision (unless `dense` is asked for)
//
// C (rows x k) and B (cols x k) are FP32; their product runs on the tcgen05 tensor cores with FP32 accuracy by
// feeding three-term BF16 splits: the six significant cross products are laid side by side along K,
//   A6[r] = [Ch | Ch | Cl | Ch | Cl2 | Cl],   B6[c] = [Bh | Bl | Bh | Bl2 | Bh | Bl]      (K = 6*kp, padded to 64s)
// so one chain of `tcgen05.mma.kind::f16` (M = 128, N = 128) accumulates all of them in tensor memory.
//
// Persistent CTAs, warp-specialised: a TMA producer streams A6 / B6 in 64-wide K chunks through a three-slot
// ring and the x tile into a double buffer; one warp issues the MMAs into a double-buffered accumulator; eight
// epilogue warps turn accumulator and x into NVFP4.  An epilogue thread owns one row and 64 of its columns:
// it subtracts in registers and encodes the blocks that run along the columns straight from registers.  For
// the blocks that run along the rows the warp transposes its 32 x 32 patch through a private piece of shared
// memory (a warp's 32 rows hold whole 16-row blocks), so the epilogue has no CTA-wide barrier at all.
// Every mbarrier wait is bounded; on expiry the kernel records METIS_DEV_TIMEOUT and unwinds.
#include <cuda.h>

#include "quant_tile.cuh"
#include "tc_ptx.cuh"

namespace {

using namespace metis_tc;
using metis_qt::QuantParams;
using metis_qt::encode_block_tab;

constexpr int TM = 128, TN = 128, BK = 64;
constexpr int RING = 3;
constexpr int SLOT_BYTES = 2 * TM * BK * 2;               // A6 chunk + B6 chunk, 16 KiB each
constexpr int X_BYTES = TM * TN * 2;                      // two 64-column boxes of 16 KiB
constexpr int N_EW = 16;                                  // epilogue warps: four TMEM lane quarters x four column quarters
constexpr int PATCH_HALF = 16 * 20 + 16;                   // 16 rows of 20 floats; the second half starts 16 banks further
constexpr int PATCH_F = 2 * PATCH_HALF;                   // floats per warp patch (32 rows x 16 columns)
constexpr int PATCH_U = 32 * 18;                          // 16-bit draws per warp patch
constexpr int NUM_THREADS = 64 + 32 * N_EW;               // producer, MMA issuer, epilogue warps
constexpr size_t SMEM_BYTES = (size_t)RING * SLOT_BYTES + 2 * X_BYTES + N_EW * (PATCH_F * 4 + PATCH_U * 2) + 1024 + 256 + metis_qt::R_TABLE * 4;

struct ResidArgs {
  QuantParams p;
  const float* amax_src;
  float* ts_out0; float* ts_out1;
  float* dense;
  int k_chunks;             // 64-wide K chunks of A6 / B6
  uint32_t* dev_status;
};

// out[i][6*kp padded to kx] for vector i: pattern A = [h|h|l|h|l2|l] (coefficients), pattern B = [h|l|h|l2|h|l] (basis).
// src element (i, j): src[i*stride_i + j*stride_j], j < k (zero beyond).  One thread per (i, group of 8 j).
__global__ void __launch_bounds__(256)
splits6_kernel(const float* __restrict__ src, int64_t n, int k, int kp, int kx, int64_t stride_i, int64_t stride_j, int pattern_b,
               __nv_bfloat16* __restrict__ out) {
  const int groups = kx / 8;
  const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (idx >= n * groups) return;
  const int64_t i = idx / groups;
  const int gq = (int)(idx % groups);
  uint4* dst = reinterpret_cast<uint4*>(out + i * kx) + gq;
  const int term = (gq * 8) / kp, j0 = (gq * 8) % kp;      // which of the six blocks, where inside it
  if (term >= 6) { *dst = make_uint4(0u, 0u, 0u, 0u); return; }
  float v[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) v[e] = (j0 + e < k) ? src[i * stride_i + (int64_t)(j0 + e) * stride_j] : 0.0f;
  uint4 h, l, l2;
  metis_split3x8(v, h, l, l2);
  // term:        0  1  2  3   4   5
  // pattern A:   h  h  l  h   l2  l
  // pattern B:   h  l  h  l2  h   l
  const int sel_a[6] = {0, 0, 1, 0, 2, 1}, sel_b[6] = {0, 1, 0, 2, 0, 1};
  const int sel = pattern_b ? sel_b[term] : sel_a[term];
  *dst = sel == 0 ? h : (sel == 1 ? l : l2);
}

// SR: stochastic rounding (compile-time, so the round-to-nearest kernel carries no draws).  FAST: the matrix is a whole
// number of 128 x 128 tiles, both scale layouts are the tiled one and no dense residual is asked for, so every
// bounds test and layout switch of the epilogue folds away.
template <bool SR, bool FAST>
__global__ void __launch_bounds__(NUM_THREADS, 1)
residual_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_a,
                   const __grid_constant__ CUtensorMap map_b, ResidArgs g) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gen_base = smem_raw + (base - raw);
  auto a_addr = [&](int s) { return base + (uint32_t)s * SLOT_BYTES; };
  auto b_addr = [&](int s) { return a_addr(s) + TM * BK * 2; };
  auto x_addr = [&](int xb) { return base + (uint32_t)RING * SLOT_BYTES + (uint32_t)xb * X_BYTES; };
  const size_t patch_off = (size_t)RING * SLOT_BYTES + 2 * X_BYTES;
  const uint32_t bar_base = base + (uint32_t)(patch_off + N_EW * (PATCH_F * 4 + PATCH_U * 2));
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (RING + s); };
  auto xfull_bar = [&](int xb) { return bar_base + 8u * (2 * RING + xb); };
  auto xempty_bar = [&](int xb) { return bar_base + 8u * (2 * RING + 2 + xb); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * RING + 4 + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * RING + 6 + a); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + patch_off + N_EW * (PATCH_F * 4 + PATCH_U * 2) + 8 * (2 * RING + 8));
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* r_tab = reinterpret_cast<float*>(gen_base + patch_off + N_EW * (PATCH_F * 4 + PATCH_U * 2) + 256);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const QuantParams& p = g.p;
  const int n_ct = (int)((p.cols + TN - 1) / TN), n_rt = (int)((p.rows + TM - 1) / TM);
  const int num_tiles = n_ct * n_rt;

  if (threadIdx.x == 0) {
    for (int s = 0; s < RING; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(xfull_bar(b), 1); mbar_init(xempty_bar(b), N_EW);
      mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), N_EW);
    }
    *dead = 0;
    fence_barrier_init();
  }
  __syncthreads();
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 256);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------- producer -------------------------------
    int s = 0; uint32_t ph = 0;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
      const int row0 = (tile / n_ct) * TM, col0 = (tile % n_ct) * TN;
      const int xb = it & 1;
      if (!mbar_wait(xempty_bar(xb), (((uint32_t)it >> 1) & 1u) ^ 1u, g.dev_status, dead)) { ok = false; break; }
      if (elect_one()) {
        mbar_expect_tx(xfull_bar(xb), (uint32_t)X_BYTES);
        tma_load_2d(x_addr(xb), &map_x, col0, row0, xfull_bar(xb));
        tma_load_2d(x_addr(xb) + X_BYTES / 2, &map_x, col0 + 64, row0, xfull_bar(xb));
      }
      __syncwarp();
      for (int ck = 0; ck < g.k_chunks; ++ck) {
        if (!mbar_wait(empty_bar(s), ph ^ 1u, g.dev_status, dead)) { ok = false; break; }
        if (elect_one()) {
          mbar_expect_tx(full_bar(s), (uint32_t)SLOT_BYTES);
          tma_load_2d(a_addr(s), &map_a, ck * BK, row0, full_bar(s));
          tma_load_2d(b_addr(s), &map_b, ck * BK, col0, full_bar(s));
        }
        __syncwarp();
        if (++s == RING) { s = 0; ph ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer -----------------------------
    constexpr uint32_t idesc = make_idesc_bf16(TM, TN);
    int s = 0; uint32_t ph = 0;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
      const int acc = it & 1;
      if (!mbar_wait(tempty_bar(acc), (((uint32_t)it >> 1) & 1u) ^ 1u, g.dev_status, dead)) { ok = false; break; }
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(acc * TN);
      for (int ck = 0; ck < g.k_chunks; ++ck) {
        if (!mbar_wait(full_bar(s), ph, g.dev_status, dead)) { ok = false; break; }
        tc_fence_after();
        if (elect_one()) {
          const uint64_t a_d = make_smem_desc(a_addr(s), 1024, SWIZZLE_128B), b_d = make_smem_desc(b_addr(s), 1024, SWIZZLE_128B);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            tc_mma_bf16(d_tmem, a_d + (uint64_t)(k * 2), b_d + (uint64_t)(k * 2), idesc, (ck | k) != 0 ? 1u : 0u);
          tc_commit(empty_bar(s));
        }
        __syncwarp();
        if (++s == RING) { s = 0; ph ^= 1u; }
      }
      if (ok && elect_one()) tc_commit(tfull_bar(acc));
      __syncwarp();
    }
  } else {
    // ------------------------------- epilogue -------------------------------
    const int ew = warp - 2;                                // 0..15
    const int quarter = warp & 3, colq = ew >> 2;           // TMEM lane quarter (fixed by the warp id), column quarter
    float* patch = reinterpret_cast<float*>(gen_base + patch_off) + ew * PATCH_F;
    uint16_t* upatch = reinterpret_cast<uint16_t*>(gen_base + patch_off + N_EW * PATCH_F * 4) + ew * PATCH_U;
    constexpr bool sr = SR;
    const int c_layout = FAST ? (int)METIS_SF_TILED : p.c_layout, r_layout = FAST ? (int)METIS_SF_TILED : p.r_layout;
    const float s_T = metis_tensor_scale(*g.amax_src);
    const float six_s_T = __fmul_rn(6.0f, s_T);
    metis_qt::fill_r_table(r_tab, s_T, (int)threadIdx.x - 64, 32 * N_EW);
    asm volatile("bar.sync 1, %0;" ::"n"(32 * N_EW) : "memory");       // the epilogue warps only
    if (blockIdx.x == 0 && threadIdx.x == 64) {
      if (g.ts_out0) *g.ts_out0 = s_T;
      if (g.ts_out1) *g.ts_out1 = s_T;
    }
    const int64_t c_kbytes = p.cols / 2, r_kbytes = p.rows / 2, c_bpr = p.cols / 16, r_bpr = p.rows / 16;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
      const int row0 = (tile / n_ct) * TM, col0 = (tile % n_ct) * TN;
      const int acc = it & 1, xb = it & 1;
      const uint32_t par = ((uint32_t)it >> 1) & 1u;
      if (!mbar_wait(xfull_bar(xb), par, g.dev_status, dead)) { ok = false; break; }
      if (!mbar_wait(tfull_bar(acc), par, g.dev_status, dead)) { ok = false; break; }
      tc_fence_after();
      const int64_t row = (int64_t)row0 + quarter * 32 + lane;              // this thread's row
      const bool row_ok = FAST || row < p.rows;
      const int64_t slab_row0 = (int64_t)row0 + quarter * 32;               // first row of the warp's 32
      const int64_t c0 = (int64_t)col0 + colq * 32;                         // first of this warp's 32 columns
      // x tile: two 64-column boxes of 128-byte rows, 16-byte chunks XOR-swizzled by the row
      const uint32_t xrow = x_addr(xb) + (uint32_t)(colq >> 1) * (X_BYTES / 2) + (uint32_t)(quarter * 32 + lane) * 128u;
      const uint32_t sw = (uint32_t)((quarter * 32 + lane) & 7);
      float v[32];
      {
        uint32_t a[32];
        tc_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * TN + colq * 32), a);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint32_t w0, w1, w2, w3;
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3)
                       : "r"(xrow + ((((uint32_t)(4 * (colq & 1) + j)) ^ sw) << 4)));
          const uint32_t ws[4] = {w0, w1, w2, w3};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            v[8 * j + 2 * e] = __uint_as_float(ws[e] << 16) - __uint_as_float(a[8 * j + 2 * e]);
            v[8 * j + 2 * e + 1] = __uint_as_float(ws[e] & 0xFFFF0000u) - __uint_as_float(a[8 * j + 2 * e + 1]);
          }
        }
      }
      // accumulator and x tile read: hand both back.  The x box was read with ordinary shared-memory loads (generic
      // proxy) and is refilled by a tensor copy (async proxy): the proxy fence orders those reads before the copy
      // that the arrival permits.  Without it the refill could land - rarely - before the warp's last load had been
      // performed, and 8 columns of 32 rows came out with the next tile's values.
      tc_fence_before();
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) { mbar_arrive(tempty_bar(acc)); mbar_arrive(xempty_bar(xb)); }
      const bool step_ok = FAST || c0 < p.cols;                                      // false: the warp's columns lie outside the matrix
      const bool blk1_ok = FAST || c0 + 16 < p.cols;
      uint32_t u[32];
      if (sr) {
        const uint64_t e0 = (uint64_t)row * (uint64_t)p.e_stride_r + (uint64_t)c0;        // multiple of 8
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          const uint4 w = metis_philox_block((e0 >> 3) + q4, p.seed, p.stream_id);
          const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) { u[8 * q4 + 2 * j] = ww[j] << 16; u[8 * q4 + 2 * j + 1] = ww[j] & 0xFFFF0000u; }   // thresholds: draw << 16
        }
      }
      if (!FAST && g.dense != nullptr && row_ok && step_ok) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (c0 + 4 * j < p.cols)
            METIS_DBG_GUARD(g.dev_status, (row * p.cols + c0 + 4 * j) * 4, 16, p.rows * p.cols * 4)
            *reinterpret_cast<float4*>(g.dense + row * p.cols + c0 + 4 * j) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
      }
      if (p.c_codes != nullptr && step_ok) {
        // blocks along the columns: two blocks of this row, from registers
        float v0[16], v1[16];
        uint32_t u0[16], u1[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) { v0[i] = v[i]; v1[i] = v[16 + i]; u0[i] = sr ? u[i] : 0u; u1[i] = sr ? u[16 + i] : 0u; }
        uint32_t pk0[2], pk1[2];
        const uint32_t sb0 = encode_block_tab(v0, u0, sr, six_s_T, r_tab, pk0);
        const uint32_t sb1 = encode_block_tab(v1, u1, sr, six_s_T, r_tab, pk1);
        if (row_ok) {
          uint8_t* cp = p.c_codes + row * c_kbytes + c0 / 2;
          METIS_DBG_GUARD(g.dev_status, row * c_kbytes + c0 / 2, blk1_ok ? 16 : 8, p.rows * c_kbytes) {
            if (blk1_ok) *reinterpret_cast<uint4*>(cp) = make_uint4(pk0[0], pk0[1], pk1[0], pk1[1]);
            else *reinterpret_cast<uint2*>(cp) = make_uint2(pk0[0], pk0[1]);
          }
        }
        if (row_ok || c_layout == METIS_SF_TILED) {                         // padded rows of a 128-row slab get zero scales
          const int64_t o = metis_sf_offset(row, c0 / 16, c_bpr, c_layout);
          METIS_DBG_GUARD(g.dev_status, o, 2, p.c_sf_bytes)
          if (FAST) {
            *reinterpret_cast<uint16_t*>(p.c_scales + o) = (uint16_t)(sb0 | (sb1 << 8));   // c0 / 16 is even: an aligned pair
          } else {
            p.c_scales[o] = row_ok ? (uint8_t)sb0 : (uint8_t)0;
            if (blk1_ok) p.c_scales[o + 1] = row_ok ? (uint8_t)sb1 : (uint8_t)0;
          }
        }
      }
      if (p.r_codes != nullptr && (step_ok || r_layout == METIS_SF_TILED)) {
        // blocks along the rows: the warp transposes its 32 x 32 values 16 columns at a time through its patch;
        // in each half lane l encodes the block of column l % 16, rows 16 * (l / 16) .. +15
        const int cb = lane & 15, rb = lane >> 4;
        const bool rb_ok = FAST || slab_row0 + 16 * rb < p.rows;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          {
            // one row of 16 values per lane as four 16-byte stores (rows 80 bytes apart: a quarter warp covers all banks)
            float4* dst = reinterpret_cast<float4*>(patch + (lane >> 4) * PATCH_HALF + (lane & 15) * 20);
#pragma unroll
            for (int j = 0; j < 4; ++j) dst[j] = make_float4(v[16 * hf + 4 * j], v[16 * hf + 4 * j + 1], v[16 * hf + 4 * j + 2], v[16 * hf + 4 * j + 3]);
          }
          if (sr) {
#pragma unroll
            for (int i = 0; i < 16; ++i) upatch[lane * 18 + i] = (uint16_t)(u[16 * hf + i] >> 16);
          }
          __syncwarp();
          const int64_t col = c0 + 16 * hf + cb;
          const bool col_ok = FAST || col < p.cols;
          float t[16];
          uint32_t d[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            t[i] = patch[rb * PATCH_HALF + i * 20 + cb];
            d[i] = sr ? (uint32_t)upatch[(16 * rb + i) * 18 + cb] << 16 : 0u;
          }
          uint32_t pk[2];
          const uint32_t sb = encode_block_tab(t, d, sr, six_s_T, r_tab, pk);
          if (col_ok && rb_ok) METIS_DBG_GUARD(g.dev_status, col * r_kbytes + (slab_row0 + 16 * rb) / 2, 8, p.cols * r_kbytes)
            *reinterpret_cast<uint2*>(p.r_codes + col * r_kbytes + (slab_row0 + 16 * rb) / 2) = make_uint2(pk[0], pk[1]);
          if (rb_ok && (col_ok || r_layout == METIS_SF_TILED))               // padded columns of a 128-slab get zero scales
            METIS_DBG_GUARD(g.dev_status, metis_sf_offset(col, slab_row0 / 16 + rb, r_bpr, r_layout), 1, p.r_sf_bytes)
            p.r_scales[metis_sf_offset(col, slab_row0 / 16 + rb, r_bpr, r_layout)] = col_ok ? (uint8_t)sb : (uint8_t)0;
          __syncwarp();
        }
      }
    }
  }

  // ------------------------------- teardown ---------------------------------
  tc_fence_before();
  __syncthreads();
  if (*dead) {
    // a wait expired: give copies already in flight time to land before the shared memory is released
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 256);
  }
}

}  // namespace

int metis_residual_kx(int kp) { return (6 * kp + 63) / 64 * 64; }

bool metis_residual_tc_usable(const void* x, int64_t cols) { return metis_aligned16(x) && cols % 8 == 0; }

// a6: [rows][kx] = per row [Ch|Ch|Cl|Ch|Cl2|Cl], b6: [cols][kx] = per column [Bh|Bl|Bh|Bl2|Bh|Bl] (BF16,
// kx = metis_residual_kx(kp)).  b6 is filled by the caller; a6 too unless `coef` ([rows][kp] FP32) is given,
// in which case it is written here first.
metis_status_t metis_residual_set_attrs() {
  METIS_CUDA_TRY(cudaFuncSetAttribute(residual_tc_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
  METIS_CUDA_TRY(cudaFuncSetAttribute(residual_tc_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
  METIS_CUDA_TRY(cudaFuncSetAttribute(residual_tc_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
  METIS_CUDA_TRY(cudaFuncSetAttribute(residual_tc_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
  return METIS_OK;
}

metis_status_t metis_launch_residual_tc(metis_context* ctx, const void* x, const float* coef, int k, int kp,
                                        const metis_qt::QuantParams& qp, const float* amax_src, float* ts_out0, float* ts_out1,
                                        float* dense, void* a6, void* b6, cudaStream_t s) {
  const int kx = metis_residual_kx(kp);
  const int64_t rows = qp.rows, cols = qp.cols;
  if (coef != nullptr) {
    splits6_kernel<<<(unsigned)metis_ceil_div(rows * (kx / 8), 256), 256, 0, s>>>(coef, rows, k, kp, kx, kp, 1, 0,
                                                                                  reinterpret_cast<__nv_bfloat16*>(a6)); METIS_COUNT_LAUNCH();
  }
  CUtensorMap mx, ma, mb;
  METIS_TRY(make_map_bf16(ctx, &mx, x, rows, cols, cols, TM));
  METIS_TRY(make_map_bf16(ctx, &ma, a6, rows, kx, kx, TM));
  METIS_TRY(make_map_bf16(ctx, &mb, b6, cols, kx, kx, TN));
  ResidArgs g{};
  g.p = qp;
  g.p.c_sf_bytes = qp.c_codes ? (int64_t)metis_sf_bytes(rows, cols, qp.c_layout) : 0;
  g.p.r_sf_bytes = qp.r_codes ? (int64_t)metis_sf_bytes(cols, rows, qp.r_layout) : 0;
  g.amax_src = amax_src; g.ts_out0 = ts_out0; g.ts_out1 = ts_out1; g.dense = dense;
  g.k_chunks = kx / BK;
  g.dev_status = ctx->dev_status;
  const bool fast = rows % TM == 0 && cols % TN == 0 && dense == nullptr &&
                    (qp.c_codes == nullptr || (qp.c_layout == METIS_SF_TILED && reinterpret_cast<uintptr_t>(qp.c_scales) % 2 == 0)) &&
                    (qp.r_codes == nullptr || qp.r_layout == METIS_SF_TILED);
  const bool sr = qp.rounding == METIS_ROUND_SR;
  const int64_t tiles = metis_ceil_div(rows, TM) * metis_ceil_div(cols, TN);
  // A persistent CTA fills its SM (216 KB of shared memory).  A few SMs are left free so that the small kernels
  // of the factor chain, which run beside this pass on another stream, and those of other operands' chains do
  // not have to wait for the whole pass to end.
  // The smaller the operand, the more of the step is those chains: up to 1024 tiles (4096 x 4096) the pass leaves
  // 40 SMs (measured best of 0 ... 100 on the three-operand layer step), up to 4096 tiles 16.  A large operand's
  // pass is long against the chains and throughput-bound: it leaves only a few SMs (with none free the factor
  // chain, which runs beside it, would simply be appended to it).
  const int reserve = tiles <= 1024 ? 40 : (tiles <= 4096 ? 16 : 4);
  const int usable = ctx->sm_count > 2 * reserve ? ctx->sm_count - reserve : ctx->sm_count;
  const int grid = (int)(tiles < usable ? tiles : usable);
  if (sr) {
    if (fast) residual_tc_kernel<true, true><<<grid, NUM_THREADS, SMEM_BYTES, s>>>(mx, ma, mb, g);
    else residual_tc_kernel<true, false><<<grid, NUM_THREADS, SMEM_BYTES, s>>>(mx, ma, mb, g);
  } else {
    if (fast) residual_tc_kernel<false, true><<<grid, NUM_THREADS, SMEM_BYTES, s>>>(mx, ma, mb, g);
    else residual_tc_kernel<false, false><<<grid, NUM_THREADS, SMEM_BYTES, s>>>(mx, ma, mb, g);
  }
  METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  return METIS_OK;
}
