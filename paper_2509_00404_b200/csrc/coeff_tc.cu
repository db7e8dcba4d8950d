// Broadcast of the sampled subspace to every row (Section 3.1) on the tcgen05 tensor cores:
//
//   part[s][r][j] = sum over the s-th slice of columns c of  x[r][c] * B[j][c]        (C = X B, split over K)
//
// x is BF16 (exact operand); the FP32 basis enters as three BF16 terms B = Bh + Bl + Bl2 that are laid side by
// side as 3*KP accumulator columns (one MMA stream, N = 3*KP) and added in the epilogue, smallest first, so
// the products keep FP32 accuracy.  The kernel streams x once from HBM: TMA loads of 128-row x 64-column boxes
// (128-byte swizzle) into a four-stage ring, `tcgen05.mma.kind::f16` (M = 128, N = 3*KP, K = 16) with the
// accumulator in tensor memory.  The four epilogue warps are idle during the main loop, so they scan every
// landed x box for amax|x| (the residual's tensor scale) before the slot is released.
// Grid: (row tiles of 128, column slices); the slices are summed in a fixed order by the caller's finish kernel.
// Every mbarrier wait is bounded; on expiry the kernel records METIS_DEV_TIMEOUT and unwinds.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace {

using namespace metis_tc;

constexpr int BM = 128, BK = 64, STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;                      // 16 KiB
constexpr int NUM_THREADS = 192;                          // producer, MMA issuer, 4 epilogue / amax warps

struct CoeffArgs {
  float* part;              // [slices][rows][kp]
  float* amax;              // running amax|x| as the bits of a non-negative float (may be NULL)
  int64_t rows;
  int kp, num_chunks, chunks_per_slice;
  int raw;                  // 1: write all 3 * kp accumulator columns as they are, part[slices][rows][3 * kp]
  int a_mn;                 // 1: the A operand is x transposed (M runs along the columns of x, K along its rows)
  uint32_t* dev_status;
};

template <int NB>                                         // accumulator columns = 3 * kp
__global__ void __launch_bounds__(NUM_THREADS, 1)
coeff_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_b, CoeffArgs g) {
  constexpr int B_BYTES = NB * BK * 2;
  constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr int TMEM_COLS = NB <= 64 ? 64 : (NB <= 128 ? 128 : 256);
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gen_base = smem_raw + (base - raw);
  auto a_addr = [&](int s) { return base + (uint32_t)s * STAGE_BYTES; };
  auto b_addr = [&](int s) { return a_addr(s) + A_BYTES; };
  const uint32_t bar_base = base + (uint32_t)STAGES * STAGE_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  const uint32_t tfull_bar = bar_base + 8u * (2 * STAGES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + (size_t)STAGES * STAGE_BYTES + 8 * (2 * STAGES + 1));
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row0 = blockIdx.x * BM;
  const int c_begin = blockIdx.y * g.chunks_per_slice;
  const int c_end = min(g.num_chunks, c_begin + g.chunks_per_slice);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 5); }   // MMA commit + 4 scanning warps
    mbar_init(tfull_bar, 1);
    *dead = 0;
    fence_barrier_init();
  }
  __syncthreads();
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------- producer -------------------------------
    int s = 0; uint32_t ph = 0;
    for (int c = c_begin; c < c_end; ++c) {
      if (!mbar_wait(empty_bar(s), ph ^ 1u, g.dev_status, dead)) break;
      if (elect_one()) {
        mbar_expect_tx(full_bar(s), (uint32_t)STAGE_BYTES);
        if (g.a_mn) {                                       // two boxes of 64 columns x 64 rows: MN-major A
          tma_load_2d(a_addr(s), &map_x, row0, c * BK, full_bar(s));
          tma_load_2d(a_addr(s) + A_BYTES / 2, &map_x, row0 + 64, c * BK, full_bar(s));
        } else {
          tma_load_2d(a_addr(s), &map_x, c * BK, row0, full_bar(s));
        }
        tma_load_2d(b_addr(s), &map_b, c * BK, 0, full_bar(s));
      }
      __syncwarp();
      if (++s == STAGES) { s = 0; ph ^= 1u; }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer -----------------------------
    constexpr uint32_t idesc_k = make_idesc_bf16(BM, NB), idesc_mn = make_idesc_bf16_a_mn(BM, NB);
    const uint32_t idesc = g.a_mn ? idesc_mn : idesc_k;
    int s = 0; uint32_t ph = 0;
    bool ok = true;
    for (int c = c_begin; c < c_end; ++c) {
      if (!mbar_wait(full_bar(s), ph, g.dev_status, dead)) { ok = false; break; }
      tc_fence_after();
      if (elect_one()) {
        const uint64_t b_d = make_smem_desc(b_addr(s), 1024, SWIZZLE_128B);
        // K-major A: 16 elements = 32 bytes per step inside the 128-byte rows.  MN-major A: a step is 16 K-rows of
        // 128 bytes (two atoms of 8 rows, 1024 bytes apart); the second 64 columns are the second box, 8 KiB on.
        const uint64_t a_d = g.a_mn ? make_smem_desc_mn(a_addr(s), A_BYTES / 2, 1024, SWIZZLE_128B) : make_smem_desc(a_addr(s), 1024, SWIZZLE_128B);
        const uint64_t a_step = g.a_mn ? (uint64_t)(16 * 128 / 16) : 2ull;
#pragma unroll
        for (int k = 0; k < BK / 16; ++k)
          tc_mma_bf16(tmem_base, a_d + (uint64_t)k * a_step, b_d + (uint64_t)(k * 2), idesc, (c > c_begin || k > 0) ? 1u : 0u);
        tc_commit(empty_bar(s));
      }
      __syncwarp();
      if (++s == STAGES) { s = 0; ph ^= 1u; }
    }
    if (ok && elect_one()) tc_commit(tfull_bar);
    __syncwarp();
  } else {
    // ------------------------------- amax scan, then epilogue ---------------
    const int te = threadIdx.x - 64;                        // 0..127: row of the box this thread scans
    uint32_t amax2 = 0u;                                    // two running |.| maxima as a BF16 pair
    int s = 0; uint32_t ph = 0;
    bool ok = true;
    for (int c = c_begin; c < c_end; ++c) {
      if (!mbar_wait(full_bar(s), ph, g.dev_status, dead)) { ok = false; break; }
      if (g.amax != nullptr) {
        const uint32_t rowp = a_addr(s) + (uint32_t)te * 128u;
#pragma unroll
        for (int j = 0; j < 8; ++j) {                       // lanes start at different 16-byte chunks: no bank conflicts
          uint32_t w0, w1, w2, w3;
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3)
                       : "r"(rowp + (uint32_t)(((j + lane) & 7) << 4)));
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const uint32_t ab = (e == 0 ? w0 : e == 1 ? w1 : e == 2 ? w2 : w3) & 0x7FFF7FFFu;
            amax2 = max(ab & 0xFFFFu, amax2 & 0xFFFFu) | (max(ab >> 16, amax2 >> 16) << 16);
          }
        }
      }
      fence_proxy_async();                                // the box was read through the generic proxy; a tensor copy refills it
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar(s));
      if (++s == STAGES) { s = 0; ph ^= 1u; }
    }
    if (g.amax != nullptr) {
      // as ordered bit patterns all the way (a NaN ranks above infinity and must survive: fmaxf would drop it)
      uint32_t am = max((amax2 & 0xFFFFu) << 16, amax2 & 0xFFFF0000u);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, o));
      if (lane == 0) atomicMax(reinterpret_cast<unsigned int*>(g.amax), am);
    }
    if (ok && c_end > c_begin && mbar_wait(tfull_bar, 0u, g.dev_status, dead)) {
      tc_fence_after();
      const int quarter = warp & 3;                         // TMEM lanes 32*quarter .. +31 belong to this warp
      const int64_t row = (int64_t)row0 + quarter * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
      if (g.raw) {
        float* dst = g.part + ((int64_t)blockIdx.y * g.rows + row) * NB;
        for (int jb = 0; jb < NB; jb += 16) {
          uint32_t r0[16];
          tc_ld16(t_row + (uint32_t)jb, r0);
          tc_wait_ld();
          if (row < g.rows) {
#pragma unroll
            for (int e = 0; e < 16; e += 4)
              *reinterpret_cast<float4*>(dst + jb + e) = make_float4(__uint_as_float(r0[e]), __uint_as_float(r0[e + 1]),
                                                                     __uint_as_float(r0[e + 2]), __uint_as_float(r0[e + 3]));
          }
        }
      }
      float* dst = g.part + ((int64_t)blockIdx.y * g.rows + row) * g.kp;
      for (int jb = 0; jb < (g.raw ? 0 : g.kp); jb += 16) {
        uint32_t r0[16], r1[16], r2[16];
        tc_ld16(t_row + (uint32_t)jb, r0);
        tc_ld16(t_row + (uint32_t)(g.kp + jb), r1);
        tc_ld16(t_row + (uint32_t)(2 * g.kp + jb), r2);
        tc_wait_ld();
        if (row < g.rows) {
#pragma unroll
          for (int e = 0; e < 16; e += 4)                   // smallest terms first
            *reinterpret_cast<float4*>(dst + jb + e) =
                make_float4((__uint_as_float(r2[e]) + __uint_as_float(r1[e])) + __uint_as_float(r0[e]),
                            (__uint_as_float(r2[e + 1]) + __uint_as_float(r1[e + 1])) + __uint_as_float(r0[e + 1]),
                            (__uint_as_float(r2[e + 2]) + __uint_as_float(r1[e + 2])) + __uint_as_float(r0[e + 2]),
                            (__uint_as_float(r2[e + 3]) + __uint_as_float(r1[e + 3])) + __uint_as_float(r0[e + 3]));
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
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

template <int NB>
constexpr size_t coeff_smem() { return (size_t)STAGES * (A_BYTES + NB * BK * 2) + 1024 + 128; }
template <int NB>
cudaError_t set_attr() { return cudaFuncSetAttribute(coeff_tc_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)coeff_smem<NB>()); }

template <int NB>
metis_status_t launch(const CUtensorMap& mx, const CUtensorMap& mb, const CoeffArgs& g, dim3 grid, cudaStream_t s) {
  constexpr size_t smem = coeff_smem<NB>();
  coeff_tc_kernel<NB><<<grid, NUM_THREADS, smem, s>>>(mx, mb, g); METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  return METIS_OK;
}

}  // namespace

metis_status_t metis_coeff_set_attrs() {
  METIS_CUDA_TRY(set_attr<48>()); METIS_CUDA_TRY(set_attr<96>()); METIS_CUDA_TRY(set_attr<144>());
  METIS_CUDA_TRY(set_attr<192>()); METIS_CUDA_TRY(set_attr<240>());
  return METIS_OK;
}

// number of column slices (grid.y) and 64-column chunks per slice: about one CTA per SM, at most 8 slices
int metis_coeff_slices(int64_t rows, int64_t cols, int* chunks_per_slice) {
  const int64_t tiles = metis_ceil_div(rows, BM), chunks = metis_ceil_div(cols, BK);
  int64_t s = metis_ceil_div(160, tiles);
  if (s > 8) s = 8;
  if (s > chunks) s = chunks;
  if (s < 1) s = 1;
  const int64_t cps = metis_ceil_div(chunks, s);
  if (chunks_per_slice) *chunks_per_slice = (int)cps;
  return (int)metis_ceil_div(chunks, cps);                // every slice has work
}

bool metis_coeff_tc_usable(const void* x, const void* bs, int64_t cols, int kp) {
  return metis_aligned16(x) && metis_aligned16(bs) && cols % 8 == 0 && (kp == 16 || kp == 32 || kp == 48 || kp == 64);
}

// part: [metis_coeff_slices(rows, cols, ..)][rows][kp] FP32; bs: [3][kp][cols] BF16 (three-term split of the basis).
// raw = 1: the operand is a single (3 * kp) x cols BF16 matrix and the accumulator columns are written unsummed,
// part[slice][rows][3 * kp] (the sketch Z = X Omega of a full-mode split).
// Projection of a full-mode split on the same kernel: part[slice][col][jp] = sum over the slice's rows r of
// x[r][col] * H[r][j], i.e. M^T = x^T H with x as an MN-major A operand (M runs along the columns of x).
// hsp: [3][jp][ldh] BF16 (three-term split of H, transposed, ldh >= rows rounded up to 64, zero padded).
bool metis_project_tc_usable(const void* x, const void* hsp, int64_t cols, int jp) {
  return metis_aligned16(x) && metis_aligned16(hsp) && cols % 8 == 0 && (jp == 16 || jp == 32 || jp == 48 || jp == 64 || jp == 80);
}

int metis_project_slices(int64_t rows, int64_t cols) { return metis_coeff_slices(cols, rows, nullptr); }

metis_status_t metis_launch_project_tc(metis_context* ctx, const void* x, int64_t rows, int64_t cols, const void* hsp, int jp,
                                       int64_t ldh, float* part, cudaStream_t s) {
  CUtensorMap mx, mb;
  METIS_TRY(make_map_bf16(ctx, &mx, x, rows, cols, cols, BK));
  METIS_TRY(make_map_bf16(ctx, &mb, hsp, 3 * (int64_t)jp, ldh, ldh, 3 * jp));
  CoeffArgs g{};
  g.part = part; g.amax = nullptr; g.rows = cols; g.kp = jp; g.raw = 0; g.a_mn = 1;
  g.num_chunks = (int)metis_ceil_div(rows, BK);
  const int slices = metis_coeff_slices(cols, rows, &g.chunks_per_slice);
  g.dev_status = ctx->dev_status;
  dim3 grid((unsigned)metis_ceil_div(cols, BM), (unsigned)slices);
  switch (jp) {
    case 16: return launch<48>(mx, mb, g, grid, s);
    case 32: return launch<96>(mx, mb, g, grid, s);
    case 48: return launch<144>(mx, mb, g, grid, s);
    case 64: return launch<192>(mx, mb, g, grid, s);
    case 80: return launch<240>(mx, mb, g, grid, s);
    default: return METIS_ERR_SHAPE;
  }
}

metis_status_t metis_launch_coeff_tc(metis_context* ctx, const void* x, int64_t rows, int64_t cols, const void* bs, int kp,
                                     float* part, float* amax, int raw, cudaStream_t s) {
  CUtensorMap mx, mb;
  METIS_TRY(make_map_bf16(ctx, &mx, x, rows, cols, cols, BM));
  METIS_TRY(make_map_bf16(ctx, &mb, bs, 3 * (int64_t)kp, cols, cols, 3 * kp));
  CoeffArgs g{};
  g.part = part; g.amax = amax; g.rows = rows; g.kp = kp; g.raw = raw; g.a_mn = 0;
  g.num_chunks = (int)metis_ceil_div(cols, BK);
  const int slices = metis_coeff_slices(rows, cols, &g.chunks_per_slice);
  g.dev_status = ctx->dev_status;
  dim3 grid((unsigned)metis_ceil_div(rows, BM), (unsigned)slices);
  switch (kp) {
    case 16: return launch<48>(mx, mb, g, grid, s);
    case 32: return launch<96>(mx, mb, g, grid, s);
    case 48: return launch<144>(mx, mb, g, grid, s);
    case 64: return launch<192>(mx, mb, g, grid, s);
    default: return METIS_ERR_SHAPE;
  }
}
