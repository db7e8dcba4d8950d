// Block-scaled NVFP4 GEMM on the 5th-generation tensor cores (tcgen05) of sm_100a.
//
//   D[M x N] = alpha * sum_k  e2m1(A[m,k]) * ue4m3(SFA[m,k/16]) * e2m1(B[n,k]) * ue4m3(SFB[n,k/16])
//
// A (M x K) and B (N x K) are K-major packed FP4 (two codes per byte) with one UE4M3 scale per 16
// elements stored in the 128 x 4 tiled layout, alpha = tensor_scale(A) * tensor_scale(B).
// These matrix products are where nearly all of the training arithmetic goes (Section 3): the
// residual x residual term of Eq. 2 / Eq. 3 / the weight gradient, and the skinny factor products.
//
// Two kernels, both persistent over output tiles and warp-specialised (TMA producer warp, MMA issuer warp,
// epilogue warps; shared-memory ring with mbarriers; FP32 accumulators in tensor memory):
//   gemm_nvfp4_kernel<BLOCK_N>       one CTA per 128 x BLOCK_N tile (skinny products)
//   two_cta::gemm_nvfp4_2cta_kernel  a CTA pair (cta_group::2) per 256 x 256 tile, optionally followed by BF16
//                                    K boxes that add a low-rank correction into the same accumulator
// The producer and issuer loops are walked by whole warps with one elected lane issuing, so that descriptors
// and addresses stay in uniform registers.  Every mbarrier wait is bounded; on expiry the kernel records
// METIS_DEV_TIMEOUT and unwinds.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace {

using namespace metis_tc;

constexpr int BLOCK_M = 128;
constexpr int BLOCK_K = 256;                  // elements per stage = 128 bytes of packed FP4 = one swizzle row
constexpr int MMA_K = 64;                     // elements per tcgen05.mma (kind::mxf4nvf4, dense)
constexpr int K_STEPS = BLOCK_K / MMA_K;      // 4
constexpr int NUM_THREADS = 192;

template <int BLOCK_N>
struct Cfg {
  static constexpr int STAGES = BLOCK_N == 128 ? 6 : 4;
  static constexpr int NUM_ACC = BLOCK_N == 128 ? 2 : 1;
  static constexpr int N_TILES_SF = BLOCK_N / 128;                 // 128-row scale tiles of B per stage
  static constexpr int A_BYTES = BLOCK_M * BLOCK_K / 2;            // 16 KiB
  static constexpr int B_BYTES = BLOCK_N * BLOCK_K / 2;
  static constexpr int SFA_BYTES = K_STEPS * 512;
  static constexpr int SFB_BYTES = N_TILES_SF * K_STEPS * 512;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + SFA_BYTES + SFB_BYTES;
  static constexpr int ACC_COLS = NUM_ACC * BLOCK_N;               // 256
  // every ring stage has its own scale columns in tensor memory, so the scale copy of stage s+1 never has to
  // wait for the MMAs of stage s to finish reading theirs
  static constexpr int SF_COLS_PER_STAGE = 4 * K_STEPS * (1 + N_TILES_SF);      // 32 or 48
  static constexpr int SF_COL0 = ACC_COLS;
  static constexpr int TMEM_COLS = 512;
  static_assert(ACC_COLS + STAGES * SF_COLS_PER_STAGE <= 512, "tensor memory budget");
  static constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};


// Instruction descriptor for kind::mxf4nvf4 with UE4M3 scales: E2M1 operands (format 1) at [7,10) and
// [10,13), both K-major, N/8 at [17,23), scale format 0 (UE4M3) at bit 23, M/16 at [24,29).
__host__ __device__ constexpr uint32_t make_idesc(int m, int n) {
  return (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

struct GemmArgs {
  const uint8_t* a_sf; const uint8_t* b_sf;
  const float* a_ts; const float* b_ts;
  void* d; int d_dtype; int64_t ldd;
  int M, N, K;
  uint32_t* dev_status;
  int tma_store;           // two-CTA kernel: the output goes through shared memory and tensor stores
  int extra_kb;            // BF16 correction boxes (64 elements of K each) appended after the FP4 K loop
};

// Writes 32 consecutive accumulator columns of one output row (scaled by alpha) as FP32 or BF16.
__device__ __forceinline__ void store_row_chunk(const GemmArgs& g, int row, int col, const uint32_t (&r)[32], float alpha) {
  if (g.d_dtype == METIS_FP32) {
    float* dst = reinterpret_cast<float*>(g.d) + (size_t)row * g.ldd + col;
    if (col + 32 <= g.N && ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0)) {
#pragma unroll
      for (int j = 0; j < 32; j += 4)
        *reinterpret_cast<float4*>(dst + j) = make_float4(__uint_as_float(r[j]) * alpha, __uint_as_float(r[j + 1]) * alpha,
                                                          __uint_as_float(r[j + 2]) * alpha, __uint_as_float(r[j + 3]) * alpha);
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) if (col + j < g.N) dst[j] = __uint_as_float(r[j]) * alpha;
    }
  } else {
    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(g.d) + (size_t)row * g.ldd + col;
    if (col + 32 <= g.N && ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0)) {
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[j + 2 * q]) * alpha,
                                                         __uint_as_float(r[j + 2 * q + 1]) * alpha);
          w[q] = *reinterpret_cast<const uint32_t*>(&h);
        }
        *reinterpret_cast<uint4*>(dst + j) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) if (col + j < g.N) dst[j] = __float2bfloat16_rn(__uint_as_float(r[j]) * alpha);
    }
  }
}

template <int BLOCK_N>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_nvfp4_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, GemmArgs g) {
  using C = Cfg<BLOCK_N>;
  metis_pdl_trigger();
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;              // 1024-byte alignment for the 128-byte swizzle
  unsigned char* gen_base = smem_raw + (base - raw);
  auto a_addr = [&](int s) { return base + (uint32_t)s * C::STAGE_BYTES; };
  auto b_addr = [&](int s) { return a_addr(s) + C::A_BYTES; };
  auto sfa_addr = [&](int s) { return b_addr(s) + C::B_BYTES; };
  auto sfb_addr = [&](int s) { return sfa_addr(s) + C::SFA_BYTES; };
  const uint32_t bar_base = base + (uint32_t)C::STAGES * C::STAGE_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (C::STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + C::NUM_ACC + a); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + (size_t)C::STAGES * C::STAGE_BYTES + 8 * (2 * C::STAGES + 2 * C::NUM_ACC));
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_m = (g.M + BLOCK_M - 1) / BLOCK_M, num_n = (g.N + BLOCK_N - 1) / BLOCK_N;
  const int num_tiles = num_m * num_n;
  const int num_kb = (g.K + BLOCK_K - 1) / BLOCK_K;
  const int sf_k_atoms = g.K / MMA_K;                        // 512-byte scale atoms per 128-row tile

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < C::NUM_ACC; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
    *dead = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // everything above touched only this CTA's shared and tensor memory: it may overlap the previous kernel's tail
  metis_pdl_wait();

  if (warp == 0) {
    // ------------------------------- producer -------------------------------
    // (the whole warp walks the loop so that addresses stay warp-uniform; one elected lane issues)
    int s = 0; uint32_t ph = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      const int mb = tile % num_m, nb = tile / num_m;
      for (int kb = 0; kb < num_kb; ++kb) {
        if (!mbar_wait(empty_bar(s), ph ^ 1u, g.dev_status, dead)) { ok = false; break; }
        if (elect_one()) {
          const int atoms = min(K_STEPS, sf_k_atoms - kb * K_STEPS);
          mbar_expect_tx(full_bar(s), (uint32_t)(C::A_BYTES + C::B_BYTES) + (uint32_t)atoms * 512u * (1 + C::N_TILES_SF));
          tma_load_2d(a_addr(s), &map_a, kb * (BLOCK_K / 2), mb * BLOCK_M, full_bar(s));
          tma_load_2d(b_addr(s), &map_b, kb * (BLOCK_K / 2), nb * BLOCK_N, full_bar(s));
          bulk_load(sfa_addr(s), g.a_sf + ((size_t)mb * sf_k_atoms + (size_t)kb * K_STEPS) * 512, atoms * 512, full_bar(s));
#pragma unroll
          for (int t = 0; t < C::N_TILES_SF; ++t)
            bulk_load(sfb_addr(s) + t * K_STEPS * 512,
                      g.b_sf + ((size_t)min(nb * C::N_TILES_SF + t, (g.N + 127) / 128 - 1) * sf_k_atoms + (size_t)kb * K_STEPS) * 512,
                      atoms * 512, full_bar(s));
        }
        __syncwarp();
        if (++s == C::STAGES) { s = 0; ph ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer -----------------------------
    constexpr uint32_t idesc = make_idesc(BLOCK_M, BLOCK_N);
    int s = 0; uint32_t ph = 0;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
      const int acc = it % C::NUM_ACC;
      const uint32_t acc_ph = (uint32_t)(it / C::NUM_ACC) & 1u;
      if (!mbar_wait(tempty_bar(acc), acc_ph ^ 1u, g.dev_status, dead)) { ok = false; break; }
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BLOCK_N);
      for (int kb = 0; kb < num_kb; ++kb) {
        if (!mbar_wait(full_bar(s), ph, g.dev_status, dead)) { ok = false; break; }
        tc_fence_after();
        if (elect_one()) {
          const int atoms = min(K_STEPS, sf_k_atoms - kb * K_STEPS);
          const uint32_t sfa_t = tmem_base + C::SF_COL0 + s * C::SF_COLS_PER_STAGE;
          const uint32_t sfb_t = sfa_t + 4 * K_STEPS;
          const uint64_t sfa_d = make_smem_desc(sfa_addr(s), 128, SWIZZLE_NONE), sfb_d = make_smem_desc(sfb_addr(s), 128, SWIZZLE_NONE);
          const uint64_t a_d = make_smem_desc(a_addr(s), 1024, SWIZZLE_128B), b_d = make_smem_desc(b_addr(s), 1024, SWIZZLE_128B);
          if (atoms == K_STEPS) {
#pragma unroll
            for (int k = 0; k < K_STEPS; ++k) {
              tc_cp_sf(sfa_t + 4 * k, sfa_d + (uint64_t)(k * 32));
#pragma unroll
              for (int t = 0; t < C::N_TILES_SF; ++t)
                tc_cp_sf(sfb_t + 4 * (k * C::N_TILES_SF + t), sfb_d + (uint64_t)((t * K_STEPS + k) * 32));
            }
#pragma unroll
            for (int k = 0; k < K_STEPS; ++k)
              tc_mma_nvf4(d_tmem, a_d + (uint64_t)(k * 2), b_d + (uint64_t)(k * 2), idesc, sfa_t + 4 * k, sfb_t + 4 * k * C::N_TILES_SF,
                          (kb | k) != 0 ? 1u : 0u);
          } else {
          for (int k = 0; k < atoms; ++k) {
            tc_cp_sf(sfa_t + 4 * k, sfa_d + (uint64_t)(k * 32));
#pragma unroll
            for (int t = 0; t < C::N_TILES_SF; ++t)
              tc_cp_sf(sfb_t + 4 * (k * C::N_TILES_SF + t), sfb_d + (uint64_t)((t * K_STEPS + k) * 32));
          }
          for (int k = 0; k < atoms; ++k)
            tc_mma_nvf4(d_tmem, a_d + (uint64_t)(k * 2), b_d + (uint64_t)(k * 2), idesc, sfa_t + 4 * k, sfb_t + 4 * k * C::N_TILES_SF,
                        (kb | k) != 0 ? 1u : 0u);
          }
          tc_commit(empty_bar(s));                           // slot reusable once these MMAs have read it
        }
        __syncwarp();
        if (++s == C::STAGES) { s = 0; ph ^= 1u; }
      }
      if (ok && elect_one()) tc_commit(tfull_bar(acc));      // accumulator complete
      __syncwarp();
    }
  } else {
    // ------------------------------- epilogue -------------------------------
    const int quarter = warp & 3;                            // TMEM lanes 32*quarter .. +31 belong to this warp
    const float alpha = (*g.a_ts) * (*g.b_ts);
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
      const int mb = tile % num_m, nb = tile / num_m;
      const int acc = it % C::NUM_ACC;
      const uint32_t acc_ph = (uint32_t)(it / C::NUM_ACC) & 1u;
      if (!mbar_wait(tfull_bar(acc), acc_ph, g.dev_status, dead)) { ok = false; break; }
      tc_fence_after();
      const int row = mb * BLOCK_M + quarter * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BLOCK_N);
#pragma unroll 1
      for (int c0 = 0; c0 < BLOCK_N; c0 += 32) {
        uint32_t r[32];
        tc_ld32(t_row + c0, r);
        const int col = nb * BLOCK_N + c0;
        if (row < g.M && col < g.N) store_row_chunk(g, row, col, r, alpha);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
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
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

// =================================================================================================
// Two-CTA variant (cta_group::2): a cluster of two CTAs on neighbouring SMs computes one 256 x 256 tile.
// Each CTA loads 128 rows of A and 128 rows of B per K block (the pair's MMA reads both halves of B),
// its own 128 rows of A scales and the scales of all 256 B rows; the leader CTA issues the scale copies and
// the MMAs for both, each CTA keeps its 128 x 256 half of the accumulator in its own tensor memory and runs
// its own epilogue.  All loads of a stage, code tiles and scale atoms alike, are TMA tensor copies in the
// cta_group::2 form that credit the LEADER's barrier, so a stage costs two barrier hand-offs in all
// (slot free -> producer, data landed -> MMA issuer): the ring of five 38 KiB stages has to cover that
// round trip, and it is this latency, not the tensor pipe, that bounds the kernel.
// =================================================================================================
namespace two_cta {

constexpr int TILE_M = 256, TILE_N = 256;
constexpr int RASTER_M = 8;                                 // row tiles per raster group (see the tile order in the kernel)
constexpr int STAGES = 5;
constexpr int A_BYTES = 128 * BLOCK_K / 2;                  // this CTA's 128 rows of A
constexpr int B_BYTES = 128 * BLOCK_K / 2;                  // this CTA's 128 rows of B
constexpr int SFA_BYTES = K_STEPS * 512;
constexpr int SFB_BYTES = 2 * K_STEPS * 512;
constexpr int STAGE_BYTES = A_BYTES + B_BYTES + SFA_BYTES + SFB_BYTES;   // 38 KiB
constexpr int ACC_COLS = 256;
constexpr int SF_COLS_PER_STAGE = 4 * K_STEPS * 3;          // 16 (A) + 32 (B): each ring stage has its own scale columns
constexpr int SF_COL0 = 256;
constexpr int TMEM_COLS = 512;
static_assert(ACC_COLS + STAGES * SF_COLS_PER_STAGE <= TMEM_COLS, "tensor memory budget");
constexpr int NUM_THREADS = 384;                            // producer, MMA issuer, two idle warps, 8 epilogue warps
constexpr int OUT_STAGE_BYTES = 8 * 4096;                   // per epilogue warp: 32 rows x 128 bytes of converted output
constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + OUT_STAGE_BYTES + 1024 + 256;

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive on the barrier at the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ void mbar_arrive_remote(uint32_t local_bar, uint32_t rank) {
  asm volatile(
      "{ .reg .b32 ra; mapa.shared::cluster.u32 ra, %0, %1;\n"
      "  mbarrier.arrive.release.cluster.shared::cluster.b64 _, [ra]; }"
      ::"r"(local_bar), "r"(rank) : "memory");
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
// Tensor load into THIS CTA's shared memory whose byte count is credited to a barrier that may live in the
// pair's other CTA (cta_group::2 form; no multicast): both CTAs of a pair report to the leader's barrier.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t cluster_bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(cluster_bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{ .reg .pred p; mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, uint32_t* dev_status, volatile int* dead) {
  for (uint32_t i = 0; i < WAIT_LIMIT; ++i) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if (i > 4096) __nanosleep(32);
    if ((i & 1023u) == 1023u && *dead) break;
  }
  *dead = 1;
  atomicOr(dev_status, METIS_DEV_TIMEOUT);
  return false;
}
__device__ __forceinline__ void tmem_alloc2(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_commit2(uint32_t bar, uint16_t mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void tc_cp_sf2(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void tc_mma_nvf4_2(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                              uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile(
      "{ .reg .pred p; setp.ne.b32 p, %4, 0;\n"
      "  tcgen05.mma.cta_group::2.kind::mxf4nvf4.block_scale.block16 [%0], %1, %2, %3, [%5], [%6], p; }"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem) : "memory");
}

// dense BF16 x BF16 -> FP32 MMA into the same accumulator (the low-rank correction of the split layer)
__device__ __forceinline__ void tc_mma_bf16_2(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{ .reg .pred p; setp.ne.b32 p, %4, 0;\n"
      "  tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p; }"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// The K loop runs over num_kb FP4 blocks (256 elements each) followed by g.extra_kb BF16 boxes (64 elements
// each, same 16 KiB + 16 KiB ring slot): the latter add  Lx Rx^T  (the rank-(ka+kb) correction of the split
// layer, pre-divided by alpha) into the same FP32 accumulator.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
gemm_nvfp4_2cta_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                       const __grid_constant__ CUtensorMap map_sfa, const __grid_constant__ CUtensorMap map_sfb,
                       const __grid_constant__ CUtensorMap map_l, const __grid_constant__ CUtensorMap map_r,
                       const __grid_constant__ CUtensorMap map_d, GemmArgs g) {
  metis_pdl_trigger();
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gen_base = smem_raw + (base - raw);
  auto a_addr = [&](int s) { return base + (uint32_t)s * STAGE_BYTES; };
  auto b_addr = [&](int s) { return a_addr(s) + A_BYTES; };
  auto sfa_addr = [&](int s) { return b_addr(s) + B_BYTES; };
  auto sfb_addr = [&](int s) { return sfa_addr(s) + SFA_BYTES; };
  const uint32_t out_base = base + (uint32_t)STAGES * STAGE_BYTES;           // 1024-byte aligned (swizzled store boxes)
  const uint32_t bar_base = out_base + (uint32_t)OUT_STAGE_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };                  // leader only: both CTAs' loads landed
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };      // slot free (per CTA, by commit multicast)
  const uint32_t tfull_bar = bar_base + 8u * (2 * STAGES);                   // accumulator complete (per CTA)
  const uint32_t tempty_bar = bar_base + 8u * (2 * STAGES + 1);              // leader only: both epilogues drained
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + (size_t)STAGES * STAGE_BYTES + OUT_STAGE_BYTES + 8 * (2 * STAGES + 2));
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int num_m = (g.M + TILE_M - 1) / TILE_M, num_n = (g.N + TILE_N - 1) / TILE_N;
  const int num_tiles = num_m * num_n;
  // Work items: whole 256 x 256 tiles, except that a last partial wave which fills at most half of the pairs is
  // cut into 256 x 128 halves (two items per tile), so that it takes half a tile time instead of a whole one.
  const int full_items = (num_tiles / num_pairs) * num_pairs;
  const bool split_tail = num_tiles > full_items && 2 * (num_tiles - full_items) <= num_pairs;
  const int num_items = split_tail ? full_items + 2 * (num_tiles - full_items) : num_tiles;
  auto decode = [&](int item, int& mb, int& nb, int& nhalf) {      // nhalf: -1 whole tile, 0 / 1 left / right half
    int tile = item;
    nhalf = -1;
    if (split_tail && item >= full_items) { tile = full_items + ((item - full_items) >> 1); nhalf = (item - full_items) & 1; }
    // Tile order: groups of RASTER_M row tiles, inside a group the row tile runs fastest and the column tile sweeps
    // the whole width.  The pairs that run at the same time then cover RASTER_M x ~9 tiles: the group's A strips stay
    // in L2 for the whole sweep and every B strip is used by RASTER_M tiles back to back.  (With the row tile
    // running fastest over ALL rows, a wave touched every A strip once, and at long contractions - 2 MB per strip,
    // more than the L2 in all - each sweep of the columns read A from DRAM again: 2 GB instead of 165 MB at
    // 16384 x 4096 x 14336.)
    const int per_group = RASTER_M * num_n;
    const int grp = tile / per_group, within = tile - grp * per_group;
    const int first_m = grp * RASTER_M, gsz = min(RASTER_M, num_m - first_m);
    mb = first_m + within % gsz; nb = within / gsz;
  };
  const int num_fp4_kb = (g.K + BLOCK_K - 1) / BLOCK_K;
  const int num_kb = num_fp4_kb + g.extra_kb;
  const int sf_k_atoms = g.K / MMA_K;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(tfull_bar, 1);
    mbar_init(tempty_bar, 16);                                // 8 epilogue warps in each of the two CTAs
    *dead = 0;
    fence_barrier_init();
  }
  cluster_sync();
  if (warp == 1) tmem_alloc2(smem_u32(tmem_slot), TMEM_COLS);
  tc_fence_before();
  cluster_sync();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // everything above touched only this CTA's shared and tensor memory: it may overlap the previous kernel's tail
  metis_pdl_wait();

  if (warp == 0) {
    // ------------------------------- producer (both CTAs) -------------------
    // The leader announces the bytes of BOTH CTAs on its barrier; the other CTA only issues its loads.  A load
    // of the other CTA may land before the announcement: the count just goes negative for a moment, and the
    // phase cannot complete before the leader's arrival.  Every box is delivered in full (rows or K beyond
    // the matrix are filled with zeros), so the byte count of a stage does not depend on the position.
    // The whole warp walks the loop so that every address stays warp-uniform; one elected lane issues.
    {
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      for (int item = pair; item < num_items && ok; item += num_pairs) {
        int mb, nb, nhalf;
        decode(item, mb, nb, nhalf);
        // a half item multiplies 128 columns: each CTA supplies 64 rows of B, the first 64 of the same 128-row
        // box (the box and byte count of a stage stay what they are), and one scale slab serves both CTAs
        const int a_row = mb * TILE_M + (int)rank * 128;
        const int b_row = nhalf < 0 ? nb * TILE_N + (int)rank * 128 : nb * TILE_N + nhalf * 128 + (int)rank * 64;
        // a 128-row slab that lies wholly outside the matrix has all-zero codes; any valid slab's scales will
        // do for it, so the index is clamped instead of reading another tensor's bytes
        const int a_sf_tile = min(mb * 2 + (int)rank, (g.M + 127) / 128 - 1);
        const int b_sf_tile0 = min(nb * 2 + max(nhalf, 0), (g.N + 127) / 128 - 1), b_sf_tile1 = min(nb * 2 + 1, (g.N + 127) / 128 - 1);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(empty_bar(s), ph ^ 1u, g.dev_status, dead)) { ok = false; break; }
          if (elect_one()) {
            const uint32_t bar = map_to_rank(full_bar(s), 0u);
            if (kb >= num_fp4_kb) {                           // BF16 correction box: 128 rows x 64 elements each
              if (leader) mbar_expect_tx(full_bar(s), 2u * (uint32_t)(A_BYTES + B_BYTES));
              tma_load_2d_pair(a_addr(s), &map_l, (kb - num_fp4_kb) * 64, a_row, bar);
              tma_load_2d_pair(b_addr(s), &map_r, (kb - num_fp4_kb) * 64, b_row, bar);
            } else {
              if (leader) mbar_expect_tx(full_bar(s), 2u * (uint32_t)STAGE_BYTES);
              tma_load_2d_pair(a_addr(s), &map_a, kb * (BLOCK_K / 2), a_row, bar);
              tma_load_2d_pair(b_addr(s), &map_b, kb * (BLOCK_K / 2), b_row, bar);
              tma_load_2d_pair(sfa_addr(s), &map_sfa, 0, a_sf_tile * sf_k_atoms + kb * K_STEPS, bar);
              tma_load_2d_pair(sfb_addr(s), &map_sfb, 0, b_sf_tile0 * sf_k_atoms + kb * K_STEPS, bar);
              tma_load_2d_pair(sfb_addr(s) + K_STEPS * 512, &map_sfb, 0, b_sf_tile1 * sf_k_atoms + kb * K_STEPS, bar);
            }
          }
          __syncwarp();
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- scale copies + MMA issue (leader CTA only) ------------
    // tcgen05.cp and tcgen05.mma issued by one thread execute in order, so the scale atoms of a stage are
    // copied shared -> tensor memory right in front of the MMAs that read them.  Each ring stage has its own
    // scale columns; they are rewritten only after the MMAs of the stage's previous use have completed (the
    // stage is reloaded only after the commit that frees it).
    if (leader) {
      // the whole warp walks the loop (so that addresses and descriptors stay warp-uniform); one elected lane issues
      constexpr uint32_t idesc = make_idesc(TILE_M, TILE_N);
      int s = 0; uint32_t ph = 0;
      int it = 0;
      bool ok = true;
      for (int item = pair; item < num_items && ok; item += num_pairs, ++it) {
        const bool narrow = split_tail && item >= full_items;
        const uint32_t idesc_i = narrow ? make_idesc(TILE_M, TILE_N / 2) : idesc;
        const uint32_t idesc_xi = narrow ? make_idesc_bf16(TILE_M, TILE_N / 2) : make_idesc_bf16(TILE_M, TILE_N);
        if (!mbar_wait_cluster(tempty_bar, ((uint32_t)it & 1u) ^ 1u, g.dev_status, dead)) { ok = false; break; }
        tc_fence_after();
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait_cluster(full_bar(s), ph, g.dev_status, dead)) { ok = false; break; }
          tc_fence_after();
          if (elect_one()) {
            if (kb >= num_fp4_kb) {
#pragma unroll
              for (int k = 0; k < 4; ++k) {                   // 64 BF16 elements = four K=16 MMAs, 32 bytes apart
                const uint64_t a_desc = make_smem_desc(a_addr(s) + k * 32, 1024, SWIZZLE_128B);
                const uint64_t b_desc = make_smem_desc(b_addr(s) + k * 32, 1024, SWIZZLE_128B);
                tc_mma_bf16_2(tmem_base, a_desc, b_desc, idesc_xi, 1u);
              }
            } else {
              const int atoms = min(K_STEPS, sf_k_atoms - kb * K_STEPS);
              const uint32_t sfa_t = tmem_base + SF_COL0 + s * SF_COLS_PER_STAGE, sfb_t = sfa_t + 4 * K_STEPS;
              const uint64_t sfa_d = make_smem_desc(sfa_addr(s), 128, SWIZZLE_NONE), sfb_d = make_smem_desc(sfb_addr(s), 128, SWIZZLE_NONE);
              const uint64_t a_d = make_smem_desc(a_addr(s), 1024, SWIZZLE_128B), b_d = make_smem_desc(b_addr(s), 1024, SWIZZLE_128B);
              if (atoms == K_STEPS) {
#pragma unroll
                for (int k = 0; k < K_STEPS; ++k) {
                  tc_cp_sf2(sfa_t + 4 * k, sfa_d + (uint64_t)(k * 32));
                  tc_cp_sf2(sfb_t + 8 * k, sfb_d + (uint64_t)(k * 32));
                  if (!narrow) tc_cp_sf2(sfb_t + 8 * k + 4, sfb_d + (uint64_t)((K_STEPS + k) * 32));
                }
#pragma unroll
                for (int k = 0; k < K_STEPS; ++k)
                  tc_mma_nvf4_2(tmem_base, a_d + (uint64_t)(k * 2), b_d + (uint64_t)(k * 2), idesc_i, sfa_t + 4 * k, sfb_t + 8 * k, (kb | k) != 0 ? 1u : 0u);
              } else {
                for (int k = 0; k < atoms; ++k) {
                  tc_cp_sf2(sfa_t + 4 * k, sfa_d + (uint64_t)(k * 32));
                  tc_cp_sf2(sfb_t + 8 * k, sfb_d + (uint64_t)(k * 32));
                  if (!narrow) tc_cp_sf2(sfb_t + 8 * k + 4, sfb_d + (uint64_t)((K_STEPS + k) * 32));
                }
                for (int k = 0; k < atoms; ++k)
                  tc_mma_nvf4_2(tmem_base, a_d + (uint64_t)(k * 2), b_d + (uint64_t)(k * 2), idesc_i, sfa_t + 4 * k, sfb_t + 8 * k, (kb | k) != 0 ? 1u : 0u);
              }
            }
            tc_commit2(empty_bar(s), 3);                      // frees the slot in both CTAs
          }
          __syncwarp();
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        if (ok && elect_one()) tc_commit2(tfull_bar, 3);      // accumulator complete in both CTAs
        __syncwarp();
      }
    }
  } else if (warp >= 4) {
    // ------------------------------- epilogue (both CTAs) --------------------
    // Eight warps: warp w drains TMEM lane quarter w % 4, column half (w - 4) / 4.  A thread pulls its 128
    // accumulator columns into registers in one go and releases the accumulator at once, so the next tile's
    // MMAs start while this tile is still being scaled, converted and stored.
    const int quarter = warp & 3, half = (warp - 4) >> 2;
    const float alpha = (*g.a_ts) * (*g.b_ts);
    const uint64_t out_policy = l2_policy_evict_first();
    int it = 0;
    bool ok = true;
    for (int item = pair; item < num_items && ok; item += num_pairs, ++it) {
      int mb, nb, nhalf;
      decode(item, mb, nb, nhalf);
      if (!mbar_wait(tfull_bar, (uint32_t)it & 1u, g.dev_status, dead)) { ok = false; break; }
      tc_fence_after();
      const int row = mb * TILE_M + (int)rank * 128 + quarter * 32 + lane;
      uint32_t r[4][32];
      if (nhalf < 0) {
        const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(half * 128);
        tc_ld32_nowait(t_row, r[0]);
        tc_ld32_nowait(t_row + 32, r[1]);
        tc_ld32_nowait(t_row + 64, r[2]);
        tc_ld32_nowait(t_row + 96, r[3]);
      } else {                                                // 128 accumulator columns: 64 per warp
        const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(half * 64);
        tc_ld32_nowait(t_row, r[0]);
        tc_ld32_nowait(t_row + 32, r[1]);
      }
      tc_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote(tempty_bar, 0u);
      const int ncols_w = nhalf < 0 ? 128 : 64;                                   // columns this warp writes
      const int col_w = nb * TILE_N + (nhalf < 0 ? half * 128 : nhalf * 128 + half * 64);
      if (g.tma_store) {
        // Each lane converts its row into a 128-byte line of the warp's staging box (16-byte chunks XOR-swizzled
        // by the row, the layout of a 128-byte-swizzled tensor store), then one lane stores the 32-row box.
        // The box is reused as soon as the previous store has finished READING it.
        const uint32_t obuf = out_base + (uint32_t)(warp - 4) * 4096u + (uint32_t)lane * 128u;
        const int row_w = mb * TILE_M + (int)rank * 128 + quarter * 32;
        const uint32_t sw = (uint32_t)(lane & 7);
        if (g.d_dtype == METIS_BF16) {
#pragma unroll
          for (int st = 0; st < 2; ++st) {
            if (st * 64 < ncols_w) {
              if (lane == 0) bulk_wait_read_all();
              __syncwarp();
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                uint32_t w[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  const int e = (j & 3) * 8 + 2 * q;
                  const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(r[2 * st + (j >> 2)][e]) * alpha,
                                                                  __uint_as_float(r[2 * st + (j >> 2)][e + 1]) * alpha);
                  w[q] = *reinterpret_cast<const uint32_t*>(&hh);
                }
                st_shared_v4(obuf + (((uint32_t)j ^ sw) << 4), w[0], w[1], w[2], w[3]);
              }
              fence_proxy_async();
              __syncwarp();
              if (lane == 0 && row_w < g.M && col_w + st * 64 < g.N) {
                tma_store_2d_hint(&map_d, obuf, col_w + st * 64, row_w, out_policy);
                bulk_commit();
              }
            }
          }
        } else {
#pragma unroll
          for (int st = 0; st < 4; ++st) {
            if (st * 32 < ncols_w) {
              if (lane == 0) bulk_wait_read_all();
              __syncwarp();
#pragma unroll
              for (int j = 0; j < 8; ++j)
                st_shared_v4(obuf + (((uint32_t)j ^ sw) << 4),
                             __float_as_uint(__uint_as_float(r[st][4 * j]) * alpha), __float_as_uint(__uint_as_float(r[st][4 * j + 1]) * alpha),
                             __float_as_uint(__uint_as_float(r[st][4 * j + 2]) * alpha), __float_as_uint(__uint_as_float(r[st][4 * j + 3]) * alpha));
              fence_proxy_async();
              __syncwarp();
              if (lane == 0 && row_w < g.M && col_w + st * 32 < g.N) {
                tma_store_2d_hint(&map_d, obuf, col_w + st * 32, row_w, out_policy);
                bulk_commit();
              }
            }
          }
        }
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int col = col_w + c * 32;
          if (c * 32 < ncols_w && row < g.M && col < g.N) store_row_chunk(g, row, col, r[c], alpha);
        }
      }
    }
    if (lane == 0) bulk_wait_all();                           // the staging boxes must outlive their stores
  }

  // ------------------------------- teardown ---------------------------------
  tc_fence_before();
  __syncthreads();
  if (*dead) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  cluster_sync();                                             // the peer may still read this CTA's shared memory until here
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc2(tmem_base, TMEM_COLS);
  }
}

}  // namespace two_cta


metis_status_t make_codes_map(metis_context* ctx, CUtensorMap* map, const metis_nvfp4_t* t, int box_rows) {
  const cuuint64_t dims[2] = {(cuuint64_t)(t->k_len / 2), (cuuint64_t)t->rows};
  const cuuint64_t strides[1] = {(cuuint64_t)(t->k_len / 2)};
  const cuuint32_t box[2] = {(cuuint32_t)(BLOCK_K / 2), (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
      map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, t->codes, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
      CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? METIS_OK : METIS_ERR_CUDA;
}

// 2-D map over the tiled scale bytes of one NVFP4 tensor: one row per 512-byte atom (128 rows x 4 blocks),
// atoms of one 128-row slab consecutive along K; a box is the K_STEPS atoms of one K block.
metis_status_t make_scales_map(metis_context* ctx, CUtensorMap* map, const metis_nvfp4_t* t) {
  const cuuint64_t atoms = (cuuint64_t)metis_ceil_div(t->rows, 128) * (cuuint64_t)(t->k_len / MMA_K);
  const cuuint64_t dims[2] = {128, atoms};
  const cuuint64_t strides[1] = {512};
  const cuuint32_t box[2] = {128, (cuuint32_t)K_STEPS};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
      map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, t->scales, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
      CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? METIS_OK : METIS_ERR_CUDA;
}

template <int BLOCK_N>
metis_status_t launch(metis_context* ctx, const metis_nvfp4_t* a, const metis_nvfp4_t* b, void* d, int d_dtype,
                      int64_t ldd, cudaStream_t s) {
  using C = Cfg<BLOCK_N>;
  CUtensorMap map_a, map_b;
  METIS_TRY(make_codes_map(ctx, &map_a, a, BLOCK_M));
  METIS_TRY(make_codes_map(ctx, &map_b, b, BLOCK_N));
  GemmArgs g{};
  g.a_sf = a->scales; g.b_sf = b->scales; g.a_ts = a->tensor_scale; g.b_ts = b->tensor_scale;
  g.d = d; g.d_dtype = d_dtype; g.ldd = ldd;
  g.M = (int)a->rows; g.N = (int)b->rows; g.K = (int)a->k_len;
  g.dev_status = ctx->dev_status;
  const int tiles = (int)(metis_ceil_div(g.M, BLOCK_M) * metis_ceil_div(g.N, BLOCK_N));
  const int grid = tiles < ctx->sm_count ? tiles : ctx->sm_count;
  METIS_CUDA_TRY(metis_launch_pdl(gemm_nvfp4_kernel<BLOCK_N>, dim3(grid), dim3(NUM_THREADS), C::SMEM_BYTES, s, map_a, map_b, g)); METIS_COUNT_LAUNCH();
  return METIS_OK;
}

// 2-D map over a row-major BF16 matrix rows x kx (kx a multiple of 64), box 64 elements x 128 rows, 128-byte swizzle
metis_status_t make_bf16_map(metis_context* ctx, CUtensorMap* map, const void* ptr, int64_t rows, int64_t kx) {
  const cuuint64_t dims[2] = {(cuuint64_t)kx, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)(kx * 2)};
  const cuuint32_t box[2] = {64, 128};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
      map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
      CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? METIS_OK : METIS_ERR_CUDA;
}

// 2-D map over the output (row-major, leading dimension ldd): box = 32 rows x 128 bytes, 128-byte swizzle
metis_status_t make_out_map(metis_context* ctx, CUtensorMap* map, void* d, int d_dtype, int64_t rows, int64_t cols, int64_t ldd) {
  const cuuint64_t es = d_dtype == METIS_BF16 ? 2 : 4;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ldd * es};
  const cuuint32_t box[2] = {(cuuint32_t)(128 / es), 32};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
      map, d_dtype == METIS_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, d, dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? METIS_OK : METIS_ERR_CUDA;
}

metis_status_t launch_2cta(metis_context* ctx, const metis_nvfp4_t* a, const metis_nvfp4_t* b, void* d, int d_dtype,
                           int64_t ldd, const void* lx, const void* rx, int kx, cudaStream_t s) {
  CUtensorMap map_a, map_b, map_sfa, map_sfb, map_l, map_r, map_d;
  METIS_TRY(make_codes_map(ctx, &map_a, a, 128));
  METIS_TRY(make_codes_map(ctx, &map_b, b, 128));
  METIS_TRY(make_scales_map(ctx, &map_sfa, a));
  METIS_TRY(make_scales_map(ctx, &map_sfb, b));
  if (kx > 0) {
    METIS_TRY(make_bf16_map(ctx, &map_l, lx, a->rows, kx));
    METIS_TRY(make_bf16_map(ctx, &map_r, rx, b->rows, kx));
  } else {
    map_l = map_a; map_r = map_b;
  }
  GemmArgs g{};
  g.a_sf = a->scales; g.b_sf = b->scales; g.a_ts = a->tensor_scale; g.b_ts = b->tensor_scale;
  g.d = d; g.d_dtype = d_dtype; g.ldd = ldd;
  g.M = (int)a->rows; g.N = (int)b->rows; g.K = (int)a->k_len;
  g.dev_status = ctx->dev_status;
  g.extra_kb = kx / 64;
  // tensor stores need a 16-byte aligned base and row pitch; anything else takes the direct stores
  g.tma_store = metis_aligned16(d) && ((ldd * (d_dtype == METIS_BF16 ? 2 : 4)) % 16 == 0) ? 1 : 0;
  if (g.tma_store) METIS_TRY(make_out_map(ctx, &map_d, d, d_dtype, a->rows, b->rows, ldd));
  else map_d = map_a;
  const int tiles = (int)(metis_ceil_div(g.M, two_cta::TILE_M) * metis_ceil_div(g.N, two_cta::TILE_N));
  const int max_pairs = ctx->max_pairs;
  const int pairs = tiles < max_pairs ? tiles : max_pairs;
  METIS_CUDA_TRY(metis_launch_pdl(two_cta::gemm_nvfp4_2cta_kernel, dim3(2 * pairs), dim3(two_cta::NUM_THREADS), two_cta::SMEM_BYTES, s,
                                  map_a, map_b, map_sfa, map_sfb, map_l, map_r, map_d, g)); METIS_COUNT_LAUNCH();
  return METIS_OK;
}

}  // namespace

metis_status_t metis_gemm_set_attrs(metis_context* ctx) {
  METIS_CUDA_TRY(cudaFuncSetAttribute(gemm_nvfp4_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<128>::SMEM_BYTES));
  METIS_CUDA_TRY(cudaFuncSetAttribute(two_cta::gemm_nvfp4_2cta_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)two_cta::SMEM_BYTES));
  // how many 2-CTA clusters can be resident at once (an odd SM count inside a GPC leaves an SM unpaired)
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * (ctx->sm_count / 2)); cfg.blockDim = dim3(two_cta::NUM_THREADS);
  cfg.dynamicSmemBytes = two_cta::SMEM_BYTES;
  cudaLaunchAttribute at; at.id = cudaLaunchAttributeClusterDimension; at.val.clusterDim.x = 2; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
  cfg.attrs = &at; cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, two_cta::gemm_nvfp4_2cta_kernel, &cfg) != cudaSuccess || n <= 0) { n = ctx->sm_count / 2; (void)cudaGetLastError(); }
  ctx->max_pairs = n < ctx->sm_count / 2 ? n : ctx->sm_count / 2;
  return METIS_OK;
}

metis_status_t metis_launch_gemm_tc(metis_context* ctx, const metis_nvfp4_t* a, const metis_nvfp4_t* b, void* d,
                                    int d_dtype, int64_t ldd, cudaStream_t s) {
  if (a->rows == 0 || b->rows == 0) return METIS_OK;
  if (a->k_len != b->k_len || a->k_len % 64 != 0 || a->k_len <= 0) return METIS_ERR_SHAPE;
  if (a->sf_layout != METIS_SF_TILED || b->sf_layout != METIS_SF_TILED) return METIS_ERR_INVALID_ARG;
  if (!metis_aligned16(a->codes) || !metis_aligned16(b->codes) || !metis_aligned16(a->scales) || !metis_aligned16(b->scales))
    return METIS_ERR_ALIGNMENT;
  if (a->rows > INT32_MAX || b->rows > INT32_MAX || a->k_len > INT32_MAX) return METIS_ERR_SHAPE;
  if (a->rows >= 256 && b->rows >= 256) return launch_2cta(ctx, a, b, d, d_dtype, ldd, nullptr, nullptr, 0, s);
  return launch<128>(ctx, a, b, d, d_dtype, ldd, s);
}

bool metis_gemm_tc_can_fuse(const metis_nvfp4_t* a, const metis_nvfp4_t* b) {
  return a->rows >= 256 && b->rows >= 256;
}

// d = alpha * (a b^T) + alpha * (lx rx^T): lx (M x kx) and rx (N x kx) are row-major BF16, kx a multiple of 64.
metis_status_t metis_launch_gemm_tc_fused(metis_context* ctx, const metis_nvfp4_t* a, const metis_nvfp4_t* b, void* d,
                                          int d_dtype, int64_t ldd, const void* lx, const void* rx, int kx, cudaStream_t s) {
  if (!metis_gemm_tc_can_fuse(a, b) || kx <= 0 || kx % 64) return METIS_ERR_INVALID_ARG;
  if (a->k_len != b->k_len || a->k_len % 64 != 0 || a->k_len <= 0) return METIS_ERR_SHAPE;
  if (a->sf_layout != METIS_SF_TILED || b->sf_layout != METIS_SF_TILED) return METIS_ERR_INVALID_ARG;
  if (!metis_aligned16(a->codes) || !metis_aligned16(b->codes) || !metis_aligned16(a->scales) || !metis_aligned16(b->scales) ||
      !metis_aligned16(lx) || !metis_aligned16(rx))
    return METIS_ERR_ALIGNMENT;
  return launch_2cta(ctx, a, b, d, d_dtype, ldd, lx, rx, kx, s);
}
