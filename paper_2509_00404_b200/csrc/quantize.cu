// Tensor amax and the stand-alone NVFP4 quantizer (Section 2.3; value set of Appendix C.1).
#include "quant_tile.cuh"

namespace {

__global__ void amax_kernel(const void* __restrict__ x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                            float* __restrict__ out) {
  // |x| as a bit pattern: non-negative floats order like their bit patterns, infinity above every number and a
  // NaN above infinity, so a non-finite element survives the reduction (fmaxf would drop a NaN)
  uint32_t m = 0u;
  const int64_t n8 = cols / 8;
  if (dtype == METIS_BF16 && (cols & 7) == 0 && (ld & 7) == 0) {
    const int64_t total = rows * n8;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
      const int64_t r = i / n8, g = i - r * n8;
      const uint4 q = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(x) + r * ld + g * 8);
      const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        m = max(m, (w[j] << 16) & 0x7FFFFFFFu);
        m = max(m, w[j] & 0x7FFF0000u);
      }
    }
  } else {
    const int64_t total = rows * cols;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
      const int64_t r = i / cols, c = i - r * cols;
      m = max(m, __float_as_uint(metis_ld_as_float(x, dtype, r * ld + c)) & 0x7FFFFFFFu);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  __shared__ uint32_t wmax[32];
  if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x < 32) {
    m = threadIdx.x < (blockDim.x >> 5) ? wmax[threadIdx.x] : 0u;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if (threadIdx.x == 0) atomicMax(reinterpret_cast<unsigned int*>(out), m);
  }
}

// Stand-alone quantizer, 128 x 128 elements per CTA.
//  pass 1  every thread loads 16 consecutive elements of a row (32 bytes of BF16) - exactly one block along the
//          columns - and, if that orientation is wanted, encodes it in registers and writes its 8 code bytes
//          straight to global memory (8 threads = 64 contiguous bytes of a row); the values (BF16 or FP32) and
//          the stochastic-rounding draws go to shared memory for pass 2
//  pass 2  blocks along the rows: a thread reads 16 values down a column from shared memory, encodes them and
//          stages the bytes; the transposed codes and both scale tiles are then written out coalesced
constexpr int QK_CP = metis_qt::TILE / 2 + 8;                     // pitch of a staged row of row-block codes, bytes
template <typename T, bool SR>   // T = __nv_bfloat16 or float: element type of the shared tile (= input type)
__global__ void __launch_bounds__(metis_qt::THREADS, SR ? 3 : 4)
quantize_kernel(const T* __restrict__ x, int64_t ld, metis_qt::QuantParams p, const float* __restrict__ tscale_src,
                int tscale_is_amax, float* ts_out0, float* ts_out1) {
  using namespace metis_qt;
  // Shared-memory layouts, chosen so that every access of a warp touches each bank once.
  //   BF16 tile and draws: rows of 256 bytes = 16 chunks of 16 bytes, chunk ch stored at ch ^ (ch >> 3): the eight
  //     lanes of a quarter warp store the even (or odd) chunks of one row, which the swizzle spreads over all banks;
  //     pass 2 reads 32 consecutive words of a row, a permutation of the chunks inside one 128-byte window.
  //   FP32 tile: pitch 129 words.
  //   staged row-block codes: 72-byte rows; a BF16 thread owns two adjacent columns, so column c is staged in row
  //     (c >> 1) + 64 (c & 1) and the 32 lanes of a store write 32 consecutive rows (18 words apart: 16 lanes cover
  //     the 32 banks with their 8 bytes each).
  constexpr int TP = sizeof(T) == 2 ? TILE : TILE + 1;           // tile pitch in elements
  extern __shared__ __align__(16) unsigned char smem[];
  T* tile = reinterpret_cast<T*>(smem);                                        // [TILE][TP]
  uint8_t* codes_s = smem + ((sizeof(T) * TILE * TP + 15) & ~(size_t)15);      // [TILE][QK_CP] row-block codes
  uint8_t* sfr = codes_s + TILE * QK_CP;                                       // [TILE][8] scales of the row blocks
  uint8_t* sfc = sfr + TILE * 8;                                               // [TILE][8] scales of the column blocks
  float* r_tab = reinterpret_cast<float*>(sfc + TILE * 8);                     // multiplier per scale byte
  uint16_t* rnd = reinterpret_cast<uint16_t*>(r_tab + R_TABLE);                // [TILE][TILE] draws (SR only)

  auto staged_row = [](int c) { return sizeof(T) == 2 ? (c >> 1) + 64 * (c & 1) : c; };
  // Scale bytes of the tile, from their staging area [stored row][8] to global memory.  The four blocks of a 64-element
  // K group are adjacent in both layouts, so they go out as one word per thread (256 words per tile and orientation;
  // in the tiled layout consecutive threads write consecutive words of a 512-byte atom, and blocks or rows of the atom
  // that lie outside the matrix are its zero padding); an unaligned linear layout takes the byte path.
  auto write_scales = [&](uint8_t* dst, int64_t extent, int layout, int64_t bpr, const uint8_t* src, bool staged, int v_rows, int v_k, int64_t g_row0, int64_t g_blk0) {
    (void)extent;
    const bool tiled = layout == METIS_SF_TILED;
    if ((tiled || (bpr & 3) == 0) && (reinterpret_cast<uintptr_t>(dst) & 3) == 0) {
      const int i = threadIdx.x;                                          // THREADS == 2 * TILE words
      const int atom = tiled ? i >> 7 : i & 1;
      const int r = tiled ? ((i & 127) >> 2) + 32 * (i & 3) : i >> 1;
      if (atom * 64 < v_k && (r < v_rows || tiled)) {
        const uint32_t w = r < v_rows ? *reinterpret_cast<const uint32_t*>(src + (staged ? staged_row(r) : r) * 8 + atom * 4) : 0u;
        const int64_t off = metis_sf_offset(g_row0 + r, g_blk0 + atom * 4, bpr, layout);
        METIS_DBG_GUARD(p.dbg, off, 4, extent) *reinterpret_cast<uint32_t*>(dst + off) = w;
      }
    } else {
      for (int i = threadIdx.x; i < TILE * 8; i += THREADS) {
        int r, b;
        if (tiled) { const int atom = i >> 9, w = i & 511; r = (w >> 4) + 32 * ((w >> 2) & 3); b = atom * 4 + (w & 3); }
        else { r = i >> 3; b = i & 7; }
        if (b * 16 < v_k && (r < v_rows || tiled))
          METIS_DBG_GUARD(p.dbg, metis_sf_offset(g_row0 + r, g_blk0 + b, bpr, layout), 1, extent) dst[metis_sf_offset(g_row0 + r, g_blk0 + b, bpr, layout)] = r < v_rows ? src[(staged ? staged_row(r) : r) * 8 + b] : (uint8_t)0;
      }
    }
  };
  const int tid = threadIdx.x;
  const int64_t row0 = (int64_t)blockIdx.y * TILE, col0 = (int64_t)blockIdx.x * TILE;
  const float s_T = tscale_is_amax ? metis_tensor_scale(*tscale_src) : *tscale_src;
  const float six_s_T = __fmul_rn(6.0f, s_T);
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) {
    if (ts_out0 != nullptr && ts_out0 != tscale_src) *ts_out0 = s_T;
    if (ts_out1 != nullptr && ts_out1 != tscale_src) *ts_out1 = s_T;
  }
  constexpr bool sr = SR;
  fill_r_table(r_tab, s_T, tid, THREADS);
  const bool want_c = p.c_codes != nullptr, want_r = p.r_codes != nullptr;
  const int vrows = (int)min((int64_t)TILE, p.rows - row0), vcols = (int)min((int64_t)TILE, p.cols - col0);
  const bool fast_draws = p.e_stride_c == 1 && (p.e_stride_r & 7) == 0;
  const bool wide_ld = sizeof(T) == 2 && (ld & 15) == 0 && (reinterpret_cast<uintptr_t>(x) & 31) == 0;   // 32-byte aligned blocks

  // ---- pass 1 ----
  // all global loads of the tile are issued before the first block is encoded: 128 bytes per thread in flight
  uint4 raw[sizeof(T) == 2 ? 8 : 1];
  if (sizeof(T) == 2) {
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int b = tid & 7, r = (tid >> 3) + 32 * it;
      raw[2 * it] = raw[2 * it + 1] = make_uint4(0u, 0u, 0u, 0u);
      if (r < vrows && b * 16 < vcols) {
        const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(x) + (row0 + r) * ld + col0 + b * 16);
        if (wide_ld) {                                     // one 32-byte load per block: consecutive lanes, consecutive 32 bytes
          asm volatile("ld.global.nc.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                       : "=r"(raw[2 * it].x), "=r"(raw[2 * it].y), "=r"(raw[2 * it].z), "=r"(raw[2 * it].w),
                         "=r"(raw[2 * it + 1].x), "=r"(raw[2 * it + 1].y), "=r"(raw[2 * it + 1].z), "=r"(raw[2 * it + 1].w)
                       : "l"(src));
        } else {
          raw[2 * it] = src[0]; raw[2 * it + 1] = src[1];
        }
      }
    }
  }
  __syncthreads();                                         // multiplier table complete (the tile loads are in flight)
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int b = tid & 7, r = (tid >> 3) + 32 * it;
    const int64_t gr = row0 + r, gc = col0 + b * 16;
    const bool in = r < vrows && b * 16 < vcols;
    float v[16];
    uint32_t u[16];
    if (sizeof(T) == 2) {
      const uint4 q0 = raw[sizeof(T) == 2 ? 2 * it : 0], q1 = raw[sizeof(T) == 2 ? 2 * it + 1 : 0];
      const uint32_t w[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
      for (int j = 0; j < 8; ++j) { v[2 * j] = __uint_as_float(w[j] << 16); v[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u); }
      if (want_r) {
        uint4* trow = reinterpret_cast<uint4*>(smem + r * 256);
        trow[(2 * b) ^ (b >> 2)] = q0;
        trow[(2 * b + 1) ^ (b >> 2)] = q1;
      }
    } else if (in) {
      const float4* src = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(x) + gr * ld + gc);
#pragma unroll
      for (int j = 0; j < 4; ++j) { const float4 q = src[j]; v[4 * j] = q.x; v[4 * j + 1] = q.y; v[4 * j + 2] = q.z; v[4 * j + 3] = q.w; }
      if (want_r) {
        float* dst = reinterpret_cast<float*>(tile) + r * TP + b * 16;
#pragma unroll
        for (int j = 0; j < 16; ++j) dst[j] = v[j];
      }
    } else {
#pragma unroll
      for (int j = 0; j < 16; ++j) v[j] = 0.0f;
      if (want_r) {
        T* dst = tile + r * TP + b * 16;
#pragma unroll
        for (int j = 0; j < 16; ++j) dst[j] = T(0.0f);
      }
    }
    if (sr) {
      if (fast_draws && in) {
        const uint64_t e = (uint64_t)gr * (uint64_t)p.e_stride_r + (uint64_t)gc;
        const uint4 w0 = metis_philox_block(e >> 3, p.seed, p.stream_id), w1 = metis_philox_block((e >> 3) + 1, p.seed, p.stream_id);
        const uint32_t ww[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) { u[2 * j] = ww[j] << 16; u[2 * j + 1] = ww[j] & 0xFFFF0000u; }   // thresholds: draw << 16
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          u[j] = in ? metis_draw_u16((uint64_t)gr * (uint64_t)p.e_stride_r + (uint64_t)(gc + j) * (uint64_t)p.e_stride_c, p.seed, p.stream_id) << 16 : 0u;
      }
      if (want_r) {
        if (sizeof(T) == 2) {
          uint4* drow = reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(rnd) + r * 256);
          drow[(2 * b) ^ (b >> 2)] = make_uint4((u[0] >> 16) | u[1], (u[2] >> 16) | u[3], (u[4] >> 16) | u[5], (u[6] >> 16) | u[7]);
          drow[(2 * b + 1) ^ (b >> 2)] = make_uint4((u[8] >> 16) | u[9], (u[10] >> 16) | u[11], (u[12] >> 16) | u[13], (u[14] >> 16) | u[15]);
        } else {
          uint32_t* dst = reinterpret_cast<uint32_t*>(rnd + r * TILE + b * 16);
#pragma unroll
          for (int j = 0; j < 8; ++j) dst[j] = (u[2 * j] >> 16) | u[2 * j + 1];
        }
      }
    }
    if (want_c) {
      uint32_t packed[2];
      const uint32_t byte = encode_block_tab(v, u, sr, six_s_T, r_tab, packed);
      if (in) METIS_DBG_GUARD(p.dbg, gr * (p.cols / 2) + gc / 2, 8, p.rows * p.cols / 2) *reinterpret_cast<uint2*>(p.c_codes + gr * (p.cols / 2) + gc / 2) = make_uint2(packed[0], packed[1]);
      sfc[r * 8 + b] = in ? (uint8_t)byte : (uint8_t)0;
    }
  }
  __syncthreads();
  // ---- pass 2 ----
  if (want_r) {
    if (sizeof(T) == 2) {
      // BF16 tile: a thread takes two adjacent columns (one 32-bit shared load per row) and four of the eight
      // row blocks, i.e. eight blocks in two rounds of four
#pragma unroll 1
      for (int it = 0; it < 2; ++it) {
        const int wd = tid & 63, b = (tid >> 6) + 4 * it;         // columns 2 wd, 2 wd + 1: word wd of a tile row
        const int pw = ((((wd >> 2) ^ (wd >> 5)) << 2) | (wd & 3));    // its swizzled position
        float v0[16], v1[16];
        uint32_t u0[16], u1[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const uint32_t w = reinterpret_cast<const uint32_t*>(smem)[(b * 16 + i) * 64 + pw];
          v0[i] = __uint_as_float(w << 16); v1[i] = __uint_as_float(w & 0xFFFF0000u);
        }
        if (sr) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const uint32_t w = reinterpret_cast<const uint32_t*>(rnd)[(b * 16 + i) * 64 + pw];
            u0[i] = w << 16; u1[i] = w & 0xFFFF0000u;
          }
        }
        uint32_t packed[2];
        uint32_t byte = encode_block_tab(v0, u0, sr, six_s_T, r_tab, packed);
        *reinterpret_cast<uint2*>(codes_s + wd * QK_CP + b * 8) = make_uint2(packed[0], packed[1]);
        sfr[wd * 8 + b] = (uint8_t)byte;
        byte = encode_block_tab(v1, u1, sr, six_s_T, r_tab, packed);
        *reinterpret_cast<uint2*>(codes_s + (64 + wd) * QK_CP + b * 8) = make_uint2(packed[0], packed[1]);
        sfr[(64 + wd) * 8 + b] = (uint8_t)byte;
      }
    } else {
#pragma unroll 1
    for (int it = 0; it < 4; ++it) {
      const int c = tid & 127, b = (tid >> 7) + 2 * it;
      float v[16];
      uint32_t u[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) v[i] = reinterpret_cast<const float*>(tile)[(b * 16 + i) * TP + c];
      if (sr) {
#pragma unroll
        for (int i = 0; i < 16; ++i) u[i] = (uint32_t)rnd[(b * 16 + i) * TILE + c] << 16;
      }
      uint32_t packed[2];
      const uint32_t byte = encode_block_tab(v, u, sr, six_s_T, r_tab, packed);
      *reinterpret_cast<uint2*>(codes_s + c * QK_CP + b * 8) = make_uint2(packed[0], packed[1]);
      sfr[c * 8 + b] = (uint8_t)byte;
    }
    }
    __syncthreads();
    const int64_t kbytes = p.rows / 2;
    for (int i = tid; i < TILE * 8; i += THREADS) {
      const int c = i >> 3, seg = i & 7;
      if (c < vcols && seg * 16 < vrows)
        METIS_DBG_GUARD(p.dbg, (col0 + c) * kbytes + row0 / 2 + seg * 8, 8, p.rows * p.cols / 2) *reinterpret_cast<uint2*>(p.r_codes + (col0 + c) * kbytes + row0 / 2 + seg * 8) = *reinterpret_cast<const uint2*>(codes_s + staged_row(c) * QK_CP + seg * 8);
    }
    write_scales(p.r_scales, p.r_sf_bytes, p.r_layout, p.rows / 16, sfr, true, vcols, vrows, col0, row0 / 16);
  }
  if (want_c) write_scales(p.c_scales, p.c_sf_bytes, p.c_layout, p.cols / 16, sfc, false, vrows, vcols, row0, col0 / 16);
}

template <typename T>
constexpr size_t quantize_smem(bool sr) {
  return ((sizeof(T) * metis_qt::TILE * (metis_qt::TILE + (sizeof(T) == 2 ? 0 : 1)) + 15) & ~(size_t)15) + metis_qt::TILE * QK_CP +
         2 * metis_qt::TILE * 8 + sizeof(float) * metis_qt::R_TABLE + (sr ? sizeof(uint16_t) * metis_qt::TILE * metis_qt::TILE : 0);
}

}  // namespace

metis_status_t metis_quantize_set_attrs() {
  using namespace metis_qt;
  METIS_CUDA_TRY(cudaFuncSetAttribute(quantize_kernel<__nv_bfloat16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)quantize_smem<__nv_bfloat16>(true)));
  METIS_CUDA_TRY(cudaFuncSetAttribute(quantize_kernel<float, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)quantize_smem<float>(true)));
  METIS_CUDA_TRY(cudaFuncSetAttribute(quantize_kernel<__nv_bfloat16, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)quantize_smem<__nv_bfloat16>(false)));
  METIS_CUDA_TRY(cudaFuncSetAttribute(quantize_kernel<float, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)quantize_smem<float>(false)));
  return METIS_OK;
}

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


// Few long rows (the transposed split factors: k x len FP32, blocks along the contiguous dimension only): one
// thread per block of 16, no tiles, no shared memory.  Threads beyond `rows` inside the last 128-row slab of the
// tiled scale layout write zero scale bytes.
__device__ __forceinline__ void rowblocks_body(const float* __restrict__ x, int64_t ld, const metis_qt::QuantParams& p,
                                               const float* __restrict__ tscale_src, int tscale_is_amax, float* ts_out) {
  const int64_t bpr = p.cols / 16;
  const int64_t rows_pad = p.c_layout == METIS_SF_TILED ? (p.rows + 127) / 128 * 128 : p.rows;
  const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (idx >= rows_pad * bpr) return;
  const int64_t r = idx / bpr, b = idx % bpr;
  if (r >= p.rows) { p.c_scales[metis_sf_offset(r, b, bpr, p.c_layout)] = 0; return; }
  const float s_T = tscale_is_amax ? metis_tensor_scale(*tscale_src) : *tscale_src;
  if (idx == 0 && ts_out != nullptr) *ts_out = s_T;
  const bool sr = p.rounding == METIS_ROUND_SR;
  float v[16];
  uint32_t u[16];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float4 q = *reinterpret_cast<const float4*>(x + r * ld + b * 16 + i * 4);
    v[4 * i] = q.x; v[4 * i + 1] = q.y; v[4 * i + 2] = q.z; v[4 * i + 3] = q.w;
  }
  if (sr) {
    if (p.e_stride_c == 1 && (p.e_stride_r & 7) == 0) {
      const uint64_t e0 = (uint64_t)r * (uint64_t)p.e_stride_r + (uint64_t)b * 16u;
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2) {
        const uint4 w = metis_philox_block((e0 >> 3) + h2, p.seed, p.stream_id);
#pragma unroll
        for (uint32_t hh = 0; hh < 8; ++hh) u[8 * h2 + hh] = metis_u16_of(w, hh);
      }
    } else {
#pragma unroll
      for (int i = 0; i < 16; ++i)
        u[i] = metis_draw_u16((uint64_t)r * (uint64_t)p.e_stride_r + (uint64_t)(b * 16 + i) * (uint64_t)p.e_stride_c, p.seed, p.stream_id);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i) u[i] = 0u;
  }
  uint32_t packed[2];
  const uint32_t byte = metis_qt::encode_block(v, u, sr, s_T, __fmul_rn(6.0f, s_T), packed);
  *reinterpret_cast<uint2*>(p.c_codes + r * (p.cols / 2) + b * 8) = make_uint2(packed[0], packed[1]);
  p.c_scales[metis_sf_offset(r, b, bpr, p.c_layout)] = (uint8_t)byte;
}

__global__ void __launch_bounds__(256)
quantize_rowblocks_kernel(const float* __restrict__ x, int64_t ld, metis_qt::QuantParams p, const float* __restrict__ tscale_src,
                          int tscale_is_amax, float* ts_out) {
  rowblocks_body(x, ld, p, tscale_src, tscale_is_amax, ts_out);
}

// ------------------------------------------------------------------------------------------------
// Comparison recipe of Section 4: random Hadamard transform of every 16-block along the columns, then NVFP4.
// y = H16 (s * x) / 4, four butterfly stages in binary32 (distance 1, 2, 4, 8; (a, b) -> (a + b, a - b)), signs
// s from bit 15 of the Philox draw of the column index (stream METIS_STREAM_SIGNS).
__device__ __forceinline__ void rht_block(const void* __restrict__ x, int dtype, int64_t ld, int64_t r, int64_t b, uint64_t seed, float (&v)[16]) {
  const uint4 w0 = metis_philox_block((uint64_t)b * 2, seed, METIS_STREAM_SIGNS), w1 = metis_philox_block((uint64_t)b * 2 + 1, seed, METIS_STREAM_SIGNS);
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const float xv = metis_ld_as_float(x, dtype, r * ld + b * 16 + i);
    const uint32_t u = metis_u16_of(i < 8 ? w0 : w1, (uint32_t)(i & 7));
    v[i] = (u & 0x8000u) ? -xv : xv;
  }
#pragma unroll
  for (int h = 1; h < 16; h <<= 1) {
#pragma unroll
    for (int i = 0; i < 16; ++i)
      if ((i & h) == 0) { const float a = v[i], c = v[i + h]; v[i] = __fadd_rn(a, c); v[i + h] = __fsub_rn(a, c); }
  }
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __fmul_rn(v[i], 0.25f);
}

__global__ void __launch_bounds__(256)
rht_amax_kernel(const void* __restrict__ x, int dtype, int64_t rows, int64_t cols, int64_t ld, uint64_t seed, float* __restrict__ amax_out) {
  const int64_t bpr = cols / 16;
  const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
  uint32_t m = 0u;
  if (idx < rows * bpr) {
    float v[16];
    rht_block(x, dtype, ld, idx / bpr, idx % bpr, seed, v);
#pragma unroll
    for (int i = 0; i < 16; ++i) m = max(m, __float_as_uint(v[i]) & 0x7FFFFFFFu);      // ordered bit patterns: a NaN survives
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  if ((threadIdx.x & 31) == 0 && m) atomicMax(reinterpret_cast<unsigned int*>(amax_out), m);
}

__global__ void __launch_bounds__(256)
rht_quantize_kernel(const void* __restrict__ x, int dtype, int64_t ld, metis_qt::QuantParams p, const float* __restrict__ amax, float* ts_out) {
  const int64_t bpr = p.cols / 16;
  const int64_t rows_pad = p.c_layout == METIS_SF_TILED ? (p.rows + 127) / 128 * 128 : p.rows;
  const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (idx >= rows_pad * bpr) return;
  const int64_t r = idx / bpr, b = idx % bpr;
  if (r >= p.rows) { p.c_scales[metis_sf_offset(r, b, bpr, p.c_layout)] = 0; return; }
  const float s_T = metis_tensor_scale(*amax);
  if (idx == 0) *ts_out = s_T;
  const bool sr = p.rounding == METIS_ROUND_SR;
  float v[16];
  uint32_t u[16];
  rht_block(x, dtype, ld, r, b, p.seed, v);
#pragma unroll
  for (int i = 0; i < 16; ++i) u[i] = 0u;
  if (sr) {
    const uint64_t e0 = (uint64_t)r * (uint64_t)p.cols + (uint64_t)b * 16u;
#pragma unroll
    for (int h2 = 0; h2 < 2; ++h2) {
      const uint4 w = metis_philox_block((e0 >> 3) + h2, p.seed, p.stream_id);
#pragma unroll
      for (uint32_t hh = 0; hh < 8; ++hh) u[8 * h2 + hh] = metis_u16_of(w, hh);
    }
  }
  uint32_t packed[2];
  const uint32_t byte = metis_qt::encode_block(v, u, sr, s_T, __fmul_rn(6.0f, s_T), packed);
  *reinterpret_cast<uint2*>(p.c_codes + r * (p.cols / 2) + b * 8) = make_uint2(packed[0], packed[1]);
  p.c_scales[metis_sf_offset(r, b, bpr, p.c_layout)] = (uint8_t)byte;
}

metis_status_t metis_launch_quantize_rht(metis_context* ctx, const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, int rounding, uint64_t seed,
                                         uint32_t stream_id, const metis_nvfp4_t* out, float* amax_ws, cudaStream_t s) {
  using namespace metis_qt;
  QuantParams p{};
  p.rows = rows; p.cols = cols; p.rounding = rounding; p.seed = seed; p.stream_id = stream_id; p.e_stride_r = cols; p.e_stride_c = 1;
  p.c_codes = out->codes; p.c_scales = out->scales; p.c_layout = out->sf_layout;
  METIS_CUDA_TRY(cudaMemsetAsync(amax_ws, 0, sizeof(float), s));
  const int64_t bpr = cols / 16;
  rht_amax_kernel<<<(unsigned)metis_ceil_div(rows * bpr, 256), 256, 0, s>>>(x, dtype, rows, cols, ld, seed, amax_ws); METIS_COUNT_LAUNCH();
  METIS_TRY(metis_launch_amax_check(ctx, amax_ws, s));
  const int64_t rows_pad = p.c_layout == METIS_SF_TILED ? (rows + 127) / 128 * 128 : rows;
  rht_quantize_kernel<<<(unsigned)metis_ceil_div(rows_pad * bpr, 256), 256, 0, s>>>(x, dtype, ld, p, amax_ws, out->tensor_scale); METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  return METIS_OK;
}

// two factor tensors in one launch (blockIdx.y selects): the left and right factors of a decomposition
struct RowblocksJob { const float* x; int64_t ld; metis_qt::QuantParams p; const float* tscale_src; float* ts_out; };
__global__ void __launch_bounds__(256)
quantize_rowblocks_pair_kernel(RowblocksJob a, RowblocksJob b) {
  const RowblocksJob& j = blockIdx.y == 0 ? a : b;
  rowblocks_body(j.x, j.ld, j.p, j.tscale_src, 1, j.ts_out);
}

metis_status_t metis_launch_quantize(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, int rounding,
                                     uint64_t seed, uint32_t stream_id, int64_t e_stride_r, int64_t e_stride_c,
                                     const float* tscale_src, int tscale_is_amax, const metis_nvfp4_t* by_cols,
                                     const metis_nvfp4_t* by_rows, cudaStream_t s, uint32_t* dbg_status) {
  using namespace metis_qt;
  if (rows == 0 || cols == 0) return METIS_OK;
  // vector loads of 16 elements per thread: the rows must start on 16-byte boundaries
  if (cols % 16 || (dtype == METIS_BF16 ? ld % 8 : ld % 4)) return METIS_ERR_ALIGNMENT;
  QuantParams p{};
  p.rows = rows; p.cols = cols; p.rounding = rounding; p.seed = seed; p.stream_id = stream_id;
  p.e_stride_r = e_stride_r; p.e_stride_c = e_stride_c;
  if (by_cols) { p.c_codes = by_cols->codes; p.c_scales = by_cols->scales; p.c_layout = by_cols->sf_layout; p.c_sf_bytes = (int64_t)metis_sf_bytes(rows, cols, p.c_layout); }
  if (by_rows) { p.r_codes = by_rows->codes; p.r_scales = by_rows->scales; p.r_layout = by_rows->sf_layout; p.r_sf_bytes = (int64_t)metis_sf_bytes(cols, rows, p.r_layout); }
  p.dbg = dbg_status;
  if (dtype == METIS_FP32 && by_cols && !by_rows && rows <= 64) {
    const int64_t rows_pad = p.c_layout == METIS_SF_TILED ? (rows + 127) / 128 * 128 : rows;
    quantize_rowblocks_kernel<<<(unsigned)metis_ceil_div(rows_pad * (cols / 16), 256), 256, 0, s>>>(
        reinterpret_cast<const float*>(x), ld, p, tscale_src, tscale_is_amax, by_cols->tensor_scale); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(cudaGetLastError());
    return METIS_OK;
  }
  const bool sr = rounding == METIS_ROUND_SR;
  dim3 grid((unsigned)metis_ceil_div(cols, TILE), (unsigned)metis_ceil_div(rows, TILE));
  float* t0 = by_cols ? by_cols->tensor_scale : nullptr; float* t1 = by_rows ? by_rows->tensor_scale : nullptr;
  if (dtype == METIS_BF16) {
    const __nv_bfloat16* xb = reinterpret_cast<const __nv_bfloat16*>(x);
    if (sr) quantize_kernel<__nv_bfloat16, true><<<grid, THREADS, quantize_smem<__nv_bfloat16>(true), s>>>(xb, ld, p, tscale_src, tscale_is_amax, t0, t1);
    else quantize_kernel<__nv_bfloat16, false><<<grid, THREADS, quantize_smem<__nv_bfloat16>(false), s>>>(xb, ld, p, tscale_src, tscale_is_amax, t0, t1);
  } else {
    const float* xf = reinterpret_cast<const float*>(x);
    if (sr) quantize_kernel<float, true><<<grid, THREADS, quantize_smem<float>(true), s>>>(xf, ld, p, tscale_src, tscale_is_amax, t0, t1);
    else quantize_kernel<float, false><<<grid, THREADS, quantize_smem<float>(false), s>>>(xf, ld, p, tscale_src, tscale_is_amax, t0, t1);
  }
  METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  return METIS_OK;
}

// The two FP32 factor tensors of a decomposition (k x rows and k x cols, k <= 64, blocks along the long dimension,
// tensor scale from each tensor's own amax) in one launch.
metis_status_t metis_launch_quantize_factors(const float* left, int64_t rows, const float* right, int64_t cols, int k, int rounding,
                                             uint64_t seed, const float* amax_left, const float* amax_right,
                                             const metis_nvfp4_t* lq, const metis_nvfp4_t* rq, cudaStream_t s) {
  using namespace metis_qt;
  if (k <= 0 || k > 256 || rows % 16 || cols % 16) return METIS_ERR_SHAPE;
  RowblocksJob a{}, b{};
  a.x = left; a.ld = rows; a.tscale_src = amax_left; a.ts_out = lq->tensor_scale;
  a.p.rows = k; a.p.cols = rows; a.p.rounding = rounding; a.p.seed = seed; a.p.stream_id = METIS_STREAM_LEFT;
  a.p.e_stride_r = rows; a.p.e_stride_c = 1; a.p.c_codes = lq->codes; a.p.c_scales = lq->scales; a.p.c_layout = lq->sf_layout;
  b.x = right; b.ld = cols; b.tscale_src = amax_right; b.ts_out = rq->tensor_scale;
  b.p.rows = k; b.p.cols = cols; b.p.rounding = rounding; b.p.seed = seed; b.p.stream_id = METIS_STREAM_RIGHT;
  b.p.e_stride_r = cols; b.p.e_stride_c = 1; b.p.c_codes = rq->codes; b.p.c_scales = rq->scales; b.p.c_layout = rq->sf_layout;
  const int64_t pad_a = a.p.c_layout == METIS_SF_TILED ? (k + 127) / 128 * 128 : k, pad_b = b.p.c_layout == METIS_SF_TILED ? (k + 127) / 128 * 128 : k;
  const int64_t work_a = pad_a * (rows / 16), work_b = pad_b * (cols / 16);
  const unsigned gx = (unsigned)metis_ceil_div(work_a > work_b ? work_a : work_b, 256);
  quantize_rowblocks_pair_kernel<<<dim3(gx, 2), 256, 0, s>>>(a, b); METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  return METIS_OK;
}
