// NVFP4 quantization of a 128 x 128 FP32 tile held in shared memory, in one or both block
// orientations (Section 2.3).  Used by the stand-alone quantizer and by the fused
// residual -> quantizer kernel of the split, so both produce identical codes for identical values.
#pragma once
#include "common.cuh"

namespace metis_qt {

constexpr int TILE = 128;
constexpr int PITCH = 132;            // floats per shared-memory tile row (conflict-free float4 access by row)
constexpr int THREADS = 256;

struct QuantParams {
  int64_t rows, cols;                 // source matrix extent
  int rounding;
  uint64_t seed;
  uint32_t stream_id;
  int64_t e_stride_r, e_stride_c;     // logical element index = r*e_stride_r + c*e_stride_c (keys the SR draw)
  // outputs (either may be absent: codes == nullptr)
  uint8_t* c_codes; uint8_t* c_scales; int c_layout;    // blocks along columns: stored rows x cols
  uint8_t* r_codes; uint8_t* r_scales; int r_layout;    // blocks along rows:    stored cols x rows
  // debug build: extents of the scale buffers (the code buffers hold rows * cols / 2 bytes) and the status word
  int64_t c_sf_bytes, r_sf_bytes;
  uint32_t* dbg;
};

struct __align__(16) Stage {
  uint8_t codes[TILE][TILE / 2];      // 8 KiB: [stored row in tile][packed k]
  uint8_t sf[TILE][TILE / 16];        // 1 KiB: [stored row in tile][block]
};

// Encodes one block of 16 values; returns the scale byte, writes 8 code bytes.
__device__ __forceinline__ uint32_t encode_block(const float (&v)[16], const uint32_t (&u)[16], bool sr, float s_T,
                                                 float six_s_T, uint32_t (&packed)[2]) {
  // maximum by a tree: four dependent steps instead of sixteen
  float m8[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) m8[i] = fmaxf(fabsf(v[i]), fabsf(v[i + 8]));
  const float amax = fmaxf(fmaxf(fmaxf(m8[0], m8[4]), fmaxf(m8[1], m8[5])), fmaxf(fmaxf(m8[2], m8[6]), fmaxf(m8[3], m8[7])));
  float t = fminf(__fdiv_rn(amax, six_s_T), 448.0f);
  float sb;
  const uint32_t byte = metis_e4m3_ceil(t, &sb);
  const float r = sb == 0.0f ? 0.0f : __fdiv_rn(1.0f, __fmul_rn(sb, s_T));
  packed[0] = packed[1] = 0u;
  if (!sr) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint32_t b = metis_e2m1x2_rne(__fmul_rn(v[2 * i], r), __fmul_rn(v[2 * i + 1], r));
      packed[i >> 2] |= b << (8 * (i & 3));
    }
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const uint32_t c = metis_e2m1_sr(__fmul_rn(v[i], r), u[i]);
      packed[i >> 3] |= c << (4 * (i & 7));
    }
  }
  return byte;
}

// The element multiplier r = 1 / (E4M3(byte) * s_T) depends only on the block's scale byte and the tensor scale, so a
// kernel can evaluate the defined operations once per byte and look the result up per block (0 for byte 0).
constexpr int R_TABLE = 128;
__device__ __forceinline__ void fill_r_table(float* tab, float s_T, int tid, int nthreads) {
  for (int b = tid; b < R_TABLE; b += nthreads)
    tab[b] = (b == 0 || b == 127) ? 0.0f : __fdiv_rn(1.0f, __fmul_rn(metis_e4m3_value((uint32_t)b), s_T));
}

// four round-to-nearest-even code bytes (eight values) packed into one word
__device__ __forceinline__ uint32_t e2m1x8_rne(float a0, float a1, float a2, float a3, float a4, float a5, float a6, float a7) {
  uint32_t w;
  asm("{ .reg .b8 t0, t1, t2, t3;\n"
      "cvt.rn.satfinite.e2m1x2.f32 t0, %2, %1;\n"
      "cvt.rn.satfinite.e2m1x2.f32 t1, %4, %3;\n"
      "cvt.rn.satfinite.e2m1x2.f32 t2, %6, %5;\n"
      "cvt.rn.satfinite.e2m1x2.f32 t3, %8, %7;\n"
      "mov.b32 %0, {t0, t1, t2, t3}; }"
      : "=r"(w) : "f"(a0), "f"(a1), "f"(a2), "f"(a3), "f"(a4), "f"(a5), "f"(a6), "f"(a7));
  return w;
}

// Eight stochastically rounded codes in one word; thr[i] = draw_i << 16.  The same decision as metis_e2m1_sr,
// arranged for the instruction mix of the SM (integer logic and compares issue at half the FP32 / IMAD rate):
//   b = max(a, RU(a/2 + 1/2)) maps a < 1 onto [1/2, 1] (the E2M1 grid {0, 1/2, 1} becomes {1/2, 3/4, 1}: one
//       mantissa bit per binade like the values from 1 up) and leaves a >= 1 alone, without a select;
//   up = (bits(b) << 10) > thr compares the 22 mantissa bits below the grid bit with the draw, no masks;
//   the magnitude code is (bits(b) >> 22) - 252 + up; the eight "- 252" are taken off the packed word at once;
//   the sign nibbles are gathered with one funnel shift per element and masked once per word.
__device__ __forceinline__ uint32_t e2m1x8_sr(const float (&y)[8], const uint32_t (&thr)[8]) {
  uint32_t mag = 0u, sgn = 0u;
#pragma unroll
  for (int i = 7; i >= 0; --i) {
    const float a = fminf(fabsf(y[i]), 6.0f);
    const uint32_t bits = __float_as_uint(fmaxf(a, __fmaf_ru(a, 0.5f, 0.5f)));
    const uint32_t t = (bits >> 22) + (((bits << 10) > thr[i]) ? 1u : 0u);
    mag = mag * 16u + t;                                   // modulo 2^32: the excess of 252 per nibble is removed below
    sgn = __funnelshift_l(__float_as_uint(y[i]), sgn, 4);  // top nibble of y (sign and three exponent bits) shifted in
  }
  return (mag - 252u * 0x11111111u) | (sgn & 0x88888888u);
}

// encode_block with the multiplier looked up in a table filled by fill_r_table (same bytes as encode_block).
// thr[i] = draw_i << 16 (only read with stochastic rounding).
__device__ __forceinline__ uint32_t encode_block_tab(const float (&v)[16], const uint32_t (&thr)[16], bool sr, float six_s_T,
                                                     const float* r_tab, uint32_t (&packed)[2]) {
  float m8[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) m8[i] = fmaxf(fabsf(v[i]), fabsf(v[i + 8]));
  const float amax = fmaxf(fmaxf(fmaxf(m8[0], m8[4]), fmaxf(m8[1], m8[5])), fmaxf(fmaxf(m8[2], m8[6]), fmaxf(m8[3], m8[7])));
  const float t = fminf(__fdiv_rn(amax, six_s_T), 448.0f);
  float sb_unused;
  const uint32_t byte = metis_e4m3_ceil(t, &sb_unused);
  const float r = r_tab[byte];
  if (!sr) {
    packed[0] = e2m1x8_rne(__fmul_rn(v[0], r), __fmul_rn(v[1], r), __fmul_rn(v[2], r), __fmul_rn(v[3], r),
                           __fmul_rn(v[4], r), __fmul_rn(v[5], r), __fmul_rn(v[6], r), __fmul_rn(v[7], r));
    packed[1] = e2m1x8_rne(__fmul_rn(v[8], r), __fmul_rn(v[9], r), __fmul_rn(v[10], r), __fmul_rn(v[11], r),
                           __fmul_rn(v[12], r), __fmul_rn(v[13], r), __fmul_rn(v[14], r), __fmul_rn(v[15], r));
  } else {
    float y0[8], y1[8];
    uint32_t t0[8], t1[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { y0[i] = __fmul_rn(v[i], r); y1[i] = __fmul_rn(v[8 + i], r); t0[i] = thr[i]; t1[i] = thr[8 + i]; }
    packed[0] = e2m1x8_sr(y0, t0);
    packed[1] = e2m1x8_sr(y1, t1);
  }
  return byte;
}

// tile:  [TILE][PITCH] floats, rows/cols outside the matrix already zero-filled
// rnd:   [TILE][TILE] 16-bit draws (only read when rounding == SR)
// stage: scratch
// All THREADS threads of the block must call this; contains __syncthreads().
__device__ __forceinline__ void quantize_tile(const float* tile, const uint16_t* rnd, Stage* stage,
                                              const QuantParams& p, int64_t row0, int64_t col0, float s_T) {
  const int tid = threadIdx.x;
  const bool sr = p.rounding == METIS_ROUND_SR;
  const float six_s_T = __fmul_rn(6.0f, s_T);
  const int vrows = (int)min((int64_t)TILE, p.rows - row0);
  const int vcols = (int)min((int64_t)TILE, p.cols - col0);

  if (p.c_codes != nullptr) {
    // blocks along columns: thread -> (row = tid % 128, blocks b = tid/128 + 2*it)
#pragma unroll 1
    for (int it = 0; it < 4; ++it) {
      const int r = tid & 127, b = (tid >> 7) + 2 * it;
      float v[16];
      uint32_t u[16];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float4 q = *reinterpret_cast<const float4*>(tile + r * PITCH + b * 16 + i * 4);
        v[4 * i] = q.x; v[4 * i + 1] = q.y; v[4 * i + 2] = q.z; v[4 * i + 3] = q.w;
      }
      if (sr) {
#pragma unroll
        for (int i = 0; i < 16; ++i) u[i] = rnd[r * TILE + b * 16 + i];
      }
      uint32_t packed[2];
      const uint32_t byte = encode_block(v, u, sr, s_T, six_s_T, packed);
      *reinterpret_cast<uint2*>(&stage->codes[r][b * 8]) = make_uint2(packed[0], packed[1]);
      stage->sf[r][b] = (uint8_t)byte;
    }
    __syncthreads();
    // coalesced write-out
    const int64_t kbytes = p.cols / 2;
    for (int i = tid; i < TILE * 8; i += THREADS) {      // 8-byte units: one block of 16 codes each
      const int r = i >> 3, seg = i & 7;
      if (r < vrows && seg * 16 < vcols) {
        *reinterpret_cast<uint2*>(p.c_codes + (row0 + r) * kbytes + col0 / 2 + seg * 8) =
            *reinterpret_cast<const uint2*>(&stage->codes[r][seg * 8]);
      }
    }
    const int64_t bpr = p.cols / 16;
    for (int i = tid; i < TILE * 8; i += THREADS) {
      int r, b;
      if (p.c_layout == METIS_SF_TILED) {   // walk the two 512-byte atoms in storage order
        const int atom = i >> 9, w = i & 511;
        r = (w >> 4) + 32 * ((w >> 2) & 3);
        b = atom * 4 + (w & 3);
      } else {
        r = i >> 3; b = i & 7;
      }
      if (b * 16 < vcols && (r < vrows || p.c_layout == METIS_SF_TILED)) {
        const uint8_t val = r < vrows ? stage->sf[r][b] : (uint8_t)0;
        p.c_scales[metis_sf_offset(row0 + r, col0 / 16 + b, bpr, p.c_layout)] = val;
      }
    }
    __syncthreads();
  }

  if (p.r_codes != nullptr) {
    // blocks along rows: stored row = source column.  thread -> (col = tid % 128, row-blocks b = tid/128 + 2*it)
#pragma unroll 1
    for (int it = 0; it < 4; ++it) {
      const int c = tid & 127, b = (tid >> 7) + 2 * it;
      float v[16];
      uint32_t u[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) v[i] = tile[(b * 16 + i) * PITCH + c];
      if (sr) {
#pragma unroll
        for (int i = 0; i < 16; ++i) u[i] = rnd[(b * 16 + i) * TILE + c];
      }
      uint32_t packed[2];
      const uint32_t byte = encode_block(v, u, sr, s_T, six_s_T, packed);
      *reinterpret_cast<uint2*>(&stage->codes[c][b * 8]) = make_uint2(packed[0], packed[1]);
      stage->sf[c][b] = (uint8_t)byte;
    }
    __syncthreads();
    const int64_t kbytes = p.rows / 2;
    for (int i = tid; i < TILE * 8; i += THREADS) {
      const int c = i >> 3, seg = i & 7;
      if (c < vcols && seg * 16 < vrows) {
        *reinterpret_cast<uint2*>(p.r_codes + (col0 + c) * kbytes + row0 / 2 + seg * 8) =
            *reinterpret_cast<const uint2*>(&stage->codes[c][seg * 8]);
      }
    }
    const int64_t bpr = p.rows / 16;
    for (int i = tid; i < TILE * 8; i += THREADS) {
      int c, b;
      if (p.r_layout == METIS_SF_TILED) {
        const int atom = i >> 9, w = i & 511;
        c = (w >> 4) + 32 * ((w >> 2) & 3);
        b = atom * 4 + (w & 3);
      } else {
        c = i >> 3; b = i & 7;
      }
      if (b * 16 < vrows && (c < vcols || p.r_layout == METIS_SF_TILED)) {
        const uint8_t val = c < vcols ? stage->sf[c][b] : (uint8_t)0;
        p.r_scales[metis_sf_offset(col0 + c, row0 / 16 + b, bpr, p.r_layout)] = val;
      }
    }
    __syncthreads();
  }
}

// Fills the tile's 16-bit draws.  Fast path: elements consecutive along a row share Philox counters.
__device__ __forceinline__ void fill_draws(uint16_t* rnd, const QuantParams& p, int64_t row0, int64_t col0) {
  const int tid = threadIdx.x;
  if (p.e_stride_c == 1 && (p.e_stride_r & 7) == 0 && (col0 & 7) == 0) {
    for (int i = tid; i < TILE * (TILE / 8); i += THREADS) {
      const int r = i >> 4, g = i & 15;
      const uint64_t e = (uint64_t)(row0 + r) * (uint64_t)p.e_stride_r + (uint64_t)(col0 + g * 8);
      const uint4 w = metis_philox_block(e >> 3, p.seed, p.stream_id);
      uint4 out;
      out.x = w.x; out.y = w.y; out.z = w.z; out.w = w.w;   // halves in order: low half of word 0 first
      *reinterpret_cast<uint4*>(rnd + r * TILE + g * 8) = out;
    }
  } else {
    for (int i = tid; i < TILE * TILE; i += THREADS) {
      const int r = i >> 7, c = i & 127;
      const uint64_t e = (uint64_t)(row0 + r) * (uint64_t)p.e_stride_r + (uint64_t)(col0 + c) * (uint64_t)p.e_stride_c;
      rnd[i] = (uint16_t)metis_draw_u16(e, p.seed, p.stream_id);
    }
  }
}

constexpr size_t smem_bytes(bool sr) {
  return sizeof(float) * TILE * PITCH + sizeof(Stage) + (sr ? sizeof(uint16_t) * TILE * TILE : 0);
}

}  // namespace metis_qt
