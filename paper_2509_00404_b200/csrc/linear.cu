// Split-FP4 linear layer: forward (Eq. 2), input gradient (Eq. 3) and weight gradient (Section 3.2).
//
// With both operands written as  Ta = Fo_a diag(sa) Fc_a^T + Res_a  (M x K) and
// Tb = Fo_b diag(sb) Fc_b^T + Res_b (N x K), where Fc_* are the factors lying along the contraction
// axis and Fo_* those lying along the output axes, the product expands into
//
//   Ta Tb^T = Res_a Res_b^T                          main FP4 GEMM           (M x N)
//           + (G1 + Fo_a sa P) sb Fo_b^T             G1 = Res_a Fc_b (M x kb), P = Fc_a^T Fc_b (ka x kb)
//           + (Fo_a sa) Wt^T                         Wt = Res_b Fc_a (N x ka)
//
// i.e. one large and three skinny block-scaled FP4 GEMMs followed by a rank-(ka+kb) FP32 update.
// All four quantized cross terms of the paper's expansion are kept.
#include "common.cuh"

bool metis_gemm_tc_can_fuse(const metis_nvfp4_t* a, const metis_nvfp4_t* b);
metis_status_t metis_launch_gemm_tc_fused(metis_context* ctx, const metis_nvfp4_t* a, const metis_nvfp4_t* b, void* d,
                                          int d_dtype, int64_t ldd, const void* lx, const void* rx, int kx, cudaStream_t s);

namespace {

__device__ __forceinline__ float deq_at(const uint8_t* codes, const uint8_t* sf, int layout, int64_t k_len, int64_t r,
                                        int64_t c) {
  const uint32_t byte = codes[r * (k_len / 2) + c / 2];
  const uint32_t code = (c & 1) ? (byte >> 4) : (byte & 15u);
  return metis_e2m1_value(code) * metis_e4m3_value(sf[metis_sf_offset(r, c / 16, k_len / 16, layout)]);
}

// Finishes the two skinny operands of the rank-(ka+kb) update, in place.  Layout: Lcat [M][kb + ka],
// Rcat [N][kb + ka].  On entry Lcat[:, :kb] holds G1 and Rcat[:, kb:] holds Wt (written there by the skinny
// GEMMs).  On exit  Lcat[:, :kb] = (G1 + Fo_a sa P) sb,  Lcat[:, kb:] = Fo_a sa,  Rcat[:, :kb] = Fo_b.
// One warp per row.  Every global load of a row is issued before the first value is used (the loads are one
// round trip instead of a chain of them), and the finished rows stay in shared memory for the BF16 pass.
__device__ __forceinline__ float deq_of(uint32_t byte, uint32_t sf_byte, int64_t c) {
  const uint32_t code = (c & 1) ? (byte >> 4) : (byte & 15u);
  return metis_e2m1_value(code) * metis_e4m3_value((uint8_t)sf_byte);
}
__global__ void __launch_bounds__(256)
lowrank_finish_kernel(int64_t M, int64_t N, int ka, int kb,
                      const uint8_t* foa_codes, const uint8_t* foa_sf, int foa_layout, const float* foa_ts,
                      const float* sa,
                      const uint8_t* fob_codes, const uint8_t* fob_sf, int fob_layout, const float* fob_ts,
                      const float* sb, const float* __restrict__ pm, float* __restrict__ lcat, float* __restrict__ rcat,
                      __nv_bfloat16* __restrict__ lx, __nv_bfloat16* __restrict__ rx, int kx,
                      const float* res_a_ts, const float* res_b_ts) {
  __shared__ float ps[64][65];
  __shared__ float fa[8][64];
  __shared__ float lrow[8][128];
  __shared__ float rrow[8][128];
  __shared__ float lraw[8][64], rraw[8][64];                // the factors as E2M1 x E4M3 products, before any FP32 scale
  metis_pdl_wait();
  metis_pdl_trigger();                                      // the large GEMM behind this kernel sets itself up meanwhile
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int kc = ka + kb;
  const int64_t i = (int64_t)blockIdx.x * 8 + warp;
  // ---- loads (ka, kb <= 64: two values per lane and operand) ----
  uint32_t a_byte[2] = {0u, 0u}, a_sfb[2] = {0u, 0u}, b_byte[2] = {0u, 0u}, b_sfb[2] = {0u, 0u};
  float sa_v[2] = {0.0f, 0.0f}, sb_v[2] = {0.0f, 0.0f}, g1[2] = {0.0f, 0.0f}, wt[2] = {0.0f, 0.0f};
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const int u = lane + 32 * j;
    if (u < ka) {
      sa_v[j] = sa[u];
      if (i < M) {
        a_byte[j] = foa_codes[(int64_t)u * (M / 2) + i / 2];
        a_sfb[j] = foa_sf[metis_sf_offset(u, i / 16, M / 16, foa_layout)];
      }
      if (i < N) wt[j] = rcat[i * kc + kb + u];
    }
    if (u < kb) {
      sb_v[j] = sb[u];
      if (i < M) g1[j] = lcat[i * kc + u];
      if (i < N) {
        b_byte[j] = fob_codes[(int64_t)u * (N / 2) + i / 2];
        b_sfb[j] = fob_sf[metis_sf_offset(u, i / 16, N / 16, fob_layout)];
      }
    }
  }
  const float tsa = ka ? *foa_ts : 0.0f, tsb = kb ? *fob_ts : 0.0f;
  const float inv_alpha = lx != nullptr ? 1.0f / ((*res_a_ts) * (*res_b_ts)) : 0.0f;
  for (int o = tid; o < ka * kb; o += 256) ps[o / kb][o % kb] = pm[o];
  __syncthreads();
  if (i < M) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int u = lane + 32 * j;
      if (u < ka) {
        const float raw = deq_of(a_byte[j], a_sfb[j], i);
        const float v = raw * tsa * sa_v[j];
        lraw[warp][u] = raw;
        fa[warp][u] = v;
        lrow[warp][kb + u] = v;
        lcat[i * kc + kb + u] = v;
      }
    }
    __syncwarp();
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int t = lane + 32 * j;
      if (t < kb) {
        float v = g1[j];
        for (int u = 0; u < ka; ++u) v = fmaf(fa[warp][u], ps[u][t], v);
        v *= sb_v[j];
        lrow[warp][t] = v;
        lcat[i * kc + t] = v;
      }
    }
  }
  if (i < N) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int t = lane + 32 * j;
      if (t < kb) {
        const float raw = deq_of(b_byte[j], b_sfb[j], i);
        const float v = raw * tsb;
        rraw[warp][t] = raw;
        rrow[warp][t] = v;
        rcat[i * kc + t] = v;
      }
      if (t < ka) rrow[warp][kb + t] = wt[j];
    }
  }
  if (lx == nullptr) return;
  // BF16 operands of the in-accumulator correction, zero padded to kx columns.  A dequantized factor entry is an
  // E2M1 x E4M3 product (six significant bits): with its FP32 scales moved to the other operand it is exact in BF16
  // and needs no low part, so each of the two rank-k terms costs two column groups instead of three:
  //   Lx = [ A hi | A lo | Fa | Fa ],  A  = (G1 + Fo_a sa P) sb ts_b / alpha     (k_b columns), Fa = Fo_a / ts_a (k_a)
  //   Rx = [ Fb   | Fb   | B hi | B lo ],  Fb = Fo_b / ts_b (k_b),  B = Wt sa ts_a / alpha          (k_a columns)
  __syncwarp();
  const float l_scale = tsb * inv_alpha, r_scale = tsa * inv_alpha;
  for (int c = lane; c < kx; c += 32) {
    float lo_ = 0.0f, ro_ = 0.0f;
    if (c < 2 * kb) {
      const int t = c < kb ? c : c - kb;
      if (i < M) {
        const float v = lrow[warp][t] * l_scale;
        const float h = __bfloat162float(__float2bfloat16_rn(v));
        lo_ = c < kb ? h : v - h;
      }
      if (i < N) ro_ = rraw[warp][t];
    } else if (c < 2 * kc) {
      const int u0 = c - 2 * kb, u = u0 < ka ? u0 : u0 - ka;
      if (i < M) lo_ = lraw[warp][u];
      if (i < N) {
        const float v = rrow[warp][kb + u] * sa[u] * r_scale;
        const float h = __bfloat162float(__float2bfloat16_rn(v));
        ro_ = u0 < ka ? h : v - h;
      }
    }
    if (i < M) lx[i * kx + c] = __float2bfloat16_rn(lo_);
    if (i < N) rx[i * kx + c] = __float2bfloat16_rn(ro_);
  }
}

// Ranks above 64: the same finishing step as three kernels that tile over the rank.
//   lowrank_deq_wide_kernel    Lcat[:, kb:] = Fo_a sa and Rcat[:, :kb] = Fo_b from the NVFP4 factors (a thread
//                              dequantizes eight consecutive rows of one vector from one 32-bit load)
//   lowrank_gemm_wide_kernel   Lcat[:, :kb] = (G1 + Lcat[:, kb:] P) sb, a 64 x 64 x 16 tiled FP32 product, 4 x 4 per thread
//   lowrank_bf16_kernel        the BF16 correction operands, eight columns per thread
constexpr int LW_MAXK = 256;
__global__ void __launch_bounds__(256)
lowrank_deq_wide_kernel(int64_t M, int64_t N, int ka, int kb,
                        const uint8_t* foa_codes, const uint8_t* foa_sf, int foa_layout, const float* foa_ts, const float* sa,
                        const uint8_t* fob_codes, const uint8_t* fob_sf, int fob_layout, const float* fob_ts,
                        float* __restrict__ lcat, float* __restrict__ rcat,
                        __nv_bfloat16* __restrict__ lx, __nv_bfloat16* __restrict__ rx, int kx) {
  metis_pdl_wait();
  const int tid = threadIdx.x, kc = ka + kb;
  const int64_t i0 = (int64_t)blockIdx.x * 32 + 8 * (tid & 3);      // this thread's eight rows (M, N are multiples of 16)
  const float tsa = ka ? *foa_ts : 0.0f, tsb = kb ? *fob_ts : 0.0f;
  for (int u = tid >> 2; u < ka; u += 64) {
    if (i0 >= M) break;
    const uint32_t word = *reinterpret_cast<const uint32_t*>(foa_codes + (int64_t)u * (M / 2) + i0 / 2);
    const float sc = metis_e4m3_value(foa_sf[metis_sf_offset(u, i0 / 16, M / 16, foa_layout)]), su = sa[u];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float raw = metis_e2m1_value((word >> (4 * j)) & 15u) * sc;
      lcat[(i0 + j) * kc + kb + u] = raw * tsa * su;
      if (lx != nullptr) {                                  // the exact factor entry, both of its column groups
        const __nv_bfloat16 e = __float2bfloat16_rn(raw);
        lx[(i0 + j) * kx + 2 * kb + u] = e;
        lx[(i0 + j) * kx + 2 * kb + ka + u] = e;
      }
    }
  }
  for (int t = tid >> 2; t < kb; t += 64) {
    if (i0 >= N) break;
    const uint32_t word = *reinterpret_cast<const uint32_t*>(fob_codes + (int64_t)t * (N / 2) + i0 / 2);
    const float sc = metis_e4m3_value(fob_sf[metis_sf_offset(t, i0 / 16, N / 16, fob_layout)]);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float raw = metis_e2m1_value((word >> (4 * j)) & 15u) * sc;
      rcat[(i0 + j) * kc + t] = raw * tsb;
      if (rx != nullptr) {
        const __nv_bfloat16 e = __float2bfloat16_rn(raw);
        rx[(i0 + j) * kx + t] = e;
        rx[(i0 + j) * kx + kb + t] = e;
      }
    }
  }
}

__global__ void __launch_bounds__(256)
lowrank_gemm_wide_kernel(int64_t M, int ka, int kb, const float* __restrict__ sb, const float* __restrict__ pm, float* __restrict__ lcat) {
  metis_pdl_wait();
  constexpr int KT = 16;
  __shared__ __align__(16) float as[KT][68], bs[KT][68];   // [u][row], [u][column]
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15, kc = ka + kb;
  const int64_t m0 = (int64_t)blockIdx.y * 64;
  const int n0 = blockIdx.x * 64;
  float acc[4][4] = {};
  for (int u0 = 0; u0 < ka; u0 += KT) {
    __syncthreads();
    for (int o = tid; o < 64 * KT; o += 256) {
      const int uu = o % KT, r = o / KT;                    // consecutive threads: consecutive u of one row (contiguous in Lcat)
      as[uu][r] = (m0 + r < M && u0 + uu < ka) ? lcat[(m0 + r) * kc + kb + u0 + uu] : 0.0f;
      const int t = o % 64, u2 = o / 64;                    // consecutive threads: consecutive columns of one row of P
      bs[u2][t] = (u0 + u2 < ka && n0 + t < kb) ? pm[(int64_t)(u0 + u2) * kb + n0 + t] : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int uu = 0; uu < KT; ++uu) {
      const float4 a = *reinterpret_cast<const float4*>(&as[uu][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&bs[uu][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t r = m0 + ty * 4 + i;
    if (r >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int t = n0 + tx * 4 + j;
      if (t < kb) lcat[r * kc + t] = (lcat[r * kc + t] + acc[i][j]) * sb[t];
    }
  }
}

// Then the general halves of the BF16 correction operands (the layout of lowrank_finish_kernel): [A hi | A lo] of Lx and
// [B hi | B lo] of Rx from the finished FP32 operands, and the zero padding up to kx columns; the exact factor groups
// were written by lowrank_deq_wide_kernel.  One thread per row and eight columns (the group boundaries 2 k_b and
// 2 (k_a + k_b) are multiples of eight).
__global__ void __launch_bounds__(256)
lowrank_bf16_kernel(int64_t M, int64_t N, int ka, int kb, int kx, const float* __restrict__ lcat, const float* __restrict__ rcat,
                    const float* foa_ts, const float* __restrict__ sa, const float* fob_ts,
                    __nv_bfloat16* __restrict__ lx, __nv_bfloat16* __restrict__ rx, const float* res_a_ts, const float* res_b_ts) {
  metis_pdl_wait();
  const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const int64_t mx = M > N ? M : N;
  const int per_row = kx / 8, kc = ka + kb;
  if (idx >= mx * per_row) return;
  const int64_t i = idx / per_row;
  const int c0 = (int)(idx - i * per_row) * 8;
  const float inv_alpha = 1.0f / ((*res_a_ts) * (*res_b_ts));
  const float l_scale = (kb ? *fob_ts : 0.0f) * inv_alpha, r_scale = (ka ? *foa_ts : 0.0f) * inv_alpha;
  __align__(16) __nv_bfloat16 o[8];
  if (c0 < 2 * kb) {                                        // [A hi | A lo]
    if (i < M) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int c = c0 + e, t = c < kb ? c : c - kb;
        const float v = lcat[i * kc + t] * l_scale;
        const float h = __bfloat162float(__float2bfloat16_rn(v));
        o[e] = __float2bfloat16_rn(c < kb ? h : v - h);
      }
      *reinterpret_cast<uint4*>(lx + i * kx + c0) = *reinterpret_cast<const uint4*>(o);
    }
  } else if (c0 < 2 * kc) {                                 // [B hi | B lo]
    if (i < N) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int u0 = c0 + e - 2 * kb, u = u0 < ka ? u0 : u0 - ka;
        const float v = rcat[i * kc + kb + u] * sa[u] * r_scale;
        const float h = __bfloat162float(__float2bfloat16_rn(v));
        o[e] = __float2bfloat16_rn(u0 < ka ? h : v - h);
      }
      *reinterpret_cast<uint4*>(rx + i * kx + c0) = *reinterpret_cast<const uint4*>(o);
    }
  } else {                                                  // padding of both operands
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    if (i < M) *reinterpret_cast<uint4*>(lx + i * kx + c0) = z;
    if (i < N) *reinterpret_cast<uint4*>(rx + i * kx + c0) = z;
  }
}

// out = y0 + Lcat Rcat^T, 64 x 64 tile per CTA
__global__ void __launch_bounds__(256)
rank_update_kernel(const float* __restrict__ y0, int64_t M, int64_t N, int kc, const float* __restrict__ lcat,
                   const float* __restrict__ rcat, void* __restrict__ out, int out_dtype, int64_t ldo) {
  extern __shared__ float sm[];
  float* ls = sm;                       // [kc][64 + 4]
  float* rs = sm + kc * 68;
  const int tid = threadIdx.x;
  const int64_t m0 = (int64_t)blockIdx.y * 64, n0 = (int64_t)blockIdx.x * 64;
  for (int i = tid; i < 64 * kc; i += 256) {
    const int r = i / kc, t = i % kc;
    ls[t * 68 + r] = (m0 + r < M) ? lcat[(m0 + r) * kc + t] : 0.0f;
    rs[t * 68 + r] = (n0 + r < N) ? rcat[(n0 + r) * kc + t] : 0.0f;
  }
  __syncthreads();
  const int ty = tid >> 4, tx = tid & 15;
  float acc[4][4] = {};
  for (int t = 0; t < kc; ++t) {
    const float4 a = *reinterpret_cast<const float4*>(ls + t * 68 + ty * 4);
    const float4 b = *reinterpret_cast<const float4*>(rs + t * 68 + tx * 4);
    const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t r = m0 + ty * 4 + i, c = n0 + tx * 4 + j;
      if (r < M && c < N) {
        const float v = y0[r * N + c] + acc[i][j];
        if (out_dtype == METIS_BF16) reinterpret_cast<__nv_bfloat16*>(out)[r * ldo + c] = __float2bfloat16_rn(v);
        else reinterpret_cast<float*>(out)[r * ldo + c] = v;
      }
    }
}


// ------------------------------------------------------------------------------------------------
// Gradients of the weight factors (Section 3.2, the derivatives listed after Eq. 3).  With the weight gradient
// G (n x m, FP32 or BF16, as produced by the wgrad product) and a dequantized factor F stored k x len:
//   TRANS = 0:  out[t][r] = scale_t * sum_c G[r][c] F[t][c]      (r over n, c over m:  dL/dV from U)
//   TRANS = 1:  out[t][r] = scale_t * sum_c G[c][r] F[t][c]      (r over m, c over n:  dL/dU from V)
// scale_t = sigma_t.  One CTA owns 32 values of r and walks c in chunks of 32; FP32 FMAs, fixed summation
// order (deterministic).  With `other` given (the factor lying along r), the CTA also writes its partial of
//   dsigma[t] = sum_r other[t][r] * (sum_c ...)   to ds_part[blockIdx.x][t].
constexpr int FG_ROWS = 32, FG_CHUNK = 32;
template <int KT, bool TRANS>                           // KT = ceil(k / 8) outputs per thread
__global__ void __launch_bounds__(256)
factor_grad_kernel(const void* __restrict__ gsrc, int g_dtype, int64_t ldg, int64_t n_r, int64_t n_c, int k, int t0, int k_all,
                   const uint8_t* f_codes, const uint8_t* f_sf, int f_layout, const float* f_ts,
                   const uint8_t* o_codes, const uint8_t* o_sf, int o_layout, const float* o_ts,
                   const float* __restrict__ sigma, float* __restrict__ out, float* __restrict__ ds_part) {
  // factor vectors t0 .. t0 + k - 1 of k_all (a launch handles at most 64 of them)
  __shared__ float gs[FG_ROWS][FG_CHUNK + 1];
  __shared__ __align__(16) float fs[FG_CHUNK][8 * KT + 4];
  __shared__ float red[8][8 * KT];
  const int tid = threadIdx.x, r = tid >> 3, tg = tid & 7;
  const int64_t r0 = (int64_t)blockIdx.x * FG_ROWS;
  const float fts = *f_ts;
  float acc[KT];
#pragma unroll
  for (int j = 0; j < KT; ++j) acc[j] = 0.0f;
  for (int64_t c0 = 0; c0 < n_c; c0 += FG_CHUNK) {
    // tile of G: element (rr, cc) of this chunk
    for (int o = tid; o < FG_ROWS * FG_CHUNK; o += 256) {
      const int a = o >> 5, b = o & 31;                 // b runs along the contiguous axis of G
      const int rr = TRANS ? b : a, cc = TRANS ? a : b;
      const int64_t gr = r0 + rr, gc = c0 + cc;
      float v = 0.0f;
      if (gr < n_r && gc < n_c) {
        const int64_t off = TRANS ? gc * ldg + gr : gr * ldg + gc;
        v = g_dtype == METIS_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(gsrc)[off])
                                  : reinterpret_cast<const float*>(gsrc)[off];
      }
      gs[rr][cc] = v;
    }
    for (int o = tid; o < FG_CHUNK * 8 * KT; o += 256) {
      const int t = o >> 5, cc = o & 31;
      fs[cc][t] = (t < k && c0 + cc < n_c) ? deq_at(f_codes, f_sf, f_layout, n_c, t0 + t, c0 + cc) : 0.0f;
    }
    __syncthreads();
#pragma unroll 8
    for (int cc = 0; cc < FG_CHUNK; ++cc) {
      const float gv = gs[r][cc];
#pragma unroll
      for (int j = 0; j < KT; ++j) acc[j] = fmaf(gv, fs[cc][tg * KT + j], acc[j]);
    }
    __syncthreads();
  }
  const int64_t gr = r0 + r;
#pragma unroll
  for (int j = 0; j < KT; ++j) {
    const int t = tg * KT + j;
    acc[j] *= fts;
    if (t < k && gr < n_r) out[(int64_t)(t0 + t) * n_r + gr] = acc[j] * sigma[t0 + t];
  }
  if (ds_part != nullptr) {
    const float ots = *o_ts;
    // sum over the CTA's 32 rows in a fixed order: 4 rows per warp by shuffles, then 8 warps through shared memory
#pragma unroll
    for (int j = 0; j < KT; ++j) {
      const int t = tg * KT + j;
      float v = (t < k && gr < n_r) ? acc[j] * deq_at(o_codes, o_sf, o_layout, n_r, t0 + t, gr) * ots : 0.0f;
      v += __shfl_xor_sync(0xFFFFFFFFu, v, 8);
      v += __shfl_xor_sync(0xFFFFFFFFu, v, 16);
      if ((tid & 31) < 8) red[tid >> 5][t] = v;
    }
    __syncthreads();
    if (tid < k) {
      float v = 0.0f;
#pragma unroll
      for (int w = 0; w < 8; ++w) v += red[w][tid];
      ds_part[(int64_t)blockIdx.x * k_all + t0 + tid] = v;
    }
  }
}

// dsigma[t] = sum over the partials, in order
__global__ void factor_grad_sigma_kernel(const float* __restrict__ part, int n_part, int k, float* __restrict__ ds) {
  const int t = threadIdx.x;
  if (t >= k) return;
  float v = 0.0f;
  for (int i = 0; i < n_part; ++i) v += part[(int64_t)i * k + t];
  ds[t] = v;
}

template <bool TRANS>
metis_status_t launch_factor_grad(cudaStream_t s, const void* g, int g_dtype, int64_t ldg, int64_t n_r, int64_t n_c, int k,
                                  const metis_nvfp4_t* f, const metis_nvfp4_t* o, const float* sigma, float* out, float* ds_part) {
  const unsigned grid = (unsigned)metis_ceil_div(n_r, FG_ROWS);
#define METIS_FG(KT) factor_grad_kernel<KT, TRANS><<<grid, 256, 0, s>>>(g, g_dtype, ldg, n_r, n_c, kg, t0, k, f->codes, f->scales, f->sf_layout, \
    f->tensor_scale, o ? o->codes : nullptr, o ? o->scales : nullptr, o ? o->sf_layout : 0, o ? o->tensor_scale : nullptr, sigma, out, ds_part)
  for (int t0 = 0; t0 < k; t0 += 64) {                  // at most 64 factor vectors per pass over the gradient
    const int kg = k - t0 < 64 ? k - t0 : 64;
    switch ((kg + 7) / 8) {
      case 1: METIS_FG(1); break; case 2: METIS_FG(2); break; case 3: METIS_FG(3); break; case 4: METIS_FG(4); break;
      case 5: METIS_FG(5); break; case 6: METIS_FG(6); break; case 7: METIS_FG(7); break; case 8: METIS_FG(8); break;
      default: return METIS_ERR_SHAPE;
    }
    METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(cudaGetLastError());
  }
#undef METIS_FG
  return METIS_OK;
}

// the host-side checks of factor_grads, callable before anything is enqueued
metis_status_t factor_grads_check(const metis_operand_t* w, const float* d_left, const float* d_sigma, const void* ws, size_t ws_bytes) {
  if (!w || w->k <= 0 || w->k > LW_MAXK || !w->sigma) return METIS_ERR_SHAPE;
  const metis_nvfp4_t *lq = &w->left_q, *rq = &w->right_q;
  if (!lq->codes || !rq->codes || lq->k_len != w->rows || rq->k_len != w->cols) return METIS_ERR_SHAPE;
  if (d_sigma && !d_left) return METIS_ERR_INVALID_ARG;          // the sigma partials ride on the d_left pass
  if (d_sigma && (!ws || ws_bytes < sizeof(float) * (size_t)metis_ceil_div(w->rows, FG_ROWS) * w->k)) return METIS_ERR_WORKSPACE;
  return METIS_OK;
}

// d_left (k x n), d_sigma (k), d_right (k x m) of the weight operand W_t = left diag(sigma) right^T from dw (n x m).
metis_status_t factor_grads(metis_context* ctx, const void* dw, int dw_dtype, int64_t lddw, const metis_operand_t* w,
                            float* d_left, float* d_sigma, float* d_right, void* ws, size_t ws_bytes, cudaStream_t s) {
  (void)ctx;
  if (!w || w->k <= 0 || w->k > LW_MAXK || !w->sigma) return METIS_ERR_SHAPE;
  const int64_t n = w->rows, m = w->cols;
  const metis_nvfp4_t *lq = &w->left_q, *rq = &w->right_q;
  if (!lq->codes || !rq->codes || lq->k_len != n || rq->k_len != m) return METIS_ERR_SHAPE;
  const int64_t n_part = metis_ceil_div(n, FG_ROWS);
  if (d_sigma && (!ws || ws_bytes < sizeof(float) * (size_t)n_part * w->k)) return METIS_ERR_WORKSPACE;
  float* part = reinterpret_cast<float*>(ws);
  // dL/dV (the paper's V = left, n x k): rows of dw against U = right; also the partials of dL/dS
  if (d_left || d_sigma) {
    if (!d_left) return METIS_ERR_INVALID_ARG;          // the sigma partials ride on the d_left pass
    METIS_TRY(launch_factor_grad<false>(s, dw, dw_dtype, lddw, n, m, w->k, rq, d_sigma ? lq : nullptr, w->sigma, d_left,
                                        d_sigma ? part : nullptr));
    if (d_sigma) {
      factor_grad_sigma_kernel<<<1, 256, 0, s>>>(part, (int)n_part, w->k, d_sigma); METIS_COUNT_LAUNCH();
      METIS_CUDA_TRY(cudaGetLastError());
    }
  }
  // dL/dU (the paper's U = right, m x k): columns of dw against V = left
  if (d_right) METIS_TRY(launch_factor_grad<true>(s, dw, dw_dtype, lddw, m, n, w->k, lq, nullptr, w->sigma, d_right, nullptr));
  return METIS_OK;
}

struct Side {
  const metis_nvfp4_t* res;   // residual, K-major along the contraction axis
  const metis_nvfp4_t* fc;    // factor along the contraction axis (k x K)
  const metis_nvfp4_t* fo;    // factor along the output axis      (k x M or k x N)
  const float* sigma;
  int k;
};

size_t align256(size_t b) { return (b + 255) & ~(size_t)255; }

metis_status_t check_nvfp4(const metis_nvfp4_t* t) {
  if (!t || !t->codes || !t->scales || !t->tensor_scale) return METIS_ERR_INVALID_ARG;
  if (t->sf_layout != METIS_SF_TILED) return METIS_ERR_INVALID_ARG;
  if (t->k_len % 64 || t->rows <= 0) return METIS_ERR_SHAPE;
  return METIS_OK;
}

// Where the intermediates of one product live inside the caller's workspace.
struct Plan {
  int64_t M, N, K;
  int ka, kb, kc, kx;
  bool fuse;
  float *pm, *lcat, *rcat, *y0;
  __nv_bfloat16 *lx, *rx;
  size_t bytes;
};

metis_status_t make_plan(const Side& a, const Side& b, void* ws, size_t ws_bytes, Plan* pl) {
  METIS_TRY(check_nvfp4(a.res));
  METIS_TRY(check_nvfp4(b.res));
  pl->M = a.res->rows; pl->N = b.res->rows; pl->K = a.res->k_len;
  if (b.res->k_len != pl->K) return METIS_ERR_SHAPE;
  pl->ka = a.k; pl->kb = b.k; pl->kc = a.k + b.k; pl->bytes = 0;
  if (pl->kc == 0) return METIS_OK;
  const int64_t M = pl->M, N = pl->N, K = pl->K;
  const int ka = a.k, kb = b.k, kc = pl->kc;
  if (ka > LW_MAXK || kb > LW_MAXK) return METIS_ERR_SHAPE;
  if (ka) { METIS_TRY(check_nvfp4(a.fc)); METIS_TRY(check_nvfp4(a.fo)); if (a.fc->k_len != K || a.fo->k_len != M || !a.sigma) return METIS_ERR_SHAPE; }
  if (kb) { METIS_TRY(check_nvfp4(b.fc)); METIS_TRY(check_nvfp4(b.fo)); if (b.fc->k_len != K || b.fo->k_len != N || !b.sigma) return METIS_ERR_SHAPE; }
  unsigned char* w = reinterpret_cast<unsigned char*>(ws);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align256(bytes); return o; };
  pl->fuse = metis_gemm_tc_can_fuse(a.res, b.res);
  if (!pl->fuse && kc > 128) return METIS_ERR_SHAPE;    // layers below 256 rows hold the update operands in shared memory
  pl->kx = (2 * kc + 63) / 64 * 64;          // two BF16 column groups per rank-k term (see lowrank_finish_kernel)
  const size_t o_pm = take(sizeof(float) * (size_t)(ka * kb > 64 * 64 ? ka * kb : 64 * 64)), o_l = take(sizeof(float) * M * kc), o_r = take(sizeof(float) * N * kc);
  const size_t o_lx = pl->fuse ? take(sizeof(__nv_bfloat16) * M * pl->kx) : 0, o_rx = pl->fuse ? take(sizeof(__nv_bfloat16) * N * pl->kx) : 0;
  const size_t o_y0 = pl->fuse ? 0 : take(sizeof(float) * M * N);
  pl->bytes = off;
  if (!ws || off > ws_bytes) return METIS_ERR_WORKSPACE;
  pl->pm = reinterpret_cast<float*>(w + o_pm); pl->lcat = reinterpret_cast<float*>(w + o_l); pl->rcat = reinterpret_cast<float*>(w + o_r);
  pl->lx = pl->fuse ? reinterpret_cast<__nv_bfloat16*>(w + o_lx) : nullptr;
  pl->rx = pl->fuse ? reinterpret_cast<__nv_bfloat16*>(w + o_rx) : nullptr;
  pl->y0 = pl->fuse ? nullptr : reinterpret_cast<float*>(w + o_y0);
  return METIS_OK;
}

// Everything of a product that comes before its large GEMM: the three skinny products (straight into their
// slots of the concatenated operands) and the finishing kernel.  The skinny products run on the handle's side
// streams `side0` and `side0 + 1` beside `s` (the caller has made those streams wait for `s`'s past already).
metis_status_t split_gemm_prologue(metis_context* ctx, const Side& a, const Side& b, const Plan& pl, int side0,
                                   cudaStream_t s) {
  if (pl.kc == 0) return METIS_OK;
  const int64_t M = pl.M, N = pl.N;
  const int ka = pl.ka, kb = pl.kb, kc = pl.kc;
  if (!pl.fuse) METIS_TRY(metis_launch_gemm_tc(ctx, a.res, b.res, pl.y0, METIS_FP32, N, s));
  cudaStream_t s1 = ctx->side[side0], s2 = ctx->side[side0 + 1];
  if (kb) METIS_TRY(metis_launch_gemm_tc(ctx, a.res, b.fc, pl.lcat, METIS_FP32, kc, s));
  if (ka) METIS_TRY(metis_launch_gemm_tc(ctx, b.res, a.fc, pl.rcat + kb, METIS_FP32, kc, s1));
  if (ka && kb) METIS_TRY(metis_launch_gemm_tc(ctx, a.fc, b.fc, pl.pm, METIS_FP32, kb, s2));
  METIS_TRY(metis_join(ctx, s, side0));
  METIS_TRY(metis_join(ctx, s, side0 + 1));
  const int64_t mx = M > N ? M : N;
  if (ka > 64 || kb > 64) {
    METIS_CUDA_TRY(metis_launch_pdl(lowrank_deq_wide_kernel, dim3((unsigned)metis_ceil_div(mx, 32)), dim3(256), 0, s,
        M, N, ka, kb, ka ? a.fo->codes : nullptr, ka ? a.fo->scales : nullptr, ka ? a.fo->sf_layout : 0,
        ka ? a.fo->tensor_scale : nullptr, a.sigma, kb ? b.fo->codes : nullptr, kb ? b.fo->scales : nullptr,
        kb ? b.fo->sf_layout : 0, kb ? b.fo->tensor_scale : nullptr, pl.lcat, pl.rcat, pl.lx, pl.rx, pl.kx)); METIS_COUNT_LAUNCH();
    if (kb) {
      METIS_CUDA_TRY(metis_launch_pdl(lowrank_gemm_wide_kernel, dim3((unsigned)metis_ceil_div(kb, 64), (unsigned)metis_ceil_div(M, 64)), dim3(256), 0, s,
          M, ka, kb, b.sigma, (const float*)pl.pm, pl.lcat)); METIS_COUNT_LAUNCH();
    }
    if (pl.lx != nullptr) {
      METIS_CUDA_TRY(metis_launch_pdl(lowrank_bf16_kernel, dim3((unsigned)metis_ceil_div(mx * (pl.kx / 8), 256)), dim3(256), 0, s, M, N, ka, kb, pl.kx,
          (const float*)pl.lcat, (const float*)pl.rcat, (const float*)(ka ? a.fo->tensor_scale : nullptr), (const float*)a.sigma,
          (const float*)(kb ? b.fo->tensor_scale : nullptr),
          pl.lx, pl.rx, (const float*)a.res->tensor_scale, (const float*)b.res->tensor_scale)); METIS_COUNT_LAUNCH();
    }
    METIS_CUDA_TRY(cudaGetLastError());
    return METIS_OK;
  }
  METIS_CUDA_TRY(metis_launch_pdl(lowrank_finish_kernel, dim3((unsigned)metis_ceil_div(mx, 8)), dim3(256), 0, s,
      M, N, ka, kb, ka ? a.fo->codes : nullptr, ka ? a.fo->scales : nullptr, ka ? a.fo->sf_layout : 0,
      ka ? a.fo->tensor_scale : nullptr, a.sigma, kb ? b.fo->codes : nullptr, kb ? b.fo->scales : nullptr,
      kb ? b.fo->sf_layout : 0, kb ? b.fo->tensor_scale : nullptr, b.sigma, pl.pm, pl.lcat, pl.rcat, pl.lx, pl.rx, pl.kx,
      a.res->tensor_scale, b.res->tensor_scale)); METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  return METIS_OK;
}

metis_status_t split_gemm_main(metis_context* ctx, const Side& a, const Side& b, const Plan& pl, void* d, int d_dtype, int64_t ldd,
                               cudaStream_t s) {
  if (pl.kc == 0) return metis_launch_gemm_tc(ctx, a.res, b.res, d, d_dtype, ldd, s);
  if (pl.fuse) {
    // residual x residual product and the rank-(ka+kb) correction accumulate into one FP32 tile in tensor memory
    return metis_launch_gemm_tc_fused(ctx, a.res, b.res, d, d_dtype, ldd, pl.lx, pl.rx, pl.kx, s);
  }
  dim3 grid((unsigned)metis_ceil_div(pl.N, 64), (unsigned)metis_ceil_div(pl.M, 64));
  const size_t smem = sizeof(float) * 2 * pl.kc * 68;
  rank_update_kernel<<<grid, 256, smem, s>>>(pl.y0, pl.M, pl.N, pl.kc, pl.lcat, pl.rcat, d, d_dtype, ldd); METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  return METIS_OK;
}

metis_status_t split_gemm(metis_context* ctx, const Side& a, const Side& b, void* d, int d_dtype, int64_t ldd, void* ws,
                          size_t ws_bytes, cudaStream_t s) {
  Plan pl;
  METIS_TRY(make_plan(a, b, ws, ws_bytes, &pl));
  METIS_TRY(metis_fork(ctx, s, 2));
  METIS_TRY(split_gemm_prologue(ctx, a, b, pl, 0, s));
  return split_gemm_main(ctx, a, b, pl, d, d_dtype, ldd, s);
}

}  // namespace

metis_status_t metis_linear_set_attrs() {
  METIS_CUDA_TRY(cudaFuncSetAttribute(rank_update_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(sizeof(float) * 2 * 128 * 68)));
  return METIS_OK;
}

size_t metis_linear_ws_bytes(int64_t M, int64_t N, int k) {
  const int kc = 2 * k;
  const int kx = (2 * kc + 63) / 64 * 64;
  // sized for either path: FP32 staging of the main product (small shapes) or the BF16 correction operands
  const size_t pm_elems = (size_t)k * k > 64 * 64 ? (size_t)k * k : 64 * 64;
  return align256(sizeof(float) * M * N) + align256(sizeof(float) * pm_elems) +
         align256(sizeof(float) * M * (kc ? kc : 1)) + align256(sizeof(float) * N * (kc ? kc : 1)) +
         align256(sizeof(__nv_bfloat16) * M * (kx ? kx : 1)) + align256(sizeof(__nv_bfloat16) * N * (kx ? kx : 1)) +
         align256(sizeof(float) * (size_t)(k > 64 ? k : 64) * (size_t)metis_ceil_div(M > N ? M : N, FG_ROWS));     // partials of the sigma gradient
}

metis_status_t metis_linear_fwd(metis_handle_t h, const metis_operand_t* x, const metis_operand_t* w, void* y,
                                int32_t y_dtype, int64_t ldy, void* ws, size_t ws_bytes, metis_stream_t stream) {
  METIS_NVTX("metis_linear_fwd");
  if (!h || !x || !w || !y) return METIS_ERR_INVALID_ARG;
  if (y_dtype != METIS_BF16 && y_dtype != METIS_FP32) return METIS_ERR_INVALID_ARG;
  if (x->cols != w->cols || ldy < w->rows) return METIS_ERR_SHAPE;
  // contraction over in-features: X (l x m) by columns, W_t (n x m) by columns
  Side a{&x->res_by_cols, &x->right_q, &x->left_q, x->sigma, x->k};
  Side b{&w->res_by_cols, &w->right_q, &w->left_q, w->sigma, w->k};
  return split_gemm(h, a, b, y, y_dtype, ldy, ws, ws_bytes, reinterpret_cast<cudaStream_t>(stream));
}

metis_status_t metis_linear_bwd(metis_handle_t h, const metis_operand_t* dy, const metis_operand_t* x,
                                const metis_operand_t* w, void* dx, int32_t dx_dtype, int64_t lddx, void* dw,
                                int32_t dw_dtype, int64_t lddw, float* d_left, float* d_sigma, float* d_right,
                                void* ws, size_t ws_bytes, metis_stream_t stream) {
  METIS_NVTX("metis_linear_bwd");
  if (!h || !dy) return METIS_ERR_INVALID_ARG;
  if ((d_left || d_sigma || d_right) && (!dw || !w)) return METIS_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  // every host-detectable error is reported before anything is enqueued
  if (dx && (!w || dy->cols != w->rows)) return METIS_ERR_SHAPE;
  if (dw && (!x || dy->rows != x->rows)) return METIS_ERR_SHAPE;
  if (dx && ((dx_dtype != METIS_BF16 && dx_dtype != METIS_FP32))) return METIS_ERR_INVALID_ARG;
  if (dw && ((dw_dtype != METIS_BF16 && dw_dtype != METIS_FP32))) return METIS_ERR_INVALID_ARG;
  if (dx && lddx < w->cols) return METIS_ERR_SHAPE;
  if (dw && lddw < x->cols) return METIS_ERR_SHAPE;
  if (dw && (d_left || d_sigma || d_right)) {
    if (w->rows != dy->cols || w->cols != x->cols) return METIS_ERR_SHAPE;
    METIS_TRY(factor_grads_check(w, d_left, d_sigma, ws, ws_bytes));
  }
  // dX (l x m) = D W_t, contraction over out-features n: D by columns, W_t by rows (stored m x n)
  Side da{&dy->res_by_cols, &dy->right_q, &dy->left_q, dy->sigma, dy->k};
  Side db = w ? Side{&w->res_by_rows, &w->left_q, &w->right_q, w->sigma, w->k} : Side{};
  // dW_t (n x m) = D^T X, contraction over tokens l: both by rows (stored n x l and m x l)
  Side wa{&dy->res_by_rows, &dy->left_q, &dy->right_q, dy->sigma, dy->k};
  Side wb = x ? Side{&x->res_by_rows, &x->left_q, &x->right_q, x->sigma, x->k} : Side{};
  if (dx && dw) {
    // Both products: with room for two sets of intermediates, everything that precedes the weight gradient's
    // large GEMM runs on a side stream underneath the input gradient.
    Plan pd, pw;
    METIS_TRY(make_plan(da, db, ws, ws_bytes, &pd));
    const size_t off = pd.bytes;
    const metis_status_t st = make_plan(wa, wb, ws ? reinterpret_cast<unsigned char*>(ws) + off : nullptr,
                                        ws_bytes > off ? ws_bytes - off : 0, &pw);
    if (st == METIS_OK) {
      // all six skinny products at once (a large GEMM, once resident, leaves no SM to a kernel that comes later)
      METIS_TRY(metis_fork(h, s, METIS_N_SIDE));
      METIS_TRY(split_gemm_prologue(h, wa, wb, pw, 3, h->side[2]));
      METIS_TRY(split_gemm_prologue(h, da, db, pd, 0, s));
      METIS_TRY(split_gemm_main(h, da, db, pd, dx, dx_dtype, lddx, s));
      METIS_TRY(metis_join(h, s, 2));
      METIS_TRY(split_gemm_main(h, wa, wb, pw, dw, dw_dtype, lddw, s));
    } else if (st == METIS_ERR_WORKSPACE) {
      METIS_TRY(split_gemm(h, da, db, dx, dx_dtype, lddx, ws, ws_bytes, s));
      METIS_TRY(split_gemm(h, wa, wb, dw, dw_dtype, lddw, ws, ws_bytes, s));
    } else {
      return st;
    }
  } else if (dx) {
    METIS_TRY(split_gemm(h, da, db, dx, dx_dtype, lddx, ws, ws_bytes, s));
  } else if (dw) {
    METIS_TRY(split_gemm(h, wa, wb, dw, dw_dtype, lddw, ws, ws_bytes, s));
  }
  if (dw && (d_left || d_sigma || d_right))
    METIS_TRY(factor_grads(h, dw, dw_dtype, lddw, w, d_left, d_sigma, d_right, ws, ws_bytes, s));
  return METIS_OK;
}
