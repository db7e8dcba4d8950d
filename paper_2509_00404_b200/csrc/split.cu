// Low-rank + residual split of one GEMM operand (Sections 3.1 and 3.2) and its NVFP4 quantization.
//
// Steps (FULL = on all rows, SAMPLED = subspace from a sparse row sample, "broadcast" to all rows):
//   amax(x) -> row sample -> sketch Z = x[S,:] Omega (Omega from Philox + quantile table, never stored)
//   -> CholeskyQR2 (FP64 Gram + Cholesky) -> M = H^T x[S,:] -> eigen-decomposition of M M^T (Jacobi,
//   FP64) -> right basis B -> [SAMPLED: C = x B, Rayleigh-Ritz on C^T C] -> residual R = x - C B^T fused
//   with the NVFP4 quantizer in both block orientations -> factor rotation, sign fix, factor quantization.
#include "quant_tile.cuh"

namespace {

constexpr int MAXQ = 64;
constexpr size_t JACOBI_SMEM = sizeof(double) * 2 * MAXQ * (MAXQ + 1);

// ------------------------------------------------------------------------------------------------
__global__ void sample_rows_kernel(int* __restrict__ idx, int n_s, int64_t rows, uint64_t seed, int full) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n_s) return;
  if (full) { idx[j] = j; return; }
  const uint32_t g = (uint32_t)(rows / n_s);
  const uint4 w = metis_philox((uint32_t)j, 0u, METIS_STREAM_SAMPLING, 0u, (uint32_t)seed, (uint32_t)(seed >> 32));
  idx[j] = (int)((uint32_t)j * g + w.x % g);          // one row per stratum of g consecutive rows
}

// ------------------------------------------------------------------------------------------------
// Sketch partials: Zp[chunk][row][j] = sum over the chunk's 256 columns of x[idx[row], col] * Omega[col, j].
constexpr int SK_ROWS = 16, SK_COLS = 256;
__global__ void __launch_bounds__(256)
sketch_kernel(const __nv_bfloat16* __restrict__ x, int64_t cols, const int* __restrict__ idx, int n_s, int q,
              uint64_t seed, const __nv_bfloat16* __restrict__ lut, float* __restrict__ zp) {
  extern __shared__ __align__(16) unsigned char smem[];
  float* om = reinterpret_cast<float*>(smem);                  // [SK_COLS * q]
  float* xs = om + SK_COLS * q;                                // [SK_ROWS][SK_COLS]
  const int tid = threadIdx.x;
  const int64_t col0 = (int64_t)blockIdx.y * SK_COLS;
  const int row0 = blockIdx.x * SK_ROWS;
  const int ncols = (int)min((int64_t)SK_COLS, cols - col0);
  // Omega rows col0 .. col0+ncols: logical indices e = col*q + j form one contiguous range
  const uint64_t e_lo = (uint64_t)col0 * q, e_hi = (uint64_t)(col0 + ncols) * q;
  for (uint64_t blk = (e_lo >> 3) + tid; blk <= ((e_hi - 1) >> 3); blk += 256) {
    const uint4 w = metis_philox_block(blk, seed, METIS_STREAM_OMEGA);
#pragma unroll
    for (uint32_t h = 0; h < 8; ++h) {
      const uint64_t e = (blk << 3) + h;
      if (e >= e_lo && e < e_hi) om[e - e_lo] = __bfloat162float(lut[metis_u16_of(w, h)]);
    }
  }
  for (int i = tid; i < SK_ROWS * SK_COLS; i += 256) {
    const int r = i / SK_COLS, c = i % SK_COLS;
    xs[i] = (row0 + r < n_s && c < ncols) ? __bfloat162float(x[(int64_t)idx[row0 + r] * cols + col0 + c]) : 0.0f;
  }
  __syncthreads();
  for (int o = tid; o < SK_ROWS * q; o += 256) {
    const int r = o / q, j = o % q;
    float acc = 0.0f;
    for (int t = 0; t < ncols; ++t) acc = fmaf(xs[r * SK_COLS + t], om[t * q + j], acc);
    if (row0 + r < n_s) zp[((int64_t)blockIdx.y * n_s + row0 + r) * q + j] = acc;
  }
}

__global__ void reduce_partials_kernel(const float* __restrict__ zp, int n_chunks, int64_t n, float* __restrict__ z) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= n) return;
  float acc = 0.0f;
  for (int c = 0; c < n_chunks; ++c) acc += zp[(int64_t)c * n + i];     // fixed order: reproducible
  z[i] = acc;
}

// ------------------------------------------------------------------------------------------------
// Gram partials in FP64: part[p][i][j] = sum over the p-th slab of rows r of v(r,i) v(r,j),
// v(r,i) = V[r*stride_row + i*stride_vec].
constexpr int GR_TILE = 32;
__global__ void __launch_bounds__(256)
gram_kernel(const float* __restrict__ v, int64_t n_rows, int n, int64_t stride_row, int64_t stride_vec,
            int64_t rows_per_part, double* __restrict__ part) {
  __shared__ float tile[GR_TILE][MAXQ + 1];
  const int tid = threadIdx.x;
  const int64_t r_begin = (int64_t)blockIdx.x * rows_per_part;
  const int64_t r_end = min(n_rows, r_begin + rows_per_part);
  double acc[(MAXQ * MAXQ + 255) / 256];
#pragma unroll
  for (int e = 0; e < (MAXQ * MAXQ + 255) / 256; ++e) acc[e] = 0.0;
  for (int64_t r0 = r_begin; r0 < r_end; r0 += GR_TILE) {
    for (int i = tid; i < GR_TILE * n; i += 256) {
      int rr, ii;
      if (stride_row == 1) { rr = i % GR_TILE; ii = i / GR_TILE; } else { ii = i % n; rr = i / n; }
      tile[rr][ii] = (r0 + rr < r_end) ? v[(r0 + rr) * stride_row + ii * stride_vec] : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int e = 0; e < (MAXQ * MAXQ + 255) / 256; ++e) {
      const int o = tid + e * 256;
      if (o < n * n) {
        const int i = o / n, j = o % n;
        double a = acc[e];
#pragma unroll 8
        for (int rr = 0; rr < GR_TILE; ++rr) a += (double)tile[rr][i] * (double)tile[rr][j];
        acc[e] = a;
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int e = 0; e < (MAXQ * MAXQ + 255) / 256; ++e) {
    const int o = tid + e * 256;
    if (o < n * n) part[(int64_t)blockIdx.x * n * n + o] = acc[e];
  }
}

// ------------------------------------------------------------------------------------------------
// One CholeskyQR pass: G = sum of Gram partials = L L^T (FP64, in shared memory, every CTA redundantly),
// then z_row <- z_row L^-T for the CTA's rows.  A pivot below 1e-13 of the largest diagonal marks a
// dependent sketch column: its output column becomes zero instead of amplified noise.
__global__ void __launch_bounds__(128)
cholqr_apply_kernel(float* __restrict__ z, int64_t n_rows, int q, const double* __restrict__ part, int n_parts,
                    uint32_t* dev_status) {
  __shared__ double L[MAXQ][MAXQ + 1];
  __shared__ double invd[MAXQ];
  __shared__ double gmax_s;
  const int tid = threadIdx.x;
  for (int o = tid; o < q * q; o += 128) {
    double s = 0.0;
    for (int p = 0; p < n_parts; ++p) s += part[(int64_t)p * q * q + o];
    L[o / q][o % q] = s;
  }
  __syncthreads();
  if (tid == 0) {
    double g = 0.0;
    for (int i = 0; i < q; ++i) g = fmax(g, L[i][i]);
    gmax_s = g;
  }
  __syncthreads();
  const double tol = 1e-13 * gmax_s;
  for (int j = 0; j < q; ++j) {
    const double d = L[j][j];
    const bool dep = !(d > tol);
    __syncthreads();
    if (dep) {
      for (int i = j + tid; i < q; i += 128) L[i][j] = 0.0;
      if (tid == 0) invd[j] = 0.0;
    } else {
      const double ljj = sqrt(d);
      for (int i = j + 1 + tid; i < q; i += 128) L[i][j] /= ljj;
      if (tid == 0) { L[j][j] = ljj; invd[j] = 1.0 / ljj; }
    }
    __syncthreads();
    if (!dep) {
      const int m = q - j - 1;
      for (int o = tid; o < m * m; o += 128) {
        const int a = j + 1 + o / m, b = j + 1 + o % m;
        if (b <= a) L[a][b] -= L[a][j] * L[b][j];
      }
    }
    __syncthreads();
  }
  const int64_t r = (int64_t)blockIdx.x * 128 + tid;
  if (r < n_rows) {
    double h[MAXQ];
    for (int j = 0; j < q; ++j) {
      double s = (double)z[r * q + j];
      for (int i = 0; i < j; ++i) s -= h[i] * L[j][i];
      h[j] = s * invd[j];
    }
    for (int j = 0; j < q; ++j) z[r * q + j] = (float)h[j];
  }
  (void)dev_status;
}

// ------------------------------------------------------------------------------------------------
// M[j][col] = sum_r H[r][j] * x[idx[r], col]     (q x cols, row j contiguous)
constexpr int PJ_COLS = 128, PJ_ROWS = 32;
__global__ void __launch_bounds__(256)
project_kernel(const __nv_bfloat16* __restrict__ x, int64_t cols, const int* __restrict__ idx, int n_s, int q,
               const float* __restrict__ h, float* __restrict__ m) {
  __shared__ float hs[PJ_ROWS][MAXQ];
  const int tid = threadIdx.x, c = tid & (PJ_COLS - 1), jg = tid >> 7;       // 2 groups of factor indices
  const int64_t col = (int64_t)blockIdx.x * PJ_COLS + c;
  float acc[MAXQ / 2];
#pragma unroll
  for (int j = 0; j < MAXQ / 2; ++j) acc[j] = 0.0f;
  for (int r0 = 0; r0 < n_s; r0 += PJ_ROWS) {
    for (int i = tid; i < PJ_ROWS * q; i += 256) {
      const int rr = i / q, jj = i % q;
      hs[rr][jj] = (r0 + rr < n_s) ? h[(int64_t)(r0 + rr) * q + jj] : 0.0f;
    }
    __syncthreads();
    const int nr = min(PJ_ROWS, n_s - r0);
    for (int rr = 0; rr < nr; ++rr) {
      const float xv = col < cols ? __bfloat162float(x[(int64_t)idx[r0 + rr] * cols + col]) : 0.0f;
#pragma unroll
      for (int j = 0; j < MAXQ / 2; ++j)
        if (2 * j + jg < q) acc[j] = fmaf(hs[rr][2 * j + jg], xv, acc[j]);
    }
    __syncthreads();
  }
  if (col < cols)
#pragma unroll
    for (int j = 0; j < MAXQ / 2; ++j)
      if (2 * j + jg < q) m[(int64_t)(2 * j + jg) * cols + col] = acc[j];
}

// ------------------------------------------------------------------------------------------------
// Symmetric eigen-decomposition (n <= 64) by parallel-order cyclic Jacobi in FP64, one CTA.
// Input: Gram partials.  Output: eigenvalues descending, eigenvectors as columns of vec[n][n].
__global__ void __launch_bounds__(256)
jacobi_eig_kernel(const double* __restrict__ part, int n_parts, int n, double* __restrict__ evals,
                  double* __restrict__ evecs) {
  extern __shared__ __align__(16) unsigned char jsm[];
  double (*A)[MAXQ + 1] = reinterpret_cast<double (*)[MAXQ + 1]>(jsm);
  double (*V)[MAXQ + 1] = reinterpret_cast<double (*)[MAXQ + 1]>(jsm + sizeof(double) * MAXQ * (MAXQ + 1));
  __shared__ double cs[MAXQ / 2][2];
  __shared__ int pr[MAXQ / 2][2];
  __shared__ double red[2];
  __shared__ int order[MAXQ];
  const int tid = threadIdx.x;
  for (int o = tid; o < n * n; o += 256) {
    double s = 0.0;
    for (int p = 0; p < n_parts; ++p) s += part[(int64_t)p * n * n + o];
    A[o / n][o % n] = s;
    V[o / n][o % n] = (o / n == o % n) ? 1.0 : 0.0;
  }
  __syncthreads();
  for (int o = tid; o < n * n; o += 256) {            // symmetrise (partials are symmetric up to summation order)
    const int i = o / n, j = o % n;
    if (i < j) { const double s = 0.5 * (A[i][j] + A[j][i]); A[i][j] = s; A[j][i] = s; }
  }
  __syncthreads();
  const int np = n + (n & 1), half = np / 2;
  for (int sweep = 0; sweep < 14; ++sweep) {
    if (tid == 0) {
      double off = 0.0, dg = 0.0;
      for (int i = 0; i < n; ++i) {
        dg += A[i][i] * A[i][i];
        for (int j = i + 1; j < n; ++j) off += A[i][j] * A[i][j];
      }
      red[0] = off; red[1] = dg;
    }
    __syncthreads();
    if (red[0] <= 1e-30 * red[1] || red[0] == 0.0) break;
    for (int step = 0; step < np - 1; ++step) {
      if (tid < half) {
        int a, b;
        if (tid == 0) { a = 0; b = (step % (np - 1)) + 1; }
        else { a = ((step + tid) % (np - 1)) + 1; b = ((step + np - 1 - tid) % (np - 1)) + 1; }
        if (a > b) { const int t = a; a = b; b = t; }
        double c = 1.0, s = 0.0;
        if (b < n) {
          const double apq = A[a][b];
          if (fabs(apq) > 1e-300) {
            const double theta = (A[b][b] - A[a][a]) / (2.0 * apq);
            const double t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
            c = 1.0 / sqrt(t * t + 1.0);
            s = t * c;
          }
        }
        pr[tid][0] = a; pr[tid][1] = b; cs[tid][0] = c; cs[tid][1] = s;
      }
      __syncthreads();
      for (int o = tid; o < half * n; o += 256) {       // rows p,q of A <- J^T A
        const int m = o / n, col = o % n;
        const int p = pr[m][0], q2 = pr[m][1];
        if (q2 < n) {
          const double c = cs[m][0], s = cs[m][1];
          const double ap = A[p][col], aq = A[q2][col];
          A[p][col] = c * ap - s * aq;
          A[q2][col] = s * ap + c * aq;
        }
      }
      __syncthreads();
      for (int o = tid; o < half * n; o += 256) {       // columns p,q of A and V <- (.) J
        const int m = o / n, row = o % n;
        const int p = pr[m][0], q2 = pr[m][1];
        if (q2 < n) {
          const double c = cs[m][0], s = cs[m][1];
          const double ap = A[row][p], aq = A[row][q2];
          A[row][p] = c * ap - s * aq;
          A[row][q2] = s * ap + c * aq;
          const double vp = V[row][p], vq = V[row][q2];
          V[row][p] = c * vp - s * vq;
          V[row][q2] = s * vp + c * vq;
        }
      }
      __syncthreads();
    }
  }
  __syncthreads();
  if (tid < n) {
    const double li = A[tid][tid];
    int rank = 0;
    for (int j = 0; j < n; ++j) {
      const double lj = A[j][j];
      rank += (lj > li) || (lj == li && j < tid);
    }
    order[rank] = tid;
  }
  __syncthreads();
  if (tid < n) evals[tid] = A[order[tid]][order[tid]];
  for (int o = tid; o < n * n; o += 256) evecs[o] = V[o / n][order[o % n]];
}

// ------------------------------------------------------------------------------------------------
// Right basis from the small SVD: B[j][col] = sum_i Ut[i][j] M[i][col] / s_j, s_j = sqrt(eval_j); j < k.
__global__ void __launch_bounds__(256)
right_basis_kernel(const float* __restrict__ m, int64_t cols, int q, int k, const double* __restrict__ evals,
                   const double* __restrict__ evecs, float* __restrict__ basis, float* __restrict__ sigma_out) {
  __shared__ double ut[MAXQ][MAXQ + 1];
  __shared__ double inv_s[MAXQ];
  const int tid = threadIdx.x;
  for (int o = tid; o < q * q; o += 256) ut[o / q][o % q] = evecs[o];
  if (tid < k) {
    const double s = sqrt(fmax(evals[tid], 0.0));
    inv_s[tid] = s > 0.0 ? 1.0 / s : 0.0;
    if (blockIdx.x == 0 && sigma_out != nullptr) sigma_out[tid] = (float)s;
  }
  __syncthreads();
  const int64_t col = (int64_t)blockIdx.x * 256 + tid;
  if (col >= cols) return;
  float mv[MAXQ];
  for (int i = 0; i < q; ++i) mv[i] = m[(int64_t)i * cols + col];
  for (int j = 0; j < k; ++j) {
    double a = 0.0;
    for (int i = 0; i < q; ++i) a += ut[i][j] * (double)mv[i];
    basis[(int64_t)j * cols + col] = (float)(a * inv_s[j]);
  }
}

// ------------------------------------------------------------------------------------------------
// Broadcast of the sampled subspace to every row: Ct[j][r] = sum_col x[r, col] * B[j][col].
constexpr int CF_ROWS = 32, CF_COLS = 128;
__global__ void __launch_bounds__(256)
coeff_kernel(const __nv_bfloat16* __restrict__ x, int64_t rows, int64_t cols, int k, const float* __restrict__ basis,
             float* __restrict__ coef_t) {
  extern __shared__ __align__(16) unsigned char smem[];
  float* xs = reinterpret_cast<float*>(smem);                 // [CF_ROWS][CF_COLS + 1]
  float* bs = xs + CF_ROWS * (CF_COLS + 1);                   // [k][CF_COLS + 1]
  const int tid = threadIdx.x, r = tid >> 3, jg = tid & 7;
  const int64_t row0 = (int64_t)blockIdx.x * CF_ROWS;
  float acc[MAXQ / 8];
#pragma unroll
  for (int j = 0; j < MAXQ / 8; ++j) acc[j] = 0.0f;
  for (int64_t c0 = 0; c0 < cols; c0 += CF_COLS) {
    for (int i = tid; i < CF_ROWS * CF_COLS; i += 256) {
      const int rr = i / CF_COLS, cc = i % CF_COLS;
      xs[rr * (CF_COLS + 1) + cc] =
          (row0 + rr < rows && c0 + cc < cols) ? __bfloat162float(x[(row0 + rr) * cols + c0 + cc]) : 0.0f;
    }
    for (int i = tid; i < k * CF_COLS; i += 256) {
      const int jj = i / CF_COLS, cc = i % CF_COLS;
      bs[jj * (CF_COLS + 1) + cc] = (c0 + cc < cols) ? basis[(int64_t)jj * cols + c0 + cc] : 0.0f;
    }
    __syncthreads();
    for (int t = 0; t < CF_COLS; ++t) {
      const float xv = xs[r * (CF_COLS + 1) + t];
#pragma unroll
      for (int j = 0; j < MAXQ / 8; ++j)
        if (j * 8 + jg < k) acc[j] = fmaf(xv, bs[(j * 8 + jg) * (CF_COLS + 1) + t], acc[j]);
    }
    __syncthreads();
  }
  if (row0 + r < rows)
#pragma unroll
    for (int j = 0; j < MAXQ / 8; ++j)
      if (j * 8 + jg < k) coef_t[(int64_t)(j * 8 + jg) * rows + row0 + r] = acc[j];
}

// ------------------------------------------------------------------------------------------------
// Fused residual + quantizer: R = x - sum_j coefT[j][r] * scale_j * basis[j][col] on a 128 x 128 tile,
// then NVFP4 in one or both block orientations straight from shared memory (the residual never goes
// to HBM unless `dense` is given).
__global__ void __launch_bounds__(metis_qt::THREADS)
residual_quant_kernel(const __nv_bfloat16* __restrict__ x, int k, const float* __restrict__ coef_t,
                      const float* __restrict__ scale, const float* __restrict__ basis, metis_qt::QuantParams p,
                      const float* __restrict__ amax_src, float* ts_out0, float* ts_out1, float* __restrict__ dense) {
  using namespace metis_qt;
  extern __shared__ __align__(16) unsigned char smem[];
  float* tile = reinterpret_cast<float*>(smem);
  Stage* stage = reinterpret_cast<Stage*>(smem + sizeof(float) * TILE * PITCH);
  unsigned char* after = smem + sizeof(float) * TILE * PITCH + sizeof(Stage);
  const bool sr = p.rounding == METIS_ROUND_SR;
  uint16_t* rnd = reinterpret_cast<uint16_t*>(after);
  float* cs = reinterpret_cast<float*>(after + (sr ? sizeof(uint16_t) * TILE * TILE : 0));   // [k][TILE]
  float* bs = cs + k * TILE;                                                                 // [k][TILE]

  const int tid = threadIdx.x;
  const int64_t row0 = (int64_t)blockIdx.y * TILE, col0 = (int64_t)blockIdx.x * TILE;
  const float s_T = metis_tensor_scale(*amax_src);
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) {
    if (ts_out0) *ts_out0 = s_T;
    if (ts_out1) *ts_out1 = s_T;
  }
  for (int i = tid; i < TILE * (TILE / 8); i += THREADS) {
    const int r = i >> 4, g = i & 15;
    const int64_t gr = row0 + r, gc = col0 + g * 8;
    float v[8];
    if (gr < p.rows && gc + 8 <= p.cols) {
      const uint4 q = *reinterpret_cast<const uint4*>(x + gr * p.cols + gc);
      const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) { v[2 * j] = __uint_as_float(w[j] << 16); v[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u); }
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = (gr < p.rows && gc + j < p.cols) ? __bfloat162float(x[gr * p.cols + gc + j]) : 0.0f;
    }
    *reinterpret_cast<float4*>(tile + r * PITCH + g * 8) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(tile + r * PITCH + g * 8 + 4) = make_float4(v[4], v[5], v[6], v[7]);
  }
  for (int i = tid; i < k * TILE; i += THREADS) {
    const int j = i >> 7, t = i & 127;
    const float sc = scale ? scale[j] : 1.0f;
    cs[i] = (row0 + t < p.rows) ? coef_t[(int64_t)j * p.rows + row0 + t] * sc : 0.0f;
    bs[i] = (col0 + t < p.cols) ? basis[(int64_t)j * p.cols + col0 + t] : 0.0f;
  }
  if (sr) fill_draws(rnd, p, row0, col0);
  __syncthreads();
  {
    const int r0 = (tid >> 4) * 8, c0 = (tid & 15) * 8;
    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[i][j] = 0.0f;
    for (int j = 0; j < k; ++j) {
      const float4 a0 = *reinterpret_cast<const float4*>(cs + j * TILE + r0), a1 = *reinterpret_cast<const float4*>(cs + j * TILE + r0 + 4);
      const float4 b0 = *reinterpret_cast<const float4*>(bs + j * TILE + c0), b1 = *reinterpret_cast<const float4*>(bs + j * TILE + c0 + 4);
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) acc[i][jj] = fmaf(a[i], b[jj], acc[i][jj]);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float* t = tile + (r0 + i) * PITCH + c0;
      float4 v0 = *reinterpret_cast<float4*>(t), v1 = *reinterpret_cast<float4*>(t + 4);
      v0.x -= acc[i][0]; v0.y -= acc[i][1]; v0.z -= acc[i][2]; v0.w -= acc[i][3];
      v1.x -= acc[i][4]; v1.y -= acc[i][5]; v1.z -= acc[i][6]; v1.w -= acc[i][7];
      *reinterpret_cast<float4*>(t) = v0; *reinterpret_cast<float4*>(t + 4) = v1;
      if (dense != nullptr && row0 + r0 + i < p.rows && col0 + c0 + 8 <= p.cols) {
        float* d = dense + (row0 + r0 + i) * p.cols + col0 + c0;
        *reinterpret_cast<float4*>(d) = v0; *reinterpret_cast<float4*>(d + 4) = v1;
      }
    }
  }
  __syncthreads();
  quantize_tile(tile, rnd, stage, p, row0, col0, s_T);
}

// ------------------------------------------------------------------------------------------------
// right[j][col] = sum_i basis[i][col] * W[i][j] (W == nullptr: identity), then the sign convention:
// the largest-magnitude entry of each right vector (lowest index on ties) is made positive.
__global__ void __launch_bounds__(256)
right_rotate_sign_kernel(const float* __restrict__ basis, int64_t cols, int n_in, const double* __restrict__ w,
                         float* __restrict__ right, float* __restrict__ sign_out) {
  __shared__ double wj[MAXQ];
  __shared__ float best_v[256];
  __shared__ long long best_i[256];
  const int j = blockIdx.x, tid = threadIdx.x;
  if (tid < n_in) wj[tid] = w ? w[tid * n_in + j] : (tid == j ? 1.0 : 0.0);
  __syncthreads();
  float bv = -1.0f, bsgn = 1.0f;
  long long bi = 0x7FFFFFFFFFFFFFFFll;
  for (int64_t col = tid; col < cols; col += 256) {
    double a = 0.0;
    if (w) { for (int i = 0; i < n_in; ++i) a += (double)basis[(int64_t)i * cols + col] * wj[i]; }
    else a = (double)basis[(int64_t)j * cols + col];
    const float v = (float)a;
    right[(int64_t)j * cols + col] = v;
    if (fabsf(v) > bv) { bv = fabsf(v); bi = col; bsgn = v < 0.0f ? -1.0f : 1.0f; }
  }
  best_v[tid] = bv; best_i[tid] = bi;
  __shared__ float sgn_s[256];
  sgn_s[tid] = bsgn;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (tid < s) {
      const bool take = best_v[tid + s] > best_v[tid] || (best_v[tid + s] == best_v[tid] && best_i[tid + s] < best_i[tid]);
      if (take) { best_v[tid] = best_v[tid + s]; best_i[tid] = best_i[tid + s]; sgn_s[tid] = sgn_s[tid + s]; }
    }
    __syncthreads();
  }
  const float sg = sgn_s[0];
  if (tid == 0) sign_out[j] = sg;
  if (sg < 0.0f)
    for (int64_t col = tid; col < cols; col += 256) right[(int64_t)j * cols + col] = -right[(int64_t)j * cols + col];
}

// left[j][r] = sign_j * scale_j * sum_i coef(i, r) * W[i][j],  coef(i, r) = c[i*stride_i + r*stride_r]
// scale_j = 1/sqrt(eval_j) when inv_sqrt_evals is given (Rayleigh-Ritz normalisation), else 1.
// Also writes sigma_out[j] = sqrt(eval_j) when asked.
__global__ void __launch_bounds__(256)
left_rotate_kernel(const float* __restrict__ c, int64_t rows, int n_in, int k, int64_t stride_i, int64_t stride_r,
                   const double* __restrict__ w, const double* __restrict__ evals_for_scale,
                   const float* __restrict__ sign, float* __restrict__ left, float* __restrict__ sigma_out) {
  __shared__ double ws[MAXQ][MAXQ + 1];
  __shared__ double scl[MAXQ];
  const int tid = threadIdx.x;
  for (int o = tid; o < n_in * n_in; o += 256) ws[o / n_in][o % n_in] = w[o];
  if (tid < k) {
    double s = 1.0;
    if (evals_for_scale) {
      const double lam = sqrt(fmax(evals_for_scale[tid], 0.0));
      s = lam > 0.0 ? 1.0 / lam : 0.0;
      if (blockIdx.x == 0 && sigma_out) sigma_out[tid] = (float)lam;
    }
    scl[tid] = s * (double)sign[tid];
  }
  __syncthreads();
  const int64_t r = (int64_t)blockIdx.x * 256 + tid;
  if (r >= rows) return;
  float cv[MAXQ];
  for (int i = 0; i < n_in; ++i) cv[i] = c[i * stride_i + r * stride_r];
  for (int j = 0; j < k; ++j) {
    double a = 0.0;
    for (int i = 0; i < n_in; ++i) a += (double)cv[i] * ws[i][j];
    left[(int64_t)j * rows + r] = (float)(a * scl[j]);
  }
}

struct SplitWs {
  size_t amax, idx, zp, z, gram, evals, evecs, m, basis, coef, sign, evals2, evecs2, total;
};

SplitWs split_ws_layout(int64_t rows, int64_t cols, int k, int p, int64_t n_s) {
  SplitWs w{};
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 255) & ~(size_t)255; return o; };
  const int q = k + p;
  const int64_t chunks = metis_ceil_div(cols, SK_COLS);
  w.amax = take(256);
  w.idx = take(sizeof(int) * (size_t)n_s);
  w.zp = take(sizeof(float) * (size_t)chunks * n_s * q);
  w.z = take(sizeof(float) * (size_t)n_s * q);
  w.gram = take(sizeof(double) * 64 * MAXQ * MAXQ);
  w.evals = take(sizeof(double) * MAXQ);
  w.evecs = take(sizeof(double) * MAXQ * MAXQ);
  w.m = take(sizeof(float) * (size_t)q * cols);
  w.basis = take(sizeof(float) * (size_t)k * cols);
  w.coef = take(sizeof(float) * (size_t)k * rows);
  w.sign = take(sizeof(float) * MAXQ);
  w.evals2 = take(sizeof(double) * MAXQ);
  w.evecs2 = take(sizeof(double) * MAXQ * MAXQ);
  w.total = off;
  return w;
}

int gram_parts(int64_t n_rows, int64_t* rows_per_part) {
  int parts = (int)metis_ceil_div(n_rows, 512);
  if (parts > 64) parts = 64;
  if (parts < 1) parts = 1;
  int64_t rpp = metis_ceil_div(n_rows, parts);
  rpp = metis_ceil_div(rpp, GR_TILE) * GR_TILE;
  *rows_per_part = rpp;
  return (int)metis_ceil_div(n_rows, rpp);
}

}  // namespace

int64_t metis_default_sample_count(int64_t rows, int32_t q) {
  int64_t want = 4 * (int64_t)q;
  const int64_t pct = (rows + 99) / 100;
  if (pct > want) want = pct;
  want = (want + 15) / 16 * 16;
  return want < rows ? want : rows;
}

size_t metis_split_ws_bytes(int64_t rows, int64_t cols, int k, int p) {
  // sized for the FULL sketch (n_s = rows), which bounds the SAMPLED one
  return split_ws_layout(rows, cols, k, p, rows).total;
}

metis_status_t metis_split(metis_handle_t h, const void* xv, int64_t rows, int64_t cols, int32_t k, int32_t p,
                           int32_t sketch, int64_t n_sample, uint64_t seed, int32_t rounding, int32_t residual_axes,
                           metis_operand_t* out, float* residual_dense, void* ws, size_t ws_bytes,
                           metis_stream_t stream) {
  using namespace metis_qt;
  if (!h || !xv || !out || !ws) return METIS_ERR_INVALID_ARG;
  if (rows <= 0 || cols <= 0 || rows % 16 || cols % 16 || k < 0 || p < 0) return METIS_ERR_SHAPE;
  if (k > 0 && (k + p > MAXQ || k % 4)) return METIS_ERR_SHAPE;
  if (out->k != k || out->rows != rows || out->cols != cols) return METIS_ERR_INVALID_ARG;
  if (!metis_aligned16(xv) || !metis_aligned16(ws)) return METIS_ERR_ALIGNMENT;
  if (rounding != METIS_ROUND_RNE && rounding != METIS_ROUND_SR) return METIS_ERR_INVALID_ARG;
  if (sketch != METIS_SKETCH_FULL && sketch != METIS_SKETCH_SAMPLED) return METIS_ERR_INVALID_ARG;
  const bool want_c = (residual_axes & METIS_BLOCKS_ALONG_COLS) != 0, want_r = (residual_axes & METIS_BLOCKS_ALONG_ROWS) != 0;
  if (want_c && (!out->res_by_cols.codes || !out->res_by_cols.scales || !out->res_by_cols.tensor_scale)) return METIS_ERR_INVALID_ARG;
  if (want_r && (!out->res_by_rows.codes || !out->res_by_rows.scales || !out->res_by_rows.tensor_scale)) return METIS_ERR_INVALID_ARG;
  if (want_c && out->res_by_cols.sf_layout == METIS_SF_TILED && cols % 64) return METIS_ERR_SHAPE;
  if (want_r && out->res_by_rows.sf_layout == METIS_SF_TILED && rows % 64) return METIS_ERR_SHAPE;
  const int q = k + p;
  const bool full = sketch == METIS_SKETCH_FULL;
  int64_t n_s = full ? rows : (n_sample > 0 ? n_sample : metis_default_sample_count(rows, q));
  if (k > 0 && (n_s > rows || n_s % 16 || q > n_s || q > cols)) return METIS_ERR_SHAPE;
  if (k == 0) n_s = 16;
  const SplitWs L = split_ws_layout(rows, cols, k, p, n_s);
  if (ws_bytes < L.total) return METIS_ERR_WORKSPACE;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  unsigned char* wsb = reinterpret_cast<unsigned char*>(ws);
  const __nv_bfloat16* x = reinterpret_cast<const __nv_bfloat16*>(xv);
  float* amax = reinterpret_cast<float*>(wsb + L.amax);

  METIS_TRY(metis_launch_amax(x, METIS_BF16, rows, cols, cols, amax, s));

  metis_nvfp4_t rc = out->res_by_cols, rr = out->res_by_rows;
  rc.rows = rows; rc.k_len = cols; rr.rows = cols; rr.k_len = rows;
  if (k == 0) {
    return metis_launch_quantize(x, METIS_BF16, rows, cols, cols, rounding, seed, METIS_STREAM_RESIDUAL, cols, 1, amax,
                                 1, want_c ? &rc : nullptr, want_r ? &rr : nullptr, s);
  }
  if (!out->left || !out->sigma || !out->right || !out->left_q.codes || !out->right_q.codes || !out->left_q.scales ||
      !out->right_q.scales || !out->left_q.tensor_scale || !out->right_q.tensor_scale)
    return METIS_ERR_INVALID_ARG;
  if (out->left_q.sf_layout == METIS_SF_TILED && rows % 64) return METIS_ERR_SHAPE;
  if (out->right_q.sf_layout == METIS_SF_TILED && cols % 64) return METIS_ERR_SHAPE;

  int* idx = reinterpret_cast<int*>(wsb + L.idx);
  float* zp = reinterpret_cast<float*>(wsb + L.zp);
  float* z = reinterpret_cast<float*>(wsb + L.z);
  double* gram = reinterpret_cast<double*>(wsb + L.gram);
  double* evals = reinterpret_cast<double*>(wsb + L.evals);
  double* evecs = reinterpret_cast<double*>(wsb + L.evecs);
  float* m = reinterpret_cast<float*>(wsb + L.m);
  float* basis = reinterpret_cast<float*>(wsb + L.basis);
  float* coef = reinterpret_cast<float*>(wsb + L.coef);
  float* sign = reinterpret_cast<float*>(wsb + L.sign);
  double* evals2 = reinterpret_cast<double*>(wsb + L.evals2);
  double* evecs2 = reinterpret_cast<double*>(wsb + L.evecs2);
  metis_context* ctx = h;

  {
    static bool attr = false;
    if (!attr) { METIS_CUDA_TRY(cudaFuncSetAttribute(jacobi_eig_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)JACOBI_SMEM)); attr = true; }
  }
  // (1) row sample, (2) sketch
  sample_rows_kernel<<<(unsigned)metis_ceil_div(n_s, 256), 256, 0, s>>>(idx, (int)n_s, rows, seed, full ? 1 : 0); METIS_COUNT_LAUNCH();
  const int chunks = (int)metis_ceil_div(cols, SK_COLS);
  {
    const size_t smem = sizeof(float) * (SK_COLS * q + SK_ROWS * SK_COLS);
    static bool attr = false;
    if (!attr) { METIS_CUDA_TRY(cudaFuncSetAttribute(sketch_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(sizeof(float) * (SK_COLS * MAXQ + SK_ROWS * SK_COLS)))); attr = true; }
    dim3 grid((unsigned)(n_s / SK_ROWS), (unsigned)chunks);
    sketch_kernel<<<grid, 256, smem, s>>>(x, cols, idx, (int)n_s, q, seed, ctx->quantile_lut, zp); METIS_COUNT_LAUNCH();
  }
  reduce_partials_kernel<<<(unsigned)metis_ceil_div(n_s * q, 256), 256, 0, s>>>(zp, chunks, n_s * q, z); METIS_COUNT_LAUNCH();
  // (3) CholeskyQR2: orthonormal basis H of range(Z), in place
  for (int pass = 0; pass < 2; ++pass) {
    int64_t rpp; const int parts = gram_parts(n_s, &rpp);
    gram_kernel<<<parts, 256, 0, s>>>(z, n_s, q, q, 1, rpp, gram); METIS_COUNT_LAUNCH();
    cholqr_apply_kernel<<<(unsigned)metis_ceil_div(n_s, 128), 128, 0, s>>>(z, n_s, q, gram, parts, ctx->dev_status); METIS_COUNT_LAUNCH();
  }
  // (4) M = H^T x[S,:], eigen-decomposition of M M^T, right basis
  project_kernel<<<(unsigned)metis_ceil_div(cols, PJ_COLS), 256, 0, s>>>(x, cols, idx, (int)n_s, q, z, m); METIS_COUNT_LAUNCH();
  {
    int64_t rpp; const int parts = gram_parts(cols, &rpp);
    gram_kernel<<<parts, 256, 0, s>>>(m, cols, q, 1, cols, rpp, gram); METIS_COUNT_LAUNCH();
    jacobi_eig_kernel<<<1, 256, JACOBI_SMEM, s>>>(gram, parts, q, evals, evecs); METIS_COUNT_LAUNCH();
  }
  right_basis_kernel<<<(unsigned)metis_ceil_div(cols, 256), 256, 0, s>>>(m, cols, q, k, evals, evecs, basis,
                                                                          full ? out->sigma : nullptr); METIS_COUNT_LAUNCH();
  // (5) factors
  const float* res_coef; const float* res_scale; const float* res_basis;
  if (full) {
    // left = H U~_k, right = basis; residual against left * sigma * right^T
    right_rotate_sign_kernel<<<k, 256, 0, s>>>(basis, cols, k, nullptr, out->right, sign); METIS_COUNT_LAUNCH();
    left_rotate_kernel<<<(unsigned)metis_ceil_div(rows, 256), 256, 0, s>>>(z, rows, q, k, 1, q, evecs, nullptr, sign,
                                                                           out->left, nullptr); METIS_COUNT_LAUNCH();
    res_coef = out->left; res_scale = out->sigma; res_basis = out->right;
  } else {
    const size_t smem = sizeof(float) * (CF_ROWS + k) * (CF_COLS + 1);
    static bool attr = false;
    if (!attr) { METIS_CUDA_TRY(cudaFuncSetAttribute(coeff_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(sizeof(float) * (CF_ROWS + MAXQ) * (CF_COLS + 1)))); attr = true; }
    coeff_kernel<<<(unsigned)metis_ceil_div(rows, CF_ROWS), 256, smem, s>>>(x, rows, cols, k, basis, coef); METIS_COUNT_LAUNCH();
    res_coef = coef; res_scale = nullptr; res_basis = basis;
  }
  // (6) fused residual + quantizer (tensor scale from the source tensor's amax)
  {
    QuantParams qp{};
    qp.rows = rows; qp.cols = cols; qp.rounding = rounding; qp.seed = seed; qp.stream_id = METIS_STREAM_RESIDUAL;
    qp.e_stride_r = cols; qp.e_stride_c = 1;
    if (want_c) { qp.c_codes = rc.codes; qp.c_scales = rc.scales; qp.c_layout = rc.sf_layout; }
    if (want_r) { qp.r_codes = rr.codes; qp.r_scales = rr.scales; qp.r_layout = rr.sf_layout; }
    const bool sr = rounding == METIS_ROUND_SR;
    const size_t smem = smem_bytes(sr) + sizeof(float) * 2 * k * TILE;
    static bool attr = false;
    if (!attr) { METIS_CUDA_TRY(cudaFuncSetAttribute(residual_quant_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(smem_bytes(true) + sizeof(float) * 2 * MAXQ * TILE))); attr = true; }
    dim3 grid((unsigned)metis_ceil_div(cols, TILE), (unsigned)metis_ceil_div(rows, TILE));
    residual_quant_kernel<<<grid, THREADS, smem, s>>>(x, k, res_coef, res_scale, res_basis, qp, amax,
                                                      want_c ? rc.tensor_scale : nullptr,
                                                      want_r ? rr.tensor_scale : nullptr, residual_dense); METIS_COUNT_LAUNCH();
  }
  if (!full) {
    // (7) Rayleigh-Ritz on C^T C, rotate both factors, singular values
    int64_t rpp; const int parts = gram_parts(rows, &rpp);
    gram_kernel<<<parts, 256, 0, s>>>(coef, rows, k, 1, rows, rpp, gram); METIS_COUNT_LAUNCH();
    jacobi_eig_kernel<<<1, 256, JACOBI_SMEM, s>>>(gram, parts, k, evals2, evecs2); METIS_COUNT_LAUNCH();
    right_rotate_sign_kernel<<<k, 256, 0, s>>>(basis, cols, k, evecs2, out->right, sign); METIS_COUNT_LAUNCH();
    left_rotate_kernel<<<(unsigned)metis_ceil_div(rows, 256), 256, 0, s>>>(coef, rows, k, k, rows, 1, evecs2, evals2, sign,
                                                                           out->left, out->sigma); METIS_COUNT_LAUNCH();
  }
  METIS_CUDA_TRY(cudaGetLastError());
  // (8) quantize the factors (stored transposed: k x rows, k x cols; blocks along the long dimension)
  metis_nvfp4_t lq = out->left_q, rq = out->right_q;
  lq.rows = k; lq.k_len = rows; rq.rows = k; rq.k_len = cols;
  METIS_TRY(metis_launch_amax(out->left, METIS_FP32, k, rows, rows, amax + 1, s));
  METIS_TRY(metis_launch_quantize(out->left, METIS_FP32, k, rows, rows, rounding, seed, METIS_STREAM_LEFT, rows, 1,
                                  amax + 1, 1, &lq, nullptr, s));
  METIS_TRY(metis_launch_amax(out->right, METIS_FP32, k, cols, cols, amax + 2, s));
  METIS_TRY(metis_launch_quantize(out->right, METIS_FP32, k, cols, cols, rounding, seed, METIS_STREAM_RIGHT, cols, 1,
                                  amax + 2, 1, &rq, nullptr, s));
  return METIS_OK;
}
