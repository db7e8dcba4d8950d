// Small dense linear algebra of a split whose sketch is wider than one CTA's shared memory (k + p above 72, up to
// 272: the rank-128 and rank-256 points of the 70B-shaped sweep).  Same steps as the one-CTA kernels of split.cu
// (Section 3.1: thin QR of the sketch, small SVD of the projected operand), as kernels that tile over the rank:
//
//   gram64_kernel            G = V^T V in FP64, 64 x 64 output tiles over slabs of rows (partials, summed in order)
//   chol_wide_kernel         blocked Cholesky factor of a q x q Gram matrix (panels of 32 columns in shared memory,
//                            the matrix in L2) and the inverses of its diagonal blocks, one CTA
//   trsm_wide_kernel         H = Z L^-T by blocked forward substitution (32 rows of Z per CTA)
//   gemm64_kernel            C = A B with FP32 A, FP64 B and FP64 accumulation, arbitrary strides (right basis,
//                            factor rotations)
//   jacobi_cluster_kernel    one-sided Jacobi eigen-solver on a cluster of eight CTAs: the columns live in the
//                            cluster's distributed shared memory, column blocks travel between CTAs by DSMEM stores
//   jacobi_collect_kernel    eigenvalues (descending) and normalised eigenvectors from the rotated columns
//   sign_rows_kernel         sign convention of the factor pairs
//   coef_sum_kernel          sums the column slices of the broadcast pass into a group of coefficient columns
// Included by split.cu only.
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"

namespace metis_wide {

namespace cg = cooperative_groups;

constexpr int MAXQ_WIDE = 272;                          // 2 * JC_P * JC_W
constexpr int MAXK_WIDE = 256;

// ------------------------------------------------------------------------------------------------
// part[p][i][j] = sum over the p-th slab of rows r of v(r, i) v(r, j),  v(r, i) = V[r * sr + i * sv], FP64.
// grid (tiles_j, tiles_i, slabs); the 16 x 16 threads of a CTA own 4 x 4 outputs each.
constexpr int G64_T = 64, G64_R = 16;
__global__ void __launch_bounds__(256)
gram64_kernel(const float* __restrict__ v, int64_t n_rows, int n, int64_t sr, int64_t sv, int64_t rows_per_part,
              double* __restrict__ part, const int* __restrict__ skip) {
  metis_pdl_wait();
  if (skip != nullptr && *skip) return;
  __shared__ __align__(16) double as[G64_R][G64_T + 2], bs[G64_R][G64_T + 2];
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int i0 = blockIdx.y * G64_T, j0 = blockIdx.x * G64_T;
  const int64_t r_begin = (int64_t)blockIdx.z * rows_per_part, r_end = min(n_rows, r_begin + rows_per_part);
  double acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;
  for (int64_t r0 = r_begin; r0 < r_end; r0 += G64_R) {
    for (int o = tid; o < G64_R * G64_T; o += 256) {
      int rr, ii;
      if (sr == 1) { rr = o % G64_R; ii = o / G64_R; } else { ii = o % G64_T; rr = o / G64_T; }
      const bool okr = r0 + rr < r_end;
      as[rr][ii] = (okr && i0 + ii < n) ? (double)v[(r0 + rr) * sr + (int64_t)(i0 + ii) * sv] : 0.0;
      bs[rr][ii] = (okr && j0 + ii < n) ? (double)v[(r0 + rr) * sr + (int64_t)(j0 + ii) * sv] : 0.0;
    }
    __syncthreads();
#pragma unroll 4
    for (int rr = 0; rr < G64_R; ++rr) {
      double av[4], bv[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) { av[a] = as[rr][ty + 16 * a]; bv[a] = bs[rr][tx + 16 * a]; }
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] += av[a] * bv[b];
    }
    __syncthreads();
  }
  double* dst = part + (int64_t)blockIdx.z * n * n;
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int i = i0 + ty + 16 * a, j = j0 + tx + 16 * b;
      if (i < n && j < n) dst[(int64_t)i * n + j] = acc[a][b];
    }
}

// ------------------------------------------------------------------------------------------------
// Cholesky factor of the n x n Gram matrix g (n <= MAXQ_WIDE), one CTA of 1024 threads, blocked by panels of
// CW_NB columns (left-looking): a panel is the Gram panel minus the product of the finished columns of its rows
// with those of its own CW_NB rows - staged through shared memory in chunks of CW_NB columns, so the finished
// part of L is read once per panel - and is then factorised inside shared memory.  The matrix itself (half a
// megabyte in FP64) stays in global memory.  A pivot not above tol_rel * (largest diagonal entry) marks a
// dependent sketch column: its column of L and its row and column of the diagonal-block inverse are zero.
//   l_out     n x n row-major lower factor (strict upper part zero)
//   dinv_out  (optional) inverses of the CW_NB x CW_NB diagonal blocks of L, [panel][CW_NB][CW_NB] row-major lower:
//             what the triangular solve H = Z L^-T needs besides L itself (trsm_wide_kernel)
//   well_conditioned  (optional) 1 when every pivot is above 1e-8 of the largest diagonal entry
constexpr int CW_NB = 32, CW_P = CW_NB + 1;
constexpr int CW_ROWS = (MAXQ_WIDE + 15) / 16 * 16 + 16;   // rows of the shared panels: every row a thread's 4 x 4 tile may read exists
constexpr size_t CW_SMEM = sizeof(double) * ((size_t)2 * CW_ROWS * CW_P + CW_NB * CW_P + MAXQ_WIDE);

// acc[a][b] += sum over kk < 32 of  A[row0 + a][kk] * Bm[col0 + 8 b][kk]:  the 4 x 4 register tile of the panel products.
// The rows of a warp's four row groups and the columns col0 + 8 b of its eight column groups fall on distinct banks
// (pitch 33 doubles), so a step costs 8 shared-memory wavefronts per 16 multiply-adds of a warp.
__device__ __forceinline__ void cw_tile_mac(const double (*A)[CW_P], const double (*Bm)[CW_P], int row0, int col0, double (&acc)[4][4]) {
#pragma unroll 4
  for (int kk = 0; kk < CW_NB; ++kk) {
    double av[4], bv[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) { av[t] = A[row0 + t][kk]; bv[t] = Bm[col0 + 8 * t][kk]; }
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b2 = 0; b2 < 4; ++b2) acc[a][b2] += av[a] * bv[b2];
  }
}

// Blocked (left-looking) Cholesky factor of the n x n matrix g (symmetrised on the fly), one CTA, panels of 32 columns:
//   1. the panel (rows j0 .. n-1) minus the products with the finished columns, in 4 x 4 register tiles, the finished
//      columns streamed from global memory (L2) in chunks of 32;
//   2. the 32 x 32 diagonal block factorised by one warp (lane = row, column by column, one warp barrier per column);
//   3. the inverse of that factor by the same warp (lane = column);
//   4. the rows below the block:  L = A X^T  with X the inverse, again in register tiles.
// A pivot at or below tol_rel * max diag gives a zero column.  l_out: the factor (lower triangle, zeros above);
// dinv_out: the inverses of the diagonal blocks (32 x 32 each) for the blocked triangular solve.
__global__ void __launch_bounds__(1024, 1)
chol_wide_kernel(const double* __restrict__ g, int n, double tol_rel, double* l_out, double* dinv_out,
                 const int* __restrict__ skip, int* __restrict__ well_conditioned) {
  metis_pdl_wait();
  if (skip != nullptr && *skip) return;
  extern __shared__ __align__(16) unsigned char cw_sm[];
  double (*P)[CW_P] = reinterpret_cast<double (*)[CW_P]>(cw_sm);                                      // the panel, rows j0 .. n-1
  double (*As)[CW_P] = reinterpret_cast<double (*)[CW_P]>(cw_sm + sizeof(double) * CW_ROWS * CW_P);   // a chunk of finished columns of those rows
  double (*Dv)[CW_P] = reinterpret_cast<double (*)[CW_P]>(cw_sm + sizeof(double) * 2 * CW_ROWS * CW_P);
  double* rinv = reinterpret_cast<double*>(cw_sm + sizeof(double) * (2 * CW_ROWS * CW_P + CW_NB * CW_P));
  __shared__ double red[32];
  __shared__ double gmax_s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int o = tid; o < n * n; o += 1024) l_out[o] = 0.0;
  for (int o = tid; o < 2 * CW_ROWS * CW_P; o += 1024) reinterpret_cast<double*>(cw_sm)[o] = 0.0;   // rows past the matrix read as zeros
  double gm = 0.0;
  for (int i = tid; i < n; i += 1024) gm = fmax(gm, g[(int64_t)i * n + i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) gm = fmax(gm, __shfl_xor_sync(0xFFFFFFFFu, gm, o));
  if (lane == 0) red[warp] = gm;
  __syncthreads();
  if (tid == 0) { double m = 0.0; for (int w2 = 0; w2 < 32; ++w2) m = fmax(m, red[w2]); gmax_s = m; }
  __syncthreads();
  const double tol = tol_rel * gmax_s;
  double dmin = 1e300;                                     // smallest accepted pivot (warp 0 keeps it)
  const int row0 = 4 * (tid >> 3), col0 = tid & 7;         // this thread's tile: rows row0 .. row0 + 3, columns col0 + 8 b
  for (int j0 = 0; j0 < n; j0 += CW_NB) {
    const int w = min(CW_NB, n - j0), nr = n - j0;
    const bool mine = row0 < nr;
    __syncthreads();                                       // the previous panel is stored
    for (int o = tid; o < nr * CW_NB; o += 1024) {
      const int i = o / CW_NB, c = o % CW_NB;
      P[i][c] = c < w ? 0.5 * (g[(int64_t)(j0 + i) * n + j0 + c] + g[(int64_t)(j0 + c) * n + j0 + i]) : 0.0;
    }
    // ---- 1. minus the products with the finished columns ----
    double acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b2 = 0; b2 < 4; ++b2) acc[a][b2] = 0.0;
    for (int k0 = 0; k0 < j0; k0 += CW_NB) {
      __syncthreads();
      for (int o = tid; o < nr * CW_NB; o += 1024) { const int i = o / CW_NB, kk = o % CW_NB; As[i][kk] = l_out[(int64_t)(j0 + i) * n + k0 + kk]; }
      __syncthreads();
      if (mine) cw_tile_mac(As, As, row0, col0, acc);      // rows j0 .. j0 + 31 of L are the first rows of the chunk
    }
    __syncthreads();
    if (mine) {
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b2 = 0; b2 < 4; ++b2)
          if (row0 + a < nr && col0 + 8 * b2 < w) P[row0 + a][col0 + 8 * b2] -= acc[a][b2];
    }
    __syncthreads();
    // ---- 2. and 3.: the diagonal block and its inverse, warp 0 ----
    if (warp == 0) {
      for (int c = 0; c < w; ++c) {
        double s0 = 0.0, s1 = 0.0;
        int k = 0;
        for (; k + 1 < c; k += 2) { s0 += P[lane][k] * P[c][k]; s1 += P[lane][k + 1] * P[c][k + 1]; }
        if (k < c) s0 += P[lane][k] * P[c][k];
        const double sv = P[lane][c] - (s0 + s1);
        const double d = __shfl_sync(0xFFFFFFFFu, sv, c);
        const double r = d > tol ? 1.0 / sqrt(d) : 0.0;
        if (lane >= c && lane < w) P[lane][c] = lane == c ? d * r : sv * r;
        if (lane == 0) { rinv[j0 + c] = r; if (d > tol) dmin = fmin(dmin, d); }
        __syncwarp();
      }
      // X = L^-1, lane = column:  X[i][j] = -r_i sum_{k < i} L[i][k] X[k][j]  (X[k][j] = 0 for k < j),  X[j][j] = r_j
      for (int i = 0; i < CW_NB; ++i) Dv[i][lane] = 0.0;
      __syncwarp();
      for (int i = 0; i < w; ++i) {
        double s0 = 0.0, s1 = 0.0;
        int k = 0;
        for (; k + 1 < i; k += 2) { s0 += P[i][k] * Dv[k][lane]; s1 += P[i][k + 1] * Dv[k + 1][lane]; }
        if (k < i) s0 += P[i][k] * Dv[k][lane];
        const double ri = rinv[j0 + i];
        Dv[i][lane] = i == lane ? ri : (i > lane ? -ri * (s0 + s1) : 0.0);
      }
    }
    __syncthreads();
    // ---- 4. rows below the block: L = A X^T (X[c][cp] = Dv[c][cp], zero for cp > c) ----
    if (nr > CW_NB) {
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b2 = 0; b2 < 4; ++b2) acc[a][b2] = 0.0;
      const bool below = mine && row0 >= CW_NB;            // a tile lies wholly inside or wholly below the block
      if (below) cw_tile_mac(P, Dv, row0, col0, acc);
      __syncthreads();                                     // every tile has read its rows
      if (below) {
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int b2 = 0; b2 < 4; ++b2)
            if (row0 + a < nr) P[row0 + a][col0 + 8 * b2] = acc[a][b2];
      }
      __syncthreads();
    }
    for (int o = tid; o < nr * w; o += 1024) {
      const int i = o / w, c = o % w;
      if (i >= c) l_out[(int64_t)(j0 + i) * n + j0 + c] = P[i][c];
    }
    if (dinv_out != nullptr)
      for (int o = tid; o < CW_NB * CW_NB; o += 1024) dinv_out[(int64_t)(j0 / CW_NB) * CW_NB * CW_NB + o] = Dv[o / CW_NB][o % CW_NB];
  }
  if (tid == 0 && well_conditioned != nullptr) *well_conditioned = (dmin > 1e-8 * gmax_s) ? 1 : 0;
}

// H = Z L^-T by blocked forward substitution, in place: for panel J of CW_NB columns
//   h_J = (z_J - sum_{K < J} h_K L[J][K]^T) Dinv_J^T.
// A CTA owns 32 rows of Z and keeps their finished part of H in shared memory (FP64); L is read in CW_NB x CW_NB
// chunks.  l, dinv: outputs of chol_wide_kernel.  FP32 in, FP64 arithmetic, FP32 out.
constexpr int TW_ROWS = 32, TW_HP = MAXQ_WIDE + 1;
constexpr size_t TW_SMEM = sizeof(double) * ((size_t)TW_ROWS * TW_HP + 3 * CW_NB * CW_P);
__global__ void __launch_bounds__(256)
trsm_wide_kernel(float* __restrict__ z, int64_t n_rows, int n, const double* __restrict__ l, const double* __restrict__ dinv,
                 const int* __restrict__ skip) {
  metis_pdl_wait();
  if (skip != nullptr && *skip) return;
  extern __shared__ __align__(16) unsigned char tw_sm[];
  double (*Hs)[TW_HP] = reinterpret_cast<double (*)[TW_HP]>(tw_sm);
  double (*Ls)[CW_P] = reinterpret_cast<double (*)[CW_P]>(tw_sm + sizeof(double) * TW_ROWS * TW_HP);
  double (*Ds)[CW_P] = Ls + CW_NB;
  double (*Ts)[CW_P] = Ls + 2 * CW_NB;
  const int tid = threadIdx.x, tr = tid >> 5, tc = tid & 31;       // rows tr + 8 m, column tc of the panel
  const int64_t r0 = (int64_t)blockIdx.x * TW_ROWS;
  for (int j0 = 0; j0 < n; j0 += CW_NB) {
    const int w = min(CW_NB, n - j0);
    double acc[4];
#pragma unroll
    for (int m = 0; m < 4; ++m) {
      const int64_t r = r0 + tr + 8 * m;
      acc[m] = (r < n_rows && tc < w) ? (double)z[r * n + j0 + tc] : 0.0;
    }
    for (int k0 = 0; k0 < j0; k0 += CW_NB) {
      __syncthreads();
      for (int o = tid; o < CW_NB * CW_NB; o += 256) { const int c = o / CW_NB, kk = o % CW_NB; Ls[c][kk] = c < w ? l[(int64_t)(j0 + c) * n + k0 + kk] : 0.0; }
      __syncthreads();
#pragma unroll 8
      for (int kk = 0; kk < CW_NB; ++kk) {
        const double lv = Ls[tc][kk];
#pragma unroll
        for (int m = 0; m < 4; ++m) acc[m] -= Hs[tr + 8 * m][k0 + kk] * lv;
      }
    }
    __syncthreads();
    for (int o = tid; o < CW_NB * CW_NB; o += 256) Ds[o / CW_NB][o % CW_NB] = dinv[(int64_t)(j0 / CW_NB) * CW_NB * CW_NB + o];
#pragma unroll
    for (int m = 0; m < 4; ++m) Ts[tr + 8 * m][tc] = acc[m];
    __syncthreads();
#pragma unroll
    for (int m = 0; m < 4; ++m) {
      double sacc = 0.0;
      for (int cp = 0; cp <= tc; ++cp) sacc += Ts[tr + 8 * m][cp] * Ds[tc][cp];
      const int64_t r = r0 + tr + 8 * m;
      if (tc < w) {
        Hs[tr + 8 * m][j0 + tc] = sacc;
        if (r < n_rows) z[r * n + j0 + tc] = (float)sacc;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// C[m][n] = scale[n] * sum_k A[m * a_m + k * a_k] * B[k * b_k + n * b_n]      (A FP32, B FP64, FP64 accumulation)
// written as FP32 to c[m * c_m + n * c_n]; optionally also c2[m * c2_m + n * c2_n] = (that value) * scale2[n], and
// amax|C| into *amax (bits of a non-negative float, atomic max).  64 x 64 tile per CTA, 4 x 4 outputs per thread.
struct Gemm64Args {
  const float* a; int64_t a_m, a_k;
  const double* b; int64_t b_k, b_n;
  const double* scale;            // per output column n, or NULL
  float* c; int64_t c_m, c_n;
  float* c2; int64_t c2_m, c2_n; const float* scale2;
  float* amax;
  int64_t M; int N, K;
  const int* skip;
};
__global__ void __launch_bounds__(256)
gemm64_kernel(Gemm64Args g) {
  metis_pdl_wait();
  if (g.skip != nullptr && *g.skip) return;
  constexpr int T = 64, KT = 16;
  __shared__ __align__(16) double as[KT][T + 2], bs[KT][T + 2];
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int64_t m0 = (int64_t)blockIdx.y * T;
  const int n0 = blockIdx.x * T;
  double acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;
  for (int k0 = 0; k0 < g.K; k0 += KT) {
    for (int o = tid; o < KT * T; o += 256) {
      int kk, mm;
      if (g.a_k == 1) { kk = o % KT; mm = o / KT; } else { mm = o % T; kk = o / T; }
      as[kk][mm] = (m0 + mm < g.M && k0 + kk < g.K) ? (double)g.a[(m0 + mm) * g.a_m + (int64_t)(k0 + kk) * g.a_k] : 0.0;
      int kb, nn;
      if (g.b_k == 1) { kb = o % KT; nn = o / KT; } else { nn = o % T; kb = o / T; }
      bs[kb][nn] = (n0 + nn < g.N && k0 + kb < g.K) ? g.b[(int64_t)(k0 + kb) * g.b_k + (int64_t)(n0 + nn) * g.b_n] : 0.0;
    }
    __syncthreads();
#pragma unroll 4
    for (int kk = 0; kk < KT; ++kk) {
      double av[4], bv[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) { av[a] = as[kk][ty + 16 * a]; bv[a] = bs[kk][tx + 16 * a]; }
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] += av[a] * bv[b];
    }
    __syncthreads();
  }
  float am = 0.0f;
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int64_t m = m0 + ty + 16 * a;
      const int n = n0 + tx + 16 * b;
      if (m < g.M && n < g.N) {
        const float v = (float)(g.scale != nullptr ? acc[a][b] * g.scale[n] : acc[a][b]);
        g.c[m * g.c_m + (int64_t)n * g.c_n] = v;
        if (g.c2 != nullptr) g.c2[m * g.c2_m + (int64_t)n * g.c2_n] = v * g.scale2[n];
        am = fmaxf(am, fabsf(v));
      }
    }
  if (g.amax != nullptr) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) am = fmaxf(am, __shfl_xor_sync(0xFFFFFFFFu, am, o));
    if ((tid & 31) == 0) atomicMax(reinterpret_cast<unsigned int*>(g.amax), __float_as_uint(am));
  }
}

// per-column scales of the rotations: mode 0: 1/sqrt(eval_j) (right basis; also writes sigma_out = sqrt(eval_j)),
// mode 1: sign_j / sqrt(eval_j) (Rayleigh-Ritz left factor; sigma_out likewise), mode 2: sign_j
__global__ void rot_scales_kernel(const double* __restrict__ evals, const float* __restrict__ sign, int k, int mode,
                                  double* __restrict__ scale, float* __restrict__ sigma_out) {
  metis_pdl_wait();
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= k) return;
  double s = 1.0;
  if (mode != 2) {
    const double lam = sqrt(fmax(evals[j], 0.0));
    s = lam > 0.0 ? 1.0 / lam : 0.0;
    if (sigma_out != nullptr) sigma_out[j] = (float)lam;
  }
  if (mode != 0) s *= (double)sign[j];
  scale[j] = s;
}

// ------------------------------------------------------------------------------------------------
// One-sided (Hestenes) Jacobi on the columns of Y = L (the Cholesky factor of the Gram matrix, so that
// G = Y Y^T and the rotated columns end as U Sigma), for n up to MAXQ_WIDE, on ONE CLUSTER of JC_P CTAs.
// The 2 * JC_P * JC_W column slots are dealt out as 2 * JC_P blocks of JC_W columns; every CTA holds two blocks in
// its shared memory (FP64, 78 KB) and orthogonalises, one warp per couple,
//   - in the first outer round of a sweep: every pair among its 2 * JC_W columns (round-robin tournament),
//   - in the other outer rounds: every pair of one column of each block,
// then the blocks move on to the neighbouring CTAs in the order of a round-robin tournament over blocks (block 0
// stays), written straight into the neighbour's second buffer through distributed shared memory, between two
// cluster barriers.  After 2 * JC_P - 1 outer rounds every pair of columns has met once: one sweep.  Arithmetic of
// a rotation as in the one-CTA solver: columns and rotation orthonormality in FP64, steering quantities in FP32.
constexpr int JC_P = 8, JC_W = 17, JC_ROWS = 288, JC_THREADS = 32 * JC_W;
constexpr int JC_RL = JC_ROWS / 32;                     // rows per lane
constexpr size_t JC_SMEM = sizeof(double) * 2 * 2 * JC_W * JC_ROWS;

__device__ __forceinline__ void jc_pair(int I, int step, int np, int* p, int* q) {
  int a, b;
  if (I == 0) { a = 0; b = (step % (np - 1)) + 1; }
  else { a = ((step + I) % (np - 1)) + 1; b = ((step + np - 1 - I) % (np - 1)) + 1; }
  *p = min(a, b); *q = max(a, b);
}

// Rotation that makes two columns with squared norms a, b and inner product c orthogonal: the smaller root of
// tan(2 theta) = 2c / (b - a), |theta| <= pi / 4.  The FP32 quantities only steer convergence (fast reciprocal square
// roots); (cs, sn) is made a unit vector to ~1e-14 by one Newton step in FP64; tf = tan(theta) updates the carried norms.
__device__ __forceinline__ void jc_rotation(float a, float b, float cf, double& cs, double& sn, float& tf) {
  const float d = b - a, c2 = 2.0f * cf;
  const float h2 = fmaf(c2, c2, d * d);
  const float rh = rsqrtf(h2);
  const float cc = fmaf(0.5f * fabsf(d), rh, 0.5f);
  const float rs = rsqrtf(cc);
  const float c32 = cc * rs, s32 = (d < 0.0f ? -c2 : c2) * (0.5f * rh) * rs;
  tf = s32 * rs;
  const double cd = (double)c32, sd = (double)s32;
  const double scale = 1.5 - 0.5 * (cd * cd + sd * sd);
  cs = cd * scale; sn = sd * scale;
}

__global__ void __cluster_dims__(JC_P, 1, 1) __launch_bounds__(JC_THREADS, 1)
jacobi_cluster_kernel(const double* __restrict__ l, int n, float exit_cos2, double* __restrict__ ycm) {
  metis_pdl_wait();
  extern __shared__ __align__(16) unsigned char jsm[];
  double* cols = reinterpret_cast<double*>(jsm);        // [buffer][slot][column][row]
  __shared__ float nrm[2][JC_W];
  __shared__ int flag_s;
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  auto col_ptr = [&](int buf, int slot, int c) { return cols + (((size_t)buf * 2 + slot) * JC_W + c) * JC_ROWS; };
  // load: slot s of this CTA starts as block 2 * rank + s, i.e. columns (2 * rank + s) * JC_W + c of Y
  for (int o = tid; o < 2 * JC_W * JC_ROWS; o += JC_THREADS) {
    const int i = o % JC_ROWS, c = (o / JC_ROWS) % JC_W, s = o / (JC_ROWS * JC_W);
    const int gc = (2 * rank + s) * JC_W + c;
    col_ptr(0, s, c)[i] = (gc < n && i < n && gc <= i) ? l[(int64_t)i * n + gc] : 0.0;
  }
  __syncthreads();
  int cur = 0;
  for (int sweep = 0; sweep < 16; ++sweep) {
    bool above = false;
    int any_above = 0;
    for (int orr = 0; orr < 2 * JC_P - 1; ++orr) {
      // exact norms of this CTA's columns at the start of every outer round (they are carried through the rounds)
      for (int sc = warp; sc < 2 * JC_W; sc += JC_W) {
        const double* y = col_ptr(cur, sc / JC_W, sc % JC_W);
        double a = 0.0;
#pragma unroll
        for (int t = 0; t < JC_RL; ++t) { const double v = y[lane + 32 * t]; a += v * v; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xFFFFFFFFu, a, o);
        if (lane == 0) nrm[sc / JC_W][sc % JC_W] = (float)a;
      }
      __syncthreads();
      if (orr == 0) {
        // every pair among the CTA's 2 * JC_W columns: round-robin tournament, both columns of a couple through shared memory
        for (int r = 0; r < 2 * JC_W - 1; ++r) {
          int p, q;
          jc_pair(warp, r, 2 * JC_W, &p, &q);
          const int ps = p / JC_W, pc = p % JC_W, qs = q / JC_W, qc = q % JC_W;
          double* yp_s = col_ptr(cur, ps, pc);
          double* yq_s = col_ptr(cur, qs, qc);
          double yp[JC_RL], yq[JC_RL];
          double c = 0.0;
#pragma unroll
          for (int t = 0; t < JC_RL; ++t) { yp[t] = yp_s[lane + 32 * t]; yq[t] = yq_s[lane + 32 * t]; c += yp[t] * yq[t]; }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
          const float a = nrm[ps][pc], b = nrm[qs][qc], cf = (float)c;
          if (cf * cf > 1e-26f * (a * b)) {
            double cs, sn; float tf;
            jc_rotation(a, b, cf, cs, sn, tf);
#pragma unroll
            for (int t = 0; t < JC_RL; ++t) {
              yp_s[lane + 32 * t] = cs * yp[t] - sn * yq[t];
              yq_s[lane + 32 * t] = sn * yp[t] + cs * yq[t];
            }
            const float tc = tf * cf;
            if (lane == 0) { nrm[ps][pc] = a - tc; nrm[qs][qc] = b + tc; }
            above |= cf * cf > exit_cos2 * (a * b);
          }
          __syncthreads();
        }
      } else {
        // every pair of one column of each block: warp w keeps column w of the first block in registers for all
        // JC_W rounds (nobody else touches it) and meets the columns of the second block one after the other
        double* yp_s = col_ptr(cur, 0, warp);
        double yp[JC_RL];
#pragma unroll
        for (int t = 0; t < JC_RL; ++t) yp[t] = yp_s[lane + 32 * t];
        float a = nrm[0][warp];
        for (int r = 0; r < JC_W; ++r) {
          const int qc = (warp + r) % JC_W;
          double* yq_s = col_ptr(cur, 1, qc);
          double yq[JC_RL];
          double c = 0.0;
#pragma unroll
          for (int t = 0; t < JC_RL; ++t) { yq[t] = yq_s[lane + 32 * t]; c += yp[t] * yq[t]; }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
          const float b = nrm[1][qc], cf = (float)c;
          if (cf * cf > 1e-26f * (a * b)) {
            double cs, sn; float tf;
            jc_rotation(a, b, cf, cs, sn, tf);
#pragma unroll
            for (int t = 0; t < JC_RL; ++t) {
              const double np_ = cs * yp[t] - sn * yq[t];
              yq_s[lane + 32 * t] = sn * yp[t] + cs * yq[t];
              yp[t] = np_;
            }
            const float tc = tf * cf;
            above |= cf * cf > exit_cos2 * (a * b);
            if (lane == 0) nrm[1][qc] = b + tc;
            a -= tc;
          }
          __syncthreads();
        }
#pragma unroll
        for (int t = 0; t < JC_RL; ++t) yp_s[lane + 32 * t] = yp[t];
        __syncthreads();
      }
      const bool last = orr == 2 * JC_P - 2;
      if (last) {
        const int any = __syncthreads_or(above ? 1 : 0);
        if (tid == 0) flag_s = any;
      }
      cluster.sync();                                    // every CTA is done with this outer round (flags are written)
      // hand the blocks on: slot 0 ("top") of CTA c goes to the top of c + 1 (the last CTA's top becomes its own
      // bottom, CTA 0's top stays); slot 1 ("bottom") of CTA c goes to the bottom of c - 1 (CTA 0's bottom becomes
      // the top of CTA 1)
      {
        int dst_rank[2], dst_slot[2];
        if (rank == 0) { dst_rank[0] = 0; dst_slot[0] = 0; dst_rank[1] = 1; dst_slot[1] = 0; }
        else {
          if (rank == JC_P - 1) { dst_rank[0] = rank; dst_slot[0] = 1; } else { dst_rank[0] = rank + 1; dst_slot[0] = 0; }
          dst_rank[1] = rank - 1; dst_slot[1] = 1;
        }
#pragma unroll
        for (int s = 0; s < 2; ++s) {
          const double2* src = reinterpret_cast<const double2*>(col_ptr(cur, s, 0));
          double2* dst = reinterpret_cast<double2*>(cluster.map_shared_rank(col_ptr(cur ^ 1, dst_slot[s], 0), dst_rank[s]));
          for (int o = tid; o < JC_W * JC_ROWS / 2; o += JC_THREADS) dst[o] = src[o];
        }
      }
      if (last) {
        for (int c = 0; c < JC_P; ++c) any_above |= *cluster.map_shared_rank(&flag_s, c);
      }
      cluster.sync();                                    // the blocks have landed; the flags have been read
      cur ^= 1;
    }
    if (!any_above) break;
  }
  // column-major result: ycm[(slot position) * n + row]; the order of the columns is irrelevant (they are sorted
  // by their norms afterwards)
  for (int o = tid; o < 2 * JC_W * n; o += JC_THREADS) {
    const int i = o % n, sc = o / n;
    ycm[((int64_t)(2 * rank) * JC_W + sc) * n + i] = col_ptr(cur, sc / JC_W, sc % JC_W)[i];
  }
}

// eigenvalues = squared column norms (descending), eigenvectors = normalised columns: evecs[i * n + t]
__global__ void __launch_bounds__(1024, 1)
jacobi_collect_kernel(const double* __restrict__ ycm, int n, double* __restrict__ evals, double* __restrict__ evecs) {
  metis_pdl_wait();
  constexpr int NC = 2 * JC_P * JC_W;
  __shared__ double lam[NC];
  __shared__ int order[NC];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int c = warp; c < NC; c += 32) {
    double a = 0.0;
    for (int i = lane; i < n; i += 32) { const double v = ycm[(int64_t)c * n + i]; a += v * v; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xFFFFFFFFu, a, o);
    if (lane == 0) { lam[c] = a; order[c] = c; }
  }
  __syncthreads();
  if (tid < NC) {
    const double li = lam[tid];
    int rank = 0;
    for (int j = 0; j < NC; ++j) rank += (lam[j] > li) || (lam[j] == li && j < tid);
    order[rank] = tid;                                  // stays a valid index if NaNs make ranks collide
  }
  __syncthreads();
  if (tid < n) evals[tid] = lam[order[tid]];
  for (int o = tid; o < n * n; o += 1024) {
    const int i = o / n, t = o % n;
    const int c = order[t];
    const double l2 = lam[c];
    evecs[o] = l2 > 0.0 ? ycm[(int64_t)c * n + i] * (1.0 / sqrt(l2)) : 0.0;
  }
}

// ------------------------------------------------------------------------------------------------
// Sign convention, one CTA per factor vector j: the entry of largest magnitude of right[j][:] (lowest index on ties)
// is made positive; sign[j] records the flip for the left factor; amax|right| into *amax_out.
__global__ void __launch_bounds__(256)
sign_rows_kernel(float* __restrict__ right, int64_t cols, float* __restrict__ sign_out, float* __restrict__ amax_out) {
  metis_pdl_wait();
  __shared__ float bv[8], bs_[8];
  __shared__ int bi[8];
  __shared__ float sg_s;
  const int j = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float* row = right + (int64_t)j * cols;
  float av = -1.0f, sv = 0.0f;
  int ai = 0x7FFFFFFF;
  for (int64_t c = tid; c < cols; c += 256) {
    const float v = row[c];
    if (fabsf(v) > av) { av = fabsf(v); sv = v; ai = (int)c; }      // increasing c: the first maximum is kept
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xFFFFFFFFu, av, o), os = __shfl_xor_sync(0xFFFFFFFFu, sv, o);
    const int oi = __shfl_xor_sync(0xFFFFFFFFu, ai, o);
    if (ov > av || (ov == av && oi < ai)) { av = ov; sv = os; ai = oi; }
  }
  if (lane == 0) { bv[warp] = av; bs_[warp] = sv; bi[warp] = ai; }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < 8; ++w)
      if (bv[w] > bv[0] || (bv[w] == bv[0] && bi[w] < bi[0])) { bv[0] = bv[w]; bs_[0] = bs_[w]; bi[0] = bi[w]; }
    const float sg = bs_[0] < 0.0f ? -1.0f : 1.0f;
    sg_s = sg;
    sign_out[j] = sg;
    if (amax_out != nullptr) atomicMax(reinterpret_cast<unsigned int*>(amax_out), __float_as_uint(fmaxf(bv[0], 0.0f)));
  }
  __syncthreads();
  if (sg_s < 0.0f)
    for (int64_t c = tid; c < cols; c += 256) row[c] = -row[c];
}

// ------------------------------------------------------------------------------------------------
// coef[r][j0 + jj] = sum over slices s of part[s][r][jj]  (jj < gw, fixed order), and the BF16 terms of those
// coefficients in the residual product's A operand: a6[r][term * kp + j0 + jj], terms [h | h | l | h | l2 | l].
// One thread per (row, group of eight columns).  The group with j0 == 0 also clears the padding of a6 beyond 6 kp.
__global__ void __launch_bounds__(256)
coef_sum_kernel(const float* __restrict__ part, int slices, int64_t rows, int gw, int j0, int kp, float* __restrict__ coef,
                __nv_bfloat16* __restrict__ a6, int kx) {
  metis_pdl_wait();
  const int g8 = gw / 8;
  const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (idx >= rows * g8) return;
  const int64_t r = idx / g8;
  const int jj = (int)(idx % g8) * 8;
  float v[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) v[e] = 0.0f;
  for (int s = 0; s < slices; ++s) {
    const float4 p0 = *reinterpret_cast<const float4*>(part + ((int64_t)s * rows + r) * gw + jj);
    const float4 p1 = *reinterpret_cast<const float4*>(part + ((int64_t)s * rows + r) * gw + jj + 4);
    v[0] += p0.x; v[1] += p0.y; v[2] += p0.z; v[3] += p0.w; v[4] += p1.x; v[5] += p1.y; v[6] += p1.z; v[7] += p1.w;
  }
  float* cd = coef + r * kp + j0 + jj;
  *reinterpret_cast<float4*>(cd) = make_float4(v[0], v[1], v[2], v[3]);
  *reinterpret_cast<float4*>(cd + 4) = make_float4(v[4], v[5], v[6], v[7]);
  if (a6 != nullptr) {
    uint4 h, l, l2;
    metis_split3x8(v, h, l, l2);
    __nv_bfloat16* dst = a6 + r * kx + j0 + jj;
    *reinterpret_cast<uint4*>(dst) = h; *reinterpret_cast<uint4*>(dst + kp) = h; *reinterpret_cast<uint4*>(dst + 2 * kp) = l;
    *reinterpret_cast<uint4*>(dst + 3 * kp) = h; *reinterpret_cast<uint4*>(dst + 4 * kp) = l2; *reinterpret_cast<uint4*>(dst + 5 * kp) = l;
    if (j0 == 0 && jj == 0)
      for (int z = 6 * kp; z < kx; z += 8) *reinterpret_cast<uint4*>(a6 + r * kx + z) = make_uint4(0u, 0u, 0u, 0u);
  }
}

// gathers the sampled rows of x into a contiguous matrix: xs[j][:] = x[idx[j]][:]   (16 bytes per thread)
__global__ void __launch_bounds__(256)
gather_rows_kernel(const __nv_bfloat16* __restrict__ x, int64_t cols, const int* __restrict__ idx, int n_s, __nv_bfloat16* __restrict__ xs) {
  metis_pdl_wait();
  const int64_t per_row = cols / 8;
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= (int64_t)n_s * per_row) return;
  const int64_t j = i / per_row, c8 = i % per_row;
  reinterpret_cast<uint4*>(xs)[i] = reinterpret_cast<const uint4*>(x + (int64_t)idx[j] * cols)[c8];
}

}  // namespace metis_wide
