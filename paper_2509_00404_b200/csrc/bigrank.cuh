// Small dense linear algebra of a split whose sketch is wider than one CTA's shared memory (k + p above 72, up to
// 272: the rank-128 and rank-256 points of the 70B-shaped sweep).  Same steps as the one-CTA kernels of split.cu
// (Section 3.1: thin QR of the sketch, small SVD of the projected operand), as kernels that tile over the rank:
//
//   gram64_kernel            G = V^T V in FP64, 64 x 64 output tiles over slabs of rows (partials, summed in order)
//   chol_wide_kernel         Cholesky factor of a q x q Gram matrix and its triangular inverse, one CTA, matrix in L2
//   gemm64_kernel            C = A B with FP32 A, FP64 B and FP64 accumulation, arbitrary strides (triangular solve
//                            H = Z L^-T as a product, right basis, factor rotations)
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
// Cholesky factor of the n x n Gram matrix g (n <= MAXQ_WIDE) and, when asked, its inverse, one CTA of 1024 threads.
// The matrix does not fit one CTA's shared memory in FP64, so it stays in global memory (it is L2-resident: half a
// megabyte) and the CTA works column by column, left-looking: column j is the Gram column minus the contributions
// of the columns before it, four lanes per row sharing the inner product.  A pivot not above tol_rel * (largest
// diagonal entry) marks a dependent sketch column: its column of L and its row and column of L^-1 are zero.
//   l_out    n x n row-major lower factor (strict upper part zero)
//   linv_out n x n row-major L^-1 (lower), or NULL
//   well_conditioned  (optional) 1 when every pivot is above 1e-8 of the largest diagonal entry
__global__ void __launch_bounds__(1024, 1)
chol_wide_kernel(const double* __restrict__ g, int n, double tol_rel, double* l_out, double* linv_out,
                 const int* __restrict__ skip, int* __restrict__ well_conditioned) {
  metis_pdl_wait();
  if (skip != nullptr && *skip) return;
  __shared__ double rowj[MAXQ_WIDE];                    // row j of L (entries before the diagonal)
  __shared__ double vbuf[MAXQ_WIDE];                    // column j before scaling
  __shared__ double rinv[MAXQ_WIDE];                    // 1 / L[j][j], or 0 for a dependent column
  __shared__ double red[32];
  __shared__ double gmax_s, dmin_s;
  const int tid = threadIdx.x, lane4 = tid & 3, rgrp = tid >> 2;      // 256 row slots of four lanes
  for (int o = tid; o < n * n; o += 1024) {
    const int i = o / n, j = o % n;
    l_out[o] = j <= i ? 0.5 * (g[(int64_t)i * n + j] + g[(int64_t)j * n + i]) : 0.0;
  }
  double gm = 0.0;
  for (int i = tid; i < n; i += 1024) gm = fmax(gm, g[(int64_t)i * n + i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) gm = fmax(gm, __shfl_xor_sync(0xFFFFFFFFu, gm, o));
  if ((tid & 31) == 0) red[tid >> 5] = gm;
  __syncthreads();
  if (tid == 0) { double m = 0.0; for (int w = 0; w < 32; ++w) m = fmax(m, red[w]); gmax_s = m; dmin_s = 1e300; }
  __syncthreads();
  const double tol = tol_rel * gmax_s;
  for (int j = 0; j < n; ++j) {
    for (int k = tid; k < j; k += 1024) rowj[k] = l_out[(int64_t)j * n + k];
    __syncthreads();
    for (int i = j + rgrp; i < n; i += 256) {
      const double* li = l_out + (int64_t)i * n;
      double s0 = 0.0, s1 = 0.0;
      int k = lane4;
      for (; k + 4 < j; k += 8) { s0 += li[k] * rowj[k]; s1 += li[k + 4] * rowj[k + 4]; }
      if (k < j) s0 += li[k] * rowj[k];
      double s = s0 + s1;
      // the four lanes of a row run this loop together; other rows of the warp may already have left it
      const unsigned grp_mask = 0xFu << ((tid & 31) & ~3);
      s += __shfl_xor_sync(grp_mask, s, 1);
      s += __shfl_xor_sync(grp_mask, s, 2);
      if (lane4 == 0) vbuf[i] = li[j] - s;
    }
    __syncthreads();
    const double d = vbuf[j];
    const double r = d > tol ? 1.0 / sqrt(d) : 0.0;
    for (int i = j + tid; i < n; i += 1024) l_out[(int64_t)i * n + j] = i == j ? d * r : vbuf[i] * r;
    if (tid == 0) { rinv[j] = r; if (d > tol) dmin_s = fmin(dmin_s, d); }
    __syncthreads();
  }
  if (tid == 0 && well_conditioned != nullptr) *well_conditioned = (dmin_s > 1e-8 * gmax_s) ? 1 : 0;
  if (linv_out == nullptr) return;
  // L^-1 row by row: X[i][i] = 1/L[i][i], X[i][j] = -X[i][i] * sum_{k=j}^{i-1} L[i][k] X[k][j]   (j < i)
  for (int o = tid; o < n * n; o += 1024) linv_out[o] = 0.0;
  __syncthreads();
  const int jj = tid & 255, sl = tid >> 8;              // column slot, one of four slices of the k range
  __shared__ double psum[4][MAXQ_WIDE];
  for (int i = 0; i < n; ++i) {
    for (int k = tid; k < i; k += 1024) rowj[k] = l_out[(int64_t)i * n + k];
    __syncthreads();
    for (int j = jj; j < i; j += 256) {
      double s0 = 0.0, s1 = 0.0;
      int k = j + sl;
      for (; k + 4 < i; k += 8) { s0 += rowj[k] * linv_out[(int64_t)k * n + j]; s1 += rowj[k + 4] * linv_out[(int64_t)(k + 4) * n + j]; }
      if (k < i) s0 += rowj[k] * linv_out[(int64_t)k * n + j];
      psum[sl][j] = s0 + s1;
    }
    __syncthreads();
    const double ri = rinv[i];
    for (int j = tid; j <= i; j += 1024)
      linv_out[(int64_t)i * n + j] = j == i ? ri : -ri * (((psum[0][j] + psum[1][j]) + psum[2][j]) + psum[3][j]);
    __syncthreads();
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
      const int rounds = orr == 0 ? 2 * JC_W - 1 : JC_W;
      for (int r = 0; r < rounds; ++r) {
        int ps, pc, qs, qc;
        if (orr == 0) {
          int p, q;
          jc_pair(warp, r, 2 * JC_W, &p, &q);
          ps = p / JC_W; pc = p % JC_W; qs = q / JC_W; qc = q % JC_W;
        } else {
          ps = 0; pc = warp; qs = 1; qc = (warp + r) % JC_W;
        }
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
          const float d = b - a, c2 = 2.0f * cf;
          const float h2 = fmaf(c2, c2, d * d);
          const float rh = rsqrtf(h2);
          const float cc = fmaf(0.5f * fabsf(d), rh, 0.5f);
          const float rs = rsqrtf(cc);
          const float c32 = cc * rs, s32 = (d < 0.0f ? -c2 : c2) * (0.5f * rh) * rs;
          const float tf = s32 * rs;
          const double cd = (double)c32, sd = (double)s32;
          const double scale = 1.5 - 0.5 * (cd * cd + sd * sd);
          const double cs = cd * scale, sn = sd * scale;
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
