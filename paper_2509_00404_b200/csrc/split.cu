// Low-rank + residual split of one GEMM operand (Sections 3.1 and 3.2) and its NVFP4 quantization.
//
// Steps (FULL = on all rows, SAMPLED = subspace from a sparse row sample, "broadcast" to all rows):
//   amax(x) -> row sample -> sketch Z = x[S,:] Omega (Omega from Philox + quantile table, never stored)
//   -> CholeskyQR2 (FP64 Gram + Cholesky) -> M = H^T x[S,:] -> eigen-decomposition of M M^T (Jacobi,
//   FP64) -> right basis B -> [SAMPLED: C = x B, Rayleigh-Ritz on C^T C] -> residual R = x - C B^T fused
//   with the NVFP4 quantizer in both block orientations -> factor rotation, sign fix, factor quantization.
#include "quant_tile.cuh"
#include "bigrank.cuh"

metis_status_t metis_launch_residual_tc(metis_context* ctx, const void* x, const float* coef, int k, int kp,
                                        const metis_qt::QuantParams& qp, const float* amax_src, float* ts_out0, float* ts_out1,
                                        float* dense, void* a6, void* b6, cudaStream_t s);

namespace {

constexpr int MAXQ = 72;                               // k + p at most (k = 64 with p = 8)
constexpr size_t JACOBI_SMEM = sizeof(double) * MAXQ * (MAXQ + 1);

// ------------------------------------------------------------------------------------------------
__global__ void sample_rows_kernel(int* __restrict__ idx, int n_s, int64_t rows, uint64_t seed, int full) {
  metis_pdl_wait();
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n_s) return;
  if (full) { idx[j] = j; return; }
  const uint32_t g = (uint32_t)(rows / n_s);
  const uint4 w = metis_philox((uint32_t)j, 0u, METIS_STREAM_SAMPLING, 0u, (uint32_t)seed, (uint32_t)(seed >> 32));
  idx[j] = (int)((uint32_t)j * g + w.x % g);          // one row per stratum of g consecutive rows
}

// ------------------------------------------------------------------------------------------------
// Device-detected conditions of a split: amax|x| not finite (a NaN or an infinity in the operand: amax is kept as
// an ordered bit pattern, so a NaN ranks above every number), a non-finite eigenvalue.  One warp.
__global__ void split_status_kernel(const float* __restrict__ amax, const double* __restrict__ evals, int k, uint32_t* dev_status) {
  metis_pdl_wait();
  uint32_t bits = 0u;
  if (threadIdx.x == 0 && !(fabsf(*amax) <= 3.0e38f)) bits |= METIS_DEV_NONFINITE;
  for (int j = threadIdx.x; j < k; j += 32)
    if (!(fabs(evals[j]) <= 1.0e300)) bits |= METIS_DEV_NUMERIC;
  if (bits) atomicOr(dev_status, bits);
}

__global__ void reduce_partials_kernel(const float* __restrict__ zp, int n_chunks, int64_t n, float* __restrict__ z) {
  metis_pdl_wait();
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= n) return;
  float acc = 0.0f;
  int c = 0;
  for (; c + 8 <= n_chunks; c += 8) {                                    // eight loads in flight; fixed order: reproducible
    float t[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) t[u] = zp[(int64_t)(c + u) * n + i];
#pragma unroll
    for (int u = 0; u < 8; ++u) acc += t[u];
  }
  for (; c < n_chunks; ++c) acc += zp[(int64_t)c * n + i];
  z[i] = acc;
}

// ------------------------------------------------------------------------------------------------
// Gram partials in FP64: part[p][i][j] = sum over the p-th slab of rows r of v(r,i) v(r,j),
// v(r,i) = V[r*stride_row + i*stride_vec].
constexpr int GR_TILE = 32;
constexpr int GR_PITCH = MAXQ + 2;                      // doubles per tile row: even, so that 4-wide groups stay 16-byte aligned
constexpr int GR_NB = (MAXQ + 3) / 4;                   // 4 x 4 output blocks per dimension
__global__ void __launch_bounds__(256)
gram_kernel(const float* __restrict__ v, int64_t n_rows, int n, int64_t stride_row, int64_t stride_vec,
            int64_t rows_per_part, double* __restrict__ part, const int* __restrict__ skip) {
  metis_pdl_wait();
  if (skip != nullptr && *skip) return;                 // second CholeskyQR pass not needed (see chol_kernel)
  // The tile is converted to FP64 once when it is staged (FP32 -> FP64 conversions are a slow-rate instruction).
  // A thread owns 4 x 4 blocks of the output: eight shared-memory loads feed sixteen multiply-adds, which keeps
  // the kernel off the shared-memory pipe that bounds a one-output-per-thread formulation.
  __shared__ __align__(16) double tile[GR_TILE][GR_PITCH];
  const int tid = threadIdx.x;
  const int64_t r_begin = (int64_t)blockIdx.x * rows_per_part;
  const int64_t r_end = min(n_rows, r_begin + rows_per_part);
  const int nb = (n + 3) / 4, n_blocks = nb * nb;
  constexpr int BPT = (GR_NB * GR_NB + 255) / 256;      // blocks per thread at the largest n
  // With at most 128 output blocks (n <= 44) two threads share a block, each taking half of the tile's rows; their
  // partial sums are added once at the end (second half first into shared memory: a fixed order).
  const bool halved = 2 * n_blocks <= 256;
  const int half = halved ? tid / n_blocks : 0;         // 0 or 1 (threads beyond 2 * n_blocks idle)
  const int rr_begin = halved ? half * (GR_TILE / 2) : 0, rr_end = halved ? rr_begin + GR_TILE / 2 : GR_TILE;
  double acc[BPT][4][4];
#pragma unroll
  for (int b = 0; b < BPT; ++b)
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[b][i][j] = 0.0;
  for (int i = tid; i < GR_TILE * (GR_PITCH - n); i += 256) {                    // columns n .. pitch-1 stay zero
    const int rr = i / (GR_PITCH - n), ii = n + i % (GR_PITCH - n);
    tile[rr][ii] = 0.0;
  }
  for (int64_t r0 = r_begin; r0 < r_end; r0 += GR_TILE) {
    for (int i = tid; i < GR_TILE * n; i += 256) {
      int rr, ii;
      if (stride_row == 1) { rr = i % GR_TILE; ii = i / GR_TILE; } else { ii = i % n; rr = i / n; }
      tile[rr][ii] = (r0 + rr < r_end) ? (double)v[(r0 + rr) * stride_row + ii * stride_vec] : 0.0;
    }
    __syncthreads();
#pragma unroll
    for (int b = 0; b < BPT; ++b) {
      const int o = halved ? tid - half * n_blocks : tid + b * 256;
      if (o < n_blocks && half < 2 && (!halved || b == 0)) {
        const int bi = o / nb, bj = o % nb;
#pragma unroll 4
        for (int rr = rr_begin; rr < rr_end; ++rr) {
          const double2 a01 = *reinterpret_cast<const double2*>(&tile[rr][4 * bi]), a23 = *reinterpret_cast<const double2*>(&tile[rr][4 * bi + 2]);
          const double2 b01 = *reinterpret_cast<const double2*>(&tile[rr][4 * bj]), b23 = *reinterpret_cast<const double2*>(&tile[rr][4 * bj + 2]);
          const double av[4] = {a01.x, a01.y, a23.x, a23.y}, bv[4] = {b01.x, b01.y, b23.x, b23.y};
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[b][i][j] += av[i] * bv[j];
        }
      }
    }
    __syncthreads();
  }
  if (halved) {
    double* scratch = &tile[0][0];                      // the tile is free now: GR_TILE * GR_PITCH >= 16 * 128 doubles
    const int o = tid - half * n_blocks;
    if (half == 1 && o < n_blocks) {
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) scratch[o * 16 + i * 4 + j] = acc[0][i][j];
    }
    __syncthreads();
    if (half == 0 && o < n_blocks) {
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[0][i][j] += scratch[o * 16 + i * 4 + j];
    }
  }
#pragma unroll
  for (int b = 0; b < BPT; ++b) {
    const int o = halved ? tid : tid + b * 256;
    if (o < n_blocks && (!halved || b == 0)) {
      const int bi = o / nb, bj = o % nb;
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (4 * bi + i < n && 4 * bj + j < n) part[(int64_t)blockIdx.x * n * n + (4 * bi + i) * n + 4 * bj + j] = acc[b][i][j];
    }
  }
}

// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ double chol_rsqrt(double x) {
  // scale into the FP32 range by an even power of two, seed with rsqrtf, two Newton steps in FP64
  int e;
  const double mant = frexp(x, &e);                     // x = mant * 2^e, mant in [0.5, 1)
  const int e2 = e & ~1;
  const double xs = ldexp(mant, e - e2);                // in [0.5, 2)
  double y = (double)rsqrtf((float)xs);
  y = y * (1.5 - 0.5 * xs * y * y);
  y = y * (1.5 - 0.5 * xs * y * y);
  return ldexp(y, -(e2 / 2));
}

__device__ __forceinline__ double fast_rsqrt_wide(double x) { return chol_rsqrt(x); }

// 1/x in FP64: the hardware's 20-bit FP64 reciprocal seed and three Newton steps
__device__ __forceinline__ double chol_rcp(double x) {
  double y;
  asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(x));
  y = y * (2.0 - x * y);
  y = y * (2.0 - x * y);
  y = y * (2.0 - x * y);
  return y;
}

// In-place Cholesky of the n x n lower triangle of Y (row pitch P doubles) by the first 256 threads of the CTA.
// Right-looking with the column scaling deferred: step j only subtracts  Y[a][j] Y[b][j] / Y[j][j]  from the
// trailing triangle (one barrier per column, a reciprocal instead of a square root in the serial chain); the
// columns are divided by sqrt(pivot) together at the end.  The matrix lives in registers for the whole
// factorisation - thread (ty, tx) of a 16 x 16 grid keeps the elements (ty + 16u, tx + 16v) - and a step reads
// only column j and the reciprocal of its pivot, which their owners publish through shared memory before the
// barrier of the step before; the step itself has no data-dependent branch.  A pivot not above `tol` marks a
// dependent column: its reciprocal is published as zero, so it takes no part in the updates, and it ends as a
// zero column with inv_out[j] = 0.
template <int P>
__device__ __forceinline__ void cta_cholesky(double (*Y)[P], int n, double tol, double* inv_out, double* dmin_out, int nthr) {
  constexpr int NB = (MAXQ + 15) / 16;
  __shared__ double colbuf[2][16 * NB];
  __shared__ double rd_s[2];
  const int tid = threadIdx.x, ty = (tid >> 4) & 15, tx = tid & 15;
  const bool worker = tid < 256;
  double r[NB][NB];
#pragma unroll
  for (int u = 0; u < NB; ++u)
#pragma unroll
    for (int v = 0; v <= u; ++v) {
      const int a = ty + 16 * u, b = tx + 16 * v;
      r[u][v] = (worker && a < n && b <= a) ? Y[a][b] : 0.0;
    }
  if (worker && tx == 0) {
#pragma unroll
    for (int u = 0; u < NB; ++u) colbuf[0][ty + 16 * u] = r[u][0];
  }
  if (tid == 0) { const double d0 = r[0][0]; rd_s[0] = d0 > tol ? chol_rcp(d0) : 0.0; }
  __syncthreads();
  // Steps in phases of sixteen: during phase w (columns 16w .. 16w+15) only the register blocks u, v >= w still
  // change, so the unrolled block loops shrink from phase to phase (an instruction stream a thread does not run
  // costs nothing; one it runs predicated-off still costs its issue slots).
#pragma unroll
  for (int w = 0; w < NB; ++w) {
    if (16 * w < n) {
      const int j_end = min(n, 16 * w + 16);
      for (int j = 16 * w; j < j_end; ++j) {
        if (worker) {
          const double* cb = colbuf[j & 1];
          const double rd = rd_s[j & 1];                // 0 for a dependent column: the step is a no-op
          const int jn = j + 1;
          double la[NB], lb[NB];
#pragma unroll
          for (int u = w; u < NB; ++u)
            if (16 * u < n) { la[u] = cb[ty + 16 * u] * rd; lb[u] = cb[tx + 16 * u]; }
#pragma unroll
          for (int u = w; u < NB; ++u)
#pragma unroll
            for (int v = w; v <= u; ++v)
              if (16 * u < n) {
                const int a = ty + 16 * u, b = tx + 16 * v;
                if (a > j && b > j && b <= a) r[u][v] -= la[u] * lb[v];
                if (b == jn) colbuf[jn & 1][a] = r[u][v];
                if (b == jn && a == jn) { const double dn = r[u][v]; rd_s[jn & 1] = dn > tol ? chol_rcp(dn) : 0.0; }
              }
        }
        __syncthreads();
      }
    }
  }
  if (worker) {
#pragma unroll
    for (int u = 0; u < NB; ++u)
#pragma unroll
      for (int v = 0; v <= u; ++v) {
        const int a = ty + 16 * u, b = tx + 16 * v;
        if (a < n && b <= a) Y[a][b] = r[u][v];
      }
  }
  __syncthreads();
  double dj = 0.0, inv = 0.0;
  if (tid < n) {
    dj = Y[tid][tid];
    inv = dj > tol ? chol_rsqrt(dj) : 0.0;
    inv_out[tid] = inv;
  }
  if (dmin_out != nullptr && tid < 32) {                // smallest accepted pivot
    double dm = 1e300;
    for (int i = tid; i < n; i += 32) { const double v = Y[i][i]; if (v > tol) dm = fmin(dm, v); }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dm = fmin(dm, __shfl_xor_sync(0xFFFFFFFFu, dm, o));
    if (tid == 0) *dmin_out = dm;
  }
  __syncthreads();
  for (int o = tid; o < n * n; o += nthr) {
    const int i = o / n, j = o % n;
    if (i > j) Y[i][j] *= inv_out[j];
  }
  if (tid < n) Y[tid][tid] = dj * inv;                  // sqrt(pivot), or 0 for a dependent column
  __syncthreads();
}

// One CholeskyQR pass, step 1 (one CTA): G (one Gram partial) = L L^T in FP64; writes L (q x q, row-major,
// upper part unused) and the reciprocal pivots.  A pivot below 1e-13 of the largest diagonal marks a
// dependent sketch column: its reciprocal is stored as zero, so the corresponding column of H = Z L^-T
// becomes zero instead of amplified noise.
__global__ void __launch_bounds__(256)
chol_kernel(const double* __restrict__ g, int q, double* __restrict__ l_out, double* __restrict__ invd_out,
            const int* __restrict__ skip, int* __restrict__ well_conditioned) {
  metis_pdl_wait();
  if (skip != nullptr && *skip) return;
  __shared__ double L[MAXQ][MAXQ + 1];
  __shared__ double gmax_s;
  __shared__ double dmin_s;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  for (int o = tid; o < q * q; o += 256) L[o / q][o % q] = g[o];
  __syncthreads();
  if (tid < 32) {
    double gm = 0.0;
    for (int i = tid; i < q; i += 32) gm = fmax(gm, L[i][i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) gm = fmax(gm, __shfl_xor_sync(0xFFFFFFFFu, gm, o));
    if (tid == 0) gmax_s = gm;
  }
  __syncthreads();
  const double tol = 1e-13 * gmax_s;
  __shared__ double inv_s[MAXQ];
  cta_cholesky<MAXQ + 1>(L, q, tol, inv_s, &dmin_s, 256);
  if (tid < q) invd_out[tid] = inv_s[tid];
  // With every pivot above 1e-8 of the largest diagonal the FP64 factorisation leaves Z L^-T orthonormal to
  // ~1e-8 already, below the FP32 rounding of its storage: the caller's second pass is then skipped.
  if (tid == 0 && well_conditioned != nullptr) *well_conditioned = (dmin_s > 1e-8 * gmax_s) ? 1 : 0;
  for (int o = tid; o < q * q; o += 256) l_out[o] = L[o / q][o % q];
}

// One CholeskyQR pass, steps 0 and 1 in one CTA, for a sketch short enough to sit in shared memory as FP64 (the
// row-sampled case: a few hundred rows): G = Z^T Z and its Cholesky factor without a trip through global memory.
// The Gram phase computes the lower 4 x 4 blocks only; S threads (adjacent lanes) share a block, each taking
// every S-th row, and add their partial sums with shuffles in a fixed order.
constexpr int GC_THREADS = 512;
constexpr size_t GC_MAX_SMEM = 144 * 1024;              // beside ~45 KiB of static shared memory
__host__ __device__ inline int gram_chol_pitch(int q) { return 4 * ((q + 3) / 4) + 2; }
__host__ inline size_t gram_chol_smem(int64_t n_s, int q) { return (size_t)n_s * gram_chol_pitch(q) * sizeof(double); }
// Well-conditioned sketch (every pivot above 1e-8 of the largest diagonal: Z L^-T is orthonormal to ~1e-8 already):
// the kernel writes L and the reciprocal pivots and clears *applied; apply_chol_kernel, on many CTAs, does the
// triangular solves.  Otherwise (rare) the whole CholeskyQR2 runs here on the FP64 copy - solve, second Gram
// matrix, second factor, second solve - H is written over z and *applied is set, which makes the apply kernel
// behind this one return at once.
__global__ void __launch_bounds__(GC_THREADS, 1)
gram_chol_kernel(float* __restrict__ z, int n_s, int q, double* __restrict__ l_out, double* __restrict__ invd_out,
                 int* __restrict__ applied) {
  metis_pdl_wait();
  extern __shared__ __align__(16) double zs[];
  __shared__ double L[MAXQ][MAXQ + 1];
  __shared__ double gmax_s;
  __shared__ double dmin_s;
  __shared__ double inv_s[MAXQ];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nb = (q + 3) / 4, zp = gram_chol_pitch(q);
  for (int o = tid; o < n_s * zp; o += GC_THREADS) {
    const int r = o / zp, c = o - r * zp;
    zs[o] = c < q ? (double)z[(int64_t)r * q + c] : 0.0;
  }
  const int blocks = nb * (nb + 1) / 2;
  int S = 1;
  while (2 * S * blocks <= GC_THREADS && S < 32) S *= 2;
  const int o = tid / S, part = tid - o * S;
  int bi = 0;
  while ((bi + 1) * (bi + 2) / 2 <= o) ++bi;
  const int bj = o - bi * (bi + 1) / 2;
  const bool active = o < blocks;
  bool solved_here = false;
  __syncthreads();
  for (int pass = 0; pass < 2; ++pass) {
    double acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;
    if (active) {
      const double* pa = zs + 4 * bi;
      const double* pb = zs + 4 * bj;
#pragma unroll 2
      for (int rr = part; rr < n_s; rr += S) {
        const double2 a01 = *reinterpret_cast<const double2*>(pa + rr * zp), a23 = *reinterpret_cast<const double2*>(pa + rr * zp + 2);
        const double2 b01 = *reinterpret_cast<const double2*>(pb + rr * zp), b23 = *reinterpret_cast<const double2*>(pb + rr * zp + 2);
        const double av[4] = {a01.x, a01.y, a23.x, a23.y}, bv[4] = {b01.x, b01.y, b23.x, b23.y};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] += av[i] * bv[j];
      }
    }
    for (int off = S >> 1; off > 0; off >>= 1) {
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] += __shfl_xor_sync(0xFFFFFFFFu, acc[i][j], off);
    }
    if (active && part == 0) {
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (4 * bi + i < q && 4 * bj + j < q) L[4 * bi + i][4 * bj + j] = acc[i][j];
    }
    __syncthreads();
    if (tid < 32) {
      double gm = 0.0;
      for (int i = tid; i < q; i += 32) gm = fmax(gm, L[i][i]);
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) gm = fmax(gm, __shfl_xor_sync(0xFFFFFFFFu, gm, off));
      if (tid == 0) gmax_s = gm;
    }
    __syncthreads();
    const double tol = 1e-13 * gmax_s;
    cta_cholesky<MAXQ + 1>(L, q, tol, inv_s, &dmin_s, GC_THREADS);
    if (pass == 0 && dmin_s > 1e-8 * gmax_s) break;
    // z_row <- z_row L^-T in shared memory, one warp per row (the recurrence of apply_chol_kernel)
    solved_here = true;
    for (int r = warp; r < n_s; r += GC_THREADS / 32) {
      double* zr = zs + r * zp;
      double z0 = lane < q ? zr[lane] : 0.0, z1 = lane + 32 < q ? zr[lane + 32] : 0.0, z2 = lane + 64 < q ? zr[lane + 64] : 0.0;
      for (int j = 0; j < q; ++j) {
        const double lj0 = lane < q ? L[lane][j] : 0.0;
        const double lj1 = lane + 32 < q ? L[lane + 32][j] : 0.0;
        const double lj2 = lane + 64 < q ? L[lane + 64][j] : 0.0;
        const double zj = __shfl_sync(0xFFFFFFFFu, j < 32 ? z0 : (j < 64 ? z1 : z2), j & 31);
        const double hj = zj * inv_s[j];
        if (lane == (j & 31)) { if (j < 32) z0 = hj; else if (j < 64) z1 = hj; else z2 = hj; }
        if (lane > j) z0 -= hj * lj0;
        if (lane + 32 > j) z1 -= hj * lj1;
        if (lane + 64 > j) z2 -= hj * lj2;
      }
      if (lane < q) zr[lane] = z0;
      if (lane + 32 < q) zr[lane + 32] = z1;
      if (lane + 64 < q) zr[lane + 64] = z2;
    }
    __syncthreads();
  }
  if (tid == 0) *applied = solved_here ? 1 : 0;
  if (solved_here) {
    for (int e = tid; e < n_s * q; e += GC_THREADS) z[e] = (float)zs[(e / q) * zp + e % q];
  } else {
    if (tid < q) invd_out[tid] = inv_s[tid];
    for (int e = tid; e < q * q; e += GC_THREADS) l_out[e] = L[e / q][e % q];
  }
}

// One CholeskyQR pass, step 2: z_row <- z_row L^-T by forward substitution, one warp per row, column-oriented:
// lane i%32 keeps z_i; step j broadcasts h_j = z_j / L[j][j] from its owner and every lane subtracts h_j L[i][j]
// from its own later entries, so a step is one shuffle and one multiply-add deep (no reduction across lanes).
__global__ void __launch_bounds__(256)
apply_chol_kernel(float* __restrict__ z, int64_t n_rows, int q, const double* __restrict__ l, const double* __restrict__ invd,
                  const int* __restrict__ skip) {
  metis_pdl_wait();
  if (skip != nullptr && *skip) return;
  __shared__ double L[MAXQ][MAXQ + 1];
  __shared__ double inv_s[MAXQ];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int o = tid; o < q * q; o += 256) L[o / q][o % q] = l[o];
  if (tid < q) inv_s[tid] = invd[tid];
  __syncthreads();
  const int64_t r = (int64_t)blockIdx.x * 8 + warp;
  if (r >= n_rows) return;
  static_assert(MAXQ <= 96, "three values per lane");
  double z0 = lane < q ? (double)z[r * q + lane] : 0.0;               // entries lane, lane + 32, lane + 64
  double z1 = lane + 32 < q ? (double)z[r * q + lane + 32] : 0.0;
  double z2 = lane + 64 < q ? (double)z[r * q + lane + 64] : 0.0;
  for (int j = 0; j < q; ++j) {
    const double lj0 = lane < q ? L[lane][j] : 0.0;                    // column j of L (zero above the diagonal is not
    const double lj1 = lane + 32 < q ? L[lane + 32][j] : 0.0;          // stored: masked by the index tests below)
    const double lj2 = lane + 64 < q ? L[lane + 64][j] : 0.0;
    const double zj = __shfl_sync(0xFFFFFFFFu, j < 32 ? z0 : (j < 64 ? z1 : z2), j & 31);
    const double hj = zj * inv_s[j];
    if (lane == (j & 31)) { if (j < 32) z0 = hj; else if (j < 64) z1 = hj; else z2 = hj; }
    if (lane > j) z0 -= hj * lj0;
    if (lane + 32 > j) z1 -= hj * lj1;
    if (lane + 64 > j) z2 -= hj * lj2;
  }
  if (lane < q) z[r * q + lane] = (float)z0;
  if (lane + 32 < q) z[r * q + lane + 32] = (float)z1;
  if (lane + 64 < q) z[r * q + lane + 64] = (float)z2;
}

// ------------------------------------------------------------------------------------------------
// Projection partials: Mp[part][j][col] = sum over the part's sampled rows r of H[r][j] * x[idx[r], col]
// (q x cols per part, row j contiguous).  Thread: two adjacent columns, every second sketch column.
constexpr int PJ_COLS = 256, PJ_ROWS = 32;
template <int NJ4>                                                  // float4 groups of sketch columns per thread
__global__ void __launch_bounds__(256)
project_kernel(const __nv_bfloat16* __restrict__ x, int64_t cols, const int* __restrict__ idx, int n_s, int q,
               const float* __restrict__ h, int rows_per_part, float* __restrict__ mp) {
  metis_pdl_wait();
  __shared__ __align__(16) float hs[2][PJ_ROWS][MAXQ / 2];
  __shared__ int ids[PJ_ROWS];
  const int tid = threadIdx.x, c2 = tid & 127, jg = tid >> 7;       // jg: sketch columns 2*j + jg
  const int64_t col = (int64_t)blockIdx.x * PJ_COLS + c2 * 2;
  const int r_begin = blockIdx.y * rows_per_part, r_end = min(n_s, r_begin + rows_per_part);
  float acc0[NJ4 * 4], acc1[NJ4 * 4];
#pragma unroll
  for (int j = 0; j < NJ4 * 4; ++j) { acc0[j] = 0.0f; acc1[j] = 0.0f; }
  for (int r0 = r_begin; r0 < r_end; r0 += PJ_ROWS) {
    for (int i = tid; i < PJ_ROWS * MAXQ; i += 256) {
      const int rr = i / MAXQ, jj = i % MAXQ;
      hs[jj & 1][rr][jj >> 1] = (r0 + rr < r_end && jj < q) ? h[(int64_t)(r0 + rr) * q + jj] : 0.0f;
    }
    if (tid < PJ_ROWS) ids[tid] = (r0 + tid < r_end) ? idx[r0 + tid] : 0;
    __syncthreads();
    const int nr = min(PJ_ROWS, r_end - r0);
    // the tile's x values first, all loads in flight (inside the loop below each was an L2 round trip per row)
    uint32_t xw[PJ_ROWS];
#pragma unroll
    for (int rr = 0; rr < PJ_ROWS; ++rr) {
      xw[rr] = 0u;
      if (rr < nr) {
        if (col + 1 < cols) xw[rr] = *reinterpret_cast<const uint32_t*>(x + (int64_t)ids[rr] * cols + col);
        else if (col < cols) xw[rr] = (uint32_t)__bfloat16_as_ushort(x[(int64_t)ids[rr] * cols + col]);
      }
    }
#pragma unroll
    for (int rr = 0; rr < PJ_ROWS; ++rr) {
      if (rr >= nr) break;
      const float x0 = __uint_as_float(xw[rr] << 16), x1 = __uint_as_float(xw[rr] & 0xFFFF0000u);
#pragma unroll
      for (int j4 = 0; j4 < NJ4; ++j4) {
        const float4 hv = *reinterpret_cast<const float4*>(&hs[jg][rr][j4 * 4]);
        acc0[j4 * 4 + 0] = fmaf(hv.x, x0, acc0[j4 * 4 + 0]); acc1[j4 * 4 + 0] = fmaf(hv.x, x1, acc1[j4 * 4 + 0]);
        acc0[j4 * 4 + 1] = fmaf(hv.y, x0, acc0[j4 * 4 + 1]); acc1[j4 * 4 + 1] = fmaf(hv.y, x1, acc1[j4 * 4 + 1]);
        acc0[j4 * 4 + 2] = fmaf(hv.z, x0, acc0[j4 * 4 + 2]); acc1[j4 * 4 + 2] = fmaf(hv.z, x1, acc1[j4 * 4 + 2]);
        acc0[j4 * 4 + 3] = fmaf(hv.w, x0, acc0[j4 * 4 + 3]); acc1[j4 * 4 + 3] = fmaf(hv.w, x1, acc1[j4 * 4 + 3]);
      }
    }
    __syncthreads();
  }
  float* dst = mp + (int64_t)blockIdx.y * q * cols;
#pragma unroll
  for (int j = 0; j < NJ4 * 4; ++j)
    if (2 * j + jg < q) {
      if (col < cols) dst[(int64_t)(2 * j + jg) * cols + col] = acc0[j];
      if (col + 1 < cols) dst[(int64_t)(2 * j + jg) * cols + col + 1] = acc1[j];
    }
}

// ------------------------------------------------------------------------------------------------
// Symmetric positive semi-definite eigen-decomposition (n <= MAXQ) in FP64, one CTA.
// G = L L^T (Cholesky, dependent columns zeroed), then one-sided (Hestenes) Jacobi on the columns of Y = L:
// plane rotations make the columns mutually orthogonal, Y J1 J2 ... = U Sigma, so G = Y Y^T = U Sigma^2 U^T:
// eigenvalues are the squared column norms and eigenvectors the normalised columns.  Working on the
// Cholesky factor needs one matrix instead of two (no separate eigenvector accumulation), one barrier per
// round, and converges in few sweeps.  Each round pairs the columns into n/2 disjoint couples (round-robin
// tournament); a couple is handled by LANES threads that split the rows, reduce the inner product with
// shuffles and rotate their rows in registers.
// Input: Gram matrix (ld x ld, leading n x n block used).  Output: eigenvalues descending, eigenvectors as
// columns of evecs[n][n].
__device__ __forceinline__ void jacobi_pair(int I, int step, int np, int* p, int* q) {
  int a, b;
  if (I == 0) { a = 0; b = (step % (np - 1)) + 1; }
  else { a = ((step + I) % (np - 1)) + 1; b = ((step + np - 1 - I) % (np - 1)) + 1; }
  *p = min(a, b); *q = max(a, b);
}

// 1/sqrt(x) in FP64 from an FP32 seed and two Newton steps (x in the FP32 range; relative error ~1e-16).
__device__ __forceinline__ double fast_rsqrt(double x) {
  double y = (double)rsqrtf((float)x);
  y = y * (1.5 - 0.5 * x * y * y);
  y = y * (1.5 - 0.5 * x * y * y);
  return y;
}

template <int R, int LANES>                             // lanes per couple (8 or 16), rows per lane: ceil(n / LANES)
__global__ void __launch_bounds__(LANES == 8 ? (R > 8 ? 288 : 256) : (128 * R > 256 ? 128 * R : 256), 1)
jacobi_eig_kernel(const double* __restrict__ g, int n, int ld, float exit_cos2, double* __restrict__ evals,
                  double* __restrict__ evecs) {
  metis_pdl_wait();
  extern __shared__ __align__(16) unsigned char jsm[];
  double (*Y)[MAXQ + 1] = reinterpret_cast<double (*)[MAXQ + 1]>(jsm);
  __shared__ double lam[MAXQ];
  __shared__ double gmax_s;
  __shared__ int order[MAXQ];
  __shared__ uint8_t pairs[MAXQ][MAXQ / 2][2];          // [round][couple] -> (p, q)
  constexpr int NTHR = LANES == 8 ? (R > 8 ? 288 : 256) : (128 * R > 256 ? 128 * R : 256);
  const int tid = threadIdx.x;
  const int np = n + (n & 1), half = np / 2;
  for (int o = tid; o < np * np; o += NTHR) {
    const int i = o / np, j = o % np;
    Y[i][j] = (i < n && j < n) ? 0.5 * (g[i * ld + j] + g[j * ld + i]) : 0.0;
  }
  for (int o = tid; o < (np - 1) * half; o += NTHR) {
    int p, q;
    jacobi_pair(o % half, o / half, np, &p, &q);
    pairs[o / half][o % half][0] = (uint8_t)p; pairs[o / half][o % half][1] = (uint8_t)q;
  }
  __syncthreads();
  // ---- Cholesky, lower factor in place; the strict upper triangle is cleared afterwards ----
  if (tid < 32) {
    double gm = 0.0;
    for (int i = tid; i < n; i += 32) gm = fmax(gm, Y[i][i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) gm = fmax(gm, __shfl_xor_sync(0xFFFFFFFFu, gm, o));
    if (tid == 0) gmax_s = gm;
  }
  __syncthreads();
  const double tol = 1e-14 * gmax_s;
  cta_cholesky<MAXQ + 1>(Y, n, tol, lam, nullptr, NTHR);
  for (int o = tid; o < np * np; o += NTHR) {
    const int i = o / np, j = o % np;
    if (j > i) Y[i][j] = 0.0;
  }
  __syncthreads();
  // ---- one-sided Jacobi on the columns of Y ----
  // FP64 is kept for what sets the accuracy of the result - the columns themselves and the orthonormality of
  // each applied rotation - and FP32 is used for what only steers convergence: the carried column norms, the
  // rotation angle and the convergence measure.  (FP64 instructions are the slow ones in this latency chain.)
  // Norms are carried along and recomputed exactly at the start of every sweep, so a round needs a single
  // inner product per couple.  A sweep whose largest cos^2 between paired columns was below exit_cos2 is the
  // last one: convergence is quadratic, so its own rotations leave the columns orthogonal to about exit_cos2.
  float* lamf = reinterpret_cast<float*>(lam);          // FP32 norms during the sweeps (lam is reused below)
  const int m = tid / LANES, sub = tid % LANES;         // couple index, row slice
  const bool active = m < half;
  const int mc = min(m, MAXQ / 2 - 1);                  // table column of this couple slot (idle slots beyond the table share the last)
  for (int sweep = 0; sweep < 16; ++sweep) {
    if (tid < np) {
      double a0 = 0.0, a1 = 0.0;
      int i = 0;
      for (; i + 1 < np; i += 2) { a0 += Y[i][tid] * Y[i][tid]; a1 += Y[i + 1][tid] * Y[i + 1][tid]; }
      if (i < np) a0 += Y[i][tid] * Y[i][tid];
      lamf[tid] = (float)(a0 + a1);
    }
    __syncthreads();
    int p = active ? pairs[0][m][0] : 0, q = active ? pairs[0][m][1] : 0;
    bool above = false;                                 // some couple of this slot had cos^2 above exit_cos2 in this sweep
    for (int step = 0; step < np - 1; ++step) {
      {
        // every lane takes part in the shuffles; lanes of couples beyond n/2 carry zeros and write nothing
        double yp[R], yq[R];
        double c = 0.0;
#pragma unroll
        for (int t = 0; t < R; ++t) {
          const int i = sub + LANES * t;
          yp[t] = (active && i < np) ? Y[i][p] : 0.0;
          yq[t] = (active && i < np) ? Y[i][q] : 0.0;
          c += yp[t] * yq[t];
        }
#pragma unroll
        for (int o = LANES / 2; o > 0; o >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
        const float a = lamf[p], b = lamf[q], cf = (float)c;
        // next round's couple, fetched early (after the last round, and for idle couple slots, the table entry is
        // unused filler: it is inside the array and never used as an index)
        const int pn = pairs[step + 1][mc][0], qn = pairs[step + 1][mc][1];
        // rotate only if the two columns are not yet orthogonal to working precision (cos^2 > 1e-26)
        if (active && cf * cf > 1e-26f * (a * b)) {
          // tan(theta) = 2c / (d + sign(d) sqrt(d^2 + 4c^2)), d = b - a: the smaller root, |theta| <= pi/4.  These
          // FP32 quantities only steer convergence, so the fast reciprocal and reciprocal square root are enough.
          // with cos(2 theta) = |d| / hyp and sin(2 theta) = +-2c / hyp:  cos^2(theta) = (1 + cos 2theta) / 2,
          // sin(theta) = sin(2 theta) / (2 cos theta): two reciprocal square roots, no division
          const float d = b - a, c2 = 2.0f * cf;
          const float h2 = fmaf(c2, c2, d * d);
          const float rh = rsqrtf(h2);
          const float cc = fmaf(0.5f * fabsf(d), rh, 0.5f);
          const float rs = rsqrtf(cc);
          const float c32 = cc * rs, s32 = (d < 0.0f ? -c2 : c2) * (0.5f * rh) * rs;
          const float tf = s32 * rs;                      // tan(theta), for the carried norms
          // (c32, s32) is a unit vector to ~1e-7; one Newton step on 1/sqrt(c^2 + s^2) in FP64 makes it one to ~1e-14
          const double cd = (double)c32, sd = (double)s32;
          const double scale = 1.5 - 0.5 * (cd * cd + sd * sd);
          const double cs = cd * scale, sn = sd * scale;
#pragma unroll
          for (int tt = 0; tt < R; ++tt) {
            const int i = sub + LANES * tt;
            if (i < np) {
              Y[i][p] = cs * yp[tt] - sn * yq[tt];
              Y[i][q] = sn * yp[tt] + cs * yq[tt];
            }
          }
          // |y_p'|^2 = a - t c, |y_q'|^2 = b + t c for the exact rotation.  Every lane of the couple holds the same
          // numbers and stores them (one value per address): no lane-dependent branch inside the round.
          const float tc = tf * cf;
          lamf[p] = a - tc;
          lamf[q] = b + tc;
          above |= cf * cf > exit_cos2 * (a * b);
        }
        p = pn; q = qn;
      }
      __syncthreads();
    }
    if (!__syncthreads_or(above ? 1 : 0)) break;        // no couple above the threshold: this was the last sweep
  }
  // ---- eigenvalues = squared column norms, eigenvectors = normalised columns ----
  if (tid < n) {
    double a = 0.0;
    for (int i = 0; i < n; ++i) a += Y[i][tid] * Y[i][tid];
    lam[tid] = a;
    order[tid] = tid;                                   // stays a valid index if NaNs make the ranks below collide
  }
  __syncthreads();
  if (tid < n) {
    const double li = lam[tid];
    int rank = 0;
    for (int j = 0; j < n; ++j) rank += (lam[j] > li) || (lam[j] == li && j < tid);
    order[rank] = tid;
  }
  __syncthreads();
  if (tid < n) evals[tid] = lam[order[tid]];
  for (int o = tid; o < n * n; o += NTHR) {
    const int i = o / n, j = order[o % n];
    const double l2 = lam[j];
    evecs[o] = l2 > 0.0 ? Y[i][j] * fast_rsqrt_wide(l2) : 0.0;
  }
}

// ------------------------------------------------------------------------------------------------
// Right basis from the small SVD: B[j][col] = sum_i Ut[i][j] M[i][col] / s_j, s_j = sqrt(eval_j); j < k.
// Block = 64 columns x 4 groups of output vectors; a thread keeps four accumulators in flight.
constexpr int RB_COLS = 32;
__global__ void __launch_bounds__(256)
right_basis_kernel(const float* __restrict__ m, int64_t cols, int q, int k, const double* __restrict__ evals,
                   const double* __restrict__ evecs, float* __restrict__ basis, float* __restrict__ sigma_out) {
  metis_pdl_wait();
  // 32 columns per CTA; the CTA's slice of M is staged in shared memory first, so that all of its loads are in
  // flight at once (read inside the accumulation loop they were one L2 round trip per term)
  __shared__ double ut[MAXQ][64 + 1];                   // eigenvectors, the k <= 64 wanted columns
  __shared__ double inv_s[64];
  __shared__ float ms[MAXQ][RB_COLS];
  const int tid = threadIdx.x, cx = tid & (RB_COLS - 1), jg = tid / RB_COLS;      // 8 groups of output vectors
  const int64_t col0 = (int64_t)blockIdx.x * RB_COLS;
  for (int o = tid; o < q * RB_COLS; o += 256) {
    const int i = o / RB_COLS, c = o % RB_COLS;
    ms[i][c] = col0 + c < cols ? m[(int64_t)i * cols + col0 + c] : 0.0f;
  }
  for (int o = tid; o < q * k; o += 256) ut[o / k][o % k] = evecs[(o / k) * q + o % k];
  if (tid < k) {
    const double s = sqrt(fmax(evals[tid], 0.0));
    inv_s[tid] = s > 0.0 ? 1.0 / s : 0.0;
    if (blockIdx.x == 0 && sigma_out != nullptr) sigma_out[tid] = (float)s;
  }
  __syncthreads();
  const int64_t col = col0 + cx;
  if (col >= cols) return;
  for (int j0 = jg * 4; j0 < k; j0 += 32) {
    double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
    for (int i = 0; i < q; ++i) {
      const double v = (double)ms[i][cx];
      a0 += ut[i][j0] * v; a1 += ut[i][j0 + 1] * v; a2 += ut[i][j0 + 2] * v; a3 += ut[i][j0 + 3] * v;
    }
    basis[(int64_t)j0 * cols + col] = (float)(a0 * inv_s[j0]);
    if (j0 + 1 < k) basis[(int64_t)(j0 + 1) * cols + col] = (float)(a1 * inv_s[j0 + 1]);
    if (j0 + 2 < k) basis[(int64_t)(j0 + 2) * cols + col] = (float)(a2 * inv_s[j0 + 2]);
    if (j0 + 3 < k) basis[(int64_t)(j0 + 3) * cols + col] = (float)(a3 * inv_s[j0 + 3]);
  }
}

// ------------------------------------------------------------------------------------------------
// Tensor-core helpers (warp-level mma.sync m16n8k16, BF16 operands, FP32 accumulate).  FP32 operands
// are fed as three BF16 terms (hi + lo + lo2 = 24 mantissa bits) so the products stay FP32-accurate.
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
// three-term BF16 split of a pair of floats: v = hi + lo + lo2 (each term BF16, packed as pairs)
__device__ __forceinline__ void split3(float x, float y, uint32_t& hi, uint32_t& lo, uint32_t& lo2) {
  const __nv_bfloat16 xh = __float2bfloat16_rn(x), yh = __float2bfloat16_rn(y);
  const float xr = x - __bfloat162float(xh), yr = y - __bfloat162float(yh);
  const __nv_bfloat16 xl = __float2bfloat16_rn(xr), yl = __float2bfloat16_rn(yr);
  const float xr2 = xr - __bfloat162float(xl), yr2 = yr - __bfloat162float(yl);
  hi = (uint32_t)__bfloat16_as_ushort(xh) | ((uint32_t)__bfloat16_as_ushort(yh) << 16);
  lo = (uint32_t)__bfloat16_as_ushort(xl) | ((uint32_t)__bfloat16_as_ushort(yl) << 16);
  lo2 = pack_bf16(xr2, yr2);
}

// BF16 splits of the right basis in both operand orientations:
//   bs[t][j][col]  (col contiguous; B operand of C = x B, contraction over col); with more than 64 vectors the
//                  layout is by groups of 64 vectors, bs[group][t][j in group][col], so that the three terms of a
//                  group are one contiguous matrix (one launch of the coefficient kernel per group)
//   bt[t][col][j]  (j contiguous, padded to kp; B operand of C B^T, contraction over j; optional)
__global__ void __launch_bounds__(128)
basis_splits_kernel(const float* __restrict__ basis, int64_t cols, int k, int kp, __nv_bfloat16* __restrict__ bs,
                    __nv_bfloat16* __restrict__ bt, __nv_bfloat16* __restrict__ b6, int kx) {
  metis_pdl_wait();
  const int64_t col = (int64_t)blockIdx.x * 128 + threadIdx.x;
  if (col >= cols) return;
  // b6 (optional): [cols][kx], per column the six K blocks [Bh | Bl | Bh | Bl2 | Bh | Bl] of the residual product
  if (b6 != nullptr && blockIdx.y == 0)
    for (int z = 6 * kp; z < kx; z += 8) *reinterpret_cast<uint4*>(b6 + col * kx + z) = make_uint4(0u, 0u, 0u, 0u);
  {
    const int j0 = blockIdx.y * 8;                        // grid.y = kp / 8: one group of eight vectors per thread
    uint32_t w[3][4];
#pragma unroll
    for (int jj = 0; jj < 8; jj += 2) {
      const float v0 = j0 + jj < k ? basis[(int64_t)(j0 + jj) * cols + col] : 0.0f;
      const float v1 = j0 + jj + 1 < k ? basis[(int64_t)(j0 + jj + 1) * cols + col] : 0.0f;
      split3(v0, v1, w[0][jj >> 1], w[1][jj >> 1], w[2][jj >> 1]);
    }
#pragma unroll
    for (int t = 0; t < 3; ++t) {
      const int grp = j0 / 64, gw = min(64, kp - 64 * grp);
      const int64_t row0 = (int64_t)3 * 64 * grp + (int64_t)t * gw + (j0 - 64 * grp);
#pragma unroll
      for (int jj = 0; jj < 8; ++jj)
        bs[(row0 + jj) * cols + col] = __ushort_as_bfloat16((unsigned short)((w[t][jj >> 1] >> (16 * (jj & 1))) & 0xFFFFu));
      if (bt != nullptr) *reinterpret_cast<uint4*>(bt + ((int64_t)t * cols + col) * kp + j0) = make_uint4(w[t][0], w[t][1], w[t][2], w[t][3]);
    }
    if (b6 != nullptr) {
      const int sel[6] = {0, 1, 0, 2, 0, 1};
#pragma unroll
      for (int term = 0; term < 6; ++term)
        *reinterpret_cast<uint4*>(b6 + col * kx + term * kp + j0) = make_uint4(w[sel[term]][0], w[sel[term]][1], w[sel[term]][2], w[sel[term]][3]);
    }
  }
}

// Broadcast of the sampled subspace to every row (Section 3.1): C[r][j] = sum_col x[r, col] * B[j][col],
// stored row-major with kp columns (zero padded).  One CTA = 32 rows; its 8 warps split the columns and
// their partial tiles are added in fixed order.  Fused by-products of the same pass over x: amax|x|
// (atomic max, order independent) and the FP64 Gram partial of the CTA's rows of C (for Rayleigh-Ritz).
template <int KP>
__global__ void __launch_bounds__(256)
coeff_mma_kernel(const __nv_bfloat16* __restrict__ x, int64_t rows, int64_t cols, const __nv_bfloat16* __restrict__ bs,
                 float* __restrict__ coef, float* __restrict__ amax_out, double* __restrict__ gram_part) {
  metis_pdl_wait();
  constexpr int NT = KP / 8;
  extern __shared__ __align__(16) unsigned char smem[];
  float* red = reinterpret_cast<float*>(smem);                 // [8 warps][32 rows][KP]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int64_t row0 = (int64_t)blockIdx.x * 32;
  const int ksteps = (int)(cols / 16);
  const int ks_begin = (int)((int64_t)ksteps * warp / 8), ks_end = (int)((int64_t)ksteps * (warp + 1) / 8);
  float acc[2][NT][4];
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[m][n][e] = 0.0f;
  uint32_t amax2 = 0u;                                         // two running |.| maxima, BF16 pair
  const bool v0 = row0 + g < rows, v1 = row0 + g + 8 < rows, v2 = row0 + g + 16 < rows, v3 = row0 + g + 24 < rows;
  const __nv_bfloat16* xr0 = x + (row0 + g) * cols;
#pragma unroll 2
  for (int ks = ks_begin; ks < ks_end; ++ks) {
    const int kk = ks * 16 + 2 * t;
    uint32_t a[2][4];
    a[0][0] = v0 ? *reinterpret_cast<const uint32_t*>(xr0 + kk) : 0u;
    a[0][1] = v1 ? *reinterpret_cast<const uint32_t*>(xr0 + 8 * cols + kk) : 0u;
    a[0][2] = v0 ? *reinterpret_cast<const uint32_t*>(xr0 + kk + 8) : 0u;
    a[0][3] = v1 ? *reinterpret_cast<const uint32_t*>(xr0 + 8 * cols + kk + 8) : 0u;
    a[1][0] = v2 ? *reinterpret_cast<const uint32_t*>(xr0 + 16 * cols + kk) : 0u;
    a[1][1] = v3 ? *reinterpret_cast<const uint32_t*>(xr0 + 24 * cols + kk) : 0u;
    a[1][2] = v2 ? *reinterpret_cast<const uint32_t*>(xr0 + 16 * cols + kk + 8) : 0u;
    a[1][3] = v3 ? *reinterpret_cast<const uint32_t*>(xr0 + 24 * cols + kk + 8) : 0u;
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t ab = a[m][e] & 0x7FFF7FFFu;             // |.| of both halves; BF16 magnitudes order like integers
        const uint32_t lo = max(ab & 0xFFFFu, amax2 & 0xFFFFu), hi = max(ab >> 16, amax2 >> 16);
        amax2 = lo | (hi << 16);
      }
#pragma unroll
    for (int sp = 0; sp < 3; ++sp) {
      const __nv_bfloat16* bsp = bs + (int64_t)sp * KP * cols;
#pragma unroll
      for (int n = 0; n < NT; ++n) {
        const __nv_bfloat16* bp = bsp + (int64_t)(n * 8 + g) * cols + kk;
        const uint32_t b0 = *reinterpret_cast<const uint32_t*>(bp), b1 = *reinterpret_cast<const uint32_t*>(bp + 8);
        mma_bf16(acc[0][n], a[0], b0, b1);
        mma_bf16(acc[1][n], a[1], b0, b1);
      }
    }
  }
  // per-warp partial tile -> shared memory
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      float* r0p = red + ((warp * 32) + m * 16 + g) * KP + n * 8 + 2 * t;
      r0p[0] = acc[m][n][0]; r0p[1] = acc[m][n][1];
      r0p[8 * KP] = acc[m][n][2]; r0p[8 * KP + 1] = acc[m][n][3];
    }
  {
    uint32_t am = max((amax2 & 0xFFFFu) << 16, amax2 & 0xFFFF0000u);      // ordered bit patterns: a NaN survives
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, o));
    if (lane == 0 && amax_out) atomicMax(reinterpret_cast<unsigned int*>(amax_out), am);
  }
  __syncthreads();
  float* cfin = red + 8 * 32 * KP;                             // [32][KP] final tile
  for (int o = tid; o < 32 * KP; o += 256) {
    float sacc = 0.0f;
#pragma unroll
    for (int w = 0; w < 8; ++w) sacc += red[w * 32 * KP + o];
    cfin[o] = sacc;
    const int64_t r = row0 + o / KP;
    if (r < rows) coef[r * KP + (o % KP)] = sacc;
  }
  __syncthreads();
  if (gram_part) {
    for (int o = tid; o < KP * KP; o += 256) {
      const int i = o / KP, j = o % KP;
      double a = 0.0;
#pragma unroll 8
      for (int r = 0; r < 32; ++r) a += (double)cfin[r * KP + i] * (double)cfin[r * KP + j];
      gram_part[(int64_t)blockIdx.x * KP * KP + o] = a;
    }
  }
}

// out[e] = sum over all partials p of in[p][e].  A CTA of four warps owns 32 elements; warp s adds every fourth
// partial (eight loads in flight), the four sums are added in a fixed order: the result does not depend on timing.
__global__ void __launch_bounds__(128)
reduce_gram_kernel(const double* __restrict__ in, int n_in, int nn, double* __restrict__ out,
                   const int* __restrict__ skip) {
  metis_pdl_wait();
  if (skip != nullptr && *skip) return;
  __shared__ double part[4][32];
  const int lane = threadIdx.x & 31, sl = threadIdx.x >> 5;
  const int e = blockIdx.x * 32 + lane;
  double a = 0.0;
  if (e < nn) {
    int p = sl;
    for (; p + 28 < n_in; p += 32) {
      double v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = in[(int64_t)(p + 4 * u) * nn + e];
#pragma unroll
      for (int u = 0; u < 8; ++u) a += v[u];
    }
    for (; p < n_in; p += 4) a += in[(int64_t)p * nn + e];
  }
  part[sl][lane] = a;
  __syncthreads();
  if (sl == 0 && e < nn) out[e] = ((part[0][lane] + part[1][lane]) + part[2][lane]) + part[3][lane];
}

// Sums the column slices of the tensor-core broadcast pass in a fixed order: coef[r][j] = sum_s part[s][r][j],
// and writes the FP64 Gram partial of the CTA's 32 rows of C (for Rayleigh-Ritz).
template <int KP>
__global__ void __launch_bounds__(256)
coef_finish_kernel(const float* __restrict__ part, int slices, int64_t rows, float* __restrict__ coef,
                   double* __restrict__ gram_part, __nv_bfloat16* __restrict__ a6, int kx) {
  metis_pdl_wait();
  __shared__ float cfin[32 * KP];
  const int tid = threadIdx.x;
  const int64_t row0 = (int64_t)blockIdx.x * 32;
  for (int o = tid; o < 32 * KP; o += 256) {
    const int64_t r = row0 + o / KP;
    float v = 0.0f;
    if (r < rows) {
      float t[8];                                          // at most eight slices; all loads in flight, fixed order of the sum
#pragma unroll
      for (int s = 0; s < 8; ++s) t[s] = s < slices ? part[((int64_t)s * rows + r) * KP + (o % KP)] : 0.0f;
#pragma unroll
      for (int s = 0; s < 8; ++s) v += t[s];
      coef[r * KP + (o % KP)] = v;
    }
    cfin[o] = v;
  }
  __syncthreads();
  if (a6 != nullptr) {
    // a6: [rows][kx], per row the six K blocks [Ch | Ch | Cl | Ch | Cl2 | Cl] of the residual product (zero padded)
    for (int o = tid; o < 32 * (KP / 8); o += 256) {
      const int rr = o / (KP / 8), j0 = (o % (KP / 8)) * 8;
      const int64_t r = row0 + rr;
      if (r >= rows) continue;
      float v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = cfin[rr * KP + j0 + e];
      uint4 h, l, l2;
      metis_split3x8(v, h, l, l2);
      __nv_bfloat16* dst = a6 + r * kx + j0;
      *reinterpret_cast<uint4*>(dst) = h; *reinterpret_cast<uint4*>(dst + KP) = h; *reinterpret_cast<uint4*>(dst + 2 * KP) = l;
      *reinterpret_cast<uint4*>(dst + 3 * KP) = h; *reinterpret_cast<uint4*>(dst + 4 * KP) = l2; *reinterpret_cast<uint4*>(dst + 5 * KP) = l;
      if (j0 == 0)
        for (int z = 6 * KP; z < kx; z += 8) *reinterpret_cast<uint4*>(a6 + r * kx + z) = make_uint4(0u, 0u, 0u, 0u);
    }
  }
  if (gram_part) {
    __shared__ double cd[32 * KP];                      // converted once: FP32 -> FP64 is a slow-rate instruction
    for (int o = tid; o < 32 * KP; o += 256) cd[o] = (double)cfin[o];
    __syncthreads();
    for (int o = tid; o < KP * KP; o += 256) {
      const int i = o / KP, j = o % KP;
      double a = 0.0;
#pragma unroll 8
      for (int r = 0; r < 32; ++r) a += cd[r * KP + i] * cd[r * KP + j];
      gram_part[(int64_t)blockIdx.x * KP * KP + o] = a;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Fused residual + quantizer: R = x - C B^T on a 128 x 128 tile (tensor cores, three-term BF16 splits of
// both FP32 operands), then NVFP4 in one or both block orientations straight from shared memory (the
// residual never goes to HBM unless `dense` is given).  coef: [rows][KP] row-major, bt: [3][cols][KP].
template <int KP>
__global__ void __launch_bounds__(metis_qt::THREADS, 2)
residual_quant_kernel(const __nv_bfloat16* __restrict__ x, const float* __restrict__ coef,
                      const __nv_bfloat16* __restrict__ bt, metis_qt::QuantParams p,
                      const float* __restrict__ amax_src, float* ts_out0, float* ts_out1, float* __restrict__ dense) {
  metis_pdl_wait();
  using namespace metis_qt;
  extern __shared__ __align__(16) unsigned char smem[];
  float* tile = reinterpret_cast<float*>(smem);
  Stage* stage = reinterpret_cast<Stage*>(smem + sizeof(float) * TILE * PITCH);
  uint16_t* rnd = reinterpret_cast<uint16_t*>(smem + sizeof(float) * TILE * PITCH + sizeof(Stage));
  const bool sr = p.rounding == METIS_ROUND_SR;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int64_t row0 = (int64_t)blockIdx.y * TILE, col0 = (int64_t)blockIdx.x * TILE;
  const float s_T = metis_tensor_scale(*amax_src);
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) {
    if (ts_out0) *ts_out0 = s_T;
    if (ts_out1) *ts_out1 = s_T;
  }
  if (sr) fill_draws(rnd, p, row0, col0);
  // this warp: rows row0 + 16*warp .. +15, all 128 columns
  const int64_t ra = row0 + warp * 16 + g, rb = ra + 8;
  const bool va = ra < p.rows, vb = rb < p.rows;
  float acc[16][4];
#pragma unroll
  for (int n = 0; n < 16; ++n)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[n][e] = 0.0f;
#pragma unroll
  for (int ks = 0; ks < KP / 16; ++ks) {
    const int kk = ks * 16 + 2 * t;
    uint32_t ah[4], al[4], al2[4];
    {
      const float2 z = make_float2(0.0f, 0.0f);
      const float2 c0 = va ? *reinterpret_cast<const float2*>(coef + ra * KP + kk) : z;
      const float2 c1 = vb ? *reinterpret_cast<const float2*>(coef + rb * KP + kk) : z;
      const float2 c2 = va ? *reinterpret_cast<const float2*>(coef + ra * KP + kk + 8) : z;
      const float2 c3 = vb ? *reinterpret_cast<const float2*>(coef + rb * KP + kk + 8) : z;
      split3(c0.x, c0.y, ah[0], al[0], al2[0]);
      split3(c1.x, c1.y, ah[1], al[1], al2[1]);
      split3(c2.x, c2.y, ah[2], al[2], al2[2]);
      split3(c3.x, c3.y, ah[3], al[3], al2[3]);
    }
#pragma unroll
    for (int n = 0; n < 16; ++n) {
      const int64_t col = col0 + n * 8 + g;
      uint32_t bh0 = 0, bh1 = 0, bl0 = 0, bl1 = 0, bm0 = 0, bm1 = 0;
      if (col < p.cols) {
        const __nv_bfloat16* bp = bt + col * KP + kk;
        bh0 = *reinterpret_cast<const uint32_t*>(bp); bh1 = *reinterpret_cast<const uint32_t*>(bp + 8);
        bl0 = *reinterpret_cast<const uint32_t*>(bp + p.cols * KP); bl1 = *reinterpret_cast<const uint32_t*>(bp + p.cols * KP + 8);
        bm0 = *reinterpret_cast<const uint32_t*>(bp + 2 * p.cols * KP); bm1 = *reinterpret_cast<const uint32_t*>(bp + 2 * p.cols * KP + 8);
      }
      // smallest terms first
      mma_bf16(acc[n], al, bl0, bl1);
      mma_bf16(acc[n], al2, bh0, bh1);
      mma_bf16(acc[n], ah, bm0, bm1);
      mma_bf16(acc[n], al, bh0, bh1);
      mma_bf16(acc[n], ah, bl0, bl1);
      mma_bf16(acc[n], ah, bh0, bh1);
    }
  }
  // R = x - acc into the shared tile (and to `dense` when asked)
#pragma unroll
  for (int n = 0; n < 16; ++n) {
    const int64_t col = col0 + n * 8 + 2 * t;
    const int lc = n * 8 + 2 * t;
    float x00 = 0.0f, x01 = 0.0f, x10 = 0.0f, x11 = 0.0f;
    if (col < p.cols) {
      if (va) { const uint32_t w = *reinterpret_cast<const uint32_t*>(x + ra * p.cols + col); x00 = __uint_as_float(w << 16); x01 = __uint_as_float(w & 0xFFFF0000u); }
      if (vb) { const uint32_t w = *reinterpret_cast<const uint32_t*>(x + rb * p.cols + col); x10 = __uint_as_float(w << 16); x11 = __uint_as_float(w & 0xFFFF0000u); }
    }
    const float2 r0v = make_float2(x00 - acc[n][0], x01 - acc[n][1]);
    const float2 r1v = make_float2(x10 - acc[n][2], x11 - acc[n][3]);
    *reinterpret_cast<float2*>(tile + (warp * 16 + g) * PITCH + lc) = (va && col < p.cols) ? r0v : make_float2(0.0f, 0.0f);
    *reinterpret_cast<float2*>(tile + (warp * 16 + g + 8) * PITCH + lc) = (vb && col < p.cols) ? r1v : make_float2(0.0f, 0.0f);
    if (dense != nullptr && col < p.cols) {
      if (va) *reinterpret_cast<float2*>(dense + ra * p.cols + col) = r0v;
      if (vb) *reinterpret_cast<float2*>(dense + rb * p.cols + col) = r1v;
    }
  }
  __syncthreads();
  quantize_tile(tile, rnd, stage, p, row0, col0, s_T);
}

// ------------------------------------------------------------------------------------------------
// Sketch of gathered rows (mma.sync): Zp[chunk][row][j] = sum over the chunk's columns of x[idx[row], col] * Omega[col, j].
// One CTA = 256 sampled rows x one column chunk (`ccols` = 64 or 256 columns, see sketch_chunk_cols); Omega's slice
// is generated once per CTA (Philox + quantile table) straight into shared memory, transposed to [j][col] BF16 (its
// values are BF16 by construction, so the products are exact and only the FP32 accumulation rounds).  Optionally also
// reduces amax|x| over the rows it reads.  A full sketch of an aligned operand does not come here: it runs on the
// tcgen05 kernel of the broadcast pass (omega_rows_kernel + metis_launch_coeff_tc in its raw mode).
constexpr int SKM_ROWS = 256, SKM_COLS = 256, SKM_PITCH = SKM_COLS + 8;
template <int NT>                                      // sketch columns / 8, rounded up
__global__ void __launch_bounds__(256)
sketch_mma_kernel(const __nv_bfloat16* __restrict__ x, int64_t cols, const int* __restrict__ idx, int n_s, int q,
                  uint64_t seed, const __nv_bfloat16* __restrict__ lut, float* __restrict__ zp, float* __restrict__ amax_out,
                  int ccols) {
  metis_pdl_wait();
  extern __shared__ __align__(16) unsigned char smem[];
  __nv_bfloat16* om = reinterpret_cast<__nv_bfloat16*>(smem);          // [NT*8][SKM_PITCH]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int64_t col0 = (int64_t)blockIdx.y * ccols;        // ccols <= SKM_COLS columns per CTA
  const int row0 = blockIdx.x * SKM_ROWS + warp * 32;
  const int ncols = (int)min((int64_t)ccols, cols - col0);
  for (int i = tid; i < NT * 8 * SKM_PITCH; i += 256) om[i] = __float2bfloat16_rn(0.0f);
  __syncthreads();
  const uint64_t e_lo = (uint64_t)col0 * q, e_hi = (uint64_t)(col0 + ncols) * q;
  for (uint64_t blk = (e_lo >> 3) + tid; blk <= ((e_hi - 1) >> 3); blk += 256) {
    const uint4 w = metis_philox_block(blk, seed, METIS_STREAM_OMEGA);
#pragma unroll
    for (uint32_t h = 0; h < 8; ++h) {
      const uint64_t e = (blk << 3) + h;
      if (e >= e_lo && e < e_hi) {
        const uint32_t rel = (uint32_t)(e - e_lo);
        om[(rel % q) * SKM_PITCH + rel / q] = lut[metis_u16_of(w, h)];
      }
    }
  }
  __syncthreads();
  float acc[2][NT][4];
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[m][n][e] = 0.0f;
  const bool v0 = row0 + g < n_s, v1 = row0 + g + 8 < n_s, v2 = row0 + g + 16 < n_s, v3 = row0 + g + 24 < n_s;
  const __nv_bfloat16* p0 = x + (int64_t)(v0 ? idx[row0 + g] : 0) * cols + col0;
  const __nv_bfloat16* p1 = x + (int64_t)(v1 ? idx[row0 + g + 8] : 0) * cols + col0;
  const __nv_bfloat16* p2 = x + (int64_t)(v2 ? idx[row0 + g + 16] : 0) * cols + col0;
  const __nv_bfloat16* p3 = x + (int64_t)(v3 ? idx[row0 + g + 24] : 0) * cols + col0;
  uint32_t amax2 = 0u;
#pragma unroll 2
  for (int ks = 0; ks < ncols / 16; ++ks) {
    const int kk = ks * 16 + 2 * t;
    uint32_t a[2][4];
    a[0][0] = v0 ? *reinterpret_cast<const uint32_t*>(p0 + kk) : 0u;
    a[0][1] = v1 ? *reinterpret_cast<const uint32_t*>(p1 + kk) : 0u;
    a[0][2] = v0 ? *reinterpret_cast<const uint32_t*>(p0 + kk + 8) : 0u;
    a[0][3] = v1 ? *reinterpret_cast<const uint32_t*>(p1 + kk + 8) : 0u;
    a[1][0] = v2 ? *reinterpret_cast<const uint32_t*>(p2 + kk) : 0u;
    a[1][1] = v3 ? *reinterpret_cast<const uint32_t*>(p3 + kk) : 0u;
    a[1][2] = v2 ? *reinterpret_cast<const uint32_t*>(p2 + kk + 8) : 0u;
    a[1][3] = v3 ? *reinterpret_cast<const uint32_t*>(p3 + kk + 8) : 0u;
    if (amax_out) {
#pragma unroll
      for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const uint32_t ab = a[m][e] & 0x7FFF7FFFu;
          amax2 = max(ab & 0xFFFFu, amax2 & 0xFFFFu) | (max(ab >> 16, amax2 >> 16) << 16);
        }
    }
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      const __nv_bfloat16* bp = om + (n * 8 + g) * SKM_PITCH + kk;
      const uint32_t b0 = *reinterpret_cast<const uint32_t*>(bp), b1 = *reinterpret_cast<const uint32_t*>(bp + 8);
      mma_bf16(acc[0][n], a[0], b0, b1);
      mma_bf16(acc[1][n], a[1], b0, b1);
    }
  }
  float* dst = zp + (int64_t)blockIdx.y * n_s * q;
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      const int r = row0 + m * 16 + g, j = n * 8 + 2 * t;
      if (r < n_s) { if (j < q) dst[(int64_t)r * q + j] = acc[m][n][0]; if (j + 1 < q) dst[(int64_t)r * q + j + 1] = acc[m][n][1]; }
      if (r + 8 < n_s) { if (j < q) dst[(int64_t)(r + 8) * q + j] = acc[m][n][2]; if (j + 1 < q) dst[(int64_t)(r + 8) * q + j + 1] = acc[m][n][3]; }
    }
  if (amax_out) {
    uint32_t am = max((amax2 & 0xFFFFu) << 16, amax2 & 0xFFFF0000u);      // ordered bit patterns: a NaN survives
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) am = max(am, __shfl_xor_sync(0xFFFFFFFFu, am, o));
    if (lane == 0) atomicMax(reinterpret_cast<unsigned int*>(amax_out), am);
  }
}

// Full-mode sketch on the tcgen05 path: Omega is written once, transposed and zero-padded to nb rows
// (omt[j][col], BF16: its values are BF16 by construction), and Z = X Omega runs on the same kernel as the
// coefficient pass.  One thread per Philox block of eight consecutive elements e = col * q + j.
__global__ void __launch_bounds__(256)
omega_rows_kernel(int64_t cols, int q, int nb, uint64_t seed, const __nv_bfloat16* __restrict__ lut, __nv_bfloat16* __restrict__ omt) {
  metis_pdl_wait();
  const uint64_t total = (uint64_t)cols * (uint64_t)q;
  const uint64_t blk = (uint64_t)blockIdx.x * 256 + threadIdx.x;
  if (blk < (total + 7) / 8) {
    const uint4 w = metis_philox_block(blk, seed, METIS_STREAM_OMEGA);
#pragma unroll
    for (uint32_t h = 0; h < 8; ++h) {
      const uint64_t e = (blk << 3) + h;
      if (e < total) omt[(e % q) * cols + e / q] = lut[metis_u16_of(w, h)];
    }
  }
  // rows q .. nb-1 are zero
  const int64_t pad = (int64_t)(nb - q) * cols;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < pad; i += (int64_t)gridDim.x * 256)
    omt[(int64_t)q * cols + i] = __float2bfloat16_rn(0.0f);
}

// m[j][col] = sum over slices s of part[s][col][j], j < q (the tensor-core projection writes M transposed, jp wide)
__global__ void __launch_bounds__(256)
reduce_proj_kernel(const float* __restrict__ part, int slices, int64_t cols, int jp, int q, float* __restrict__ m) {
  metis_pdl_wait();
  __shared__ float t[32][33];
  const int64_t c0 = (int64_t)blockIdx.x * 32;
  const int j0 = blockIdx.y * 32, tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int r = ty; r < 32; r += 8) {                     // r: column of x inside the tile, tx: sketch index
    float acc = 0.0f;
    if (c0 + r < cols && j0 + tx < q) {
      float v[8];                                           // at most eight slices
#pragma unroll
      for (int s = 0; s < 8; ++s) v[s] = s < slices ? part[((int64_t)s * cols + c0 + r) * jp + j0 + tx] : 0.0f;
#pragma unroll
      for (int s = 0; s < 8; ++s) acc += v[s];
    }
    t[r][tx] = acc;
  }
  __syncthreads();
  for (int r = ty; r < 32; r += 8)                        // r: sketch index, tx: column
    if (j0 + r < q && c0 + tx < cols) m[(int64_t)(j0 + r) * cols + c0 + tx] = t[tx][r];
}

// z[r * ldz + j] = sum over slices s of part[s][r][j], j < q (part rows are nb wide); fixed order
__global__ void __launch_bounds__(256)
reduce_sketch_kernel(const float* __restrict__ part, int slices, int64_t rows, int nb, int q, float* __restrict__ z, int ldz) {
  metis_pdl_wait();
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= rows * q) return;
  const int64_t r = i / q;
  const int j = (int)(i % q);
  float t[8], acc = 0.0f;                                 // at most eight slices
#pragma unroll
  for (int s = 0; s < 8; ++s) t[s] = s < slices ? part[((int64_t)s * rows + r) * nb + j] : 0.0f;
#pragma unroll
  for (int s = 0; s < 8; ++s) acc += t[s];
  z[r * ldz + j] = acc;
}

// Tensor-core projection: Mp[part][j][col] = sum over the part's sampled rows r of H[r][j] * x[idx[r], col].
// The contraction runs over rows of the row-major x, so x tiles are staged in shared memory and read back
// transposed with ldmatrix; H (FP32) is fed as three BF16 terms.  CTA = 128 columns x one slab of rows.
// ------------------------------------------------------------------------------------------------
// Projection M = H^T x over many rows (every row in FULL mode), software-pipelined: the CTA owns 128 columns and
// a slab of rows, and walks the slab in chunks of 64 rows through a three-stage cp.async ring (x rows gathered
// by idx, the three BF16 terms of H pre-split and transposed by h_splits_kernel), so the loads of chunk c + 2
// overlap the MMAs of chunk c.  Same partial layout as project_kernel: Mp[part][j][col].
constexpr int PP_COLS = 128, PP_K = 64, PP_STAGES = 3, PP_XP = PP_COLS + 8, PP_HP = PP_K + 8;

// hsp[sp][j][r] (r contiguous, ldh >= rows rounded up to 64, zero padded): three-term BF16 split of H[r][j]
__global__ void __launch_bounds__(256)
h_splits_kernel(const float* __restrict__ h, int n_s, int q, int jp, int ldh, __nv_bfloat16* __restrict__ hsp, int pitch_h) {
  metis_pdl_wait();
  const int r = blockIdx.x * 256 + threadIdx.x, j = blockIdx.y;
  if (r >= ldh) return;
  const float v = (r < n_s && j < q) ? h[(int64_t)r * pitch_h + j] : 0.0f;
  const __nv_bfloat16 hh = __float2bfloat16_rn(v);
  const float r1 = v - __bfloat162float(hh);
  const __nv_bfloat16 hl = __float2bfloat16_rn(r1);
  hsp[((int64_t)0 * jp + j) * ldh + r] = hh;
  hsp[((int64_t)1 * jp + j) * ldh + r] = hl;
  hsp[((int64_t)2 * jp + j) * ldh + r] = __float2bfloat16_rn(r1 - __bfloat162float(hl));
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int bytes = valid ? 16 : 0;                      // 0: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}

template <int MT>                                      // sketch columns / 16, rounded up
__global__ void __launch_bounds__(256)
project_pipe_kernel(const __nv_bfloat16* __restrict__ x, int64_t cols, const int* __restrict__ idx, int n_s, int q,
                    const __nv_bfloat16* __restrict__ hsp, int ldh, int rows_per_part, float* __restrict__ mp) {
  metis_pdl_wait();
  extern __shared__ __align__(16) unsigned char psm[];
  constexpr int XS_BYTES = PP_K * PP_XP * 2, HS_BYTES = 3 * MT * 16 * PP_HP * 2, STAGE = XS_BYTES + HS_BYTES;
  const uint32_t sbase = (uint32_t)__cvta_generic_to_shared(psm);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int64_t col0 = (int64_t)blockIdx.x * PP_COLS;
  const int r_begin = blockIdx.y * rows_per_part, r_end = min(n_s, r_begin + rows_per_part);
  const int n_chunks = (r_end - r_begin + PP_K - 1) / PP_K;
  float acc[MT][2][4];
#pragma unroll
  for (int m = 0; m < MT; ++m)
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[m][n][e] = 0.0f;

  auto load_chunk = [&](int c) {
    const int st = c % PP_STAGES;
    const int r0 = r_begin + c * PP_K;
    const uint32_t xs = sbase + (uint32_t)st * STAGE, hs = xs + XS_BYTES;
    for (int i = tid; i < PP_K * (PP_COLS / 8); i += 256) {
      const int rr = i >> 4, c8 = (i & 15) * 8;
      const bool ok = r0 + rr < r_end && col0 + c8 + 8 <= cols;
      const __nv_bfloat16* src = ok ? x + (int64_t)idx[r0 + rr] * cols + col0 + c8 : x;
      cp_async16(xs + (uint32_t)(rr * PP_XP + c8) * 2u, src, ok);
    }
    for (int i = tid; i < 3 * MT * 16 * (PP_K / 8); i += 256) {
      const int row = i >> 3, k8 = (i & 7) * 8;          // row = sp * MT*16 + j
      cp_async16(hs + (uint32_t)(row * PP_HP + k8) * 2u, hsp + (int64_t)row * ldh + r0 + k8, true);
    }
  };

  for (int c = 0; c < PP_STAGES - 1; ++c) {
    if (c < n_chunks) load_chunk(c);
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  for (int c = 0; c < n_chunks; ++c) {
    asm volatile("cp.async.wait_group %0;" ::"n"(PP_STAGES - 2) : "memory");
    __syncthreads();                                     // chunk c has landed; everyone is done with chunk c - 1
    if (c + PP_STAGES - 1 < n_chunks) load_chunk(c + PP_STAGES - 1);
    asm volatile("cp.async.commit_group;" ::: "memory");
    const int st = c % PP_STAGES;
    const uint32_t xs = sbase + (uint32_t)st * STAGE, hs = xs + XS_BYTES;
#pragma unroll
    for (int ks = 0; ks < PP_K / 16; ++ks) {
      uint32_t b[2][2];
#pragma unroll
      for (int n = 0; n < 2; ++n) {
        const uint32_t addr = xs + (uint32_t)((ks * 16 + (lane & 15)) * PP_XP + (warp * 2 + n) * 8) * 2u;
        asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];" : "=r"(b[n][0]), "=r"(b[n][1]) : "r"(addr));
      }
#pragma unroll
      for (int sp = 0; sp < 3; ++sp)
#pragma unroll
        for (int m = 0; m < MT; ++m) {
          uint32_t a[4];
          const uint32_t addr = hs + (uint32_t)(((sp * MT + m) * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * PP_HP + ks * 16 + (lane >> 4) * 8) * 2u;
          asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                       : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]) : "r"(addr));
          mma_bf16(acc[m][0], a, b[0][0], b[0][1]);
          mma_bf16(acc[m][1], a, b[1][0], b[1][1]);
        }
    }
  }
  float* dst = mp + (int64_t)blockIdx.y * q * cols;
#pragma unroll
  for (int m = 0; m < MT; ++m)
#pragma unroll
    for (int n = 0; n < 2; ++n) {
      const int j = m * 16 + g;
      const int64_t col = col0 + (warp * 2 + n) * 8 + 2 * t;
      if (col + 1 < cols) {
        if (j < q) *reinterpret_cast<float2*>(dst + (int64_t)j * cols + col) = make_float2(acc[m][n][0], acc[m][n][1]);
        if (j + 8 < q) *reinterpret_cast<float2*>(dst + (int64_t)(j + 8) * cols + col) = make_float2(acc[m][n][2], acc[m][n][3]);
      }
    }
}


// right[j][col] = sum_i basis[i][col] * W[i][j] (W == nullptr: identity).  One thread per column; each CTA
// also records, for every j, its entry of largest magnitude (signed value and column, lowest column on ties)
// for the sign convention.
__global__ void __launch_bounds__(256)
right_rotate_kernel(const float* __restrict__ basis, int64_t cols, int k, const double* __restrict__ w,
                    float* __restrict__ right, float* __restrict__ cand_v, int* __restrict__ cand_i) {
  metis_pdl_wait();
  __shared__ float wsm[MAXQ][MAXQ + 1];
  __shared__ float red_v[8][MAXQ];
  __shared__ int red_i[8][MAXQ];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (w) for (int o = tid; o < k * k; o += 256) wsm[o / k][o % k] = (float)w[o];
  __syncthreads();
  const int64_t col = (int64_t)blockIdx.x * 256 + tid;
  // blockIdx.y owns the output vectors j = 8*blockIdx.y .. +7 (a CTA per 256 columns alone leaves most SMs idle)
  const int j_begin = blockIdx.y * 8, j_end = min(k, j_begin + 8);
  float bv[MAXQ];
#pragma unroll
  for (int i = 0; i < MAXQ; ++i) bv[i] = (i < k && col < cols) ? basis[(int64_t)i * cols + col] : 0.0f;
  for (int j = j_begin; j < j_end; ++j) {
    float v;
    if (w) {
      v = 0.0f;
#pragma unroll
      for (int i = 0; i < MAXQ; ++i) if (i < k) v = fmaf(bv[i], wsm[i][j], v);
    } else {
      v = 0.0f;
#pragma unroll
      for (int i = 0; i < MAXQ; ++i) if (i == j) v = bv[i];
    }
    if (col < cols) right[(int64_t)j * cols + col] = v;
    float av = col < cols ? fabsf(v) : -1.0f, sv = v;            // magnitude for the contest, signed value for the decision
    int ai = (int)min(col, (int64_t)0x7FFFFFFF);
#pragma unroll
    for (int sft = 16; sft > 0; sft >>= 1) {
      const float ov = __shfl_xor_sync(0xFFFFFFFFu, av, sft);
      const float os = __shfl_xor_sync(0xFFFFFFFFu, sv, sft);
      const int oi = __shfl_xor_sync(0xFFFFFFFFu, ai, sft);
      if (ov > av || (ov == av && oi < ai)) { av = ov; ai = oi; sv = os; }
    }
    if (lane == 0) { red_v[warp][j] = sv; red_i[warp][j] = ai; }
  }
  __syncthreads();
  if (tid >= j_begin && tid < j_end) {
    float sv = red_v[0][tid]; int ai = red_i[0][tid];
    for (int wv = 1; wv < 8; ++wv) {
      const float ov = red_v[wv][tid];
      if (fabsf(ov) > fabsf(sv) || (fabsf(ov) == fabsf(sv) && red_i[wv][tid] < ai)) { sv = ov; ai = red_i[wv][tid]; }
    }
    cand_v[(int64_t)blockIdx.x * k + tid] = sv;                  // signed winner of this column chunk
    cand_i[(int64_t)blockIdx.x * k + tid] = ai;
  }
}

// Sign convention: the largest-magnitude entry of each right vector (lowest index on ties) is made positive.
// grid (column chunks, k).  Every CTA re-derives the winner of its vector from the per-chunk candidates, whose
// signed values were recorded before any flipping (the flips of other CTAs must not influence the decision).
__global__ void __launch_bounds__(256)
sign_fix_kernel(float* __restrict__ right, int64_t cols, int k, const float* __restrict__ cand_v,
                const int* __restrict__ cand_i, int n_cand, float* __restrict__ sign_out, float* __restrict__ amax_out) {
  metis_pdl_wait();
  const int j = blockIdx.y;
  float sv = 0.0f; int ai = 0x7FFFFFFF;
  for (int c = 0; c < n_cand; ++c) {
    const float v = cand_v[(int64_t)c * k + j]; const int i = cand_i[(int64_t)c * k + j];
    if (fabsf(v) > fabsf(sv) || (fabsf(v) == fabsf(sv) && i < ai)) { sv = v; ai = i; }
  }
  const float sg = sv < 0.0f ? -1.0f : 1.0f;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    sign_out[j] = sg;
    // the winner's magnitude is the vector's amax: the factor's tensor scale needs the max over all vectors
    if (amax_out != nullptr) atomicMax(reinterpret_cast<unsigned int*>(amax_out), __float_as_uint(fabsf(sv)));
  }
  const int64_t col = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (sg < 0.0f && col < cols) right[(int64_t)j * cols + col] = -right[(int64_t)j * cols + col];
}

// left[j][r] = sign_j * scale_j * sum_i coef(i, r) * W[i][j],  coef(i, r) = c[i*stride_i + r*stride_r]
// scale_j = 1/sqrt(eval_j) when inv_sqrt_evals is given (Rayleigh-Ritz normalisation), else 1.
// Also writes sigma_out[j] = sqrt(eval_j) when asked, and coef_rm[r][j] = left[j][r] * sigma_for_coef[j]
// (row-major, kp columns, zero padded) when asked.
__global__ void __launch_bounds__(256)
left_rotate_kernel(const float* __restrict__ c, int64_t rows, int n_in, int k, int64_t stride_i, int64_t stride_r,
                   const double* __restrict__ w, const double* __restrict__ evals_for_scale,
                   const float* __restrict__ sign, float* __restrict__ left, float* __restrict__ sigma_out,
                   float* __restrict__ coef_rm, int kp, const float* __restrict__ sigma_for_coef,
                   float* __restrict__ amax_out) {
  metis_pdl_wait();
  __shared__ double ws[MAXQ][MAXQ + 1];
  __shared__ double scl[MAXQ];
  const int tid = threadIdx.x, rx = tid & 63, jg = tid >> 6;
  for (int o = tid; o < n_in * n_in; o += 256) ws[o / n_in][o % n_in] = w[o];
  if (tid < k) {
    double s = 1.0;
    if (evals_for_scale) {
      const double lam = sqrt(fmax(evals_for_scale[tid], 0.0));
      s = lam > 0.0 ? 1.0 / lam : 0.0;
      if (blockIdx.x == 0 && blockIdx.y == 0 && sigma_out) sigma_out[tid] = (float)lam;
    }
    scl[tid] = s * (double)sign[tid];
  }
  __syncthreads();
  const int64_t r = (int64_t)blockIdx.x * 64 + rx;
  float am = 0.0f;
  if (r < rows) {
    for (int j0 = jg * 4 + 16 * blockIdx.y; j0 < kp; j0 += 16 * gridDim.y) {   // blockIdx.y: every gridDim.y-th group of 16 outputs
      double a[4] = {0.0, 0.0, 0.0, 0.0};
      if (j0 < k) {
#pragma unroll 4
        for (int i = 0; i < n_in; ++i) {
          const double v = (double)c[i * stride_i + r * stride_r];
          a[0] += v * ws[i][j0]; a[1] += v * ws[i][j0 + 1]; a[2] += v * ws[i][j0 + 2]; a[3] += v * ws[i][j0 + 3];
        }
      }
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int j = j0 + t;
        if (j < k) {
          const float v = (float)(a[t] * scl[j]);
          left[(int64_t)j * rows + r] = v;
          am = fmaxf(am, fabsf(v));
          if (coef_rm) coef_rm[r * kp + j] = v * sigma_for_coef[j];
        } else if (coef_rm && j < kp) {
          coef_rm[r * kp + j] = 0.0f;
        }
      }
    }
  }
  // amax|left| for the factor's tensor scale (order-independent atomic max on the float bits)
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) am = fmaxf(am, __shfl_xor_sync(0xFFFFFFFFu, am, o));
  if ((tid & 31) == 0 && amax_out != nullptr) atomicMax(reinterpret_cast<unsigned int*>(amax_out), __float_as_uint(am));
}

// Columns per sketch CTA: a sampled sketch has few rows, so narrow chunks are what gives it enough CTAs; a full
// sketch has one CTA per 256 rows already and wide chunks keep the partial buffer small.
// accumulator columns of the tensor-core sketch: k + p rounded up to what the coefficient kernel is built for
int sketch_tc_cols(int q) { return q <= 48 ? 48 : 96; }

int sketch_chunk_cols(int64_t n_s) { return n_s <= 512 ? 64 : SKM_COLS; }

struct SplitWs {
  size_t amax, idx, zp, omt, z, gram, gram1, linv, evals, evecs, mp, m, basis, coef, sign, cand_v, cand_i, evals2, evecs2, bs, bt,
      gram_c, part, a6, b6, hsp, total;
};

constexpr int PJ_MAX_PARTS = 16;

int project_parts(int64_t n_s, int64_t cols, int* rows_per_part) {
  const int64_t col_chunks = metis_ceil_div(cols, PJ_COLS);
  int64_t parts = metis_ceil_div(2 * 148, col_chunks);          // aim at two CTAs per SM
  if (parts > PJ_MAX_PARTS) parts = PJ_MAX_PARTS;
  if (parts > metis_ceil_div(n_s, 16)) parts = metis_ceil_div(n_s, 16);
  if (parts < 1) parts = 1;
  int64_t rpp = metis_ceil_div(n_s, parts);
  rpp = metis_ceil_div(rpp, 16) * 16;
  *rows_per_part = (int)rpp;
  return (int)metis_ceil_div(n_s, rpp);
}

SplitWs split_ws_layout(int64_t rows, int64_t cols, int k, int p, int64_t n_s) {
  SplitWs w{};
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 255) & ~(size_t)255; return o; };
  const int q = k + p;
  const int64_t chunks = metis_ceil_div(cols, sketch_chunk_cols(n_s));
  w.amax = take(256);
  w.idx = take(sizeof(int) * (size_t)n_s);
  // the full-mode tensor-core sketch writes slices x rows x nb partials into the same buffer
  const int nb_sk = sketch_tc_cols(q);
  const size_t zp_mma = (size_t)chunks * n_s * q, zp_tc = (size_t)metis_coeff_slices(rows, cols, nullptr) * rows * nb_sk;
  w.zp = take(sizeof(float) * (zp_mma > zp_tc ? zp_mma : zp_tc));
  w.omt = take(sizeof(__nv_bfloat16) * (size_t)nb_sk * cols);
  w.z = take(sizeof(float) * (size_t)n_s * q);
  w.gram = take(sizeof(double) * 64 * MAXQ * MAXQ);
  w.linv = take(sizeof(double) * (MAXQ * MAXQ + MAXQ));
  w.gram1 = take(sizeof(double) * MAXQ * MAXQ);
  w.evals = take(sizeof(double) * MAXQ);
  w.evecs = take(sizeof(double) * MAXQ * MAXQ);
  {
    const size_t per_col_mma = (size_t)PJ_MAX_PARTS * q, per_col_tc = (size_t)8 * ((q + 15) / 16 * 16);   // tensor-core projection: <= 8 slices x jp
    w.mp = take(sizeof(float) * (per_col_mma > per_col_tc ? per_col_mma : per_col_tc) * cols);
  }
  w.m = take(sizeof(float) * (size_t)q * cols);
  w.basis = take(sizeof(float) * (size_t)k * cols);
  const int kp = (k + 15) / 16 * 16;
  w.coef = take(sizeof(float) * (size_t)kp * rows);
  w.part = take(sizeof(float) * (size_t)metis_coeff_slices(rows, cols, nullptr) * kp * rows);
  w.a6 = take(sizeof(__nv_bfloat16) * (size_t)metis_residual_kx(kp) * rows);
  w.b6 = take(sizeof(__nv_bfloat16) * (size_t)metis_residual_kx(kp) * cols);
  w.hsp = take(n_s >= 1024 ? sizeof(__nv_bfloat16) * 3 * (size_t)((q + 15) / 16 * 16) * (size_t)((n_s + 63) / 64 * 64) : 0);
  w.bs = take(sizeof(__nv_bfloat16) * 3 * (size_t)kp * cols);
  w.bt = take(sizeof(__nv_bfloat16) * 3 * (size_t)kp * cols);
  w.gram_c = take(sizeof(double) * (size_t)metis_ceil_div(rows, 32) * kp * kp);
  w.sign = take(sizeof(float) * MAXQ);
  w.cand_v = take(sizeof(float) * MAXQ * (size_t)metis_ceil_div(cols, 256));
  w.cand_i = take(sizeof(int) * MAXQ * (size_t)metis_ceil_div(cols, 256));
  w.evals2 = take(sizeof(double) * MAXQ);
  w.evecs2 = take(sizeof(double) * MAXQ * MAXQ);
  w.total = off;
  return w;
}

int gram_parts(int64_t n_rows, int64_t* rows_per_part) {
  int parts = (int)metis_ceil_div(n_rows, 64);
  if (parts > 64) parts = 64;
  if (parts < 1) parts = 1;
  int64_t rpp = metis_ceil_div(n_rows, parts);
  rpp = metis_ceil_div(rpp, GR_TILE) * GR_TILE;
  *rows_per_part = rpp;
  return (int)metis_ceil_div(n_rows, rpp);
}

void launch_jacobi(cudaStream_t s, const double* g, int n, int ld, float exit_cos2, double* evals, double* evecs) {
  // sixteen lanes per couple: 8 lanes (longer per-thread instruction streams) and 32 lanes (five shuffle stages, up
  // to 1024 threads at the barrier) both measured slower
  const int np = n + (n & 1);
  switch ((np + 15) / 16) {
    case 1: (void)(metis_launch_pdl((jacobi_eig_kernel<1, 16>), dim3(1), dim3(256), (size_t)(JACOBI_SMEM), s, g, n, ld, exit_cos2, evals, evecs)); break;
    case 2: (void)(metis_launch_pdl((jacobi_eig_kernel<2, 16>), dim3(1), dim3(256), (size_t)(JACOBI_SMEM), s, g, n, ld, exit_cos2, evals, evecs)); break;
    case 3: (void)(metis_launch_pdl((jacobi_eig_kernel<3, 16>), dim3(1), dim3(384), (size_t)(JACOBI_SMEM), s, g, n, ld, exit_cos2, evals, evecs)); break;
    case 4: (void)(metis_launch_pdl((jacobi_eig_kernel<4, 16>), dim3(1), dim3(512), (size_t)(JACOBI_SMEM), s, g, n, ld, exit_cos2, evals, evecs)); break;
    default: (void)(metis_launch_pdl((jacobi_eig_kernel<5, 16>), dim3(1), dim3(640), (size_t)(JACOBI_SMEM), s, g, n, ld, exit_cos2, evals, evecs)); break;
  }
  METIS_COUNT_LAUNCH();
}

template <int NJ4>
void launch_project(dim3 grid, cudaStream_t s, const __nv_bfloat16* x, int64_t cols, const int* idx, int n_s, int q,
                    const float* h, int rpp, float* mp) {
  (void)(metis_launch_pdl((project_kernel<NJ4>), dim3(grid), dim3(256), (size_t)(0), s, x, cols, idx, n_s, q, h, rpp, mp)); METIS_COUNT_LAUNCH();
}

int jacobi_threads(int n) {
  const int half = (n + 1) / 2;
  int t = (half * half + 31) / 32 * 32;
  return t < 64 ? 64 : t;
}


// ------------------------------------------------------------------------------------------------
// Wide sketches (k + p above MAXQ or k above 64, up to 272 / 256): the same decomposition on kernels that tile over
// the rank (bigrank.cuh).  The range finder works on a contiguous matrix - the operand itself (FULL) or its sampled
// rows gathered once (SAMPLED) - so that sketch and projection both run on the tcgen05 kernel of the broadcast
// pass, in groups of sketch columns.
struct WideWs {
  size_t amax, idx, xs, omt, zp, z, gram, gram1, l, linv, evals, evecs, ycm, scale, hsp, mp, m, basis, bs, coef, part,
      a6, b6, sign, evals2, evecs2, total;
};
constexpr int WIDE_GRAM_PARTS = 32;
constexpr int WIDE_SK = 96;                              // sketch columns per launch of the tensor-core sketch
constexpr int WIDE_PJ = 80;                              // sketch columns per launch of the tensor-core projection
constexpr int WIDE_CG = 64;                              // basis vectors per launch of the broadcast pass

WideWs wide_ws_layout(int64_t rows, int64_t cols, int k, int p, int64_t n_s, bool full) {
  WideWs w{};
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 255) & ~(size_t)255; return o; };
  const int q = k + p, kp = (k + 15) / 16 * 16;
  const int64_t n_r = full ? rows : n_s;
  const int nbq = (q + WIDE_SK - 1) / WIDE_SK * WIDE_SK;
  const int64_t ldh = (n_r + 63) / 64 * 64;
  w.amax = take(256);
  w.idx = take(sizeof(int) * (size_t)n_s);
  w.xs = take(full ? 0 : sizeof(__nv_bfloat16) * (size_t)n_s * cols);
  w.omt = take(sizeof(__nv_bfloat16) * (size_t)nbq * cols);
  w.zp = take(sizeof(float) * (size_t)metis_coeff_slices(n_r, cols, nullptr) * n_r * WIDE_SK);
  w.z = take(sizeof(float) * (size_t)n_r * q);
  w.gram = take(sizeof(double) * (size_t)WIDE_GRAM_PARTS * q * q);
  w.gram1 = take(sizeof(double) * (size_t)q * q);
  w.l = take(sizeof(double) * (size_t)q * q);
  w.linv = take(sizeof(double) * (size_t)q * q);                 // inverses of the factor's diagonal blocks (fewer than q * q entries)
  w.evals = take(sizeof(double) * (size_t)q);
  w.evecs = take(sizeof(double) * (size_t)q * q);
  w.ycm = take(sizeof(double) * (size_t)metis_wide::MAXQ_WIDE * q);
  w.scale = take(sizeof(double) * (size_t)q);
  w.hsp = take(sizeof(__nv_bfloat16) * 3 * (size_t)WIDE_PJ * ldh);
  w.mp = take(sizeof(float) * (size_t)8 * cols * WIDE_PJ);
  w.m = take(sizeof(float) * (size_t)q * cols);
  w.basis = take(sizeof(float) * (size_t)k * cols);
  w.bs = take(sizeof(__nv_bfloat16) * 3 * (size_t)kp * cols);
  w.coef = take(sizeof(float) * (size_t)kp * rows);
  w.part = take(sizeof(float) * (size_t)metis_coeff_slices(rows, cols, nullptr) * rows * WIDE_CG);
  w.a6 = take(sizeof(__nv_bfloat16) * (size_t)metis_residual_kx(kp) * rows);
  w.b6 = take(sizeof(__nv_bfloat16) * (size_t)metis_residual_kx(kp) * cols);
  w.sign = take(sizeof(float) * (size_t)kp);
  w.evals2 = take(sizeof(double) * (size_t)k);
  w.evecs2 = take(sizeof(double) * (size_t)k * k);
  w.total = off;
  return w;
}

bool split_is_wide(int k, int p) { return k > 64 || k + p > MAXQ; }

metis_status_t launch_gemm64(cudaStream_t s, const metis_wide::Gemm64Args& g) {
  dim3 grid((unsigned)metis_ceil_div(g.N, 64), (unsigned)metis_ceil_div(g.M, 64));
  METIS_CUDA_TRY(metis_launch_pdl(metis_wide::gemm64_kernel, grid, dim3(256), (size_t)0, s, g)); METIS_COUNT_LAUNCH();
  return METIS_OK;
}

// FP64 Gram matrix of n vectors (element (r, i) at v[r * sr + i * sv]) into gram1 (n x n), by slabs of rows
metis_status_t launch_gram64(cudaStream_t s, const float* v, int64_t n_rows, int n, int64_t sr, int64_t sv, double* parts, double* gram1,
                             const int* skip = nullptr) {
  int64_t rpp = metis_ceil_div(metis_ceil_div(n_rows, WIDE_GRAM_PARTS), metis_wide::G64_R) * metis_wide::G64_R;
  if (rpp < 64) rpp = 64;
  const int n_parts = (int)metis_ceil_div(n_rows, rpp);
  const unsigned t = (unsigned)metis_ceil_div(n, metis_wide::G64_T);
  METIS_CUDA_TRY(metis_launch_pdl(metis_wide::gram64_kernel, dim3(t, t, (unsigned)n_parts), dim3(256), (size_t)0, s, v, n_rows, n, sr, sv, rpp, parts,
                                  skip)); METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(metis_launch_pdl((reduce_gram_kernel), dim3((unsigned)metis_ceil_div(n * n, 32)), dim3(128), (size_t)(0), s, (const double*)parts, n_parts, n * n, gram1,
                                  skip)); METIS_COUNT_LAUNCH();
  return METIS_OK;
}

// eigen-decomposition of the n x n Gram matrix gram1: Cholesky factor, cluster Jacobi on its columns, collection
metis_status_t launch_eig_wide(cudaStream_t s, const double* gram1, int n, float exit_cos2, double* l, double* ycm, double* evals, double* evecs) {
  METIS_CUDA_TRY(metis_launch_pdl(metis_wide::chol_wide_kernel, dim3(1), dim3(1024), metis_wide::CW_SMEM, s, gram1, n, 1e-14, l, (double*)nullptr, (const int*)nullptr,
                                  (int*)nullptr)); METIS_COUNT_LAUNCH();
  metis_wide::jacobi_cluster_kernel<<<metis_wide::JC_P, metis_wide::JC_THREADS, metis_wide::JC_SMEM, s>>>(l, n, exit_cos2, ycm); METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  metis_wide::jacobi_collect_kernel<<<1, 1024, 0, s>>>(ycm, n, evals, evecs); METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  return METIS_OK;
}

metis_status_t split_wide(metis_context* ctx, const __nv_bfloat16* x, int64_t rows, int64_t cols, int k, int p, bool full, int64_t n_s,
                          uint64_t seed, int rounding, bool want_c, bool want_r, const float* src_amax, metis_operand_t* out, float* residual_dense,
                          unsigned char* wsb, const WideWs& L, cudaStream_t s) {
  using namespace metis_qt;
  using metis_wide::Gemm64Args;
  const int q = k + p, kp = (k + 15) / 16 * 16, kx6 = metis_residual_kx(kp);
  const int64_t n_r = full ? rows : n_s;
  const int64_t ldh = (n_r + 63) / 64 * 64;
  float* amax = reinterpret_cast<float*>(wsb + L.amax);
  int* idx = reinterpret_cast<int*>(wsb + L.idx);
  __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(wsb + L.xs);
  __nv_bfloat16* omt = reinterpret_cast<__nv_bfloat16*>(wsb + L.omt);
  float* zp = reinterpret_cast<float*>(wsb + L.zp);
  float* z = reinterpret_cast<float*>(wsb + L.z);
  double* gram = reinterpret_cast<double*>(wsb + L.gram);
  double* gram1 = reinterpret_cast<double*>(wsb + L.gram1);
  double* lf = reinterpret_cast<double*>(wsb + L.l);
  double* linv = reinterpret_cast<double*>(wsb + L.linv);
  double* evals = reinterpret_cast<double*>(wsb + L.evals);
  double* evecs = reinterpret_cast<double*>(wsb + L.evecs);
  double* ycm = reinterpret_cast<double*>(wsb + L.ycm);
  double* scale = reinterpret_cast<double*>(wsb + L.scale);
  __nv_bfloat16* hsp = reinterpret_cast<__nv_bfloat16*>(wsb + L.hsp);
  float* mp = reinterpret_cast<float*>(wsb + L.mp);
  float* m = reinterpret_cast<float*>(wsb + L.m);
  float* basis = reinterpret_cast<float*>(wsb + L.basis);
  __nv_bfloat16* bs = reinterpret_cast<__nv_bfloat16*>(wsb + L.bs);
  float* coef = reinterpret_cast<float*>(wsb + L.coef);
  float* part = reinterpret_cast<float*>(wsb + L.part);
  __nv_bfloat16* a6 = reinterpret_cast<__nv_bfloat16*>(wsb + L.a6);
  __nv_bfloat16* b6 = reinterpret_cast<__nv_bfloat16*>(wsb + L.b6);
  float* sign = reinterpret_cast<float*>(wsb + L.sign);
  double* evals2 = reinterpret_cast<double*>(wsb + L.evals2);
  double* evecs2 = reinterpret_cast<double*>(wsb + L.evecs2);

  METIS_CUDA_TRY(cudaMemsetAsync(amax, 0, 64, s));
  if (src_amax != nullptr) METIS_CUDA_TRY(cudaMemcpyAsync(amax, src_amax, sizeof(float), cudaMemcpyDeviceToDevice, s));
  const __nv_bfloat16* xr = x;
  if (!full) {
    METIS_CUDA_TRY(metis_launch_pdl((sample_rows_kernel), dim3((unsigned)metis_ceil_div(n_s, 256)), dim3(256), (size_t)(0), s, idx, (int)n_s, rows, seed, 0)); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(metis_launch_pdl(metis_wide::gather_rows_kernel, dim3((unsigned)metis_ceil_div(n_s * (cols / 8), 256)), dim3(256), (size_t)0, s, x, cols,
                                    (const int*)idx, (int)n_s, xs)); METIS_COUNT_LAUNCH();
    xr = xs;
  }
  // (2) sketch Z = xr Omega on the tensor cores, WIDE_SK sketch columns per launch
  const int nbq = (q + WIDE_SK - 1) / WIDE_SK * WIDE_SK;
  {
    const uint64_t blocks = ((uint64_t)cols * q + 7) / 8;
    METIS_CUDA_TRY(metis_launch_pdl((omega_rows_kernel), dim3((unsigned)metis_ceil_div((int64_t)blocks, 256)), dim3(256), (size_t)(0), s, cols, q, nbq, seed, ctx->quantile_lut, omt)); METIS_COUNT_LAUNCH();
    const int slices = metis_coeff_slices(n_r, cols, nullptr);
    for (int j0 = 0; j0 < q; j0 += WIDE_SK) {
      const int qg = q - j0 < WIDE_SK ? q - j0 : WIDE_SK;
      METIS_TRY(metis_launch_coeff_tc(ctx, xr, n_r, cols, omt + (int64_t)j0 * cols, WIDE_SK / 3, zp, (full && j0 == 0) ? amax : nullptr, 1, s));
      METIS_CUDA_TRY(metis_launch_pdl((reduce_sketch_kernel), dim3((unsigned)metis_ceil_div(n_r * qg, 256)), dim3(256), (size_t)(0), s, (const float*)zp, slices, n_r, WIDE_SK, qg,
                                      z + j0, q)); METIS_COUNT_LAUNCH();
    }
  }
  // (3) CholeskyQR (FP64 Gram matrix, blocked factorisation, blocked triangular solve).  The first factorisation
  // reports whether its smallest pivot is above 1e-8 of the largest diagonal entry; if so H is orthonormal to FP32
  // rounding already and the kernels of the second pass return at once.
  {
    float* src = z;
    int* cond_flag = reinterpret_cast<int*>(amax + 8);
    for (int pass = 0; pass < 2; ++pass) {
      const int* skip = pass ? cond_flag : nullptr;
      METIS_TRY(launch_gram64(s, src, n_r, q, q, 1, gram, gram1, skip));
      METIS_CUDA_TRY(metis_launch_pdl(metis_wide::chol_wide_kernel, dim3(1), dim3(1024), metis_wide::CW_SMEM, s, (const double*)gram1, q, 1e-13, lf, linv, skip,
                                      pass ? (int*)nullptr : cond_flag)); METIS_COUNT_LAUNCH();
      METIS_CUDA_TRY(metis_launch_pdl(metis_wide::trsm_wide_kernel, dim3((unsigned)metis_ceil_div(n_r, metis_wide::TW_ROWS)), dim3(256), metis_wide::TW_SMEM, s, src, n_r, q,
                                      (const double*)lf, (const double*)linv, skip)); METIS_COUNT_LAUNCH();
    }
  }                                                      // H = Z L^-T, in place
  // (4) M = H^T xr on the tensor cores, WIDE_PJ sketch columns per launch; eigen-decomposition of M M^T
  {
    const int slices = metis_project_slices(n_r, cols);
    for (int j0 = 0; j0 < q; j0 += WIDE_PJ) {
      const int qg = q - j0 < WIDE_PJ ? q - j0 : WIDE_PJ;
      const int jp = (qg + 15) / 16 * 16;
      METIS_CUDA_TRY(metis_launch_pdl(h_splits_kernel, dim3((unsigned)metis_ceil_div(ldh, 256), (unsigned)jp), dim3(256), (size_t)0, s, (const float*)(z + j0), (int)n_r, qg, jp,
                                      (int)ldh, hsp, q)); METIS_COUNT_LAUNCH();
      METIS_TRY(metis_launch_project_tc(ctx, xr, n_r, cols, hsp, jp, ldh, mp, s));
      dim3 rgrid((unsigned)metis_ceil_div(cols, 32), (unsigned)metis_ceil_div(qg, 32));
      METIS_CUDA_TRY(metis_launch_pdl((reduce_proj_kernel), rgrid, dim3(256), (size_t)(0), s, (const float*)mp, slices, cols, jp, qg, m + (int64_t)j0 * cols)); METIS_COUNT_LAUNCH();
    }
    METIS_TRY(launch_gram64(s, m, cols, q, 1, cols, gram, gram1));
    METIS_TRY(launch_eig_wide(s, gram1, q, 1e-8f, lf, ycm, evals, evecs));
  }
  // right basis: basis[j][col] = sum_i evecs[i][j] M[i][col] / sqrt(eval_j),  j < k
  float* rb = full ? out->right : basis;
  {
    METIS_CUDA_TRY(metis_launch_pdl(metis_wide::rot_scales_kernel, dim3((unsigned)metis_ceil_div(k, 128)), dim3(128), (size_t)0, s, (const double*)evals, (const float*)nullptr, k, 0,
                                    scale, full ? out->sigma : (float*)nullptr)); METIS_COUNT_LAUNCH();
    Gemm64Args g{};
    g.a = m; g.a_m = 1; g.a_k = cols; g.b = evecs; g.b_k = q; g.b_n = 1; g.scale = scale; g.c = rb; g.c_m = 1; g.c_n = cols; g.M = cols; g.N = k; g.K = q;
    METIS_TRY(launch_gemm64(s, g));
  }
  QuantParams qp{};
  metis_nvfp4_t rc = out->res_by_cols, rr = out->res_by_rows;
  rc.rows = rows; rc.k_len = cols; rr.rows = cols; rr.k_len = rows;
  qp.rows = rows; qp.cols = cols; qp.rounding = rounding; qp.seed = seed; qp.stream_id = METIS_STREAM_RESIDUAL;
  qp.e_stride_r = cols; qp.e_stride_c = 1;
  if (want_c) { qp.c_codes = rc.codes; qp.c_scales = rc.scales; qp.c_layout = rc.sf_layout; }
  if (want_r) { qp.r_codes = rr.codes; qp.r_scales = rr.scales; qp.r_layout = rr.sf_layout; }
  float* t0 = want_c ? rc.tensor_scale : nullptr; float* t1 = want_r ? rr.tensor_scale : nullptr;
  const dim3 bs_grid((unsigned)metis_ceil_div(cols, 128), (unsigned)(kp / 8));
  cudaStream_t sf = ctx->side[0];
  if (full) {
    // right = basis with the sign convention, left = H U~_k (same flips), coefficients = left * sigma
    METIS_CUDA_TRY(metis_launch_pdl(metis_wide::sign_rows_kernel, dim3((unsigned)k), dim3(256), (size_t)0, s, out->right, cols, sign, amax + 2)); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(metis_launch_pdl((basis_splits_kernel), bs_grid, dim3(128), (size_t)(0), s, (const float*)out->right, cols, k, kp, bs, (__nv_bfloat16*)nullptr, b6, kx6)); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(metis_launch_pdl(metis_wide::rot_scales_kernel, dim3((unsigned)metis_ceil_div(k, 128)), dim3(128), (size_t)0, s, (const double*)evals, (const float*)sign, k, 2,
                                    scale, (float*)nullptr)); METIS_COUNT_LAUNCH();
    if (kp > k) METIS_CUDA_TRY(cudaMemsetAsync(coef, 0, sizeof(float) * (size_t)kp * rows, s));
    Gemm64Args g{};
    g.a = z; g.a_m = q; g.a_k = 1; g.b = evecs; g.b_k = q; g.b_n = 1; g.scale = scale; g.c = out->left; g.c_m = 1; g.c_n = rows;
    g.c2 = coef; g.c2_m = kp; g.c2_n = 1; g.scale2 = out->sigma; g.amax = amax + 1; g.M = rows; g.N = k; g.K = q;
    METIS_TRY(launch_gemm64(s, g));
    METIS_TRY(metis_fork(ctx, s, 1));
    METIS_TRY(metis_launch_residual_tc(ctx, x, coef, k, kp, qp, amax, t0, t1, residual_dense, a6, b6, s));
  } else {
    METIS_CUDA_TRY(metis_launch_pdl((basis_splits_kernel), bs_grid, dim3(128), (size_t)(0), s, (const float*)basis, cols, k, kp, bs, (__nv_bfloat16*)nullptr, b6, kx6)); METIS_COUNT_LAUNCH();
    // (5) broadcast C = x B, WIDE_CG basis vectors per pass over x
    const int slices = metis_coeff_slices(rows, cols, nullptr);
    for (int j0 = 0; j0 < kp; j0 += WIDE_CG) {
      const int gw = kp - j0 < WIDE_CG ? kp - j0 : WIDE_CG;
      METIS_TRY(metis_launch_coeff_tc(ctx, x, rows, cols, bs + (int64_t)3 * j0 * cols, gw, part, j0 == 0 ? amax : nullptr, 0, s));
      METIS_CUDA_TRY(metis_launch_pdl(metis_wide::coef_sum_kernel, dim3((unsigned)metis_ceil_div(rows * (gw / 8), 256)), dim3(256), (size_t)0, s, (const float*)part, slices, rows, gw, j0,
                                      kp, coef, a6, kx6)); METIS_COUNT_LAUNCH();
    }
    METIS_TRY(metis_fork(ctx, s, 1));
    METIS_TRY(metis_launch_residual_tc(ctx, x, nullptr, k, kp, qp, amax, t0, t1, residual_dense, a6, b6, s));
    // (7) Rayleigh-Ritz on C^T C, rotate both factors (side stream, beside the residual pass)
    METIS_TRY(launch_gram64(sf, coef, rows, k, kp, 1, gram, gram1));
    METIS_TRY(launch_eig_wide(sf, gram1, k, 1e-6f, lf, ycm, evals2, evecs2));
    {
      Gemm64Args g{};
      g.a = basis; g.a_m = 1; g.a_k = cols; g.b = evecs2; g.b_k = k; g.b_n = 1; g.c = out->right; g.c_m = 1; g.c_n = cols; g.M = cols; g.N = k; g.K = k;
      METIS_TRY(launch_gemm64(sf, g));
    }
    METIS_CUDA_TRY(metis_launch_pdl(metis_wide::sign_rows_kernel, dim3((unsigned)k), dim3(256), (size_t)0, sf, out->right, cols, sign, amax + 2)); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(metis_launch_pdl(metis_wide::rot_scales_kernel, dim3((unsigned)metis_ceil_div(k, 128)), dim3(128), (size_t)0, sf, (const double*)evals2, (const float*)sign, k, 1,
                                    scale, out->sigma)); METIS_COUNT_LAUNCH();
    {
      Gemm64Args g{};
      g.a = coef; g.a_m = kp; g.a_k = 1; g.b = evecs2; g.b_k = k; g.b_n = 1; g.scale = scale; g.c = out->left; g.c_m = 1; g.c_n = rows; g.amax = amax + 1;
      g.M = rows; g.N = k; g.K = k;
      METIS_TRY(launch_gemm64(sf, g));
    }
  }
  METIS_CUDA_TRY(metis_launch_pdl((split_status_kernel), dim3(1), dim3(32), (size_t)(0), s, (const float*)amax, (const double*)evals, k, ctx->dev_status)); METIS_COUNT_LAUNCH();
  METIS_CUDA_TRY(cudaGetLastError());
  metis_nvfp4_t lq = out->left_q, rq = out->right_q;
  lq.rows = k; lq.k_len = rows; rq.rows = k; rq.k_len = cols;
  METIS_TRY(metis_launch_quantize_factors(out->left, rows, out->right, cols, k, rounding, seed, amax + 1, amax + 2, &lq, &rq, sf));
  return metis_join(ctx, s, 0);
}

}  // namespace

int64_t metis_default_sample_count(int64_t rows, int32_t q) {
  int64_t want = 4 * (int64_t)q;
  const int64_t pct = (rows + 99) / 100;
  if (pct > want) want = pct;
  want = (want + 15) / 16 * 16;
  return want < rows ? want : rows;
}

metis_status_t metis_split_set_attrs() {
  using namespace metis_qt;
  METIS_CUDA_TRY(cudaFuncSetAttribute(jacobi_eig_kernel<1, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)JACOBI_SMEM));
  METIS_CUDA_TRY(cudaFuncSetAttribute(jacobi_eig_kernel<2, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)JACOBI_SMEM));
  METIS_CUDA_TRY(cudaFuncSetAttribute(jacobi_eig_kernel<3, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)JACOBI_SMEM));
  METIS_CUDA_TRY(cudaFuncSetAttribute(jacobi_eig_kernel<4, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)JACOBI_SMEM));
  METIS_CUDA_TRY(cudaFuncSetAttribute(jacobi_eig_kernel<5, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)JACOBI_SMEM));
  METIS_CUDA_TRY(cudaFuncSetAttribute(coeff_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(sizeof(float) * 9 * 32 * 64)));
  METIS_CUDA_TRY(cudaFuncSetAttribute(coeff_mma_kernel<48>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(sizeof(float) * 9 * 32 * 48)));
  METIS_CUDA_TRY(cudaFuncSetAttribute(residual_quant_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes(true)));
  METIS_CUDA_TRY(cudaFuncSetAttribute(residual_quant_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes(true)));
  METIS_CUDA_TRY(cudaFuncSetAttribute(residual_quant_kernel<48>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes(true)));
  METIS_CUDA_TRY(cudaFuncSetAttribute(residual_quant_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes(true)));
  METIS_CUDA_TRY(cudaFuncSetAttribute(gram_chol_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GC_MAX_SMEM));
  METIS_CUDA_TRY(cudaFuncSetAttribute(metis_wide::jacobi_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)metis_wide::JC_SMEM));
  METIS_CUDA_TRY(cudaFuncSetAttribute(metis_wide::chol_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)metis_wide::CW_SMEM));
  METIS_CUDA_TRY(cudaFuncSetAttribute(metis_wide::trsm_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)metis_wide::TW_SMEM));
#define METIS_PP_ATTR(MTV) METIS_CUDA_TRY(cudaFuncSetAttribute(project_pipe_kernel<MTV>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
      (int)((size_t)PP_STAGES * (PP_K * PP_XP * 2 + 3 * (MTV) * 16 * PP_HP * 2))))
  METIS_PP_ATTR(1); METIS_PP_ATTR(2); METIS_PP_ATTR(3); METIS_PP_ATTR(4); METIS_PP_ATTR(5);
#undef METIS_PP_ATTR
  return METIS_OK;
}

// flags METIS_DEV_NONFINITE when *amax (the amax of a tensor about to be quantized) is not a finite number
metis_status_t metis_launch_amax_check(metis_context* ctx, const float* amax, cudaStream_t s) {
  METIS_CUDA_TRY(metis_launch_pdl((split_status_kernel), dim3(1), dim3(32), (size_t)(0), s, amax, (const double*)nullptr, 0, ctx->dev_status));
  METIS_COUNT_LAUNCH();
  return METIS_OK;
}

namespace {
// contiguous BF16 copy of a strided BF16 or FP32 operand (FP32 rounded to nearest even), eight elements per thread
__global__ void __launch_bounds__(256)
pack_bf16_kernel(const void* __restrict__ x, int dtype, int64_t rows, int64_t cols, int64_t ld, __nv_bfloat16* __restrict__ out) {
  metis_pdl_wait();
  const int64_t g = (int64_t)blockIdx.x * 256 + threadIdx.x, per_row = cols / 8;
  if (g >= rows * per_row) return;
  const int64_t r = g / per_row, c = (g - r * per_row) * 8;
  uint4 o;
  if (dtype == METIS_BF16) {
    o = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(x) + r * ld + c);
  } else {
    const float4* src = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(x) + r * ld + c);
    const float4 a = src[0], b = src[1];
    __nv_bfloat162 h0 = __floats2bfloat162_rn(a.x, a.y), h1 = __floats2bfloat162_rn(a.z, a.w);
    __nv_bfloat162 h2 = __floats2bfloat162_rn(b.x, b.y), h3 = __floats2bfloat162_rn(b.z, b.w);
    o.x = *reinterpret_cast<uint32_t*>(&h0); o.y = *reinterpret_cast<uint32_t*>(&h1);
    o.z = *reinterpret_cast<uint32_t*>(&h2); o.w = *reinterpret_cast<uint32_t*>(&h3);
  }
  *reinterpret_cast<uint4*>(out + r * cols + c) = o;
}
metis_status_t launch_pack_bf16(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, __nv_bfloat16* out, cudaStream_t s) {
  METIS_CUDA_TRY(metis_launch_pdl(pack_bf16_kernel, dim3((unsigned)metis_ceil_div(rows * (cols / 8), 256)), dim3(256), (size_t)0, s, x, dtype, rows, cols, ld, out));
  METIS_COUNT_LAUNCH();
  return METIS_OK;
}
}  // namespace

size_t metis_split_ws_bytes(int64_t rows, int64_t cols, int k, int p) {
  if (k > 0 && split_is_wide(k, p)) {
    // the larger of the FULL layout and the SAMPLED layout with the default sample count
    const size_t a = wide_ws_layout(rows, cols, k, p, rows, true).total;
    const size_t b = wide_ws_layout(rows, cols, k, p, metis_default_sample_count(rows, k + p), false).total;
    return a > b ? a : b;
  }
  // Every buffer grows with the sample count except the sketch partials, whose chunk width steps from 64 to 256
  // columns above 512 sampled rows: the FULL sketch (n_s = rows) and a 512-row sample bound every other case.
  const size_t full = split_ws_layout(rows, cols, k, p, rows).total;
  const size_t narrow = split_ws_layout(rows, cols, k, p, rows < 512 ? rows : 512).total;
  return full > narrow ? full : narrow;
}

metis_status_t metis_split(metis_handle_t h, const void* xv, int32_t dtype, int64_t rows, int64_t cols, int64_t ld, int32_t k, int32_t p,
                           int32_t sketch, int64_t n_sample, uint64_t seed, int32_t rounding, int32_t residual_axes,
                           const float* src_amax, metis_operand_t* out, float* residual_dense, void* ws, size_t ws_bytes,
                           metis_stream_t stream) {
  METIS_NVTX("metis_split");
  using namespace metis_qt;
  if (!h || !xv || !out || !ws) return METIS_ERR_INVALID_ARG;
  if (dtype != METIS_BF16 && dtype != METIS_FP32) return METIS_ERR_INVALID_ARG;
  if (rows <= 0 || cols <= 0 || rows % 16 || cols % 16 || k < 0 || p < 0 || ld < cols) return METIS_ERR_SHAPE;
  if (ld % (dtype == METIS_BF16 ? 8 : 4)) return METIS_ERR_ALIGNMENT;          // every row starts on a 16-byte boundary
  // anything but a contiguous BF16 operand is packed (and rounded) into the tail of the workspace first
  const bool packed = k > 0 && (dtype != METIS_BF16 || ld != cols);
  const size_t pack_bytes = packed ? (((size_t)rows * (size_t)cols * sizeof(__nv_bfloat16) + 255) & ~(size_t)255) : 0;
  if (k > 0 && (k > metis_wide::MAXK_WIDE || k + p > metis_wide::MAXQ_WIDE || k % 4)) return METIS_ERR_SHAPE;
  const bool wide = k > 0 && split_is_wide(k, p);
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
  if (wide) {
    // the tensor-core passes carry the wide path: 16-byte aligned rows of x, whole 64-column chunks
    if (cols % 64 || rows % 64 || (!packed && !metis_residual_tc_usable(xv, cols))) return METIS_ERR_SHAPE;
    const WideWs W = wide_ws_layout(rows, cols, k, p, n_s, full);
    if (ws_bytes < W.total + pack_bytes) return METIS_ERR_WORKSPACE;
    if (!out->left || !out->sigma || !out->right || !out->left_q.codes || !out->right_q.codes || !out->left_q.scales ||
        !out->right_q.scales || !out->left_q.tensor_scale || !out->right_q.tensor_scale)
      return METIS_ERR_INVALID_ARG;
    const __nv_bfloat16* xw = reinterpret_cast<const __nv_bfloat16*>(xv);
    if (packed) {
      __nv_bfloat16* xp = reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<unsigned char*>(ws) + ((W.total + 255) & ~(size_t)255));
      METIS_TRY(launch_pack_bf16(xv, dtype, rows, cols, ld, xp, reinterpret_cast<cudaStream_t>(stream)));
      xw = xp;
    }
    return split_wide(h, xw, rows, cols, k, p, full, n_s, seed, rounding, want_c, want_r, src_amax, out,
                      residual_dense, reinterpret_cast<unsigned char*>(ws), W, reinterpret_cast<cudaStream_t>(stream));
  }
  const SplitWs L = split_ws_layout(rows, cols, k, p, n_s);
  if (ws_bytes < L.total + pack_bytes) return METIS_ERR_WORKSPACE;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  unsigned char* wsb = reinterpret_cast<unsigned char*>(ws);
  const __nv_bfloat16* x = reinterpret_cast<const __nv_bfloat16*>(xv);
  if (packed) {
    __nv_bfloat16* xp = reinterpret_cast<__nv_bfloat16*>(wsb + ((L.total + 255) & ~(size_t)255));
    METIS_TRY(launch_pack_bf16(xv, dtype, rows, cols, ld, xp, s));
    x = xp;
  }
  float* amax = reinterpret_cast<float*>(wsb + L.amax);

  metis_nvfp4_t rc = out->res_by_cols, rr = out->res_by_rows;
  rc.rows = rows; rc.k_len = cols; rr.rows = cols; rr.k_len = rows;
  if (k == 0) {
    if (src_amax != nullptr) METIS_CUDA_TRY(cudaMemcpyAsync(amax, src_amax, sizeof(float), cudaMemcpyDeviceToDevice, s));
    else METIS_TRY(metis_launch_amax(xv, dtype, rows, cols, ld, amax, s));
    METIS_TRY(metis_launch_quantize(xv, dtype, rows, cols, ld, rounding, seed, METIS_STREAM_RESIDUAL, cols, 1, amax,
                                    1, want_c ? &rc : nullptr, want_r ? &rr : nullptr, s, h->dev_status));
    METIS_CUDA_TRY(metis_launch_pdl((split_status_kernel), dim3(1), dim3(32), (size_t)(0), s, amax, (const double*)nullptr, 0, h->dev_status)); METIS_COUNT_LAUNCH();
    return METIS_OK;
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
  double* linv = reinterpret_cast<double*>(wsb + L.linv);
  double* invd = linv + MAXQ * MAXQ;
  int* cond_flag = reinterpret_cast<int*>(amax + 8);
  double* gram1 = reinterpret_cast<double*>(wsb + L.gram1);
  double* evals = reinterpret_cast<double*>(wsb + L.evals);
  double* evecs = reinterpret_cast<double*>(wsb + L.evecs);
  float* mp = reinterpret_cast<float*>(wsb + L.mp);
  float* m = reinterpret_cast<float*>(wsb + L.m);
  float* basis = reinterpret_cast<float*>(wsb + L.basis);
  float* coef = reinterpret_cast<float*>(wsb + L.coef);
  float* sign = reinterpret_cast<float*>(wsb + L.sign);
  float* cand_v = reinterpret_cast<float*>(wsb + L.cand_v);
  int* cand_i = reinterpret_cast<int*>(wsb + L.cand_i);
  double* evals2 = reinterpret_cast<double*>(wsb + L.evals2);
  double* evecs2 = reinterpret_cast<double*>(wsb + L.evecs2);
  __nv_bfloat16* bs = reinterpret_cast<__nv_bfloat16*>(wsb + L.bs);
  __nv_bfloat16* bt = reinterpret_cast<__nv_bfloat16*>(wsb + L.bt);
  double* gram_c = reinterpret_cast<double*>(wsb + L.gram_c);
  float* part = reinterpret_cast<float*>(wsb + L.part);
  __nv_bfloat16* hsp = reinterpret_cast<__nv_bfloat16*>(wsb + L.hsp);
  void* a6 = wsb + L.a6;
  void* b6 = wsb + L.b6;
  // the residual kernel's K-concatenated BF16 operands are written by the kernels that produce coefficients and basis
  const bool resid_tc = metis_residual_tc_usable(x, cols);
  const int kx6 = metis_residual_kx((k + 15) / 16 * 16);
  __nv_bfloat16* a6p = resid_tc ? reinterpret_cast<__nv_bfloat16*>(a6) : nullptr;
  __nv_bfloat16* b6p = resid_tc ? reinterpret_cast<__nv_bfloat16*>(b6) : nullptr;
  bool a6_ready = false;
  metis_context* ctx = h;
  const int kp = (k + 15) / 16 * 16;
  // amax|x| for the residual's tensor scale: fused into the sketch pass (FULL) or the broadcast pass (SAMPLED)
  METIS_CUDA_TRY(cudaMemsetAsync(amax, 0, 64, s));       // amax slots of x, left, right and the condition flag
  if (src_amax != nullptr) METIS_CUDA_TRY(cudaMemcpyAsync(amax, src_amax, sizeof(float), cudaMemcpyDeviceToDevice, s));

  // (1) row sample, (2) sketch (tensor cores; Omega generated per CTA into shared memory)
  METIS_CUDA_TRY(metis_launch_pdl((sample_rows_kernel), dim3((unsigned)metis_ceil_div(n_s, 256)), dim3(256), (size_t)(0), s, idx, (int)n_s, rows, seed, full ? 1 : 0)); METIS_COUNT_LAUNCH();
  const int ccols = sketch_chunk_cols(n_s);
  const int chunks = (int)metis_ceil_div(cols, ccols);
  __nv_bfloat16* omt = reinterpret_cast<__nv_bfloat16*>(wsb + L.omt);
  const int nb_sk = sketch_tc_cols(q);
  const bool sketch_tc = full && q <= 96 && metis_coeff_tc_usable(x, omt, cols, nb_sk / 3);
  if (sketch_tc) {
    const uint64_t blocks = ((uint64_t)cols * q + 7) / 8;
    METIS_CUDA_TRY(metis_launch_pdl((omega_rows_kernel), dim3((unsigned)metis_ceil_div((int64_t)blocks, 256)), dim3(256), (size_t)(0), s, cols, q, nb_sk, seed, ctx->quantile_lut, omt)); METIS_COUNT_LAUNCH();
    METIS_TRY(metis_launch_coeff_tc(ctx, x, rows, cols, omt, nb_sk / 3, zp, amax, 1, s));
    const int slices = metis_coeff_slices(rows, cols, nullptr);
    METIS_CUDA_TRY(metis_launch_pdl((reduce_sketch_kernel), dim3((unsigned)metis_ceil_div(rows * q, 256)), dim3(256), (size_t)(0), s, zp, slices, rows, nb_sk, q, z, q)); METIS_COUNT_LAUNCH();
  } else {
    const int nt = (q + 7) / 8;
    const size_t smem = sizeof(__nv_bfloat16) * nt * 8 * SKM_PITCH;
    dim3 grid((unsigned)metis_ceil_div(n_s, SKM_ROWS), (unsigned)chunks);
    float* am = full ? amax : nullptr;                  // FULL mode: amax|x| comes out of this pass
    switch (nt) {
      case 1: METIS_CUDA_TRY(metis_launch_pdl((sketch_mma_kernel<1>), dim3(grid), dim3(256), (size_t)(smem), s, x, cols, idx, (int)n_s, q, seed, ctx->quantile_lut, zp, am, ccols)); break;
      case 2: METIS_CUDA_TRY(metis_launch_pdl((sketch_mma_kernel<2>), dim3(grid), dim3(256), (size_t)(smem), s, x, cols, idx, (int)n_s, q, seed, ctx->quantile_lut, zp, am, ccols)); break;
      case 3: METIS_CUDA_TRY(metis_launch_pdl((sketch_mma_kernel<3>), dim3(grid), dim3(256), (size_t)(smem), s, x, cols, idx, (int)n_s, q, seed, ctx->quantile_lut, zp, am, ccols)); break;
      case 4: METIS_CUDA_TRY(metis_launch_pdl((sketch_mma_kernel<4>), dim3(grid), dim3(256), (size_t)(smem), s, x, cols, idx, (int)n_s, q, seed, ctx->quantile_lut, zp, am, ccols)); break;
      case 5: METIS_CUDA_TRY(metis_launch_pdl((sketch_mma_kernel<5>), dim3(grid), dim3(256), (size_t)(smem), s, x, cols, idx, (int)n_s, q, seed, ctx->quantile_lut, zp, am, ccols)); break;
      case 6: METIS_CUDA_TRY(metis_launch_pdl((sketch_mma_kernel<6>), dim3(grid), dim3(256), (size_t)(smem), s, x, cols, idx, (int)n_s, q, seed, ctx->quantile_lut, zp, am, ccols)); break;
      case 7: METIS_CUDA_TRY(metis_launch_pdl((sketch_mma_kernel<7>), dim3(grid), dim3(256), (size_t)(smem), s, x, cols, idx, (int)n_s, q, seed, ctx->quantile_lut, zp, am, ccols)); break;
      case 8: METIS_CUDA_TRY(metis_launch_pdl((sketch_mma_kernel<8>), dim3(grid), dim3(256), (size_t)(smem), s, x, cols, idx, (int)n_s, q, seed, ctx->quantile_lut, zp, am, ccols)); break;
      default: METIS_CUDA_TRY(metis_launch_pdl((sketch_mma_kernel<9>), dim3(grid), dim3(256), (size_t)(smem), s, x, cols, idx, (int)n_s, q, seed, ctx->quantile_lut, zp, am, ccols)); break;
    }
    METIS_COUNT_LAUNCH();
  }
  if (!sketch_tc) {
    METIS_CUDA_TRY(metis_launch_pdl((reduce_partials_kernel), dim3((unsigned)metis_ceil_div(n_s * q, 256)), dim3(256), (size_t)(0), s, zp, chunks, n_s * q, z)); METIS_COUNT_LAUNCH();
  }
  // (3) CholeskyQR2: orthonormal basis H of range(Z), in place
  if (gram_chol_smem(n_s, q) <= GC_MAX_SMEM) {
    // a short sketch: Gram matrix and factorisation in one CTA; the triangular solves on many CTAs unless the sketch
    // was ill-conditioned, in which case the first kernel has done both passes itself and the second returns at once
    METIS_CUDA_TRY(metis_launch_pdl((gram_chol_kernel), dim3(1), dim3(GC_THREADS), gram_chol_smem(n_s, q), s, z, (int)n_s, q, linv, invd, cond_flag)); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(metis_launch_pdl((apply_chol_kernel), dim3((unsigned)metis_ceil_div(n_s, 8)), dim3(256), (size_t)(0), s, z, n_s, q, linv, invd, (const int*)cond_flag)); METIS_COUNT_LAUNCH();
  } else {
  for (int pass = 0; pass < 2; ++pass) {
    int64_t rpp; const int parts = gram_parts(n_s, &rpp);
    const int* skip = pass == 0 ? nullptr : cond_flag;
    METIS_CUDA_TRY(metis_launch_pdl((gram_kernel), dim3(parts), dim3(256), (size_t)(0), s, z, n_s, q, q, 1, rpp, gram, skip)); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(metis_launch_pdl((reduce_gram_kernel), dim3((unsigned)metis_ceil_div(q * q, 32)), dim3(128), (size_t)(0), s, gram, parts, q * q, gram1, skip)); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(metis_launch_pdl((chol_kernel), dim3(1), dim3(256), (size_t)(0), s, gram1, q, linv, invd, skip, pass == 0 ? cond_flag : nullptr)); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(metis_launch_pdl((apply_chol_kernel), dim3((unsigned)metis_ceil_div(n_s, 8)), dim3(256), (size_t)(0), s, z, n_s, q, linv, invd, skip)); METIS_COUNT_LAUNCH();
  }
  }
  // (4) M = H^T x[S,:], eigen-decomposition of M M^T, right basis
  {
    int rpp; int parts;
    bool project_tc = false;
    if (n_s >= 1024 && cols % 8 == 0) {
      parts = (int)metis_ceil_div(n_s, 512);
      if (parts > PJ_MAX_PARTS) parts = PJ_MAX_PARTS;
      rpp = (int)(metis_ceil_div(metis_ceil_div(n_s, parts), PP_K) * PP_K);
      parts = (int)metis_ceil_div(n_s, rpp);
      const int mt = (q + 15) / 16, jp = mt * 16, ldh = (int)((n_s + 63) / 64 * 64);
      METIS_CUDA_TRY(metis_launch_pdl(h_splits_kernel, dim3((unsigned)metis_ceil_div(ldh, 256), (unsigned)jp), dim3(256), (size_t)0, s, z, (int)n_s, q, jp, ldh, hsp, q)); METIS_COUNT_LAUNCH();
      project_tc = full && metis_project_tc_usable(x, hsp, cols, jp);
      if (project_tc) {
        // every row, in order: M^T = x^T H on the tcgen05 kernel of the broadcast pass (x as an MN-major operand)
        METIS_TRY(metis_launch_project_tc(ctx, x, rows, cols, hsp, jp, ldh, mp, s));
        dim3 rgrid((unsigned)metis_ceil_div(cols, 32), (unsigned)metis_ceil_div(q, 32));
        METIS_CUDA_TRY(metis_launch_pdl((reduce_proj_kernel), rgrid, dim3(256), (size_t)(0), s, mp, metis_project_slices(rows, cols), cols, jp, q, m)); METIS_COUNT_LAUNCH();
      } else {
      dim3 grid((unsigned)metis_ceil_div(cols, PP_COLS), (unsigned)parts);
      const size_t psmem = (size_t)PP_STAGES * (PP_K * PP_XP * 2 + 3 * jp * PP_HP * 2);
#define METIS_PP(MTV) { \
        METIS_CUDA_TRY(metis_launch_pdl((project_pipe_kernel<MTV>), grid, dim3(256), psmem, s, x, cols, idx, (int)n_s, q, hsp, ldh, rpp, mp)); }
      switch (mt) {
        case 1: METIS_PP(1); break;
        case 2: METIS_PP(2); break;
        case 3: METIS_PP(3); break;
        case 4: METIS_PP(4); break;
        default: METIS_PP(5); break;
      }
#undef METIS_PP
      METIS_COUNT_LAUNCH();
      }
    } else {
    parts = project_parts(n_s, cols, &rpp);
    dim3 grid((unsigned)metis_ceil_div(cols, PJ_COLS), (unsigned)parts);
    const int nj4 = (q + 7) / 8;
    switch (nj4) {
      case 1: launch_project<1>(grid, s, x, cols, idx, (int)n_s, q, z, rpp, mp); break;
      case 2: launch_project<2>(grid, s, x, cols, idx, (int)n_s, q, z, rpp, mp); break;
      case 3: launch_project<3>(grid, s, x, cols, idx, (int)n_s, q, z, rpp, mp); break;
      case 4: launch_project<4>(grid, s, x, cols, idx, (int)n_s, q, z, rpp, mp); break;
      case 5: launch_project<5>(grid, s, x, cols, idx, (int)n_s, q, z, rpp, mp); break;
      case 6: launch_project<6>(grid, s, x, cols, idx, (int)n_s, q, z, rpp, mp); break;
      case 7: launch_project<7>(grid, s, x, cols, idx, (int)n_s, q, z, rpp, mp); break;
      case 8: launch_project<8>(grid, s, x, cols, idx, (int)n_s, q, z, rpp, mp); break;
      default: launch_project<9>(grid, s, x, cols, idx, (int)n_s, q, z, rpp, mp); break;
    }
    }
    if (!project_tc) {
      METIS_CUDA_TRY(metis_launch_pdl((reduce_partials_kernel), dim3((unsigned)metis_ceil_div((int64_t)q * cols, 256)), dim3(256), (size_t)(0), s, mp, parts, (int64_t)q * cols, m)); METIS_COUNT_LAUNCH();
    }
  }
  {
    int64_t rpp; const int parts = gram_parts(cols, &rpp);
    METIS_CUDA_TRY(metis_launch_pdl((gram_kernel), dim3(parts), dim3(256), (size_t)(0), s, m, cols, q, 1, cols, rpp, gram, nullptr)); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(metis_launch_pdl((reduce_gram_kernel), dim3((unsigned)metis_ceil_div(q * q, 32)), dim3(128), (size_t)(0), s, gram, parts, q * q, gram1, nullptr)); METIS_COUNT_LAUNCH();
    launch_jacobi(s, gram1, q, q, 1e-8f, evals, evecs);
  }
  METIS_CUDA_TRY(metis_launch_pdl((right_basis_kernel), dim3((unsigned)metis_ceil_div(cols, RB_COLS)), dim3(256), (size_t)(0), s, m, cols, q, k, evals, evecs, basis,
                                                                          full ? out->sigma : nullptr)); METIS_COUNT_LAUNCH();
  // (5) coefficients of every row in the basis, (6) fused residual + quantizer
  const int n_cand = (int)metis_ceil_div(cols, 256);
  const int n_cta_c = (int)metis_ceil_div(rows, 32);
  if (full) {
    // left = H U~_k, right = basis (sign fixed); coefficients = left * sigma
    METIS_CUDA_TRY(metis_launch_pdl((right_rotate_kernel), dim3(dim3(n_cand, (k + 7) / 8)), dim3(256), (size_t)(0), s, basis, cols, k, nullptr, out->right, cand_v, cand_i)); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(metis_launch_pdl((sign_fix_kernel), dim3(dim3(n_cand, k)), dim3(256), (size_t)(0), s, out->right, cols, k, cand_v, cand_i, n_cand, sign, amax + 2)); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(metis_launch_pdl((basis_splits_kernel), dim3((unsigned)metis_ceil_div(cols, 128), (unsigned)(kp / 8)), dim3(128), (size_t)(0), s, out->right, cols, k, kp, bs, bt, b6p, kx6)); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(metis_launch_pdl((left_rotate_kernel), dim3(dim3((unsigned)metis_ceil_div(rows, 64), (unsigned)((kp + 15) / 16))), dim3(256), (size_t)(0), s, z, rows, q, k, 1, q, evecs, nullptr, sign,
                                                                            out->left, nullptr, coef, kp, out->sigma, amax + 1)); METIS_COUNT_LAUNCH();
  } else {
    METIS_CUDA_TRY(metis_launch_pdl((basis_splits_kernel), dim3((unsigned)metis_ceil_div(cols, 128), (unsigned)(kp / 8)), dim3(128), (size_t)(0), s, basis, cols, k, kp, bs, bt, b6p, kx6)); METIS_COUNT_LAUNCH();
    if (metis_coeff_tc_usable(x, bs, cols, kp)) {
      // tensor-core pass over x (column slices), then the slices are summed and the Gram partials formed
      METIS_TRY(metis_launch_coeff_tc(ctx, x, rows, cols, bs, kp, part, amax, 0, s));
      a6_ready = resid_tc;
      const int slices = metis_coeff_slices(rows, cols, nullptr);
      switch (kp) {
        case 16: METIS_CUDA_TRY(metis_launch_pdl((coef_finish_kernel<16>), dim3(n_cta_c), dim3(256), (size_t)(0), s, part, slices, rows, coef, gram_c, a6p, kx6)); break;
        case 32: METIS_CUDA_TRY(metis_launch_pdl((coef_finish_kernel<32>), dim3(n_cta_c), dim3(256), (size_t)(0), s, part, slices, rows, coef, gram_c, a6p, kx6)); break;
        case 48: METIS_CUDA_TRY(metis_launch_pdl((coef_finish_kernel<48>), dim3(n_cta_c), dim3(256), (size_t)(0), s, part, slices, rows, coef, gram_c, a6p, kx6)); break;
        default: METIS_CUDA_TRY(metis_launch_pdl((coef_finish_kernel<64>), dim3(n_cta_c), dim3(256), (size_t)(0), s, part, slices, rows, coef, gram_c, a6p, kx6)); break;
      }
    } else {
      const size_t smem = sizeof(float) * 9 * 32 * kp;
      switch (kp) {
        case 16: METIS_CUDA_TRY(metis_launch_pdl((coeff_mma_kernel<16>), dim3(n_cta_c), dim3(256), (size_t)(smem), s, x, rows, cols, bs, coef, amax, gram_c)); break;
        case 32: METIS_CUDA_TRY(metis_launch_pdl((coeff_mma_kernel<32>), dim3(n_cta_c), dim3(256), (size_t)(smem), s, x, rows, cols, bs, coef, amax, gram_c)); break;
        case 48: METIS_CUDA_TRY(metis_launch_pdl((coeff_mma_kernel<48>), dim3(n_cta_c), dim3(256), (size_t)(smem), s, x, rows, cols, bs, coef, amax, gram_c)); break;
        default: METIS_CUDA_TRY(metis_launch_pdl((coeff_mma_kernel<64>), dim3(n_cta_c), dim3(256), (size_t)(smem), s, x, rows, cols, bs, coef, amax, gram_c)); break;
      }
    }
    METIS_COUNT_LAUNCH();
  }
  {
    QuantParams qp{};
    qp.rows = rows; qp.cols = cols; qp.rounding = rounding; qp.seed = seed; qp.stream_id = METIS_STREAM_RESIDUAL;
    qp.e_stride_r = cols; qp.e_stride_c = 1;
    if (want_c) { qp.c_codes = rc.codes; qp.c_scales = rc.scales; qp.c_layout = rc.sf_layout; }
    if (want_r) { qp.r_codes = rr.codes; qp.r_scales = rr.scales; qp.r_layout = rr.sf_layout; }
    const size_t smem = smem_bytes(rounding == METIS_ROUND_SR);
    dim3 grid((unsigned)metis_ceil_div(cols, TILE), (unsigned)metis_ceil_div(rows, TILE));
    float* t0 = want_c ? rc.tensor_scale : nullptr; float* t1 = want_r ? rr.tensor_scale : nullptr;
    // the big residual pass and the small factor chain below are independent from here on: the factor chain
    // goes to a (high-priority) side stream and is joined back at the end of the call
    METIS_TRY(metis_fork(ctx, s, 1));
    cudaStream_t sr = s;
    if (resid_tc) {
      METIS_TRY(metis_launch_residual_tc(ctx, x, a6_ready ? nullptr : coef, k, kp, qp, amax, t0, t1, residual_dense, a6, b6, sr));
    } else {
      switch (kp) {
        case 16: METIS_CUDA_TRY(metis_launch_pdl((residual_quant_kernel<16>), dim3(grid), dim3(THREADS), (size_t)(smem), sr, x, coef, bt, qp, amax, t0, t1, residual_dense)); break;
        case 32: METIS_CUDA_TRY(metis_launch_pdl((residual_quant_kernel<32>), dim3(grid), dim3(THREADS), (size_t)(smem), sr, x, coef, bt, qp, amax, t0, t1, residual_dense)); break;
        case 48: METIS_CUDA_TRY(metis_launch_pdl((residual_quant_kernel<48>), dim3(grid), dim3(THREADS), (size_t)(smem), sr, x, coef, bt, qp, amax, t0, t1, residual_dense)); break;
        default: METIS_CUDA_TRY(metis_launch_pdl((residual_quant_kernel<64>), dim3(grid), dim3(THREADS), (size_t)(smem), sr, x, coef, bt, qp, amax, t0, t1, residual_dense)); break;
      }
      METIS_COUNT_LAUNCH();
    }
    METIS_CUDA_TRY(metis_launch_pdl((split_status_kernel), dim3(1), dim3(32), (size_t)(0), sr, amax, evals, k, ctx->dev_status)); METIS_COUNT_LAUNCH();
  }
  cudaStream_t sf = ctx->side[0];
  if (!full) {
    // (7) Rayleigh-Ritz on C^T C (Gram partials came out of the broadcast pass), rotate both factors
    METIS_CUDA_TRY(metis_launch_pdl((reduce_gram_kernel), dim3((unsigned)metis_ceil_div(kp * kp, 32)), dim3(128), (size_t)(0), sf, gram_c, n_cta_c, kp * kp, gram1, nullptr)); METIS_COUNT_LAUNCH();
    launch_jacobi(sf, gram1, k, kp, 1e-6f, evals2, evecs2);
    METIS_CUDA_TRY(metis_launch_pdl((right_rotate_kernel), dim3(dim3(n_cand, (k + 7) / 8)), dim3(256), (size_t)(0), sf, basis, cols, k, evecs2, out->right, cand_v, cand_i)); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(metis_launch_pdl((sign_fix_kernel), dim3(dim3(n_cand, k)), dim3(256), (size_t)(0), sf, out->right, cols, k, cand_v, cand_i, n_cand, sign, amax + 2)); METIS_COUNT_LAUNCH();
    METIS_CUDA_TRY(metis_launch_pdl((left_rotate_kernel), dim3(dim3((unsigned)metis_ceil_div(rows, 64), (unsigned)((kp + 15) / 16))), dim3(256), (size_t)(0), sf, coef, rows, k, k, 1, kp, evecs2, evals2, sign,
                                                                            out->left, out->sigma, nullptr, kp, nullptr, amax + 1)); METIS_COUNT_LAUNCH();
  }
  METIS_CUDA_TRY(cudaGetLastError());
  // (8) quantize the factors (stored transposed: k x rows, k x cols; blocks along the long dimension)
  metis_nvfp4_t lq = out->left_q, rq = out->right_q;
  lq.rows = k; lq.k_len = rows; rq.rows = k; rq.k_len = cols;
  METIS_TRY(metis_launch_quantize_factors(out->left, rows, out->right, cols, k, rounding, seed, amax + 1, amax + 2, &lq, &rq, sf));
  return metis_join(ctx, s, 0);
}
