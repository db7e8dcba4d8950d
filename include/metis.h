/*
 * metis.h - C ABI of the B200 (sm_100a) spectral-split NVFP4 linear layer.
 *
 * The library implements the hot path of "Metis: Training LLMs with FP4 Quantization":
 * every GEMM operand T (activation X, weight W, output gradient D) is written as
 *
 *        T = L diag(sigma) R^T + Res                        (Section 3.2, Eq. 1)
 *
 * with the top-k factors found by sparse row sampling plus a Gaussian random projection
 * (Section 3.1), the factors and the residual are quantized independently to NVFP4
 * (Section 2.3, Appendix C.1) and the products of Eq. 2 (forward), Eq. 3 (input gradient) and
 * the weight gradient of Section 3.2 are evaluated with block-scaled FP4 tensor-core GEMMs
 * accumulating in FP32.
 *
 * General rules
 *  - Every pointer is a DEVICE pointer unless its comment says "host".  The caller owns every
 *    buffer (inputs, outputs, workspace); the library allocates device memory only inside
 *    metis_create (a 128 KiB quantile table and a status word; it also creates five streams and six
 *    events there and sets the per-device kernel attributes) and frees it in metis_destroy.
 *  - All work is enqueued on the caller's stream (a cudaStream_t passed as void*); calls return
 *    without synchronising.  Inside a call, independent sub-chains may run on streams the handle owns;
 *    they start after the work already on the caller's stream and are joined back into it before the
 *    call returns, so the caller sees ordinary stream order.  One handle serves one stream at a time.  Host-detectable errors (null or misaligned pointer, unsupported shape,
 *    workspace too small) are returned at once and nothing is enqueued.  Device-detected conditions
 *    (a bounded wait that expired, a Cholesky breakdown) are OR-ed into the handle's device status
 *    word, read with metis_last_device_status after the caller has synchronised the stream.
 *  - Matrices are row-major.  "K-major" below means the contraction axis is the contiguous axis.
 *  - No function throws, aborts or calls exit.
 *
 * NVFP4 storage (metis_nvfp4_t)
 *  - codes: 4-bit E2M1 codes, sign in bit 3, two per byte, element 2j in the low nibble; the tensor
 *    is stored K-major: `rows` x `k_len`/2 bytes where the 16-element blocks lie along k_len.
 *    Quantizing with blocks along the ROWS of a source matrix therefore stores the transposed
 *    matrix (rows = source cols, k_len = source rows).
 *  - scales: one unsigned E4M3 byte per block.  METIS_SF_LINEAR: scales[r][b], b = k/16.
 *    METIS_SF_TILED: the tensor-core layout: tiles of 128 rows x 4 blocks, 512 bytes each, tile
 *    (r/128, b/4) at offset ((r/128)*(k_len/64) + b/4)*512, byte (r%32)*16 + ((r%128)/32)*4 + b%4
 *    inside it.  Needs k_len % 64 == 0; rows are padded to a multiple of 128 (metis_sf_bytes).
 *  - tensor_scale: one FP32 device scalar; value = E2M1(code) * E4M3(scale) * tensor_scale.
 */
#ifndef METIS_H_
#define METIS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct metis_context* metis_handle_t;
typedef void* metis_stream_t;                 /* a cudaStream_t */

typedef enum {
  METIS_OK = 0,
  METIS_ERR_INVALID_ARG = 1,
  METIS_ERR_SHAPE = 2,
  METIS_ERR_ALIGNMENT = 3,
  METIS_ERR_WORKSPACE = 4,
  METIS_ERR_ARCH = 5,
  METIS_ERR_CUDA = 6,
  METIS_ERR_NONFINITE = 7,
  METIS_ERR_NUMERIC = 8,
  METIS_ERR_TIMEOUT = 9
} metis_status_t;

/* bits of the device status word */
#define METIS_DEV_TIMEOUT 1u     /* a bounded wait inside a kernel expired                      */
#define METIS_DEV_NUMERIC 2u     /* the small eigen-decomposition of a split produced a non-finite value */
#define METIS_DEV_NONFINITE 4u   /* the operand of a split or of an amax-scaled quantization holds a NaN or an infinity */
#define METIS_DEV_INDEX 8u       /* debug build only: a kernel was about to store outside an output buffer (the store was skipped) */

typedef enum { METIS_BF16 = 0, METIS_FP32 = 1 } metis_dtype_t;
typedef enum { METIS_ROUND_RNE = 0, METIS_ROUND_SR = 1 } metis_round_t;
typedef enum { METIS_BLOCKS_ALONG_COLS = 1, METIS_BLOCKS_ALONG_ROWS = 2, METIS_BLOCKS_BOTH = 3 } metis_axis_t;
typedef enum { METIS_TSCALE_AMAX_SELF = 0, METIS_TSCALE_GIVEN = 1 } metis_tscale_t;
typedef enum { METIS_SKETCH_FULL = 0, METIS_SKETCH_SAMPLED = 1 } metis_sketch_t;
typedef enum { METIS_SF_LINEAR = 0, METIS_SF_TILED = 1 } metis_sf_layout_t;

/* Philox stream identifiers (third counter word) used by the library's own draws. */
#define METIS_STREAM_RESIDUAL 0x10u
#define METIS_STREAM_LEFT     0x11u
#define METIS_STREAM_RIGHT    0x12u
#define METIS_STREAM_OMEGA    0x100u
#define METIS_STREAM_SAMPLING 0x200u
#define METIS_STREAM_SIGNS    0x300u

typedef struct {
  uint8_t* codes;          /* rows * k_len / 2 bytes, K-major, 16-byte aligned                        */
  uint8_t* scales;         /* metis_sf_bytes(rows, k_len, sf_layout) bytes, 16-byte aligned           */
  float*   tensor_scale;   /* one device float                                                        */
  int64_t  rows;           /* stored rows                                                             */
  int64_t  k_len;          /* stored contraction length (multiple of 16; of 64 for METIS_SF_TILED)    */
  int32_t  sf_layout;      /* metis_sf_layout_t                                                       */
  int32_t  reserved;
} metis_nvfp4_t;

/* One split + quantized operand T (rows x cols) = left diag(sigma) right^T + residual.
 * k == 0 means plain NVFP4: the factor fields are ignored.
 * left / right are the FP32 factors stored TRANSPOSED (k x rows, k x cols: each factor vector
 * contiguous); left_q / right_q their NVFP4 forms (rows = k, k_len = rows resp. cols), i.e. blocks
 * along the long dimension.  res_by_cols is the residual with blocks along its columns (stored
 * rows x cols), res_by_rows with blocks along its rows (stored cols x rows).  Either residual may
 * be absent (codes == NULL) if no product needs it. */
typedef struct {
  int32_t k;
  int32_t reserved;
  int64_t rows, cols;
  float* left;             /* k x rows  */
  float* sigma;            /* k         */
  float* right;            /* k x cols  */
  metis_nvfp4_t left_q, right_q;
  metis_nvfp4_t res_by_cols, res_by_rows;
} metis_operand_t;

/* ---- life cycle -------------------------------------------------------------------------- */

/* Creates a context on `device` (cudaSetDevice is called; the device stays current).  Builds the
 * 65536-entry standard-normal quantile table used by the sketch (Section 3.1).  Fails with
 * METIS_ERR_ARCH unless the device has compute capability 10.x. */
metis_status_t metis_create(metis_handle_t* out, int device);
metis_status_t metis_destroy(metis_handle_t h);

/* Copies the device status word (METIS_DEV_* bits, 0 = clean) to *out (host) and clears it.
 * Synchronises `stream` first. */
metis_status_t metis_last_device_status(metis_handle_t h, uint32_t* out, metis_stream_t stream);

/* Test hook: copies the 65536 bfloat16 quantile-table entries (bit patterns) to host memory.
 * Entry u is the standard normal quantile at level (u + 0.5)/65536 (Section 3.1: the Gaussian test
 * matrix of the random projection is drawn through this table). */
metis_status_t metis_debug_quantile_table(metis_handle_t h, uint16_t* host_out);

/* Benchmark hook: enqueues a one-thread kernel that writes the GPU's nanosecond timer (%globaltimer) to
 * *device_slot when `stream` reaches it; usable inside a stream capture, where events cannot be timed. */
metis_status_t metis_debug_timestamp(metis_handle_t h, uint64_t* device_slot, metis_stream_t stream);

/* Failure-detection hook (the library's kernels bound every wait on an mbarrier and report an expired one through
 * METIS_DEV_TIMEOUT instead of hanging): enqueues a two-warp kernel whose first warp waits at most `polls`
 * (1 .. 2^20) polls on a barrier that is never completed, and whose second warp waits on another one until it
 * sees the first warp's give-up flag.  Afterwards the status word holds METIS_DEV_TIMEOUT and device_seen[0..1]
 * (device, two words) hold, per warp, bit 0 = "my wait expired", bit 1 = "the give-up flag was set".  The kernel
 * returns normally; the context stays usable. */
metis_status_t metis_debug_wait_timeout(metis_handle_t h, uint32_t polls, uint32_t* device_seen, metis_stream_t stream);

/* Debug build (compiled with METIS_DEBUG_BUILD; the Python binding loads it when METIS_DEBUG=1): the quantizing kernels
 * check every global store of codes and scales against the extent of its output buffer and, instead of storing out
 * of range, skip the store and set METIS_DEV_INDEX in the device status word.  metis_debug_build() tells which
 * library this is (1 = debug).  metis_debug_index_check runs the same check in a one-thread kernel on a made-up
 * store of nbytes at `offset` into a buffer of `extent` bytes (nothing is accessed): the self-test of the mechanism. */
int32_t metis_debug_build(void);
metis_status_t metis_debug_index_check(metis_handle_t h, int64_t offset, int64_t nbytes, int64_t extent, metis_stream_t stream);

/* Test / benchmark hook: kernels launched by the library in this process so far (host counter, atomic). */
uint64_t metis_debug_launch_count(void);

/* Bytes of scale storage for a stored rows x k_len NVFP4 tensor (host-only helper, no handle). */
size_t metis_sf_bytes(int64_t rows, int64_t k_len, int32_t sf_layout);

/* Workspace sizes (host-only helpers).  op: 0 quantize, 1 split, 2 linear_fwd, 3 linear_bwd, 4 split of an
 * FP32 or strided operand (op 1 plus a contiguous BF16 copy of the operand).
 * rows/cols describe the largest operand (for the linear ops: rows = max(l, n), cols = max(m, n)). */
metis_status_t metis_workspace_bytes(int32_t op, int64_t rows, int64_t cols, int32_t k, int32_t p, size_t* bytes);

/* Number of rows the SAMPLED sketch reads for a rows-row operand with k+p sketch columns
 * (Section 3.1 samples under one in a hundred sequences; here at least 4(k+p) rows, a multiple of 16). */
int64_t metis_default_sample_count(int64_t rows, int32_t q);

/* ---- NVFP4 quantizer (Section 2.3; value set of Appendix C.1) ----------------------------- */

/* Quantizes x (rows x cols, leading dimension ld elements, BF16 or FP32) into blocks of 16 along
 * its columns (out_by_cols) and/or its rows (out_by_rows); an output pointer may be NULL.
 * Block scale = smallest E4M3 value >= block amax / (6 * tensor_scale) ("rounded up"), elements
 * rounded to nearest even or stochastically (16 random bits per element from Philox4x32-10 keyed
 * by (seed, stream_id, row*cols + col), so both orientations use the same draw).
 * tscale == METIS_TSCALE_AMAX_SELF: tensor_scale <- amax(x)/2688 (1 if x == 0), written to both
 * outputs' tensor_scale; METIS_TSCALE_GIVEN: the outputs' tensor_scale already hold the value.
 * Requires cols % 16 == 0, rows % 16 == 0 when blocks along rows are asked for, tiled scales need % 64 along
 * their block axis, and ld % 8 == 0 (BF16) or ld % 4 == 0 (FP32) so that every row starts 16-byte aligned.
 * Workspace: metis_workspace_bytes(0, ...). */
metis_status_t metis_quantize_nvfp4(metis_handle_t h, const void* x, int32_t dtype, int64_t rows, int64_t cols,
                                    int64_t ld, int32_t rounding, uint64_t seed, uint32_t stream_id,
                                    int32_t tscale, metis_nvfp4_t* out_by_cols, metis_nvfp4_t* out_by_rows,
                                    void* ws, size_t ws_bytes, metis_stream_t stream);

/* Comparison recipe of Section 4 (the paper sets Metis against "a random Hadamard transform alongside SR"): every
 * block of 16 consecutive elements of a row is rotated, y = H16 (s * x) / 4 with H16 the Sylvester Hadamard matrix
 * and s random signs per column (bit 15 of the Philox draw of the column index, stream METIS_STREAM_SIGNS, so two
 * operands quantized with the same seed share them and (x H D)(w H D)^T = x w^T), then quantized like
 * metis_quantize_nvfp4 with blocks along the columns and tensor_scale = amax(y)/2688.  The transform is four
 * butterfly stages in binary32 (distance 1, 2, 4, 8) and one multiplication by 1/4.  x: rows x cols (ld), BF16 or
 * FP32, cols % 16 == 0 (% 64 for tiled scales).  Workspace: 256 bytes.  A same-box comparator for the spectral
 * fidelity figures; not part of the split-FP4 layer. */
metis_status_t metis_quantize_rht_nvfp4(metis_handle_t h, const void* x, int32_t dtype, int64_t rows, int64_t cols,
                                        int64_t ld, int32_t rounding, uint64_t seed, uint32_t stream_id,
                                        metis_nvfp4_t* out, void* ws, size_t ws_bytes, metis_stream_t stream);

/* ---- split (Sections 3.1, 3.2) ------------------------------------------------------------ */

/* Splits x (rows x cols, leading dimension ld elements, BF16 or FP32) into rank-k factors and a residual and
 * quantizes all of them into `out` (whose buffers the caller has allocated; out->k, rows, cols are checked).
 * The decomposition runs on BF16 tensor-core passes over a contiguous operand: an FP32 operand is rounded to BF16
 * (nearest even) and a strided one (ld > cols) is gathered, in one extra pass into the workspace, before anything
 * else - ask metis_workspace_bytes for op 4 instead of 1 in those cases; ld % 8 == 0 (BF16) or ld % 4 == 0 (FP32).
 * With k == 0 nothing is packed or rounded: x is quantized as metis_quantize_nvfp4 would.
 *  sketch = METIS_SKETCH_FULL:    Z = x Omega, thin QR, M = H^T x, small SVD, top k, residual
 *                                 x - A Lambda B^T.
 *  sketch = METIS_SKETCH_SAMPLED: the same on n_sample sampled rows (0 = default rule) to get the
 *                                 right basis B, then C = x B for all rows, Rayleigh-Ritz on C^T C,
 *                                 residual x - C B^T.
 * Omega (cols x (k+p)) is generated on the fly from Philox (seed, METIS_STREAM_OMEGA) through the
 * quantile table (per thread block in shared memory for sampled sketches, once per call into the
 * workspace for full ones); it is never an input or an output.  The residual is quantized with the tensor
 * scale amax(x)/2688 of the SOURCE tensor; factors with their own.  `residual_axes` selects which
 * residual orientations are produced.  `residual_dense` (optional, rows x cols FP32) receives the
 * unquantized residual the quantizer saw.  k == 0 quantizes x itself.
 * src_amax (optional device scalar): amax|x| (of the BF16-rounded values, for an FP32 operand with k > 0) as the producer of x already knows it (e.g. from the epilogue of the
 * kernel that wrote x).  NULL: the library finds it - for k > 0 inside a pass it makes anyway, for k == 0 with a
 * reduction of its own, i.e. a second read of x that a supplied value saves.  The value is trusted: a value below
 * the true maximum makes the largest elements saturate.
 * Requires rows % 16 == 0, cols % 64 == 0 (tiled scales), k % 4 == 0, k <= 256 and k + p <= 272.
 * Up to k = 64 and k + p = 72 the orthonormalisation and the two small eigen-solvers each run in one CTA's
 * shared memory; above that (the 1.5 % rank of an 8192-wide layer is 128) they run on FP64 kernels tiled over the
 * rank and on an eight-CTA cluster, which additionally needs rows % 64 == 0.  Larger ranks are refused with
 * METIS_ERR_SHAPE.
 * Workspace: metis_workspace_bytes(1, rows, cols, k, p) (for the wide ranks: sized for the default sample count;
 * a larger n_sample may need more and is then refused with METIS_ERR_WORKSPACE). */
metis_status_t metis_split(metis_handle_t h, const void* x, int32_t dtype, int64_t rows, int64_t cols, int64_t ld,
                           int32_t k, int32_t p, int32_t sketch, int64_t n_sample, uint64_t seed, int32_t rounding,
                           int32_t residual_axes, const float* src_amax, metis_operand_t* out, float* residual_dense,
                           void* ws, size_t ws_bytes, metis_stream_t stream);

/* Re-quantization of a stored operand (Section 3.2: a weight is kept as separately stored U, S, V and W_R, which the
 * optimizer updates; per step only their NVFP4 forms are refreshed - no decomposition).  `op` holds the stored FP32
 * factors (op->left k x rows, op->right k x cols, op->sigma; read, never written) and receives left_q, right_q
 * (own amax/2688 tensor scales, draws of METIS_STREAM_LEFT / _RIGHT) and the residual orientations selected by
 * `residual_axes`, quantized from `residual` (rows x cols, leading dimension ld_res elements, BF16 or FP32) with
 * draws of METIS_STREAM_RESIDUAL.  res_tscale == METIS_TSCALE_AMAX_SELF: the residual's tensor scale is
 * amax(residual)/2688 (there is no source tensor to take it from); METIS_TSCALE_GIVEN: the requested outputs'
 * tensor_scale already hold the value (e.g. the one the initial split produced).  k == 0: residual only.
 * Five launches (three amax reductions, one kernel for both residual orientations, one for both factors).
 * Workspace: 256 bytes. */
metis_status_t metis_requantize_operand(metis_handle_t h, const void* residual, int32_t res_dtype, int64_t ld_res,
                                        int32_t rounding, uint64_t seed, int32_t residual_axes, int32_t res_tscale,
                                        metis_operand_t* op, void* ws, size_t ws_bytes, metis_stream_t stream);

/* ---- linear layer (Eq. 2, Eq. 3, weight gradient) ----------------------------------------- */

/* y (l x n, ldy) = Xq Wq^T, Eq. 2.  x: l x m operand with res_by_cols; w: W_t, n x m operand with
 * res_by_cols.  y is BF16 or FP32.  Scales must be METIS_SF_TILED. */
metis_status_t metis_linear_fwd(metis_handle_t h, const metis_operand_t* x, const metis_operand_t* w,
                                void* y, int32_t y_dtype, int64_t ldy, void* ws, size_t ws_bytes,
                                metis_stream_t stream);

/* Forward layer without a caller workspace.  (No counterpart in the paper: this is an integration aid.)
 * Same result as metis_linear_fwd, bit for bit, but the intermediates live in a METIS_STATIC_WS_BYTES array
 * built into the library image (each GPU that loads the library carries it until the process exits).  It is
 * meant for callers that own inputs and outputs but cannot obtain scratch memory: a process whose memory
 * pool already holds every free byte of the device, or a plug-in that is not allowed to call an allocator.
 * The call allocates nothing on host or device.
 *  - Limit: the layer's intermediates must fit METIS_STATIC_WS_BYTES, else METIS_ERR_WORKSPACE is returned and
 *    nothing is enqueued.  With k = k_x + k_w they are 4 (l + n) k bytes of FP32 skinny operands plus, when l and
 *    n are both at least 256, 2 (l + n) roundup64(3 k) bytes of BF16 correction operands, or else (a smaller
 *    layer) 4 l n bytes of FP32 staging for the main product; plain NVFP4 operands (k = 0) need nothing.
 *  - h's device must be the current device (else METIS_ERR_INVALID_ARG).
 *  - The first call on each device looks up the array's device address (a one-time runtime query); make that
 *    first call during start-up, before any stream capture is begun.
 *  - All calls on a device share the one array, which keeps whatever the last call left in it; the layer
 *    needs no zeroed scratch, so nothing is cleared.  Two calls whose kernels overlap on the GPU (different
 *    streams, or different threads) race on it: serialise them. */
#define METIS_STATIC_WS_BYTES (4u << 20)
metis_status_t metis_linear_fwd_static_ws(metis_handle_t h, const metis_operand_t* x, const metis_operand_t* w,
                                          void* y, int32_t y_dtype, int64_t ldy, metis_stream_t stream);

/* dx (l x m) = Dq Wq' (Eq. 3; needs dy->res_by_cols, w->res_by_rows) and
 * dw (n x m) = Dq''^T Xq'' (weight gradient; needs dy->res_by_rows, x->res_by_rows).
 * Either output may be NULL to skip it.
 *
 * Factor gradients (Section 3.2, the derivatives that follow Eq. 3), optional, each may be NULL: with the
 * weight operand W_t = left diag(sigma) right^T + Res (left = the paper's V, n x k; right = the paper's U,
 * m x k) and dw as just computed,
 *   d_left  (k x n, like w->left)   = sigma_t * sum_i dw[j][i] * right_q[t][i]      (the paper's dL/dV),
 *   d_right (k x m, like w->right)  = sigma_t * sum_j dw[j][i] * left_q[t][j]       (the paper's dL/dU),
 *   d_sigma (k)                     = sum_ij left_q[t][j] dw[j][i] right_q[t][i]    (diagonal of dL/dS),
 * using the dequantized NVFP4 factors and FP32 accumulation in a fixed order.  The gradient of the residual
 * W_R is dw itself.  They need dw and w non-NULL (else METIS_ERR_INVALID_ARG) and d_sigma needs d_left;
 * dw is read back in the type it was written in. */
metis_status_t metis_linear_bwd(metis_handle_t h, const metis_operand_t* dy, const metis_operand_t* x,
                                const metis_operand_t* w, void* dx, int32_t dx_dtype, int64_t lddx, void* dw,
                                int32_t dw_dtype, int64_t lddw, float* d_left, float* d_sigma, float* d_right,
                                void* ws, size_t ws_bytes, metis_stream_t stream);

/* Plain block-scaled FP4 GEMM on already quantized tensors: d (M x N, ldd) = a b^T * (a.ts * b.ts),
 * a: M x K, b: N x K, both K-major with METIS_SF_TILED scales.  Exposed for tests and benchmarks of
 * the tensor-core kernel on identical codes.  impl: 0 = tcgen05 kernel, 1 = scalar check kernel. */
metis_status_t metis_gemm_nvfp4(metis_handle_t h, const metis_nvfp4_t* a, const metis_nvfp4_t* b, void* d,
                                int32_t d_dtype, int64_t ldd, int32_t impl, metis_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* METIS_H_ */
