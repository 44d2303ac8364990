/*
 * fmm_b200 — low-precision fast bilinear matrix multiplication on one B200 (sm_100a).
 *
 * C ABI.  No C++ or framework types cross this boundary: plain pointers and sizes only.
 * Every pointer argument says whether it is HOST or DEVICE memory.
 *
 * The operation (paper Section 2.1, Eq. 1).  An algorithm <m,k,n;R> with coefficients
 * U[R][m][k], V[R][k][n], W[R][m][n] splits A (M x K) into an m x k grid of blocks A_il
 * and B (K x N) into a k x n grid B_lj (contiguous blocks, Section 3.2) and computes
 *     Ahat_r = rnd_Pd( (sum_{i,l} u_{r,il} A_il) / sA_r )        "encode A"
 *     Bhat_r = rnd_Pd( (sum_{l,j} v_{r,lj} B_lj) / sB_r )        "encode B"
 *     M_r    = Ahat_r * Bhat_r                    (fp32 accumulation, tensor cores)
 *     C_ij   = rnd_O( sum_r w_{r,ij} sA_r sB_r M_r )             "decode"
 * The rounding of the block sums to the product dtype Pd is the step whose effect the
 * paper studies (Section 2.3, Appendix B.1); products stay fp32 and are combined in fp32
 * (Appendix B.1).  Coefficients are used as fp32 values of the fp64 numbers held in the
 * handle.  Block sums are formed as an fp32 fused-multiply-add chain over the nonzero
 * coefficients in ascending row-major (i,l) resp. (l,j) order; decode adds in ascending r.
 *
 * Conventions
 *   - every call returns an fmm_status; nothing throws, aborts or prints;
 *   - out-parameters are written only when FMM_OK is returned;
 *   - scheme handles are created by the library (host memory only, no GPU needed),
 *     are immutable, and are released with scheme_free; gauge/kron results are
 *     independent objects;
 *   - operand, result and workspace buffers are caller-owned DEVICE memory, 256-byte
 *     aligned, row-major, leading dimensions in elements and a multiple of 16 bytes;
 *   - calls that take a stream only enqueue work on it (no synchronisation, no device
 *     allocation), except error_sweep, which synchronises the stream once at its end
 *     because it returns host numbers;
 *   - M % m, K % k, N % n must be 0, K/k must be a multiple of 16 and N/n a multiple
 *     of 8 (FMM_ERR_SHAPE otherwise): zero padding is the caller's job, as in the paper
 *     (Appendix B.2 pads 40 rows to 48);
 *   - maximum sizes: one block may hold fewer than 2^31 - 4096 sixteen-byte vectors of the source
 *     ((M/m) * (K/k) * storage bytes / 16, likewise for B) and fewer than that many quads of products
 *     ((M/m) * (N/n) / 4); M/m, N/n < 2^31 - 4096 and K/k < 2^30.  Larger shapes, empty shapes
 *     (M, K or N <= 0) included, return FMM_ERR_SHAPE (the workspace queries return 0) and launch nothing;
 *   - NaN/Inf in operands propagate; e4m3 conversion saturates at +-448.
 *   - devices and threads: a call works on the current device of the calling thread; kernels are configured per
 *     device on first use.  The library keeps process-wide state (two helper streams with an event ring for
 *     error_sweep, the launch counter, the phase-timing record), created on the device that first needs it: use
 *     one device per process (the multi-GPU model here is one process per GPU) and do not call into the library
 *     from two host threads at once.  Scheme handles are immutable after creation and may be shared.
 */
#ifndef FMM_B200_H
#define FMM_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fmm_scheme fmm_scheme; /* opaque, library-owned, immutable */

typedef enum {
  FMM_OK = 0,
  FMM_ERR_ARG = 1,       /* null pointer, bad enum, bad size */
  FMM_ERR_SHAPE = 2,     /* divisibility / alignment of M,K,N,ld* violated */
  FMM_ERR_BRENT = 3,     /* coefficients do not satisfy the Brent equations within tolerance */
  FMM_ERR_SINGULAR = 4,  /* gauge matrix singular or above the condition limit */
  FMM_ERR_DTYPE = 5,     /* unsupported storage/product/output combination */
  FMM_ERR_WORKSPACE = 6, /* workspace null, misaligned or too small */
  FMM_ERR_CUDA = 7,      /* a CUDA runtime/driver call failed (incl. no device) */
  FMM_ERR_TIMEOUT = 8,   /* a bounded device-side wait expired; results are invalid */
  FMM_ERR_LIMIT = 9,     /* scheme larger than the library's table limits */
  FMM_ERR_CERTIFICATE = 10 /* Proposition 1 does not hold for this algorithm, code bound and tiling */
} fmm_status;

typedef enum { FMM_F32 = 0, FMM_BF16 = 1, FMM_E4M3 = 2 } fmm_dtype;

/* Limits of the coefficient tables a handle may hold. */
#define FMM_MAX_GRID 4    /* m, k, n <= 4 */
#define FMM_MAX_R 64      /* R <= 64 */

/* flags of fmm_gemm_desc */
#define FMM_FLAG_REUSE_BHAT 1 /* the workspace already holds Bhat (and sB) written by an earlier
                                 scheme_gemm call with the same scheme, desc and workspace: skip
                                 "encode B".  Weights are static, so their block sums can be
                                 formed once (the paper prepares weight block sums offline,
                                 Section 3.1 / Appendix C).                                   */
#define FMM_FLAG_PRODUCTS_BF16 2 /* every block product M_r is rounded to bf16 before the combination,
                                 as in the paper's model schedule, whose product kernel "returns each
                                 product in bf16" (Appendix B.1); the combination stays in fp32.  Halves
                                 the bytes the products move.  With scale_mode 1 the product of the codes
                                 is rounded (the power-of-two scales commute with the rounding); with
                                 scale_mode 2 the rounding follows the row / column scales.            */

#define FMM_FLAG_SWEEP_SERIAL 4 /* error_sweep only: run the stages of every gauge back to back on the caller's
                                 stream instead of pipelining consecutive gauges over the library's helper
                                 streams.  Same results bit for bit (the arithmetic and the order of every sum
                                 are the same); slower.  For callers that want one stream only, and for checking
                                 the pipelined path against.                                              */

#define FMM_FLAG_SWEEP_UNFUSED 16 /* error_sweep only: do not use the fused launches.  By default, where it applies (bf16
                                 storage and products, no scales, one-level algorithms on a 2 x 2 grid, blocks larger
                                 than 128 x 128), each batch's block products run as ONE kernel launch together with
                                 the decode of the batch before it and the encode of the batch after it: the CTAs
                                 carry the tensor-core roles and, beside them, warps that stream the other two passes.
                                 Every algorithm's C is the same bits either way; its error sum is added over another
                                 partition of the outputs (ratios agree to 1e-8; each path is bit-reproducible run to
                                 run).  With this flag such sweeps take the three-stream pipeline that all other
                                 sweeps use.                                                                    */
#define FMM_FLAG_ROUND_PER_LEVEL 8 /* scheme_gemm on a handle made by scheme_kron (or "strassen444"): round the block
                                 sums at EVERY level.  The outer factor's block sums of A (and of B) are scaled
                                 and rounded to the product dtype; the inner factor's block sums are formed of
                                 those rounded values and rounded again; products and decode are unchanged
                                 (decode uses the flat coefficients w1 w2 in ascending r).  This is "the algorithm
                                 applied to its own blocks" (Section 1) taken literally — a different operator
                                 from the default, flat one, which rounds each of the R1 R2 block sums of the
                                 Kronecker coefficients once (what the paper's two-level algorithm does).
                                 scale_mode 0 or 1 (mode 1: one power-of-two scale per outer tensor, then one per
                                 inner tensor in units of it; sA_r is their product).  FMM_ERR_ARG for a flat
                                 handle and in error_sweep.                                                  */

/* The float-path "quantisation specification" (Section 2.2 treats these choices as part of the
 * operator): shapes, dtypes, layout of B, scale rule. */
typedef struct {
  int64_t M, K, N;       /* C[M x N] = A[M x K] * B[K x N] */
  int64_t lda, ldb, ldc; /* leading dimensions in elements */
  int32_t storage;       /* fmm_dtype of A and B in memory: FMM_F32 or FMM_BF16 */
  int32_t product;       /* fmm_dtype the block sums are rounded to: FMM_BF16 or FMM_E4M3 */
  int32_t output;        /* fmm_dtype of C: FMM_F32 or FMM_BF16 */
  int32_t b_is_weight_layout; /* 0: B stored [K x N] (N contiguous); 1: B stored [N x K]
                                 (K contiguous, the nn.Linear weight layout) */
  int32_t scale_mode;    /* 0: no scales.  1 (e4m3 only): one power-of-two scale per encoded
                            tensor, s = 2^ceil(log2(amax/448)), s = 1 for an all-zero tensor;
                            classical_gemm uses one such scale per operand.
                            2 (e4m3 only): the simplified synthetic schedule of Appendix B.1, one
                            scale per row of each block sum of A and per column of each block sum of
                            B, s = amax / 448 in fp32 (1 for an all-zero row), code = x / s in fp32,
                            then rounded; each product is stored as (M_r * s_row) * s_col.  In the
                            workspace the scales are then [R][M/m] and [R][N/n] arrays.
                            3 (e4m3 only): the model schedule of Appendix B.1: block sums of A get one
                            scale per row and per 128 consecutive inner indices; block sums of B are
                            first rounded to bf16, then get one scale per 128 x 128 block (128 inner
                            indices x 128 output columns); s = amax / 448 as in mode 2.  The product
                            kernel accumulates every 128-group on its own, multiplies it by the two
                            scales and adds the groups in ascending order in fp32 (the last group may be
                            shorter).  Scales in the workspace: [R][M/m][G] and [R][ceil(N/n/128)][G],
                            G = ceil(K/k/128).  classical_gemm applies the same schedule to
                            the operands themselves (the deployed FP8 kernel's layout of scales) */
  int32_t flags;         /* FMM_FLAG_* */
} fmm_gemm_desc;

/* Summary of a sweep (Table 3 caption: smallest, median = upper of the two middle values when the
 * count is even, largest; spread = largest / smallest; number of ratios above 2). */
typedef struct {
  double min, median, max, spread;
  int64_t count_gt2;
  int64_t G;
  double e_classical_rel; /* relative Frobenius error of the classical product vs fp64 */
  double norm_ref;        /* Frobenius norm of the fp64 reference */
} fmm_sweep_summary;

/* ---- scheme handles (HOST only; usable without a GPU) ---------------------------------- */

/* Create a handle from coefficient arrays U[R][m][k], V[R][k][n], W[R][m][n] (HOST, fp64,
 * row-major; w indexed by the C block it feeds, Eq. 1).  The Brent equations (all unwanted
 * cross terms cancel, Section 2.1) are checked: FMM_ERR_BRENT if the largest residual
 * exceeds brent_tol * max(1, R * max|u| * max|v| * max|w|).  brent_tol <= 0 selects 1e-12.
 * The arrays are copied.  FMM_ERR_LIMIT if m,k,n > FMM_MAX_GRID or R > FMM_MAX_R.       */
fmm_status scheme_load(int m, int k, int n, int R, const double* U, const double* V, const double* W,
                       double brent_tol, fmm_scheme** out);

/* Built-in algorithms: "strassen222" (the seven products of the paper's Appendix A.1 table),
 * "strassen444" (its nesting with itself, 49 products, Section 1), "classical111",
 * "classical222" (the mkn-product classical algorithm written as a scheme).                */
fmm_status scheme_builtin(const char* name, fmm_scheme** out);

/* Nesting: `outer` applied to blocks multiplied by `inner`; block index = outer*dim_inner + inner
 * (contiguous blocks, Section 3.2), product index r = r_outer * R_inner + r_inner.  The result
 * remembers its factors (see gauge_apply, level 1).                                         */
fmm_status scheme_kron(const fmm_scheme* outer, const fmm_scheme* inner, fmm_scheme** out);

/* The same algorithm with its products renumbered: product r of *out is product perm[r] of `in` (perm: HOST,
 * a permutation of 0..R-1, else FMM_ERR_ARG).  The decode adds the products in ascending r, so the order of the
 * fp32 additions is part of the operator (Appendix B.1 reports perplexity spans from the summation order alone):
 * in exact arithmetic nothing changes, in fp32 the result may move in its last bits.  The handle is flat (no
 * outer / inner factors for gauge_apply at level 1).                                                        */
fmm_status scheme_permute_products(const fmm_scheme* in, const int* perm, fmm_scheme** out);

/* Gauge transform (Section 2.1).  With P[m][m], Q[k][k], S[n][n] (HOST, fp64, row-major,
 * invertible):  U'_r = P^T U_r Q^-T,  V'_r = Q^T V_r S^-T,  W'_r = P^-1 W_r S, which for diagonal
 * sign matrices D,E,F is the paper's sign variant d_i e_l u, e_l f_j v, d_i f_j w.
 * level 0: P,Q,S act on the handle's own m x k x n grid.
 * level 1: the handle must come from scheme_kron; P,Q,S have the OUTER factor's dimensions and
 *          transform the outer factor only.
 * FMM_ERR_SINGULAR if a matrix is singular or its 2-norm condition number exceeds cond_limit
 * (cond_limit <= 0: no limit).  Sign gauges are exact: every operation on 0, +-1 entries is. */
fmm_status gauge_apply(const fmm_scheme* in, int level, const double* P, const double* Q, const double* S,
                       double cond_limit, fmm_scheme** out);

/* dims[4] = {m,k,n,R}.  meta[8] = {L_A, L_B, L_W (Section 4.2), Phi, number of nonzero
 * coefficients, largest |coefficient|, Q, E (Appendix B.1)}.  Either pointer may be NULL. */
fmm_status scheme_info(const fmm_scheme* s, int dims[4], double meta[8]);

/* Copy the coefficients out (HOST buffers of R*m*k, R*k*n, R*m*n doubles; any may be NULL). */
fmm_status scheme_coefficients(const fmm_scheme* s, double* U, double* V, double* W);

void scheme_free(fmm_scheme* s);

/* ---- device work ------------------------------------------------------------------------ */

/* Bytes of DEVICE workspace scheme_gemm needs for this scheme and problem (0 on bad args). */
size_t scheme_gemm_workspace(const fmm_scheme* s, const fmm_gemm_desc* d);

/* Where scheme_gemm leaves its intermediates inside the workspace, so that a caller (or a test) can inspect
 * each step of Eq. 1 after the call.  Byte offsets from d_ws:
 *   off[0] Ahat_r  R blocks [M/m][K/k], product dtype      off[1] Bhat_r  R blocks [N/n][K/k], product dtype (K-major)
 *   off[2] M_r     R blocks [M/m][N/n], fp32               off[3] sA[R] fp32    off[4] sB[R] fp32 (scale_mode 1 only)
 * and the distance, in ELEMENTS, between consecutive blocks r and r+1 of each array (block size plus a small
 * padding that keeps the R streams off the same memory channels):
 *   off[5] Ahat    off[6] Bhat    off[7] M                                                                  */
fmm_status scheme_gemm_workspace_layout(const fmm_scheme* s, const fmm_gemm_desc* d, size_t off[8]);

/* C = scheme(A, B) as defined at the top of this file (Eq. 1 with rounded block sums).
 * dA, dB, dC: DEVICE.  d_ws: DEVICE, >= scheme_gemm_workspace bytes, 256-byte aligned; its
 * contents are scratch except that Bhat persists for FMM_FLAG_REUSE_BHAT.  Asynchronous on
 * `cuda_stream` (a cudaStream_t passed as void*; NULL = default stream).  Device-side waits
 * are bounded; a wait that expires is reported by fmm_device_status.                       */
fmm_status scheme_gemm(const fmm_scheme* s, const fmm_gemm_desc* d, const void* dA, const void* dB,
                       void* dC, void* d_ws, size_t ws_bytes, void* cuda_stream);

/* Read (after synchronising the stream) the device status word the kernels of the last call
 * on this workspace left: FMM_OK or FMM_ERR_TIMEOUT.                                        */
fmm_status fmm_device_status(const void* d_ws, void* cuda_stream);

/* Self-test of device-side failure reporting.  Launches ONE block of the block-product kernel on a 128 x 128 x 64
 * tile held in the workspace, with its copy-issuing warp switched off and every wait bounded by wait_ms
 * (1..2000 ms) instead of the default 2 s: the consumer's wait can never be satisfied, so it must expire, the
 * block must record FMM_ERR_TIMEOUT in the status word, release its resources and return normally.  The call only
 * enqueues; fmm_device_status(d_ws, stream) then reports FMM_ERR_TIMEOUT and the context stays usable.
 * d_ws: DEVICE, >= 128 KiB, 256-byte aligned.  Nothing in this test faults, traps or spins without bound.      */
fmm_status fmm_selftest_timeout(void* d_ws, size_t ws_bytes, unsigned wait_ms, void* cuda_stream);

size_t classical_gemm_workspace(const fmm_gemm_desc* d);

/* The classical product at the same dtypes (the paper's control, Section 3.1):
 * C = rnd_O( sA sB * rnd_Pd(A/sA) * rnd_Pd(B/sB) ), fp32 accumulation on the same tensor-core
 * kernel.  With storage == product == bf16 the operands are read in place.  Operands that are already e4m3 codes
 * (storage == product == FMM_E4M3, scale_mode 0, weight layout; one byte per element, leading dimensions a
 * multiple of 16) are multiplied in place too: the tensor-core product of the codes alone, which is also how
 * the library's own fp8 tensor rate is measured.                                                          */
fmm_status classical_gemm(const fmm_gemm_desc* d, const void* dA, const void* dB, void* dC,
                          void* d_ws, size_t ws_bytes, void* cuda_stream);

/* Exact reference (Appendix B.1, "a float64 reference"): dCstar[M x N] (DEVICE, fp64, ld = N)
 * = fp64 product of the stored operand values.  desc->product/output are ignored.          */
fmm_status exact_gemm_f64(const fmm_gemm_desc* d, const void* dA, const void* dB, double* dCstar,
                          void* cuda_stream);

size_t error_frobenius_workspace(void);

/* Squared Frobenius error against the fp64 reference (Appendix B.1): d_out[0] = sum (C - C*)^2,
 * d_out[1] = sum C*^2 (DEVICE, 2 doubles).  dC has dtype desc->output and leading dimension
 * desc->ldc; dCstar is M x N fp64 with ld = N.  Per-block partial sums go to the workspace and are
 * added in a fixed order, so the result is reproducible run to run.                         */
fmm_status error_frobenius(const fmm_gemm_desc* d, const void* dC, const double* dCstar, double* d_out,
                           void* d_ws, size_t ws_bytes, void* cuda_stream);

/* error_frobenius without any allocation or caller-supplied workspace.  (The paper has no counterpart: this
 * entry point exists for callers, not for the method.)
 *
 * Some callers may not allocate device memory at the point where they need the error: they are inside a
 * CUDA-graph capture or another no-allocation region, their memory pool is fully committed, or their host
 * application forbids libraries from growing their device footprint after start-up.  error_frobenius asks
 * such a caller for a workspace; this variant instead keeps its per-block partial sums in a fixed 32 KiB
 * array that is part of the library itself, so every GPU that loads the library carries that array until
 * the process exits.
 *
 * Same arguments and result as error_frobenius (d_out[0] = sum (C - C*)^2, d_out[1] = sum C*^2; DEVICE), minus
 * the workspace.  It calls no cudaMalloc / cudaFree and no routine that allocates.
 *   - Size limit: M * N <= error_frobenius_noalloc_max_elements() (67,108,864); larger problems return
 *     FMM_ERR_LIMIT and nothing is launched.
 *   - First call on a device: looks up the array's device address (once per device, with that device
 *     current).  Make that first call outside any stream capture.  The address is kept for the life of the
 *     process and does not survive a cudaDeviceReset of that device.
 *   - All calls on a device share the one array.  Nothing in it needs clearing between calls (each block
 *     overwrites its own slot), but two calls whose kernels overlap on the GPU — different streams without an
 *     ordering between them — race on it: order such calls yourself.                                        */
fmm_status error_frobenius_noalloc(const fmm_gemm_desc* d, const void* dC, const double* dCstar, double* d_out,
                                   void* cuda_stream);
int64_t error_frobenius_noalloc_max_elements(void);

/* scheme_gemm for operands in HOST memory — the end-to-end form of the path (Eq. 1, Appendix B.1): on `cuda_stream`,
 * A and B are copied into dense device buffers inside the workspace, scheme_gemm runs on them, and C is copied back.
 * hA, hB, hC: HOST, laid out as d says (lda / ldb / ldc in elements; pinned memory makes the copies asynchronous and
 * lets calls on different streams overlap; pageable memory works and serialises).  With FMM_FLAG_REUSE_BHAT the
 * weight is neither copied nor encoded (hB may be NULL): the previous call on this workspace left its block sums.
 * d_ws: DEVICE, >= scheme_gemm_host_workspace bytes (the three device copies plus a scheme_gemm workspace), 256-byte
 * aligned, owned by the caller; one workspace per stream in flight.  The call only enqueues; hC is valid once the
 * stream has been synchronised.  scheme_gemm_host_status synchronises the stream and reports the device status of
 * the calls on this workspace (FMM_OK or FMM_ERR_TIMEOUT), as fmm_device_status does for scheme_gemm.
 * Errors as scheme_gemm.                                                                                       */
size_t scheme_gemm_host_workspace(const fmm_scheme* s, const fmm_gemm_desc* d);
fmm_status scheme_gemm_host_status(const fmm_scheme* s, const fmm_gemm_desc* d, const void* d_ws, void* cuda_stream);
fmm_status scheme_gemm_host(const fmm_scheme* s, const fmm_gemm_desc* d, const void* hA, const void* hB, void* hC,
                            void* d_ws, size_t ws_bytes, void* cuda_stream);

size_t error_sweep_workspace(const fmm_scheme* base, const fmm_gemm_desc* d, int G);

/* Sweep over G gauge-equivalent copies of one scheme (Section 3.3 / Table 3, model-free form of
 * Appendix B.1).  For g = 0..G-1 the scheme gauge_apply(base, level, P_g, Q_g, S_g) is run on the
 * same operands; its squared Frobenius error against the fp64 reference is reduced on the device
 * (C_g is not stored).  The error-amplification ratio is
 *     rho_g = ||C_g - C*||_F / ||C_cl - C*||_F ,
 * C_cl the classical product at the same dtypes (rho = 1 if both errors vanish, +inf if only the
 * classical one does).
 * P, Q, S: HOST, G stacked row-major matrices (dimension of the gauged grid).  dCstar: DEVICE fp64
 * M x N reference, or NULL to have it computed.  h_ratios: HOST, G doubles (may be NULL).
 * out: HOST.  Synchronises the stream once before returning.
 * Errors: every gauge matrix is inverted on the host before anything is enqueued, so FMM_ERR_SINGULAR leaves the
 * device untouched; a failure after that point returns only once the caller's stream is ordered behind all work the
 * call enqueued on the library's helper streams (the workspace may then be reused or freed in stream order).
 * NaN: ratios of operands that hold NaN are NaN; if any ratio is NaN, min / median / max / spread are NaN and
 * count_gt2 counts the comparable ratios above 2.
 * Execution: equivalent algorithms share their operands, so up to eight of them (as many as fit the table limits:
 * products of the batch <= FMM_MAX_R) run as one encode, one product launch and one error-only decode; every
 * algorithm's arithmetic and summation order are those of a scheme_gemm call on it, and the call is bit-reproducible
 * run to run.                                                                                              */
fmm_status error_sweep(const fmm_scheme* base, int level, int G, const double* P, const double* Q,
                       const double* S, const fmm_gemm_desc* d, const void* dA, const void* dB,
                       const double* dCstar, double* h_ratios, fmm_sweep_summary* out, void* d_ws,
                       size_t ws_bytes, void* cuda_stream);

/* ---- Certified realisation on bounded integer codes (Section 4.2, Proposition 1; Appendix D) ------------
 *
 * The int8 operator of the quantisation specification: inputs in fp32 (or bf16), one fp32 scale per row and
 * per group of 128 consecutive inner indices, d = max|x| / b (d = 1 for an all-zero group), codes = x / d
 * rounded to nearest even, no clipping; per group in ascending order the exact integer product P of the codes is
 * converted to fp32, multiplied by the row's scale, then by the column's scale (two fp32 multiplications) and
 * added to a zero-initialised fp32 output, which is cast once to the output dtype.  K must be a multiple of
 * 128 (the caller pads with zeros, as the specification says).                                              */

/* Proposition 1 from the coefficients, the code bounds, the block inner length h, the group size g and the
 * accumulator width alone.  cert[4] (HOST, may be NULL) = {L_A*bA, L_B*bB, max{L_W*h*(L_A*bA)*(L_B*bB),
 * g*bA*bB}, 1 if a call (k blocks of length h) spans exactly one group}.  Returns 1 when the coefficients are
 * integers, (i) both block-sum bounds are <= 127, (ii) the largest bound is < 2^acc_bits and (iii) holds;
 * 0 otherwise.  s == NULL means the classical algorithm <1,1,1;1>.  Host only.                              */
int scheme_certificate(const fmm_scheme* s, int bA, int bB, int h, int g, int acc_bits, double cert[4]);

/* Quantiser.  d_X: DEVICE, rows x K of `storage` (FMM_F32 or FMM_BF16), leading dimension ldx (elements,
 * multiple of 4, pointer aligned to 4 elements).  d_codes: DEVICE int8 [rows][K]; d_scales: DEVICE fp32
 * [rows][K/128].  For B pass the weight layout [N][K] (one row per output column).  1 <= code_bound <= 127.
 * Asynchronous on the stream.                                                                                */
fmm_status int8_quantize(const void* d_X, int storage, int64_t rows, int64_t K, int64_t ldx, int code_bound,
                         int8_t* d_codes, float* d_scales, void* cuda_stream);

size_t int8_gemm_workspace(const fmm_scheme* s, int64_t M, int64_t K, int64_t N);

/* The int8 operator on quantised operands: d_cA int8 [M][K] with scales d_dA [M][K/128], d_cB int8 [N][K]
 * with d_dB [N][K/128] (all DEVICE, code pointers 16-byte aligned); d_C: DEVICE [M][ldc] of `output` (FMM_F32
 * or FMM_BF16, 16-byte aligned rows).  s == NULL computes every group's integer product classically, in one kernel
 * (int8 tensor-core products with int32 accumulators, the rescale in its epilogue).  Otherwise each group's product is
 * computed by one call of s on the group's 128 inner indices split into k blocks of length 128/k (which must be 32,
 * 64 or 128), rows into m and columns into n contiguous blocks — also in one kernel (Figure 3): the block sums of the
 * codes are formed as int8 (certificate (i): they fit), a CTA owns 128 row positions and 16 column positions of every
 * C block, multiplies the R pairs of block sums on the tensor cores (kind::i8, one int32 accumulator per product in
 * tensor memory, at most 16 products at a time), combines them with the integer w, and applies the group's two scales —
 * no block product leaves the SM.  When the certificate holds the output is bit-identical to the classical operator's for every such s.
 * Returns FMM_ERR_CERTIFICATE, launching nothing, if scheme_certificate(s, code_bound, code_bound, 128/k, 128,
 * 24) fails; the caller vouches that |code| <= code_bound.  Requires M % m == 0, N % n == 0, (N/n) % 8 == 0,
 * K % 128 == 0.  d_ws: DEVICE, >= int8_gemm_workspace bytes, 256-byte aligned; it holds a status word that
 * fmm_device_status reads.  Asynchronous on the stream.
 * int8_gemm_materialised: the same operator with every per-group block product written to memory (pack, encode,
 * grouped block products on bf16 copies of the integers with fp32 accumulators, grouped decode) — an independent
 * implementation of the same bits, twice as slow at layer sizes and with a workspace of R * K/128 fp32 blocks; s == NULL runs the classical algorithm through that pipeline.                                       */
fmm_status int8_gemm(const fmm_scheme* s, int code_bound, const int8_t* d_cA, const float* d_dA,
                     const int8_t* d_cB, const float* d_dB, int64_t M, int64_t K, int64_t N, int output, void* d_C,
                     int64_t ldc, void* d_ws, size_t ws_bytes, void* cuda_stream);
size_t int8_gemm_materialised_workspace(const fmm_scheme* s, int64_t M, int64_t K, int64_t N);
fmm_status int8_gemm_materialised(const fmm_scheme* s, int code_bound, const int8_t* d_cA, const float* d_dA,
                                  const int8_t* d_cB, const float* d_dB, int64_t M, int64_t K, int64_t N, int output,
                                  void* d_C, int64_t ldc, void* d_ws, size_t ws_bytes, void* cuda_stream);

/* ---- Full-range codes with an overflow correction (Section 4.3, Eq. 2; certificate in Appendix D) --------
 *
 * At code bound 127 the block sums of codes reach L_A * 127 (508 for two-level Strassen) and no longer fit the
 * multiplier's range.  Each is split exactly, X = X0 + 256 R with R = floor((X + 128) / 256) and X0 in
 * [-128, 127], and every block product is rebuilt from the four products of Eq. 2,
 *     Ahat Bhat = A0 B0 + 256 (R_A B0 + A0 R_B) + 256^2 R_A R_B,
 * here as one contraction over rows [A0 | 256 R_A | A0 | 256 R_A] and [B0 | B0 | 256 R_B | 256 R_B] (all entries
 * exact in bf16).  Same operands, layouts, requirements and output as int8_gemm at code bound 127; the result is
 * bit-identical to int8_gemm(NULL, 127, ...).  s must not be NULL.
 *
 * scheme_certificate_corrected: cert[4] (HOST, may be NULL) = {largest block sum L*127, largest |R|, bound
 * h (128 + 256 |R|max)^2 on the summed magnitudes inside one rebuilt product, L_W times that}.  Returns 1 when
 * the coefficients are integers, the third value is below 2^24 (fp32 accumulators), the fourth below 2^31 (int32
 * combination) and k * h == 128; int8_gemm_corrected returns FMM_ERR_CERTIFICATE otherwise.               */
int scheme_certificate_corrected(const fmm_scheme* s, int h, double cert[4]);
size_t int8_gemm_corrected_workspace(const fmm_scheme* s, int64_t M, int64_t K, int64_t N);
fmm_status int8_gemm_corrected(const fmm_scheme* s, const int8_t* d_cA, const float* d_dA, const int8_t* d_cB,
                               const float* d_dB, int64_t M, int64_t K, int64_t N, int output, void* d_C, int64_t ldc,
                               void* d_ws, size_t ws_bytes, void* cuda_stream);

/* The control of the row-pair test that BREAKS condition (iii) of Proposition 1 (Section 4.2): scales on fine groups
 * of h = call / k inner indices (one per block column of a call) while a call of the algorithm spans `call` indices.
 * The operands are quantised here (rows of d_A and of d_B, the latter in the weight layout [N][K]; d = max|x| /
 * code_bound per row and fine group, 1 if all zero, codes rounded to nearest even).  A block sum then mixes codes
 * with different scales: it is formed of the dequantised values code * scale (fp32 chain, ascending block order) and
 * rounded again with ONE scale per block sum and call, s = max|x| / second_bound (a reading: the paper names neither
 * the rule nor the bound of this second rounding; this is its quantiser's rule).  Products of the new codes are exact
 * integers, rescaled (P * sA) * sB and combined with w in fp32, ascending r within a call, calls ascending; one
 * rounding to `output`.  Because a block sum's largest magnitude depends on every row it reads, changing one token
 * row can move every output row: the paper counts all 496 pairs.  A demonstration on tiles (M * K, N * K < 2^31),
 * plain kernels, not a fast path.  d_A [M][lda], d_B [N][ldb]: DEVICE fp32; d_C: DEVICE [M][ldc] of `output`
 * (FMM_F32 / FMM_BF16).  Requires M % m == 0, N % n == 0, call % k == 0, K % call == 0.  Copies the coefficients to the
 * workspace and synchronises the stream once before enqueueing its kernels.                                      */
size_t int8_finegroup_control_workspace(const fmm_scheme* s, int64_t M, int64_t K, int64_t N, int call);
fmm_status int8_finegroup_control(const fmm_scheme* s, int code_bound, int second_bound, const float* d_A, int64_t lda,
                                  const float* d_B, int64_t ldb, int64_t M, int64_t K, int64_t N, int call, int output,
                                  void* d_C, int64_t ldc, void* d_ws, size_t ws_bytes, void* cuda_stream);

/* Randomised Hadamard rotation of the inner dimension (Appendix B, "A rotation, other summation orders and repeated
 * runs": A -> A H, B -> H^T B with H orthogonal leaves A B unchanged and changes what a fast algorithm's block sums
 * round).  A pre-pass outside scheme_gemm: rotate both operands with the same h and signs, then call any product.
 *     Y[t, :] = rnd_storage( (X[t, :] * signs) . blockdiag(H_h, ..., H_h) / sqrt(h) ),
 * H_h Sylvester's Hadamard matrix of order h (H[i][j] = (-1)^popcount(i & j)).  Arithmetic: the fast Walsh-Hadamard
 * recursion in fp32 (strides ascending), one multiplication by fl(1/sqrt(h)), one rounding to `storage`.
 * dX, dY: DEVICE [rows][ld*] of `storage` (FMM_F32 or FMM_BF16), the inner dimension contiguous — A as stored, B in
 * its [N, K] layout (rows = N); 16-byte aligned, ld* >= K and a multiple of 16 bytes; dY == dX rotates in place,
 * any other overlap is undefined.  d_signs: DEVICE, K entries of +1 / -1 (only the sign is read), 16-byte aligned,
 * or NULL for all +1.  h: a power of two, 2 <= h <= 1024, dividing K (K < 2^31).  The caller owns every buffer; the
 * call only enqueues one kernel on `cuda_stream` (the current device's).  FMM_ERR_ARG: null operand;
 * FMM_ERR_DTYPE: storage; FMM_ERR_SHAPE: sizes, divisibility or alignment (nothing is launched).             */
fmm_status hadamard_rotate(int storage, const void* dX, int64_t ldx, int64_t rows, int64_t K, int h,
                           const signed char* d_signs, void* dY, int64_t ldy, void* cuda_stream);

/* The repair rules of Appendix C ("The repair rules").
 *
 * Rule 1, row scale.  row_pow2_scale: for every row x_t of X (rows x K, `storage` FMM_F32 / FMM_BF16, DEVICE, ldx >= K)
 * d_scale[t] = 2^ceil(log2(max(RMS(x_t), 1e-3))) (DEVICE fp32 [rows]; RMS over the full row, sum of squares in fp64)
 * and Y[t, :] = X[t, :] / d_scale[t] (exact: a power of two; dY may equal dX).  row_unscale: C[t, :] *= d_scale[t] in
 * place (C rows x N of `output`, DEVICE, ldc >= N) — applied to the product of the scaled rows it restores the scale
 * of every output row; the multiplication commutes with the rounding to `output`, so it may follow scheme_gemm.
 *
 * Rule 2, joint rounding of the weight's block sums (model schedule only: d->scale_mode == 3, product FMM_E4M3, else
 * FMM_ERR_DTYPE).  scheme_joint_round_weights fills the weight side of a scheme_gemm workspace — the e4m3 codes of
 * the R block sums of B and their 128 x 128 block scales — and a following scheme_gemm with FMM_FLAG_REUSE_BHAT on
 * the same descriptor and workspace multiplies with them.  Per position, every code starts at the nearer of the two
 * e4m3 codes whose decoded values bracket the block sum's bf16 value (the code the plain schedule gives) and, in
 * sweeps over r = 1..R, is switched to the other one when that lowers e^T H e, e_r = decoded - bf16 value,
 * H_rs = <w_r, w_s> <u_r, u_s>; fp32 arithmetic: (He)_r an FMA chain over s ascending, the change
 * fma(delta^2, H_rr, 2 delta (He)_r); a sweep without a switch ends the search, at most max_sweeps (the paper: 12;
 * 0 gives the plain codes).  dB and d exactly as for scheme_gemm; d_ws: DEVICE, >= scheme_gemm_workspace bytes.
 * A weight-only pass: no activations enter.                                                                     */
fmm_status row_pow2_scale(int storage, const void* dX, int64_t ldx, int64_t rows, int64_t K, float* d_scale,
                          void* dY, int64_t ldy, void* cuda_stream);
fmm_status row_unscale(int output, void* dC, int64_t ldc, int64_t rows, int64_t N, const float* d_scale,
                       void* cuda_stream);
fmm_status scheme_joint_round_weights(const fmm_scheme* s, const fmm_gemm_desc* d, const void* dB, int max_sweeps,
                                      void* d_ws, size_t ws_bytes, void* cuda_stream);

const char* fmm_status_string(fmm_status st);

/* Number of kernels this library has launched in this process (for benchmarks' accounting). */
int64_t fmm_launch_count(void);

/* Phase timing.  While enabled, every device call brackets each step of the path with CUDA events on
 * the caller's stream (events only; no synchronisation, no change to the kernels).  Phases:
 *   0 encode A   1 encode B (incl. the transpose of a K x N operand)   2 block products (scheme)
 *   3 decode (+ error reduction)   4 block products of classical_gemm   5 everything else.
 * fmm_profile_collect synchronises the recorded events, adds their durations (milliseconds) to ms[8]
 * and the number of bracketed regions to count[8] (HOST arrays, overwritten), and clears the record. */
void fmm_profile_enable(int on);
fmm_status fmm_profile_collect(double ms[8], int64_t count[8]);

#ifdef __cplusplus
}
#endif
#endif /* FMM_B200_H */
