// Launch wrappers of the streaming (HBM-bound) kernels and of the tensor-core block products.
#pragma once
#include <cuda_runtime.h>

#include "fmm_internal.h"

// Device-resident status word at the start of every workspace.
struct DeviceStatus {
  int code;       // 0 ok, FMM_ERR_TIMEOUT when a bounded wait expired
  int where;      // which wait gave up (role id * 16 + barrier kind), for diagnosis
  int pad[62];
};

int64_t& fmm_launch_counter();

// Programmatic dependent launch: a kernel launched with launch_dependent may begin (prologue: barrier set-up,
// TMEM allocation, table loads) while the previous kernel of the same stream drains; it must execute
// grid_dependency_wait() before it touches anything that kernel wrote.  Kernels that may be followed by such a launch
// call grid_launch_dependents() early.  Both are no-ops when the launch carries no programmatic dependency.

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per (kernel, device): `done_mask` is the caller's static word for
// one kernel, bit d set once device d has been configured (devices beyond 63 are configured on every call).
template <typename Kernel>
cudaError_t fmm_allow_dynamic_smem(Kernel kernel, int bytes, unsigned long long* done_mask) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 64 && (*done_mask >> dev) & 1ull) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && dev < 64) *done_mask |= 1ull << dev;
  return e;
}
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// Joint rounding of the weight's block sums under the model schedule (Appendix C, "The repair rules"): X, the grid and
// d_tab as for launch_encode (the weight read K-major); amax_bits [R][ceil(br/128)][ceil(bc/128)] from the amax pass of
// the model schedule; d_H: R x R fp32, H_rs = <w_r, w_s> <u_r, u_s>; writes the e4m3 codes to out (R blocks [br][bc],
// out_stride elements apart) and the scales to scale_out (laid out like amax_bits).
cudaError_t launch_joint_round(int storage, const void* X, int64_t ldx, int gr, int gc, int64_t br, int64_t bc,
                               const CoefTable* d_tab, const float* d_H, const unsigned* amax_bits, float* scale_out,
                               void* out, int64_t out_stride, int max_sweeps, cudaStream_t st);

// X: source matrix (storage dtype), rows x cols with leading dimension ldx, split into a gr x gc grid of
// br x bc blocks.  out: R blocks [br][bc] in the product dtype, out_stride elements apart.  With amax_only the kernel only accumulates
// max|block sum| per product into amax_bits[R] (fp32 bit patterns of non-negative values).
// With use_scale == 1, scale[r] is derived from amax_bits[r] (2^ceil(log2(amax/448)), 1 if amax==0),
// written to scale[R] and divided out before rounding.  With use_scale == 2 there is one scale per row of every
// block sum: amax_bits and scale are [R][br]; scale = amax / 448 in fp32 (1 for an all-zero row).  use_scale == 3 (model
// schedule): one scale per 128 consecutive entries of a row, see EncodeOperand::scale_rows.
// storage may also be FMM_E4M3 with product FMM_E4M3 (use_scale 0 or 1): the source holds codes, sixteen per vector.
// h_tab = host copy of the same table (its list lengths size the kernel's shared memory).
cudaError_t launch_encode(int storage, int product, const void* X, int64_t ldx, int gr, int gc, int64_t br,
                          int64_t bc, const CoefTable* d_tab, const CoefTable* h_tab, void* out, int64_t out_stride,
                          unsigned* amax_bits, float* scale, bool amax_only, int use_scale, cudaStream_t st);

// The same decisions for a whole operand taken as one block with coefficient 1 (the classical control): rows x cols
// of `storage` -> `product` dtype, mode 0 / 1 / 2 as use_scale above (amax_bits, scale: one word, or one per row).
cudaError_t launch_quantize_plain(int storage, int product, const void* X, int64_t ldx, int64_t rows, int64_t cols,
                                  void* out, unsigned* amax_bits, float* scale, bool amax_only, int mode, int scale_rows,
                                  int bf16_first, cudaStream_t st);

// Two operands in one launch (A and B of one product, encoded side by side); b may be null.  Fields as the arguments
// of launch_encode.
struct EncodeOperand {
  const void* X; int64_t ldx; int gr, gc; int64_t br, bc;
  const CoefTable* d_tab; const CoefTable* h_tab; void* out; int64_t out_stride; unsigned* amax_bits; float* scale;
  int scale_rows;   // use_scale 3 only: rows sharing a scale (1 or 128); amax_bits / scale are [R][ceil(br/scale_rows)][ceil(bc/128)]
  int bf16_first;   // use_scale 3 only: round the block sum to bf16 before it is quantised
  const float* pre_scale = nullptr;   // use_scale 1 only: DEVICE, one float; the source's codes are in units of it and
                                      // scale[r] receives (this pass's scale) * pre_scale[0]
};
cudaError_t launch_encode_pair(int storage, int product, const EncodeOperand& a, const EncodeOperand* b, bool amax_only,
                               int use_scale, cudaStream_t st);

// One operand of an encode launch.  A launch carries up to two (A and B of one product): blocks [0, a.blocks) work
// on the first, the rest on the second, so both operands are encoded side by side without a second stream.
struct EncodeJob {
  const void* X; int64_t ldx; int gc; int64_t br, bc;
  const CoefTable* tab; void* out; unsigned* amax_bits; float* scale_out;
  int tiles_per_block; int64_t rstride; int stream_out; int blocks;
  int scale_rows;    // use_scale 3: rows of a block sum that share a scale (1: the input's 1 x 128 scales; 128: the weight's 128 x 128)
  int bf16_first;    // use_scale 3: the block sum is first rounded to bf16 (weights are stored in bf16 before they are quantised)
  const float* pre_scale;   // use_scale 1: the source holds codes in units of *pre_scale (an outer level's scale); the
                            // scale written out is the product of the two.  Null: 1.
};

// The two jobs of a bf16 -> bf16 encode without scales whose work is spread over `nblocks` blocks of 256 threads that
// exist already (the streaming groups of the fused sweep kernel) instead of a grid of its own: blocks [0, ja->blocks)
// take operand a, the next jb->blocks take b, in proportion to their sizes.  *smem_bytes: shared memory one block
// needs; *dense: every list reads the four cells of a 2 x 2 grid in one order (the register-chain variant applies).
// False if the tables do not fit this path (more than four cells per grid, positions beyond 32-bit indexing).
bool fmm_encode_jobs_for_blocks(const EncodeOperand& a, const EncodeOperand& b, int nblocks, EncodeJob* ja, EncodeJob* jb,
                                size_t* smem_bytes, int* dense);

// Bt[N x K] = B[K x N]^T for 2- or 4-byte elements.
cudaError_t launch_transpose(int elem_bytes, const void* B, int64_t ldb, int64_t K, int64_t N, void* Bt,
                             cudaStream_t st);

// Decode (+ optional error reduction).  prod: R blocks [bm][bn] of prod_dtype (FMM_F32 or FMM_BF16), prod_stride elements apart.  If C != nullptr the rounded result is stored
// (dtype `output`, leading dimension ldc).  If cstar32 != nullptr the per-block partial sums of
// (rnd_O(c) - C*)^2 are written to partials[gridDim.x] and *n_partials receives gridDim.x.
// d_tab is the CELL-MAJOR decode table (list c = the (r, w) pairs feeding C block c, ascending r); R is the
// number of products; h_tab is the host copy of d_tab (its list lengths size the shared memory).
// gauges > 1 (error reduction only, 1 / 2 / 4): the table holds that many equivalent algorithms, list c feeding C block
// c / gauges of algorithm c % gauges with product indices offset by the algorithm; partials are [algorithm][block].
cudaError_t launch_decode(int output, const void* prod, int prod_dtype, int64_t prod_stride, const CoefTable* d_tab,
                          const CoefTable* h_tab, int R, const float* sA, const float* sB, int m, int n, int64_t bm,
                          int64_t bn, void* C, int64_t ldc, const float* cstar32, double* partials, int* n_partials,
                          cudaStream_t st, int gauges = 1);
int decode_grid(int64_t bm, int64_t bn);

// out[0] = sum of partials[0..n) in a fixed order (single block).
// out[b] = sum of partials[b*n .. b*n+n), b < count
cudaError_t launch_sum_partials(const double* partials, int n, double* out, cudaStream_t st, int count = 1);

// C*(fp64) -> fp32 copy, and partial sums of C*^2.
cudaError_t launch_cstar_prepare(const double* cstar, int64_t count, float* cstar32, double* partials,
                                 int* n_partials, cudaStream_t st);
// partial sums of (C - C*)^2 and of C*^2 (two arrays of n_partials doubles, the second may be null).
cudaError_t launch_frob_err(int output, const void* C, int64_t ldc, const double* cstar, int64_t M, int64_t N,
                            double* part_err, double* part_ref, int* n_partials, cudaStream_t st);
int stream_grid(int64_t count);
// same kernel, caller-chosen number of blocks (= number of partial sums written to each array)
cudaError_t launch_frob_err_fixed_grid(int output, const void* C, int64_t ldc, const double* cstar, int64_t M,
                                       int64_t N, double* part_err, double* part_ref, int grid, cudaStream_t st);

cudaError_t launch_exact_f64(int storage, const void* A, int64_t lda, const void* B, int64_t ldb,
                             int b_weight_layout, int64_t M, int64_t K, int64_t N, double* C, cudaStream_t st);

// Batched block products on tcgen05 tensor cores:
//   D_r[rows_a x rows_b] = A_r[rows_a x kdim] * B_r[rows_b x kdim]^T   (both operands K-major)
// product dtype bf16 or e4m3, fp32 accumulation in TMEM.
//   out_mode 0: store fp32 to out (float*, row stride ldo, batch stride ldo_batch elements)
//   out_mode 1: store rnd(alpha * acc) as `output` dtype (alpha = sA[0]*sB[0] when given, else 1).
struct BlockProductArgs {
  int product;               // FMM_BF16 / FMM_E4M3
  const void* A; int64_t lda; int64_t a_batch;   // elements
  const void* B; int64_t ldb; int64_t b_batch;
  int64_t rows_a, rows_b, kdim; int batches;
  int groups;                // > 1: each batch entry holds `groups` row groups of rows_a (rows_b) rows; product (r, g)
                             // multiplies group g of A_r with group g of B_r and lands at out + (r*groups + g)*o_batch
  void* out; int64_t ldo; int64_t o_batch; int out_mode; int output;
  const float* sA; const float* sB;
  // optional per-row / per-column factors applied to the fp32 accumulator before it is stored:
  // out[r][row][col] = (acc * row_scale[r*rs_batch + row]) * col_scale[r*cs_batch + col]   (null: none)
  const float* row_scale; const float* col_scale; int64_t rs_batch, cs_batch;
  DeviceStatus* status;
  int selftest_no_producer;            // 1: the producer issues no copies (failure-reporting self-test)
  unsigned long long wait_limit_ns;    // 0: default (2 s)
};
fmm_status launch_block_products(const BlockProductArgs& a, cudaStream_t st);

// One launch of a pipelined gauge sweep (bf16 storage and products, no scales, batches of four or eight one-level
// algorithms): the block products of one batch on the tensor cores and, in the same CTAs, the error-only decode of the
// batch before it and the encode of the batch after it.  Each of the three parts may be absent (pipeline head and tail).
struct FusedSweepArgs {
  int groups;                   // streaming groups (of eight warps) per CTA: 1 or 2
  int output;                   // FMM_F32 / FMM_BF16: the dtype the decoded result is rounded to before the error is taken
  int have_products;            // products: operands, batch count and output as for launch_block_products (bf16, out_mode 0)
  BlockProductArgs products;
  int dec_gauges;               // 0: no decode; 4 / 8: algorithms in the decoded batch
  const float* dec_prod; int64_t dec_prod_stride; const CoefTable* dec_tab; int dec_RB;
  int n; int64_t bm, bn;        // C grid columns and block size
  const float* cstar32;
  double* partials;             // [dec_gauges][fused_sweep_blocks(groups)] error partials of the decoded batch
  int have_encode;              // encode: the two operands as for launch_encode_pair (bf16 -> bf16, 2 x 2 grids)
  EncodeOperand enc_a, enc_b;
};
int fused_sweep_blocks(int groups);   // number of streaming blocks (= partial sums per algorithm) of a fused launch
fmm_status launch_fused_sweep(const FusedSweepArgs& f, cudaStream_t st);

// Batched block products under the model schedule (scale mode 3): e4m3 codes A [batches][rows_a][kdim] (K-major, lda) and
// B [batches][rows_b][kdim]; G = ceil(kdim / 128) groups; scales sA [batches][rows_a][G], sB [batches][ceil(rows_b/128)][G];
// out [batches][rows_a][ldo] of `output` (FMM_F32 / FMM_BF16), o_batch elements apart.
struct Fp8GroupArgs {
  const void* A; int64_t lda, a_batch; const void* B; int64_t ldb, b_batch;
  int64_t rows_a, rows_b, kdim; int batches;
  void* out; int64_t ldo, o_batch; int output;
  const float* sA; const float* sB;
  DeviceStatus* status;
};
fmm_status launch_fp8_group_gemm(const Fp8GroupArgs& a, cudaStream_t st);

// The group-scaled int8 operator in one kernel (tcgen05 kind::i8, int32 accumulators in TMEM, rescale in the epilogue):
// cA [M][K], cB [N][K] int8 codes (K % 128 == 0, rows 16-byte aligned), dAt [K/128][M] and dBt [K/128][N] fp32 scales,
// C [M][ldc] of `output` (FMM_F32 / FMM_BF16).  N must be a multiple of 4.
fmm_status launch_int8_group_gemm(const int8_t* cA, const int8_t* cB, const float* dAt, const float* dBt, int64_t M,
                                  int64_t K, int64_t N, int output, void* C, int64_t ldc, DeviceStatus* status, cudaStream_t st);

// The certified int8 realisation in one kernel (tcgen05 kind::i8 block products of the int8 block sums, integer decode
// and group rescale in the epilogue).  Ahat: int8 [ceil(R / per)][G * bm][128], per = 128 / h products side by side in a
// row (product r at byte (r % per) * h of row g * bm + p of slab r / per); Bhat likewise with bn.  d_owned: [4][4], the blocks of C
// (i * n + j, or -1) that each of the four decode warps of a TMEM lane quarter combines; d_entries: decode lists ordered
// by (decode warp, pass, owned block, r): (TMEM column of the product inside its pass, integer w); d_pass_off: first
// entry of every such list and one terminal element; passes as int8_certified_passes() gives them.  dAt [G][M],
// dBt [G][N]: scales, group-major.
struct Int8CertArgs {
  const int8_t* Ahat; const int8_t* Bhat;
  int m, n, R, h; int64_t bm, bn; int G; int64_t M, N;
  const float* dAt; const float* dBt;
  const int2* d_entries; const int* d_pass_off; const int* d_owned; int n_entries;
  int output; void* C; int64_t ldc; DeviceStatus* status;
};
void int8_certified_passes(int R, int per, int* passes, int* pass_len);
int int8_certified_tile_columns();   // columns of a tile per block of C = TMEM columns of one product
int int8_certified_decode_warps();   // decode warps per TMEM lane quarter (each owns 16 / that many blocks of C)
fmm_status launch_int8_certified(const Int8CertArgs& a, cudaStream_t st);

// Phase timing (see fmm_profile_enable): RAII bracket of a region of the caller's stream.
struct ProfScope {
  ProfScope(int kind, cudaStream_t st);
  ~ProfScope();
  int slot;
  cudaStream_t st;
};
