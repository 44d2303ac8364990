// Streaming kernels of the scheme GEMM: encode (block sums -> product dtype), transpose,
// decode (+ error reduction), Frobenius error, fp64 reference.  All are HBM-bound passes;
// each thread moves 16-byte vectors and the grid covers the data once.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include <algorithm>
#include <cmath>
#include <cstdlib>

#include "kernels_stream.cuh"
#include "stream_bodies.cuh"

int64_t& fmm_launch_counter() {
  static int64_t c = 0;
  return c;
}


namespace {


template <typename SrcT, typename DstT, bool kAmaxOnly, int kEncSplit, bool kM3, bool kDense = false>
__global__ void __launch_bounds__(kEncThreads)
encode_kernel(const EncodeJob job_a, const EncodeJob job_b, int use_scale) {
  grid_launch_dependents();   // the block products may set up while this grid drains; they wait before reading
  extern __shared__ __align__(16) unsigned char smem_raw[];
  encode_body<SrcT, DstT, kAmaxOnly, kEncSplit, kM3, kDense>(StreamRole{(int)threadIdx.x, (int)blockIdx.x, (int)gridDim.x, 0},
                                                             smem_raw, job_a, job_b, use_scale);
}


// ------------------------------------------------------------------------------------------
// Plain quantisation of one operand (the classical control: one cell, coefficient 1): rows x cols of SrcT ->
// DstT with no scale (mode 0), one power-of-two scale per tensor (mode 1) or one scale per row (mode 2), the same
// decisions as encode_kernel takes for a 1 x 1 grid.  A pure stream: each thread keeps four independent 16-byte
// loads in flight, no shared memory.
// ------------------------------------------------------------------------------------------
template <typename SrcT, typename DstT, bool kAmaxOnly>
__global__ void __launch_bounds__(256)
quantize_plain_kernel(const SrcT* __restrict__ X, int64_t ldx, int64_t rows, int64_t cols, DstT* __restrict__ out,
                      unsigned* __restrict__ amax_bits, float* __restrict__ scale_out, int mode, int scale_rows,
                      int bf16_first) {
  constexpr int VE = Vec16<SrcT>::kElems;
  constexpr int NP = VE / 2;
  constexpr int kU = 4;
  __shared__ unsigned s_amax;
  const int64_t vec_per_row = cols / VE;
  const int64_t nvec = rows * vec_per_row;
  const int64_t stride = (int64_t)gridDim.x * 256;
  float s = 1.0f, inv = 1.0f;
  bool use_mul = true;
  if (!kAmaxOnly && mode == 1) {
    s = pow2_scale_448(__uint_as_float(amax_bits[0]));
    inv = 1.0f / s;
    use_mul = isfinite(inv) && inv * s == 1.0f && fabsf(inv) >= 1.17549435e-38f;
    if (blockIdx.x == 0 && threadIdx.x == 0 && scale_out) scale_out[0] = s;
  }
  if (kAmaxOnly && threadIdx.x == 0) s_amax = 0u;
  if (kAmaxOnly) __syncthreads();
  float tmax = 0.0f;
  for (int64_t base = (int64_t)blockIdx.x * 256 + threadIdx.x; base < nvec; base += kU * stride) {
    uint4 raw[kU];
    int64_t row[kU];
    int col[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int64_t i = base + u * stride;
      const bool on = i < nvec;
      row[u] = on ? i / vec_per_row : 0;
      col[u] = on ? (int)(i - row[u] * vec_per_row) * VE : 0;
      raw[u] = on ? __ldcs(reinterpret_cast<const uint4*>(X + row[u] * ldx + col[u])) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const bool on = base + u * stride < nvec;
      float2 v[NP];
      Vec16<SrcT>::unpack(raw[u], v);
      // model schedule (mode 3): one scale per 128 consecutive entries of a row, shared by scale_rows rows
      const int64_t sidx3 = (row[u] / scale_rows) * ((cols + 127) >> 7) + (col[u] >> 7);
      if (mode == 3 && bf16_first) {
#pragma unroll
        for (int i = 0; i < NP; ++i) {
          v[i].x = __bfloat162float(__float2bfloat16_rn(v[i].x));
          v[i].y = __bfloat162float(__float2bfloat16_rn(v[i].y));
        }
      }
      if (kAmaxOnly) {
        float a = 0.0f;
#pragma unroll
        for (int i = 0; i < NP; ++i) a = fmaxf(a, fmaxf(fabsf(v[i].x), fabsf(v[i].y)));
        if (mode == 3) {
          constexpr int kLanesPerGroup = 128 / VE;
          if ((vec_per_row & 31) == 0) {   // a warp's 32 consecutive vectors lie in one row
            const unsigned mask = kLanesPerGroup == 32 ? 0xffffffffu : (0xffffu << (threadIdx.x & 16));
            const unsigned wmax = __reduce_max_sync(mask, on ? __float_as_uint(a) : 0u);
            if ((threadIdx.x & (kLanesPerGroup - 1)) == 0 && wmax != 0u) atomicMax(&amax_bits[sidx3], wmax);
          } else if (on && a > 0.0f) {
            atomicMax(&amax_bits[sidx3], __float_as_uint(a));
          }
        } else if (mode == 2) {
          if ((vec_per_row & 31) == 0) {   // a warp's 32 consecutive vectors lie in one row
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
            if ((threadIdx.x & 31) == 0 && on && a > 0.0f) atomicMax(&amax_bits[row[u]], __float_as_uint(a));
          } else if (on && a > 0.0f) {
            atomicMax(&amax_bits[row[u]], __float_as_uint(a));
          }
        } else {
          tmax = fmaxf(tmax, a);
        }
      } else if (on) {
        if (mode == 3) {
          const float amax = __uint_as_float(amax_bits[sidx3]);
          const float sc = amax > 0.0f ? __fdiv_rn(amax, 448.0f) : 1.0f;
          if constexpr (sizeof(DstT) == 1) {
            divide_for_e4m3<NP>(v, sc);
          } else {
#pragma unroll
            for (int i = 0; i < NP; ++i) { v[i].x = __fdiv_rn(v[i].x, sc); v[i].y = __fdiv_rn(v[i].y, sc); }
          }
          if ((col[u] & 127) == 0 && (row[u] % scale_rows) == 0 && scale_out) scale_out[sidx3] = sc;
        } else if (mode == 2) {
          const float amax = __uint_as_float(amax_bits[row[u]]);
          const float sc = amax > 0.0f ? __fdiv_rn(amax, 448.0f) : 1.0f;
          if constexpr (sizeof(DstT) == 1) {
            divide_for_e4m3<NP>(v, sc);
          } else {
#pragma unroll
            for (int i = 0; i < NP; ++i) { v[i].x = __fdiv_rn(v[i].x, sc); v[i].y = __fdiv_rn(v[i].y, sc); }
          }
          if (col[u] == 0 && scale_out) scale_out[row[u]] = sc;
        } else if (mode == 1) {
          if (use_mul) {
#pragma unroll
            for (int i = 0; i < NP; ++i) { v[i].x *= inv; v[i].y *= inv; }
          } else {
#pragma unroll
            for (int i = 0; i < NP; ++i) { v[i].x = __fdiv_rn(v[i].x, s); v[i].y = __fdiv_rn(v[i].y, s); }
          }
        }
        store_vec<NP>(out + row[u] * cols + col[u], v, true);
      }
    }
  }
  if (kAmaxOnly && mode != 2 && mode != 3) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
    if ((threadIdx.x & 31) == 0 && tmax > 0.0f) atomicMax(&s_amax, __float_as_uint(tmax));
    __syncthreads();
    if (threadIdx.x == 0 && s_amax != 0u) atomicMax(&amax_bits[0], s_amax);
  }
}

template <typename SrcT, typename DstT>
static cudaError_t launch_quantize_plain_t(const void* X, int64_t ldx, int64_t rows, int64_t cols, void* out,
                                           unsigned* amax_bits, float* scale, bool amax_only, int mode, int scale_rows,
                                           int bf16_first, cudaStream_t st) {
  constexpr int VE = Vec16<SrcT>::kElems;
  const int64_t nvec = rows * (cols / VE);
  if (nvec == 0) return cudaSuccess;
  const int grid = (int)std::min<int64_t>((nvec + 256 * 4 - 1) / (256 * 4), 148 * 16);
  if (amax_only)
    quantize_plain_kernel<SrcT, DstT, true><<<grid, 256, 0, st>>>((const SrcT*)X, ldx, rows, cols, (DstT*)out, amax_bits, scale, mode, scale_rows > 0 ? scale_rows : 1, bf16_first);
  else
    quantize_plain_kernel<SrcT, DstT, false><<<grid, 256, 0, st>>>((const SrcT*)X, ldx, rows, cols, (DstT*)out, amax_bits, scale, mode, scale_rows > 0 ? scale_rows : 1, bf16_first);
  ++fmm_launch_counter();
  return cudaGetLastError();
}

// Blocks of a streaming pass: enough to fill the machine about four times over, each block walking a
// contiguous run of tiles so that its table set-up is paid once.
static void split_tiles(int64_t tiles, int* grid, int* tiles_per_block) {
  const int64_t target = 148 * 4;
  const int64_t tpb = (tiles + target - 1) / target;
  *tiles_per_block = (int)(tpb < 1 ? 1 : tpb);
  *grid = (int)((tiles + *tiles_per_block - 1) / *tiles_per_block);
}

static int padded_entries(const CoefTable& t) { return t.off[t.R]; }   // lists arrive padded from the host

// Host description of one operand of an encode launch (see launch_encode_pair).
template <typename SrcT, typename DstT, int kSplit>
static bool make_job(const EncodeOperand& o, EncodeJob* j, size_t* smem) {
  constexpr int VE = Vec16<SrcT>::kElems;
  constexpr int kEncPos = kEncThreads / kSplit;
  const int padded = padded_entries(*o.h_tab);
  *smem = ((sizeof(EncSmemHead) + (size_t)padded * 8 + 15) / 16) * 16 + 2 * (size_t)(o.gr * o.gc + 1) * kEncPos * 16;
  const int64_t vecs = o.br * (o.bc / VE);
  if (vecs + kEncThreads * 8 >= (int64_t)1 << 31) return false;   // kernels index positions in 32 bits
  int grid = 0, tpb = 1;
  if (vecs > 0) split_tiles((vecs + kEncPos - 1) / kEncPos, &grid, &tpb);
  // outputs larger than the part of L2 that keeps shared data (~60 MB) will have left it before they are read
  int stream_out = (int64_t)o.h_tab->R * o.out_stride * (int64_t)sizeof(DstT) > ((int64_t)48 << 20) ? 1 : 0;
  *j = EncodeJob{o.X, o.ldx, o.gc, o.br, o.bc, o.d_tab, o.out, o.amax_bits, o.scale, tpb, o.out_stride, stream_out, grid,
                 o.scale_rows > 0 ? o.scale_rows : 1, o.bf16_first, o.pre_scale};
  return true;
}

// every list of the table has exactly four entries over the four cells of the grid, in the same cell order
static bool dense_four_cells(const CoefTable& t);
}  // namespace

bool fmm_encode_jobs_for_blocks(const EncodeOperand& a, const EncodeOperand& b, int nblocks, EncodeJob* ja, EncodeJob* jb,
                                size_t* smem_bytes, int* dense) {
  constexpr int kSplit = 4, kEncPos = kEncThreads / kSplit, VE = 8;   // bf16 source: eight elements per vector
  if (nblocks < 2 || a.gr * a.gc > 4 || b.gr * b.gc > 4) return false;
  size_t sm_a = 0, sm_b = 0;
  if (!make_job<__nv_bfloat16, __nv_bfloat16, kSplit>(a, ja, &sm_a)) return false;
  if (!make_job<__nv_bfloat16, __nv_bfloat16, kSplit>(b, jb, &sm_b)) return false;
  const int64_t tiles_a = (a.br * (a.bc / VE) + kEncPos - 1) / kEncPos, tiles_b = (b.br * (b.bc / VE) + kEncPos - 1) / kEncPos;
  if (tiles_a < 1 || tiles_b < 1) return false;
  // blocks in proportion to the bytes each operand writes (tiles x products)
  const double wa = (double)tiles_a * a.h_tab->R, wb = (double)tiles_b * b.h_tab->R;
  int na = (int)(nblocks * wa / (wa + wb) + 0.5);
  na = std::min(std::max(na, 1), nblocks - 1);
  const int nb = nblocks - na;
  ja->tiles_per_block = (int)((tiles_a + na - 1) / na);
  ja->blocks = (int)((tiles_a + ja->tiles_per_block - 1) / ja->tiles_per_block);
  jb->tiles_per_block = (int)((tiles_b + nb - 1) / nb);
  jb->blocks = (int)((tiles_b + jb->tiles_per_block - 1) / jb->tiles_per_block);
  *smem_bytes = std::max(sm_a, sm_b);
  *dense = dense_four_cells(*a.h_tab) && dense_four_cells(*b.h_tab) ? 1 : 0;
  return true;
}

namespace {
static bool dense_four_cells(const CoefTable& t) {
  if (t.ncell != 4 || t.R < 1 || t.off[t.R] != 4 * t.R) return false;
  bool seen[4] = {false, false, false, false};
  for (int c = 0; c < 4; ++c) {
    if (t.cell[c] < 0 || t.cell[c] > 3 || seen[t.cell[c]]) return false;
    seen[t.cell[c]] = true;
  }
  for (int r = 0; r < t.R; ++r) {
    if (t.off[r] != 4 * r) return false;
    for (int c = 0; c < 4; ++c)
      if (t.cell[4 * r + c] != t.cell[c]) return false;
  }
  return true;
}

template <typename SrcT, typename DstT, bool kAmaxOnly, int kSplit, bool kM3, bool kDense = false>
static cudaError_t launch_encode_k(int grid, size_t smem, cudaStream_t st, const EncodeJob& ja, const EncodeJob& jb, int use_scale) {
  auto k = encode_kernel<SrcT, DstT, kAmaxOnly, kSplit, kM3, kDense>;
  static unsigned long long smem_ok = 0;   // per template instantiation, one bit per device
  cudaError_t e = fmm_allow_dynamic_smem(k, 200 * 1024, &smem_ok);
  if (e != cudaSuccess) return e;
  k<<<grid, kEncThreads, smem, st>>>(ja, jb, use_scale);
  return cudaSuccess;
}

template <typename SrcT, typename DstT, int kSplit>
cudaError_t launch_encode_t(const EncodeOperand& a, const EncodeOperand* b, bool amax_only, int use_scale, cudaStream_t st) {
  EncodeJob ja{}, jb{};
  size_t smem_a = 0, smem_b = 0;
  if (!make_job<SrcT, DstT, kSplit>(a, &ja, &smem_a)) return cudaErrorInvalidValue;
  if (b && !make_job<SrcT, DstT, kSplit>(*b, &jb, &smem_b)) return cudaErrorInvalidValue;
  const int grid = ja.blocks + jb.blocks;
  if (grid == 0) return cudaSuccess;
  const size_t smem = std::max(smem_a, smem_b);
  // the model schedule exists for e4m3 block sums of bf16 / fp32 sources only
  constexpr bool kCanM3 = sizeof(DstT) == 1 && sizeof(SrcT) > 1;
  if (use_scale == 3 && !kCanM3) return cudaErrorInvalidValue;
  cudaError_t e;
  if (use_scale == 3)
    e = amax_only ? launch_encode_k<SrcT, DstT, true, kSplit, kCanM3>(grid, smem, st, ja, jb, use_scale)
                  : launch_encode_k<SrcT, DstT, false, kSplit, kCanM3>(grid, smem, st, ja, jb, use_scale);
  else if (kSplit == 4 && dense_four_cells(*a.h_tab) && (b == nullptr || dense_four_cells(*b->h_tab)))
    e = amax_only ? launch_encode_k<SrcT, DstT, true, kSplit, false, true>(grid, smem, st, ja, jb, use_scale)
                  : launch_encode_k<SrcT, DstT, false, kSplit, false, true>(grid, smem, st, ja, jb, use_scale);
  else
    e = amax_only ? launch_encode_k<SrcT, DstT, true, kSplit, false>(grid, smem, st, ja, jb, use_scale)
                  : launch_encode_k<SrcT, DstT, false, kSplit, false>(grid, smem, st, ja, jb, use_scale);
  if (e != cudaSuccess) return e;
  ++fmm_launch_counter();
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// transpose (only when B is given K x N): 32 x 32 tiles through padded shared memory
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) transpose_kernel(const T* __restrict__ B, int64_t ldb, int64_t K, int64_t N,
                                                        T* __restrict__ Bt) {
  __shared__ T tile[32][33];
  const int64_t n0 = (int64_t)blockIdx.x * 32, k0 = (int64_t)blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int r = ty; r < 32; r += 8) {
    const int64_t kk = k0 + r, nn = n0 + tx;
    if (kk < K && nn < N) tile[r][tx] = B[kk * ldb + nn];
  }
  __syncthreads();
  for (int r = ty; r < 32; r += 8) {
    const int64_t nn = n0 + r, kk = k0 + tx;
    if (kk < K && nn < N) Bt[nn * K + kk] = tile[tx][r];
  }
}

// (the error-reducing variants are held to 64 registers: four blocks per SM, as many as their shared memory allows)
template <typename OutT, bool kStore, bool kErr, int kDecSplit, typename ProdT>
__global__ void __launch_bounds__(kDecThreads, (kErr && !kStore && kDecSplit == 4) ? 4 : 0)
decode_kernel(const ProdT* __restrict__ prod, const CoefTable* __restrict__ d_tab, int R,
              const float* __restrict__ sA, const float* __restrict__ sB, int n, int64_t bm, int64_t bn,
              OutT* __restrict__ C, int64_t ldc, const float* __restrict__ cstar32, int64_t ldcs,
              double* __restrict__ partials, int tiles_per_block, int64_t rstride, int gauges) {
  grid_dependency_wait();     // the products (and scales) come from the previous kernel of the stream
  extern __shared__ __align__(16) unsigned char smem_raw[];
  decode_body<OutT, kStore, kErr, kDecSplit, ProdT>(StreamRole{(int)threadIdx.x, (int)blockIdx.x, (int)gridDim.x, 0}, smem_raw, prod,
                                                    d_tab, R, sA, sB, n, bm, bn, C, ldc, cstar32, ldcs, partials,
                                                    tiles_per_block, rstride, gauges);
}


template <typename OutT, typename ProdT, int kGauges>
__global__ void __launch_bounds__(kDecThreads)
decode_batch_kernel(const ProdT* __restrict__ prod, const CoefTable* __restrict__ d_tab, int RB,
                    const float* __restrict__ sA, const float* __restrict__ sB, int n, int64_t bm, int64_t bn,
                    const float* __restrict__ cstar32, int64_t ldcs, double* __restrict__ partials,
                    int tiles_per_block, int64_t rstride) {
  grid_dependency_wait();
  __shared__ DecBatchSmem<kGauges> sm;
  decode_batch_body<OutT, ProdT, kGauges>(StreamRole{(int)threadIdx.x, (int)blockIdx.x, (int)gridDim.x, 0}, sm, prod, d_tab, RB, sA, sB, n,
                                          bm, bn, cstar32, ldcs, partials, tiles_per_block, rstride);
}


// ------------------------------------------------------------------------------------------
// block b sums partials[b * n .. b * n + n) into out[b]
__global__ void __launch_bounds__(256) sum_partials_kernel(const double* __restrict__ partials, int n,
                                                           double* __restrict__ out) {
  __shared__ double red[8];
  double v = 0.0;
  for (int i = threadIdx.x; i < n; i += 256) v += partials[(size_t)blockIdx.x * n + i];
  const double tot = block_sum_double(v, red);
  if (threadIdx.x == 0) out[blockIdx.x] = tot;
}

__global__ void __launch_bounds__(256) cstar_prepare_kernel(const double* __restrict__ cstar, int64_t count,
                                                            float* __restrict__ cstar32,
                                                            double* __restrict__ partials) {
  __shared__ double red[8];
  double s = 0.0;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < count; i += (int64_t)gridDim.x * 256) {
    const double v = cstar[i];
    cstar32[i] = (float)v;
    s += v * v;
  }
  const double tot = block_sum_double(s, red);
  if (threadIdx.x == 0) partials[blockIdx.x] = tot;
}

template <typename OutT>
__global__ void __launch_bounds__(256) frob_err_kernel(const OutT* __restrict__ C, int64_t ldc,
                                                       const double* __restrict__ cstar, int64_t M, int64_t N,
                                                       double* __restrict__ part_err, double* __restrict__ part_ref) {
  __shared__ double red[8];
  double e = 0.0, s = 0.0;
  const int64_t count = M * N;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < count; i += (int64_t)gridDim.x * 256) {
    const int64_t r = i / N, c = i - r * N;
    const double v = cstar[i];
    const double d = (double)(float)C[r * ldc + c] - v;
    e += d * d;
    s += v * v;
  }
  const double te = block_sum_double(e, red);
  if (threadIdx.x == 0) part_err[blockIdx.x] = te;
  if (part_ref != nullptr) {
    const double ts = block_sum_double(s, red);
    if (threadIdx.x == 0) part_ref[blockIdx.x] = ts;
  }
}

// ------------------------------------------------------------------------------------------
// fp64 reference product: 128 x 128 tile per block of 256 threads, 8 x 8 outputs per thread (rows ty + 16 a,
// columns tx + 16 b: a half-warp reads 16 consecutive doubles of the staged operands), inner index ascending,
// one fused multiply-add per term; operands converted to fp64 when they are staged.
// ------------------------------------------------------------------------------------------
constexpr int kExT = 128, kExK = 16;
template <typename T>
__global__ void __launch_bounds__(256) exact_f64_kernel(const T* __restrict__ A, int64_t lda,
                                                        const T* __restrict__ B, int64_t ldb, int b_weight,
                                                        int64_t M, int64_t K, int64_t N, double* __restrict__ C) {
  __shared__ double As[kExK][kExT];
  __shared__ double Bs[kExK][kExT];
  const int64_t m0 = (int64_t)blockIdx.y * kExT, n0 = (int64_t)blockIdx.x * kExT;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  double acc[8][8];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int b = 0; b < 8; ++b) acc[a][b] = 0.0;
  for (int64_t k0 = 0; k0 < K; k0 += kExK) {
    for (int i = threadIdx.x; i < kExT * kExK; i += 256) {
      {  // A tile: consecutive threads along the inner dimension
        const int kk = i & (kExK - 1), r = i >> 4;
        const int64_t row = m0 + r, t = k0 + kk;
        As[kk][r] = (row < M && t < K) ? (double)(float)A[row * lda + t] : 0.0;
      }
      if (b_weight) {
        const int kk = i & (kExK - 1), c = i >> 4;
        const int64_t col = n0 + c, t = k0 + kk;
        Bs[kk][c] = (col < N && t < K) ? (double)(float)B[col * ldb + t] : 0.0;
      } else {
        const int c = i & (kExT - 1), kk = i >> 7;
        const int64_t col = n0 + c, t = k0 + kk;
        Bs[kk][c] = (col < N && t < K) ? (double)(float)B[t * ldb + col] : 0.0;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kExK; ++kk) {
      double a[8], b[8];
#pragma unroll
      for (int x = 0; x < 8; ++x) { a[x] = As[kk][ty + 16 * x]; b[x] = Bs[kk][tx + 16 * x]; }
#pragma unroll
      for (int x = 0; x < 8; ++x)
#pragma unroll
        for (int y = 0; y < 8; ++y) acc[x][y] = fma(a[x], b[y], acc[x][y]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int x = 0; x < 8; ++x)
#pragma unroll
    for (int y = 0; y < 8; ++y) {
      const int64_t row = m0 + ty + 16 * x, col = n0 + tx + 16 * y;
      if (row < M && col < N) C[row * N + col] = acc[x][y];
    }
}

}  // namespace

cudaError_t launch_quantize_plain(int storage, int product, const void* X, int64_t ldx, int64_t rows, int64_t cols,
                                  void* out, unsigned* amax_bits, float* scale, bool amax_only, int mode, int scale_rows,
                                  int bf16_first, cudaStream_t st) {
  if (storage == FMM_F32 && product == FMM_BF16)
    return launch_quantize_plain_t<float, __nv_bfloat16>(X, ldx, rows, cols, out, amax_bits, scale, amax_only, mode, scale_rows, bf16_first, st);
  if (storage == FMM_BF16 && product == FMM_BF16)
    return launch_quantize_plain_t<__nv_bfloat16, __nv_bfloat16>(X, ldx, rows, cols, out, amax_bits, scale, amax_only, mode, scale_rows, bf16_first, st);
  if (storage == FMM_F32 && product == FMM_E4M3)
    return launch_quantize_plain_t<float, __nv_fp8_storage_t>(X, ldx, rows, cols, out, amax_bits, scale, amax_only, mode, scale_rows, bf16_first, st);
  if (storage == FMM_BF16 && product == FMM_E4M3)
    return launch_quantize_plain_t<__nv_bfloat16, __nv_fp8_storage_t>(X, ldx, rows, cols, out, amax_bits, scale, amax_only, mode, scale_rows, bf16_first, st);
  return cudaErrorInvalidValue;
}


// ------------------------------------------------------------------------------------------
// launch wrappers
// ------------------------------------------------------------------------------------------
template <int kSplit>
static cudaError_t launch_encode_split(int storage, int product, const EncodeOperand& a, const EncodeOperand* b, bool amax_only,
                                       int use_scale, cudaStream_t st) {
  if (storage == FMM_F32 && product == FMM_BF16)
    return launch_encode_t<float, __nv_bfloat16, kSplit>(a, b, amax_only, use_scale, st);
  if (storage == FMM_BF16 && product == FMM_BF16)
    return launch_encode_t<__nv_bfloat16, __nv_bfloat16, kSplit>(a, b, amax_only, use_scale, st);
  if (storage == FMM_F32 && product == FMM_E4M3)
    return launch_encode_t<float, __nv_fp8_storage_t, kSplit>(a, b, amax_only, use_scale, st);
  if (storage == FMM_BF16 && product == FMM_E4M3)
    return launch_encode_t<__nv_bfloat16, __nv_fp8_storage_t, kSplit>(a, b, amax_only, use_scale, st);
  if (storage == FMM_E4M3 && product == FMM_E4M3 && use_scale != 2 && use_scale != 3)
    return launch_encode_t<__nv_fp8_storage_t, __nv_fp8_storage_t, kSplit>(a, b, amax_only, use_scale, st);
  return cudaErrorInvalidValue;
}

cudaError_t launch_encode_pair(int storage, int product, const EncodeOperand& a, const EncodeOperand* b, bool amax_only,
                               int use_scale, cudaStream_t st) {
  // both operands of a product share the thread split: small schemes (at most 4 cells in either grid and at most 8
  // products): one thread per position vector; otherwise four threads share one (a batch of algorithms on a 2 x 2
  // grid has 28 products: 28.8 against 36.5 us per algorithm with four threads per vector)
  const int cells = std::max(a.gr * a.gc, b ? b->gr * b->gc : 0);
  const int products = std::max(a.h_tab->R, b ? b->h_tab->R : 0);
  if (cells <= 4 && products <= 8) return launch_encode_split<1>(storage, product, a, b, amax_only, use_scale, st);
  return launch_encode_split<4>(storage, product, a, b, amax_only, use_scale, st);
}

cudaError_t launch_encode(int storage, int product, const void* X, int64_t ldx, int gr, int gc, int64_t br,
                          int64_t bc, const CoefTable* d_tab, const CoefTable* h_tab, void* out, int64_t out_stride,
                          unsigned* amax_bits, float* scale, bool amax_only, int use_scale, cudaStream_t st) {
  const EncodeOperand a{X, ldx, gr, gc, br, bc, d_tab, h_tab, out, out_stride, amax_bits, scale, 1, 0, nullptr};
  return launch_encode_pair(storage, product, a, nullptr, amax_only, use_scale, st);
}

cudaError_t launch_transpose(int elem_bytes, const void* B, int64_t ldb, int64_t K, int64_t N, void* Bt,
                             cudaStream_t st) {
  dim3 grid((unsigned)((N + 31) / 32), (unsigned)((K + 31) / 32));
  if (elem_bytes == 2)
    transpose_kernel<uint16_t><<<grid, 256, 0, st>>>((const uint16_t*)B, ldb, K, N, (uint16_t*)Bt);
  else if (elem_bytes == 4)
    transpose_kernel<uint32_t><<<grid, 256, 0, st>>>((const uint32_t*)B, ldb, K, N, (uint32_t*)Bt);
  else
    return cudaErrorInvalidValue;
  ++fmm_launch_counter();
  return cudaGetLastError();
}

// upper bound of the number of decode blocks (= partial sums) over both thread splits
int decode_grid(int64_t bm, int64_t bn) {
  int grid, tpb;
  split_tiles((bm * (bn >> 2) + 63) / 64, &grid, &tpb);
  return grid;
}

template <typename OutT, int kSplit, typename ProdT>
static cudaError_t launch_decode_t(const ProdT* prod, int64_t prod_stride, const CoefTable* d_tab, int R, int nnz, const float* sA,
                                   const float* sB, int m, int n, int64_t bm, int64_t bn, void* C, int64_t ldc,
                                   const float* cstar32, double* partials, int* n_partials, int gauges, cudaStream_t st) {
  if (gauges < 1 || kSplit % gauges != 0 || (gauges > 1 && C != nullptr)) return cudaErrorInvalidValue;
  constexpr int kDecPos = kDecThreads / kSplit;
  const size_t smem = ((sizeof(DecSmemHead) + (size_t)nnz * 8 + 15) / 16) * 16 + (size_t)(R + 1) * kDecPos * 4 * sizeof(ProdT);
  const size_t smem_cs = (cstar32 != nullptr && kSplit > 1 && gauges == kSplit) ? (size_t)(16 / kSplit) * kDecPos * 16 : 0;
  if (bm * (bn >> 2) + kDecThreads * 8 >= (int64_t)1 << 31) return cudaErrorInvalidValue;   // 32-bit position index
  int grid, tpb;
  split_tiles((bm * (bn >> 2) + kDecPos - 1) / kDecPos, &grid, &tpb);
  if (n_partials) *n_partials = grid;
  const int64_t ldcs = (int64_t)n * bn;
  static unsigned long long smem_ok[3] = {0, 0, 0};   // per template instantiation, one bit per device
#define FMM_DECODE_LAUNCH(STORE, ERR, SLOT)                                                                      \
  {                                                                                                              \
    auto k = decode_kernel<OutT, STORE, ERR, kSplit, ProdT>;                                                         \
    {                                                                                                            \
      cudaError_t e = fmm_allow_dynamic_smem(k, 200 * 1024, &smem_ok[SLOT]);                                     \
      if (e != cudaSuccess) return e;                                                                            \
    }                                                                                                            \
    cudaError_t le = launch_dependent(k, dim3(grid), dim3(kDecThreads), smem + smem_cs, st, prod, d_tab, R, sA, sB, n, bm, bn, (OutT*)C, ldc, \
                                      cstar32, ldcs, partials, tpb, prod_stride, gauges);                         \
    if (le != cudaSuccess) return le;                                                                            \
  }
  if (C != nullptr && cstar32 != nullptr) FMM_DECODE_LAUNCH(true, true, 0)
  else if (C != nullptr) FMM_DECODE_LAUNCH(true, false, 1)
  else FMM_DECODE_LAUNCH(false, true, 2)
#undef FMM_DECODE_LAUNCH
  (void)m;
  ++fmm_launch_counter();
  return cudaGetLastError();
}

template <typename ProdT>
static cudaError_t launch_decode_p(int output, const ProdT* prod, int64_t prod_stride, const CoefTable* d_tab, const CoefTable* h_tab, int R,
                                   const float* sA, const float* sB, int m, int n, int64_t bm, int64_t bn, void* C,
                                   int64_t ldc, const float* cstar32, double* partials, int* n_partials, int gauges,
                                   cudaStream_t st) {
  const int nnz = padded_entries(*h_tab);
  if (C == nullptr && cstar32 == nullptr) return cudaErrorInvalidValue;
  // a batch of four small algorithms, error only: products straight into registers (decode_batch_kernel)
  if ((gauges == 4 || gauges == 8) && C == nullptr && R % gauges == 0 && R / gauges <= kBatchR && m * n <= 4 &&
      h_tab->R == gauges * m * n) {
    if (bm * (bn >> 2) + kDecThreads * 8 >= (int64_t)1 << 31) return cudaErrorInvalidValue;
    const int pos = kDecThreads / gauges;
    int grid, tpb;
    split_tiles((bm * (bn >> 2) + pos - 1) / pos, &grid, &tpb);
    if (n_partials) *n_partials = grid;
    const int64_t ldcs = (int64_t)n * bn;
    const int RB = R / gauges;
    cudaError_t le;
    if (output == FMM_F32 && gauges == 4)
      le = launch_dependent(decode_batch_kernel<float, ProdT, 4>, dim3(grid), dim3(kDecThreads), 0, st, prod, d_tab, RB, sA, sB, n,
                            bm, bn, cstar32, ldcs, partials, tpb, prod_stride);
    else if (output == FMM_F32)
      le = launch_dependent(decode_batch_kernel<float, ProdT, 8>, dim3(grid), dim3(kDecThreads), 0, st, prod, d_tab, RB, sA, sB, n,
                            bm, bn, cstar32, ldcs, partials, tpb, prod_stride);
    else if (output == FMM_BF16 && gauges == 4)
      le = launch_dependent(decode_batch_kernel<__nv_bfloat16, ProdT, 4>, dim3(grid), dim3(kDecThreads), 0, st, prod, d_tab, RB, sA,
                            sB, n, bm, bn, cstar32, ldcs, partials, tpb, prod_stride);
    else if (output == FMM_BF16)
      le = launch_dependent(decode_batch_kernel<__nv_bfloat16, ProdT, 8>, dim3(grid), dim3(kDecThreads), 0, st, prod, d_tab, RB, sA,
                            sB, n, bm, bn, cstar32, ldcs, partials, tpb, prod_stride);
    else
      return cudaErrorInvalidValue;
    if (le != cudaSuccess) return le;
    ++fmm_launch_counter();
    return cudaGetLastError();
  }
  // small schemes (at most 8 products, 4 output cells): one thread per position quad; otherwise four share one
  const bool small = R <= 8 && m * n * gauges <= 4 && gauges == 1;
  if (output == FMM_F32)
    return small ? launch_decode_t<float, 1, ProdT>(prod, prod_stride, d_tab, R, nnz, sA, sB, m, n, bm, bn, C, ldc, cstar32, partials, n_partials, gauges, st)
                 : launch_decode_t<float, 4, ProdT>(prod, prod_stride, d_tab, R, nnz, sA, sB, m, n, bm, bn, C, ldc, cstar32, partials, n_partials, gauges, st);
  if (output == FMM_BF16)
    return small ? launch_decode_t<__nv_bfloat16, 1, ProdT>(prod, prod_stride, d_tab, R, nnz, sA, sB, m, n, bm, bn, C, ldc, cstar32, partials, n_partials, gauges, st)
                 : launch_decode_t<__nv_bfloat16, 4, ProdT>(prod, prod_stride, d_tab, R, nnz, sA, sB, m, n, bm, bn, C, ldc, cstar32, partials, n_partials, gauges, st);
  return cudaErrorInvalidValue;
}

cudaError_t launch_decode(int output, const void* prod, int prod_dtype, int64_t prod_stride, const CoefTable* d_tab,
                          const CoefTable* h_tab, int R, const float* sA, const float* sB, int m, int n, int64_t bm,
                          int64_t bn, void* C, int64_t ldc, const float* cstar32, double* partials, int* n_partials,
                          cudaStream_t st, int gauges) {
  if (prod_dtype == FMM_BF16)
    return launch_decode_p<__nv_bfloat16>(output, (const __nv_bfloat16*)prod, prod_stride, d_tab, h_tab, R, sA, sB, m, n, bm, bn, C, ldc,
                                          cstar32, partials, n_partials, gauges, st);
  return launch_decode_p<float>(output, (const float*)prod, prod_stride, d_tab, h_tab, R, sA, sB, m, n, bm, bn, C, ldc, cstar32,
                                partials, n_partials, gauges, st);
}

cudaError_t launch_sum_partials(const double* partials, int n, double* out, cudaStream_t st, int count) {
  sum_partials_kernel<<<count, 256, 0, st>>>(partials, n, out);
  ++fmm_launch_counter();
  return cudaGetLastError();
}

int stream_grid(int64_t count) {
  int64_t g = (count + 256 * 8 - 1) / (256 * 8);
  if (g < 1) g = 1;
  if (g > 148 * 8) g = 148 * 8;
  return (int)g;
}

cudaError_t launch_cstar_prepare(const double* cstar, int64_t count, float* cstar32, double* partials,
                                 int* n_partials, cudaStream_t st) {
  const int grid = stream_grid(count);
  if (n_partials) *n_partials = grid;
  cstar_prepare_kernel<<<grid, 256, 0, st>>>(cstar, count, cstar32, partials);
  ++fmm_launch_counter();
  return cudaGetLastError();
}

cudaError_t launch_frob_err(int output, const void* C, int64_t ldc, const double* cstar, int64_t M, int64_t N,
                            double* part_err, double* part_ref, int* n_partials, cudaStream_t st) {
  const int grid = stream_grid(M * N);
  if (n_partials) *n_partials = grid;
  if (output == FMM_F32)
    frob_err_kernel<float><<<grid, 256, 0, st>>>((const float*)C, ldc, cstar, M, N, part_err, part_ref);
  else if (output == FMM_BF16)
    frob_err_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)C, ldc, cstar, M, N, part_err, part_ref);
  else
    return cudaErrorInvalidValue;
  ++fmm_launch_counter();
  return cudaGetLastError();
}

cudaError_t launch_frob_err_fixed_grid(int output, const void* C, int64_t ldc, const double* cstar, int64_t M,
                                       int64_t N, double* part_err, double* part_ref, int grid, cudaStream_t st) {
  if (grid < 1) return cudaErrorInvalidValue;
  if (output == FMM_F32)
    frob_err_kernel<float><<<grid, 256, 0, st>>>((const float*)C, ldc, cstar, M, N, part_err, part_ref);
  else if (output == FMM_BF16)
    frob_err_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)C, ldc, cstar, M, N, part_err, part_ref);
  else
    return cudaErrorInvalidValue;
  ++fmm_launch_counter();
  return cudaGetLastError();
}

cudaError_t launch_exact_f64(int storage, const void* A, int64_t lda, const void* B, int64_t ldb,
                             int b_weight_layout, int64_t M, int64_t K, int64_t N, double* C, cudaStream_t st) {
  dim3 grid((unsigned)((N + kExT - 1) / kExT), (unsigned)((M + kExT - 1) / kExT));
  if (storage == FMM_F32)
    exact_f64_kernel<float><<<grid, 256, 0, st>>>((const float*)A, lda, (const float*)B, ldb, b_weight_layout, M, K, N, C);
  else if (storage == FMM_BF16)
    exact_f64_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)A, lda, (const __nv_bfloat16*)B, ldb, b_weight_layout, M, K, N, C);
  else
    return cudaErrorInvalidValue;
  ++fmm_launch_counter();
  return cudaGetLastError();
}
