// Streaming kernels of the scheme GEMM: encode (block sums -> product dtype), transpose,
// decode (+ error reduction), Frobenius error, fp64 reference.  All are HBM-bound passes;
// each thread moves 16-byte (8-byte for bf16 sources) vectors and the grid covers the data once.
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include <cmath>

#include "kernels_stream.cuh"

int64_t& fmm_launch_counter() {
  static int64_t c = 0;
  return c;
}

namespace {

constexpr int kThreads = 256;

// ------------------------------------------------------------------------------------------
// small device helpers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
  const uint2 raw = *reinterpret_cast<const uint2*>(p);
  float4 v;
  v.x = __uint_as_float(raw.x << 16);
  v.y = __uint_as_float(raw.x & 0xFFFF0000u);
  v.z = __uint_as_float(raw.y << 16);
  v.w = __uint_as_float(raw.y & 0xFFFF0000u);
  return v;
}

__device__ __forceinline__ void store4(__nv_bfloat16* p, float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 raw;
  raw.x = *reinterpret_cast<uint32_t*>(&lo);
  raw.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = raw;
}
__device__ __forceinline__ void store4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
// e4m3: round to nearest even, saturate to +-448 (NaN stays NaN)
__device__ __forceinline__ void store4(__nv_fp8_storage_t* p, float4 v) {
  const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(v.x, v.y), __NV_SATFINITE, __NV_E4M3);
  const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(v.z, v.w), __NV_SATFINITE, __NV_E4M3);
  *reinterpret_cast<uint32_t*>(p) = lo | (hi << 16);
}

__device__ __forceinline__ float round_out(float x, float*) { return x; }
__device__ __forceinline__ float round_out(float x, __nv_bfloat16*) { return __bfloat162float(__float2bfloat16_rn(x)); }

// Power-of-two scale of an encoded tensor: s = 2^ceil(log2(amax/448)), 1 when amax is 0 / not finite.
// Done in fp64 so the decision at exact powers of two is the same as a plain frexp on the host.
__device__ __forceinline__ float pow2_scale_448(float amax) {
  if (!(amax > 0.0f) || isinf(amax)) return 1.0f;
  int e;
  const double f = frexp((double)amax / 448.0, &e);
  if (f == 0.5) e -= 1;
  return (float)ldexp(1.0, e);
}

__device__ __forceinline__ double block_sum_double(double v, double* red /* >= 8 doubles smem */) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  double tot = 0.0;
  if (threadIdx.x == 0)
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += red[w];
  return tot;  // valid in thread 0
}

// ------------------------------------------------------------------------------------------
// encode: block sums of Eq. 1 (inner parentheses), scale, one rounding to the product dtype.
// Each thread owns 4 consecutive inner-dimension elements of one block row; it stages the
// 4-vectors of all grid cells at that position in shared memory (used as an indexable register
// file, [cell][thread] so accesses are conflict free) and then walks the sparse coefficient list
// of every product: an fp32 FMA chain in list order.
// ------------------------------------------------------------------------------------------
struct EncSmem {
  CoefTable tab;
  float scale[FMM_MAX_R];
  float inv_scale[FMM_MAX_R];
  int use_mul[FMM_MAX_R];
  unsigned amax[FMM_MAX_R];
};

template <typename SrcT, typename DstT, bool kAmaxOnly>
__global__ void __launch_bounds__(kThreads)
encode_kernel(const SrcT* __restrict__ X, int64_t ldx, int gc, int64_t br, int64_t bc,
              const CoefTable* __restrict__ d_tab, DstT* __restrict__ out, unsigned* __restrict__ amax_bits,
              float* __restrict__ scale_out, int use_scale) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  EncSmem& sm = *reinterpret_cast<EncSmem*>(smem_raw);
  float4* stage = reinterpret_cast<float4*>(smem_raw + ((sizeof(EncSmem) + 15) / 16) * 16);

  {  // cooperative copy of the table
    const int* src = reinterpret_cast<const int*>(d_tab);
    int* dst = reinterpret_cast<int*>(&sm.tab);
    for (int i = threadIdx.x; i < (int)(sizeof(CoefTable) / 4); i += kThreads) dst[i] = src[i];
  }
  __syncthreads();
  const int R = sm.tab.R, ncell = sm.tab.ncell;
  if (threadIdx.x < R) {
    float s = 1.0f;
    if (!kAmaxOnly && use_scale) s = pow2_scale_448(__uint_as_float(amax_bits[threadIdx.x]));
    sm.scale[threadIdx.x] = s;
    const float inv = 1.0f / s;
    sm.use_mul[threadIdx.x] = (isfinite(inv) && inv * s == 1.0f && fabsf(inv) >= 1.17549435e-38f);
    sm.inv_scale[threadIdx.x] = inv;
    sm.amax[threadIdx.x] = 0u;
    if (!kAmaxOnly && use_scale && blockIdx.x == 0 && scale_out) scale_out[threadIdx.x] = s;
  }
  __syncthreads();

  const int64_t vec_per_row = bc >> 2;
  const int64_t idx = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  const bool live = idx < br * vec_per_row;
  const int64_t p = live ? idx / vec_per_row : 0;
  const int64_t t = live ? (idx - p * vec_per_row) << 2 : 0;

  if (live) {
    for (int c = 0; c < ncell; ++c) {
      const int gi = c / gc, gj = c - gi * gc;
      stage[c * kThreads + threadIdx.x] = load4(X + (gi * br + p) * ldx + gj * bc + t);
    }
  }
  // (each thread reads back only what it wrote: no barrier needed)
  for (int r = 0; r < R; ++r) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (live) {
      const int e0 = sm.tab.off[r], e1 = sm.tab.off[r + 1];
      for (int e = e0; e < e1; ++e) {
        const float c = sm.tab.coef[e];
        const float4 v = stage[sm.tab.cell[e] * kThreads + threadIdx.x];
        acc.x = __fmaf_rn(c, v.x, acc.x);
        acc.y = __fmaf_rn(c, v.y, acc.y);
        acc.z = __fmaf_rn(c, v.z, acc.z);
        acc.w = __fmaf_rn(c, v.w, acc.w);
      }
    }
    if (kAmaxOnly) {
      float a = fmaxf(fmaxf(fabsf(acc.x), fabsf(acc.y)), fmaxf(fabsf(acc.z), fabsf(acc.w)));
      if (!(a == a)) a = 0.0f;  // NaN does not set a scale
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
      if ((threadIdx.x & 31) == 0 && a > 0.0f) atomicMax(&sm.amax[r], __float_as_uint(a));
    } else if (live) {
      if (use_scale) {
        if (sm.use_mul[r]) {
          const float inv = sm.inv_scale[r];
          acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        } else {
          const float s = sm.scale[r];
          acc.x = __fdiv_rn(acc.x, s); acc.y = __fdiv_rn(acc.y, s);
          acc.z = __fdiv_rn(acc.z, s); acc.w = __fdiv_rn(acc.w, s);
        }
      }
      store4(out + ((int64_t)r * br + p) * bc + t, acc);
    }
  }
  if (kAmaxOnly) {
    __syncthreads();
    if (threadIdx.x < R && sm.amax[threadIdx.x] != 0u) atomicMax(&amax_bits[threadIdx.x], sm.amax[threadIdx.x]);
  }
}

template <typename SrcT, typename DstT>
cudaError_t launch_encode_t(const void* X, int64_t ldx, int gr, int gc, int64_t br, int64_t bc,
                            const CoefTable* d_tab, void* out, unsigned* amax_bits, float* scale, bool amax_only,
                            bool use_scale, cudaStream_t st) {
  const size_t smem = ((sizeof(EncSmem) + 15) / 16) * 16 + (size_t)gr * gc * kThreads * sizeof(float4);
  const int64_t vecs = br * (bc >> 2);
  const int grid = (int)((vecs + kThreads - 1) / kThreads);
  if (grid == 0) return cudaSuccess;
  cudaError_t e;
  if (amax_only) {
    auto k = encode_kernel<SrcT, DstT, true>;
    e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k<<<grid, kThreads, smem, st>>>((const SrcT*)X, ldx, gc, br, bc, d_tab, (DstT*)out, amax_bits, scale, use_scale);
  } else {
    auto k = encode_kernel<SrcT, DstT, false>;
    e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k<<<grid, kThreads, smem, st>>>((const SrcT*)X, ldx, gc, br, bc, d_tab, (DstT*)out, amax_bits, scale, use_scale);
  }
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

// ------------------------------------------------------------------------------------------
// decode: C_ij = rnd_O( sum_r w_{r,ij} sA_r sB_r M_r ), ascending r, fp32 FMA chain; optional
// error reduction sum (rnd_O(c) - C*)^2 per block (fp32 per thread -> fp64 shuffle tree -> one fp64
// partial per block).  Accumulators of the m*n output cells live in shared memory [cell][thread].
// ------------------------------------------------------------------------------------------
struct DecSmem {
  CoefTable tab;
  double red[kThreads / 32];
};

template <typename OutT, bool kStore, bool kErr>
__global__ void __launch_bounds__(kThreads)
decode_kernel(const float* __restrict__ prod, const CoefTable* __restrict__ d_tab, const float* __restrict__ sA,
              const float* __restrict__ sB, int n, int64_t bm, int64_t bn, OutT* __restrict__ C, int64_t ldc,
              const float* __restrict__ cstar32, int64_t ldcs, double* __restrict__ partials) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  DecSmem& sm = *reinterpret_cast<DecSmem*>(smem_raw);
  float4* acc = reinterpret_cast<float4*>(smem_raw + ((sizeof(DecSmem) + 15) / 16) * 16);
  {
    const int* src = reinterpret_cast<const int*>(d_tab);
    int* dst = reinterpret_cast<int*>(&sm.tab);
    for (int i = threadIdx.x; i < (int)(sizeof(CoefTable) / 4); i += kThreads) dst[i] = src[i];
  }
  __syncthreads();
  const int R = sm.tab.R, ncell = sm.tab.ncell;
  if (sA != nullptr) {  // fold the (power-of-two) scales into the coefficients: w * (sA_r * sB_r)
    for (int r = threadIdx.x; r < R; r += kThreads) {
      const float s = sA[r] * sB[r];
      for (int e = sm.tab.off[r]; e < sm.tab.off[r + 1]; ++e) sm.tab.coef[e] *= s;
    }
    __syncthreads();
  }
  const int64_t vec_per_row = bn >> 2;
  const int64_t idx = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  const bool live = idx < bm * vec_per_row;
  const int64_t p = live ? idx / vec_per_row : 0;
  const int64_t q = live ? (idx - p * vec_per_row) << 2 : 0;

  float err = 0.0f;
  if (live) {
    for (int c = 0; c < ncell; ++c) acc[c * kThreads + threadIdx.x] = make_float4(0.f, 0.f, 0.f, 0.f);
    const float* src = prod + p * bn + q;
    const int64_t rstride = bm * bn;
    for (int r = 0; r < R; ++r) {
      const float4 v = __ldcs(reinterpret_cast<const float4*>(src + r * rstride));
      const int e0 = sm.tab.off[r], e1 = sm.tab.off[r + 1];
      for (int e = e0; e < e1; ++e) {
        const float w = sm.tab.coef[e];
        float4* a = &acc[sm.tab.cell[e] * kThreads + threadIdx.x];
        float4 x = *a;
        x.x = __fmaf_rn(w, v.x, x.x);
        x.y = __fmaf_rn(w, v.y, x.y);
        x.z = __fmaf_rn(w, v.z, x.z);
        x.w = __fmaf_rn(w, v.w, x.w);
        *a = x;
      }
    }
    for (int c = 0; c < ncell; ++c) {
      const int i = c / n, j = c - i * n;
      float4 x = acc[c * kThreads + threadIdx.x];
      const int64_t row = i * bm + p, col = j * bn + q;
      if (kStore) store4(C + row * ldc + col, x);
      if (kErr) {
        const float4 cs = __ldcs(reinterpret_cast<const float4*>(cstar32 + row * ldcs + col));
        const float d0 = round_out(x.x, (OutT*)nullptr) - cs.x, d1 = round_out(x.y, (OutT*)nullptr) - cs.y;
        const float d2 = round_out(x.z, (OutT*)nullptr) - cs.z, d3 = round_out(x.w, (OutT*)nullptr) - cs.w;
        err = __fmaf_rn(d0, d0, err); err = __fmaf_rn(d1, d1, err);
        err = __fmaf_rn(d2, d2, err); err = __fmaf_rn(d3, d3, err);
      }
    }
  }
  if (kErr) {
    const double tot = block_sum_double((double)err, sm.red);
    if (threadIdx.x == 0) partials[blockIdx.x] = tot;
  }
}

// ------------------------------------------------------------------------------------------
// reductions
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) sum_partials_kernel(const double* __restrict__ partials, int n,
                                                           double* __restrict__ out) {
  __shared__ double red[8];
  double v = 0.0;
  for (int i = threadIdx.x; i < n; i += 256) v += partials[i];
  const double tot = block_sum_double(v, red);
  if (threadIdx.x == 0) out[0] = tot;
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
// fp64 reference product: 64 x 64 tile per block, 4 x 4 per thread, ascending inner index
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) exact_f64_kernel(const T* __restrict__ A, int64_t lda,
                                                        const T* __restrict__ B, int64_t ldb, int b_weight,
                                                        int64_t M, int64_t K, int64_t N, double* __restrict__ C) {
  __shared__ double As[16][64 + 1];
  __shared__ double Bs[16][64 + 1];
  const int64_t m0 = (int64_t)blockIdx.y * 64, n0 = (int64_t)blockIdx.x * 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  double acc[4][4] = {};
  for (int64_t k0 = 0; k0 < K; k0 += 16) {
    for (int i = threadIdx.x; i < 64 * 16; i += 256) {
      {  // A tile: consecutive threads along the inner dimension
        const int kk = i & 15, r = i >> 4;
        const int64_t row = m0 + r, t = k0 + kk;
        As[kk][r] = (row < M && t < K) ? (double)(float)A[row * lda + t] : 0.0;
      }
      if (b_weight) {
        const int kk = i & 15, c = i >> 4;
        const int64_t col = n0 + c, t = k0 + kk;
        Bs[kk][c] = (col < N && t < K) ? (double)(float)B[col * ldb + t] : 0.0;
      } else {
        const int c = i & 63, kk = i >> 6;
        const int64_t col = n0 + c, t = k0 + kk;
        Bs[kk][c] = (col < N && t < K) ? (double)(float)B[t * ldb + col] : 0.0;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      double a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; b[i] = Bs[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fma(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
  for (int i = 0; i < 4; ++i)
    for (int j = 0; j < 4; ++j) {
      const int64_t row = m0 + ty * 4 + i, col = n0 + tx * 4 + j;
      if (row < M && col < N) C[row * N + col] = acc[i][j];
    }
}

}  // namespace

// ------------------------------------------------------------------------------------------
// launch wrappers
// ------------------------------------------------------------------------------------------
cudaError_t launch_encode(int storage, int product, const void* X, int64_t ldx, int gr, int gc, int64_t br,
                          int64_t bc, const CoefTable* d_tab, void* out, unsigned* amax_bits, float* scale,
                          bool amax_only, bool use_scale, cudaStream_t st) {
  if (storage == FMM_F32 && product == FMM_BF16)
    return launch_encode_t<float, __nv_bfloat16>(X, ldx, gr, gc, br, bc, d_tab, out, amax_bits, scale, amax_only, use_scale, st);
  if (storage == FMM_BF16 && product == FMM_BF16)
    return launch_encode_t<__nv_bfloat16, __nv_bfloat16>(X, ldx, gr, gc, br, bc, d_tab, out, amax_bits, scale, amax_only, use_scale, st);
  if (storage == FMM_F32 && product == FMM_E4M3)
    return launch_encode_t<float, __nv_fp8_storage_t>(X, ldx, gr, gc, br, bc, d_tab, out, amax_bits, scale, amax_only, use_scale, st);
  if (storage == FMM_BF16 && product == FMM_E4M3)
    return launch_encode_t<__nv_bfloat16, __nv_fp8_storage_t>(X, ldx, gr, gc, br, bc, d_tab, out, amax_bits, scale, amax_only, use_scale, st);
  return cudaErrorInvalidValue;
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

int decode_grid(int64_t bm, int64_t bn) { return (int)((bm * (bn >> 2) + kThreads - 1) / kThreads); }

template <typename OutT>
static cudaError_t launch_decode_t(const float* prod, const CoefTable* d_tab, const float* sA, const float* sB, int m,
                                   int n, int64_t bm, int64_t bn, void* C, int64_t ldc, const float* cstar32,
                                   double* partials, cudaStream_t st) {
  const size_t smem = ((sizeof(DecSmem) + 15) / 16) * 16 + (size_t)m * n * kThreads * sizeof(float4);
  const int grid = decode_grid(bm, bn);
  const int64_t ldcs = (int64_t)n * bn;
#define FMM_DECODE_LAUNCH(STORE, ERR)                                                                         \
  {                                                                                                           \
    auto k = decode_kernel<OutT, STORE, ERR>;                                                                 \
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);          \
    if (e != cudaSuccess) return e;                                                                           \
    k<<<grid, kThreads, smem, st>>>(prod, d_tab, sA, sB, n, bm, bn, (OutT*)C, ldc, cstar32, ldcs, partials);  \
  }
  if (C != nullptr && cstar32 != nullptr) FMM_DECODE_LAUNCH(true, true)
  else if (C != nullptr) FMM_DECODE_LAUNCH(true, false)
  else FMM_DECODE_LAUNCH(false, true)
#undef FMM_DECODE_LAUNCH
  ++fmm_launch_counter();
  return cudaGetLastError();
}

cudaError_t launch_decode(int output, const float* prod, const CoefTable* d_tab, const float* sA, const float* sB,
                          int m, int n, int64_t bm, int64_t bn, void* C, int64_t ldc, const float* cstar32,
                          double* partials, int* n_partials, cudaStream_t st) {
  if (C == nullptr && cstar32 == nullptr) return cudaErrorInvalidValue;
  if (n_partials) *n_partials = decode_grid(bm, bn);
  if (output == FMM_F32) return launch_decode_t<float>(prod, d_tab, sA, sB, m, n, bm, bn, C, ldc, cstar32, partials, st);
  if (output == FMM_BF16) return launch_decode_t<__nv_bfloat16>(prod, d_tab, sA, sB, m, n, bm, bn, C, ldc, cstar32, partials, st);
  return cudaErrorInvalidValue;
}

cudaError_t launch_sum_partials(const double* partials, int n, double* out, cudaStream_t st) {
  sum_partials_kernel<<<1, 256, 0, st>>>(partials, n, out);
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

cudaError_t launch_exact_f64(int storage, const void* A, int64_t lda, const void* B, int64_t ldb,
                             int b_weight_layout, int64_t M, int64_t K, int64_t N, double* C, cudaStream_t st) {
  dim3 grid((unsigned)((N + 63) / 64), (unsigned)((M + 63) / 64));
  if (storage == FMM_F32)
    exact_f64_kernel<float><<<grid, 256, 0, st>>>((const float*)A, lda, (const float*)B, ldb, b_weight_layout, M, K, N, C);
  else if (storage == FMM_BF16)
    exact_f64_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)A, lda, (const __nv_bfloat16*)B, ldb, b_weight_layout, M, K, N, C);
  else
    return cudaErrorInvalidValue;
  ++fmm_launch_counter();
  return cudaGetLastError();
}
