// The two repair rules of Appendix C ("The repair rules"):
//   1. every token row x_t of the input is divided by d_t = 2^ceil(log2(max(RMS(x_t), 1e-3))) before the block sums
//      and its output row is multiplied by d_t after the combination (row_pow2_scale / row_unscale);
//   2. the e4m3 codes of the weight's block sums are chosen jointly: per position, each of the R codes starts at the
//      nearer of the two codes that bracket its bf16 value and is switched to the other one whenever that lowers
//      e^T H e, H_rs = <w_r, w_s> <u_r, u_s>, in sweeps over r (joint_round_kernel, a weight-only offline pass).
#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/fmm_b200.h"
#include "kernels_stream.cuh"

namespace {

__device__ __forceinline__ float load_f32(const float* p) { return *p; }
__device__ __forceinline__ float load_f32(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void store_f32(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_f32(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// ------------------------------------------------------------------------------------------
// rule 1: one warp per row.  The sum of squares is taken in fp64 (squares of fp32 / bf16 values are exact there), so
// the integer decision ceil(log2(.)) agrees with an fp64 evaluation of the definition except when the RMS lies
// within an fp64 rounding of a power of two.
// ------------------------------------------------------------------------------------------
template <typename T> struct RowVec;              // 16 bytes of a row
template <> struct RowVec<float> { static constexpr int kElems = 4; };
template <> struct RowVec<__nv_bfloat16> { static constexpr int kElems = 8; };

template <typename T>
__device__ __forceinline__ void unpack16(const uint4& raw, float (&v)[RowVec<T>::kElems]) {
  if constexpr (sizeof(T) == 4) {
    v[0] = __uint_as_float(raw.x); v[1] = __uint_as_float(raw.y); v[2] = __uint_as_float(raw.z); v[3] = __uint_as_float(raw.w);
  } else {
    const unsigned w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { v[2 * i] = __uint_as_float(w[i] << 16); v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
  }
}
template <typename T>
__device__ __forceinline__ uint4 pack16(const float (&v)[RowVec<T>::kElems]) {
  uint4 raw;
  if constexpr (sizeof(T) == 4) {
    raw = make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
  } else {
    unsigned w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      w[i] = *reinterpret_cast<const unsigned*>(&h);
    }
    raw = make_uint4(w[0], w[1], w[2], w[3]);
  }
  return raw;
}

// kVec: rows are read and written as 16-byte vectors (the host checks alignment and divisibility)
template <typename T, bool kVec>
__global__ void __launch_bounds__(256)
row_scale_kernel(const T* X, int64_t ldx, int64_t rows, int64_t K, float* __restrict__ d_out, T* Y, int64_t ldy) {   // Y may be X
  constexpr int VE = RowVec<T>::kElems;
  const int lane = threadIdx.x & 31;
  const int64_t warps = (int64_t)gridDim.x * 8;
  for (int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); row < rows; row += warps) {
    const T* x = X + row * ldx;
    double ss = 0.0;
    if (kVec && K <= 16 * 32 * VE) {
      // rows of up to 8 KB stay in registers between the two passes: every load is issued before the first use
      if constexpr (kVec) {
        uint4 keep[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int64_t t = ((int64_t)j * 32 + lane) * VE;
          keep[j] = t < K ? *reinterpret_cast<const uint4*>(x + t) : make_uint4(0u, 0u, 0u, 0u);
        }
        double part[4] = {0.0, 0.0, 0.0, 0.0};           // four chains; the order of an fp64 sum of exact squares
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          float v[VE];
          unpack16<T>(keep[j], v);
#pragma unroll
          for (int i = 0; i < VE; ++i) part[j & 3] = fma((double)v[i], (double)v[i], part[j & 3]);
        }
        ss = (part[0] + part[1]) + (part[2] + part[3]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        const double rms = fmax(sqrt(ss / (double)K), 1e-3);
        int e;
        const double f = frexp(rms, &e);
        const float d = ldexpf(1.0f, f == 0.5 ? e - 1 : e);
        if (lane == 0) d_out[row] = d;
        const float inv = 1.0f / d;
        T* y = Y + row * ldy;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int64_t t = ((int64_t)j * 32 + lane) * VE;
          if (t < K) {
            float v[VE];
            unpack16<T>(keep[j], v);
#pragma unroll
            for (int i = 0; i < VE; ++i) v[i] = __fmul_rn(v[i], inv);
            *reinterpret_cast<uint4*>(y + t) = pack16<T>(v);
          }
        }
      }
      continue;
    }
    if constexpr (kVec) {
      for (int64_t t = (int64_t)lane * VE; t < K; t += 32 * VE) {
        float v[VE];
        unpack16<T>(*reinterpret_cast<const uint4*>(x + t), v);
#pragma unroll
        for (int i = 0; i < VE; ++i) ss = fma((double)v[i], (double)v[i], ss);
      }
    } else {
      for (int64_t t = lane; t < K; t += 32) {
        const double v = (double)load_f32(x + t);
        ss = fma(v, v, ss);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    const double rms = fmax(sqrt(ss / (double)K), 1e-3);
    int e;
    const double f = frexp(rms, &e);                  // rms = f 2^e, f in [0.5, 1)
    const float d = ldexpf(1.0f, f == 0.5 ? e - 1 : e);
    if (lane == 0) d_out[row] = d;
    const float inv = 1.0f / d;                        // a power of two: exact
    T* y = Y + row * ldy;
    if constexpr (kVec) {
      for (int64_t t = (int64_t)lane * VE; t < K; t += 32 * VE) {
        float v[VE];
        unpack16<T>(*reinterpret_cast<const uint4*>(x + t), v);
#pragma unroll
        for (int i = 0; i < VE; ++i) v[i] = __fmul_rn(v[i], inv);
        *reinterpret_cast<uint4*>(y + t) = pack16<T>(v);
      }
    } else {
      for (int64_t t = lane; t < K; t += 32) store_f32(y + t, __fmul_rn(load_f32(x + t), inv));
    }
  }
}

template <typename T, bool kVec>
__global__ void __launch_bounds__(256)
row_unscale_kernel(T* __restrict__ C, int64_t ldc, int64_t rows, int64_t N, const float* __restrict__ d) {
  constexpr int VE = kVec ? RowVec<T>::kElems : 1;
  const int64_t per_row = N / VE, total = rows * per_row;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < total; i += (int64_t)gridDim.x * 256) {
    const int64_t row = i / per_row, col = (i - row * per_row) * VE;
    T* p = C + row * ldc + col;
    const float dr = d[row];
    if constexpr (kVec) {
      float v[RowVec<T>::kElems];
      unpack16<T>(*reinterpret_cast<const uint4*>(p), v);
#pragma unroll
      for (int k = 0; k < RowVec<T>::kElems; ++k) v[k] = __fmul_rn(v[k], dr);
      *reinterpret_cast<uint4*>(p) = pack16<T>(v);
    } else {
      store_f32(p, __fmul_rn(load_f32(p), dr));
    }
  }
}

// ------------------------------------------------------------------------------------------
// rule 2
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float e4m3_value(unsigned c) {
  const unsigned mag = c & 0x7Fu, e = mag >> 3, mnt = mag & 7u;
  const float v = e == 0 ? ldexpf((float)mnt, -9) : ldexpf((float)(8u + mnt), (int)e - 10);
  return (c & 0x80u) ? -v : v;
}
// the next code above (dir > 0) or below (dir < 0) in value order; 0xFF if there is none (beyond +-448)
__device__ __forceinline__ unsigned e4m3_neighbour(unsigned c, int dir) {
  unsigned mag = c & 0x7Fu;
  const bool neg = (c & 0x80u) != 0 && mag != 0;
  if (mag == 0) return dir > 0 ? 0x01u : 0x81u;
  const bool away = neg ? dir < 0 : dir > 0;           // larger magnitude
  if (away) return mag >= 0x7Eu ? 0xFFu : ((neg ? 0x80u : 0u) | (mag + 1));
  return mag == 1 ? 0x00u : ((neg ? 0x80u : 0u) | (mag - 1));
}

constexpr int kJointThreads = 128;

template <typename SrcT>
__global__ void __launch_bounds__(kJointThreads)
joint_round_kernel(const SrcT* __restrict__ X, int64_t ldx, int gc, int64_t br, int64_t bc,
                   const CoefTable* __restrict__ d_tab, const float* __restrict__ d_H,
                   const unsigned* __restrict__ amax_bits, float* __restrict__ scale_out,
                   __nv_fp8_storage_t* __restrict__ out, int64_t rstride, int max_sweeps) {
  __shared__ float H[FMM_MAX_R * FMM_MAX_R];
  __shared__ int s_off[FMM_MAX_R + 1];
  __shared__ int s_cell[kMaxNnz];
  __shared__ float s_coef[kMaxNnz];
  const int R = d_tab->R, ncell = d_tab->ncell;
  const int total = d_tab->off[R];
  for (int i = threadIdx.x; i < R * R; i += kJointThreads) H[i] = d_H[i];
  for (int i = threadIdx.x; i <= R; i += kJointThreads) s_off[i] = d_tab->off[i];
  for (int i = threadIdx.x; i < total; i += kJointThreads) { s_cell[i] = d_tab->cell[i]; s_coef[i] = d_tab->coef[i]; }
  __syncthreads();
  const int64_t idx = (int64_t)blockIdx.x * kJointThreads + threadIdx.x;
  if (idx >= br * bc) return;
  const int64_t p = idx / bc, t = idx - p * bc;
  const int64_t gk = (bc + 127) >> 7, row_groups = (br + 127) >> 7;

  float x[kMaxCells];
#pragma unroll
  for (int c = 0; c < kMaxCells; ++c) {
    x[c] = 0.0f;
    if (c < ncell) {
      const int gi = c / gc, gj = c - gi * gc;
      x[c] = load_f32(X + ((int64_t)gi * br + p) * ldx + (int64_t)gj * bc + t);
    }
  }
  float b[FMM_MAX_R], sc[FMM_MAX_R], e[FMM_MAX_R];
  unsigned char qc[FMM_MAX_R], ac[FMM_MAX_R];            // current code, the other candidate (0xFF: none)
  for (int r = 0; r < R; ++r) {
    float acc = 0.0f;
    for (int i = s_off[r]; i < s_off[r + 1]; ++i) {
      const int c = s_cell[i];
      if (c < ncell) acc = __fmaf_rn(s_coef[i], x[c], acc);   // padding entries point at the zero slab
    }
    const float bv = __bfloat162float(__float2bfloat16_rn(acc));   // the block sum as first stored, in bf16
    const int64_t sidx = ((int64_t)r * row_groups + (p >> 7)) * gk + (t >> 7);
    const float amax = __uint_as_float(amax_bits[sidx]);
    const float s = amax > 0.0f ? __fdiv_rn(amax, 448.0f) : 1.0f;
    if ((t & 127) == 0 && (p & 127) == 0) scale_out[sidx] = s;
    unsigned q = (unsigned)__nv_cvt_float_to_fp8(__fdiv_rn(bv, s), __NV_SATFINITE, __NV_E4M3) & 0xFFu;
    if ((q & 0x7Fu) == 0) q = 0;                          // -0 -> 0
    const float dq = __fmul_rn(s, e4m3_value(q));
    unsigned a = 0xFFu;
    if (dq < bv) a = e4m3_neighbour(q, +1);
    if (dq > bv) a = e4m3_neighbour(q, -1);
    b[r] = bv; sc[r] = s; qc[r] = (unsigned char)q; ac[r] = (unsigned char)a;
    e[r] = __fsub_rn(dq, bv);
  }
  for (int sweep = 0; sweep < max_sweeps; ++sweep) {
    bool changed = false;
    for (int r = 0; r < R; ++r) {
      if (ac[r] == 0xFFu) continue;
      const float d_alt = __fmul_rn(sc[r], e4m3_value(ac[r]));
      const float delta = __fsub_rn(d_alt, __fmul_rn(sc[r], e4m3_value(qc[r])));
      float he = 0.0f;
      const float* Hr = H + r * R;
      for (int s2 = 0; s2 < R; ++s2) he = __fmaf_rn(Hr[s2], e[s2], he);
      const float change = __fmaf_rn(__fmul_rn(delta, delta), Hr[r], __fmul_rn(__fmul_rn(2.0f, delta), he));
      if (change < 0.0f) {
        const unsigned char tmp = qc[r]; qc[r] = ac[r]; ac[r] = tmp;
        e[r] = __fsub_rn(d_alt, b[r]);
        changed = true;
      }
    }
    if (!changed) break;
  }
  for (int r = 0; r < R; ++r) out[(int64_t)r * rstride + p * bc + t] = (__nv_fp8_storage_t)qc[r];
}

int sm_count() {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  return sms;
}

}  // namespace

cudaError_t launch_joint_round(int storage, const void* X, int64_t ldx, int gr, int gc, int64_t br, int64_t bc,
                               const CoefTable* d_tab, const float* d_H, const unsigned* amax_bits, float* scale_out,
                               void* out, int64_t out_stride, int max_sweeps, cudaStream_t st) {
  (void)gr;
  const int64_t n = br * bc;
  if (n <= 0) return cudaSuccess;
  const unsigned grid = (unsigned)((n + kJointThreads - 1) / kJointThreads);
  if (storage == FMM_F32)
    joint_round_kernel<float><<<grid, kJointThreads, 0, st>>>((const float*)X, ldx, gc, br, bc, d_tab, d_H, amax_bits,
                                                              scale_out, (__nv_fp8_storage_t*)out, out_stride, max_sweeps);
  else if (storage == FMM_BF16)
    joint_round_kernel<__nv_bfloat16><<<grid, kJointThreads, 0, st>>>((const __nv_bfloat16*)X, ldx, gc, br, bc, d_tab, d_H,
                                                                      amax_bits, scale_out, (__nv_fp8_storage_t*)out,
                                                                      out_stride, max_sweeps);
  else
    return cudaErrorInvalidValue;
  ++fmm_launch_counter();
  return cudaGetLastError();
}

extern "C" fmm_status row_pow2_scale(int storage, const void* dX, int64_t ldx, int64_t rows, int64_t K, float* d_scale,
                                     void* dY, int64_t ldy, void* cuda_stream) {
  if (!dX || !dY || !d_scale) return FMM_ERR_ARG;
  if (storage != FMM_F32 && storage != FMM_BF16) return FMM_ERR_DTYPE;
  if (rows <= 0 || K <= 0 || ldx < K || ldy < K) return FMM_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int64_t want = (rows + 7) / 8, cap = (int64_t)sm_count() * 8;
  const unsigned grid = (unsigned)(want < cap ? want : cap);
  const int64_t eb = storage == FMM_F32 ? 4 : 2;
  const bool vec = (((uintptr_t)dX | (uintptr_t)dY) & 15u) == 0 && (ldx * eb) % 16 == 0 && (ldy * eb) % 16 == 0 &&
                   (K * eb) % 16 == 0;
  if (storage == FMM_F32) {
    if (vec) row_scale_kernel<float, true><<<grid, 256, 0, st>>>((const float*)dX, ldx, rows, K, d_scale, (float*)dY, ldy);
    else row_scale_kernel<float, false><<<grid, 256, 0, st>>>((const float*)dX, ldx, rows, K, d_scale, (float*)dY, ldy);
  } else {
    if (vec) row_scale_kernel<__nv_bfloat16, true><<<grid, 256, 0, st>>>((const __nv_bfloat16*)dX, ldx, rows, K, d_scale, (__nv_bfloat16*)dY, ldy);
    else row_scale_kernel<__nv_bfloat16, false><<<grid, 256, 0, st>>>((const __nv_bfloat16*)dX, ldx, rows, K, d_scale, (__nv_bfloat16*)dY, ldy);
  }
  ++fmm_launch_counter();
  return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

extern "C" fmm_status row_unscale(int output, void* dC, int64_t ldc, int64_t rows, int64_t N, const float* d_scale,
                                  void* cuda_stream) {
  if (!dC || !d_scale) return FMM_ERR_ARG;
  if (output != FMM_F32 && output != FMM_BF16) return FMM_ERR_DTYPE;
  if (rows <= 0 || N <= 0 || ldc < N) return FMM_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int64_t eb = output == FMM_F32 ? 4 : 2;
  const bool vec = ((uintptr_t)dC & 15u) == 0 && (ldc * eb) % 16 == 0 && (N * eb) % 16 == 0;
  const int64_t items = vec ? rows * (N * eb / 16) : rows * N;
  const int64_t want = (items + 255) / 256, cap = (int64_t)sm_count() * 16;
  const unsigned grid = (unsigned)(want < cap ? want : cap);
  if (output == FMM_F32) {
    if (vec) row_unscale_kernel<float, true><<<grid, 256, 0, st>>>((float*)dC, ldc, rows, N, d_scale);
    else row_unscale_kernel<float, false><<<grid, 256, 0, st>>>((float*)dC, ldc, rows, N, d_scale);
  } else {
    if (vec) row_unscale_kernel<__nv_bfloat16, true><<<grid, 256, 0, st>>>((__nv_bfloat16*)dC, ldc, rows, N, d_scale);
    else row_unscale_kernel<__nv_bfloat16, false><<<grid, 256, 0, st>>>((__nv_bfloat16*)dC, ldc, rows, N, d_scale);
  }
  ++fmm_launch_counter();
  return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}
