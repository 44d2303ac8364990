// Randomised Hadamard rotation of the inner dimension (Appendix B, "A rotation, other summation orders and
// repeated runs"): A -> A H and B -> H^T B with H orthogonal leave A B unchanged while changing what the block
// sums of a fast algorithm round.  Here H = diag(signs) . blockdiag(H_h, ..., H_h) / sqrt(h), H_h Sylvester's
// Hadamard matrix, applied to rows whose inner dimension is contiguous (A as stored; B in its [N, K] layout).
//
// A streaming pass (one read, one write per element): a group of h / E lanes of a warp owns one h-block, each lane
// E consecutive elements.  The transform is the fast Walsh-Hadamard recursion in fp32, strides ascending —
// strides below E inside a lane's registers, the rest with xor shuffles — then one multiplication by
// fl(1 / sqrt(h)) and one rounding to the storage type.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>

#include "../../include/fmm_b200.h"
#include "kernels_stream.cuh"

namespace {

constexpr int kRotThreads = 256;

template <int kBytes>
__device__ __forceinline__ void copy_bytes(void* dst, const void* src) {
  if constexpr (kBytes >= 16) {
#pragma unroll
    for (int i = 0; i < kBytes / 16; ++i) reinterpret_cast<uint4*>(dst)[i] = reinterpret_cast<const uint4*>(src)[i];
  } else if constexpr (kBytes == 8) {
    *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(src);
  } else if constexpr (kBytes == 4) {
    *reinterpret_cast<uint32_t*>(dst) = *reinterpret_cast<const uint32_t*>(src);
  } else {
    *reinterpret_cast<uint16_t*>(dst) = *reinterpret_cast<const uint16_t*>(src);
  }
}

// raw storage values and their sign bytes -> fp32 pairs with the sign applied (an exact flip of the sign bit)
template <typename T, int E>
__device__ __forceinline__ void load_signed(const T* raw, const signed char* sg, bool has_signs, bool live, float2* v) {
#pragma unroll
  for (int p = 0; p < E / 2; ++p) {
    uint32_t x0, x1;
    if constexpr (sizeof(T) == 2) {
      const uint32_t two = reinterpret_cast<const uint32_t*>(raw)[p];      // bf16 pair: fp32 bits are the halves shifted up
      x0 = two << 16;
      x1 = two & 0xffff0000u;
    } else {
      x0 = reinterpret_cast<const uint32_t*>(raw)[2 * p];
      x1 = reinterpret_cast<const uint32_t*>(raw)[2 * p + 1];
    }
    if (has_signs) {
      const uint32_t s0 = (uint32_t)(unsigned char)sg[2 * p], s1 = (uint32_t)(unsigned char)sg[2 * p + 1];
      x0 ^= (s0 & 0x80u) << 24;
      x1 ^= (s1 & 0x80u) << 24;
    }
    v[p] = live ? make_float2(__uint_as_float(x0), __uint_as_float(x1)) : make_float2(0.0f, 0.0f);
  }
}
__device__ __forceinline__ void store_pair(float2 x, float* y) { y[0] = x.x; y[1] = x.y; }
__device__ __forceinline__ void store_pair(float2 x, __nv_bfloat16* y) {
  *reinterpret_cast<__nv_bfloat162*>(y) = __float22bfloat162_rn(x);
}

// E elements per lane, L = h / E lanes per h-block (a power of two <= 32), 32 / L blocks per warp pass; a warp takes U
// passes per loop iteration and issues all their loads before it transforms the first (bytes in flight).
template <typename T, int E, int U>
__global__ void __launch_bounds__(kRotThreads)
hadamard_rotate_kernel(const T* __restrict__ X, int64_t ldx, int64_t n_blocks, int blocks_per_row, int h,
                       const signed char* __restrict__ signs, float inv_sqrt_h, T* __restrict__ Y, int64_t ldy) {
  const int L = h / E;
  const int lane = threadIdx.x & 31;
  const int l = lane & (L - 1);            // lane inside its block
  const int sub = lane / L;                // which of the warp's blocks
  const int per_warp = 32 / L;
  const int64_t warps = (int64_t)gridDim.x * (kRotThreads / 32);
  const int64_t warp0 = (int64_t)blockIdx.x * (kRotThreads / 32) + (threadIdx.x >> 5);
  const int64_t passes = (n_blocks + per_warp - 1) / per_warp;
  for (int64_t first = warp0 * U; first < passes; first += warps * U) {     // whole warps iterate together (shuffles below)
    alignas(16) T raw[U][E];
    alignas(16) signed char sg[U][E];
    int64_t off_y[U];
    bool live[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int64_t b = (first + u) * per_warp + sub;
      live[u] = first + u < passes && b < n_blocks;
      const int64_t row = live[u] ? b / blocks_per_row : 0;
      const int col = live[u] ? (int)(b - row * blocks_per_row) * h + l * E : 0;
      off_y[u] = row * ldy + col;
      if (live[u]) {
        copy_bytes<E * (int)sizeof(T)>(raw[u], X + row * ldx + col);
        if (signs != nullptr) copy_bytes<E>(sg[u], signs + col);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float2 v[E / 2];          // (even, odd) neighbours: strides >= 2 and the lane exchanges run as packed fp32 pairs
      load_signed<T, E>(raw[u], sg[u], signs != nullptr, live[u], v);
#pragma unroll
      for (int p = 0; p < E / 2; ++p) {          // stride 1: inside each pair
        const float a = v[p].x, c = v[p].y;
        v[p] = make_float2(__fadd_rn(a, c), __fsub_rn(a, c));
      }
#pragma unroll
      for (int s = 1; s < E / 2; s <<= 1) {      // strides 2 .. E/2 (pair index stride s)
#pragma unroll
        for (int p = 0; p < E / 2; ++p) {
          if ((p & s) == 0) {
            const float2 a = v[p], c = v[p + s];
            v[p] = __fadd2_rn(a, c);
            v[p + s] = __ffma2_rn(c, make_float2(-1.0f, -1.0f), a);     // a - c, one rounding
          }
        }
      }
      for (int s = 1; s < L; s <<= 1) {          // strides E .. h/2: partner lane l ^ s; fma(v, +-1, o) = o +- v exactly once rounded
        const float sgn = (l & s) != 0 ? -1.0f : 1.0f;
        const float2 sg2 = make_float2(sgn, sgn);
#pragma unroll
        for (int p = 0; p < E / 2; ++p) {
          float2 o;
          o.x = __shfl_xor_sync(0xffffffffu, v[p].x, s);
          o.y = __shfl_xor_sync(0xffffffffu, v[p].y, s);
          v[p] = __ffma2_rn(v[p], sg2, o);
        }
      }
      if (live[u]) {
        const float2 r2 = make_float2(inv_sqrt_h, inv_sqrt_h);
#pragma unroll
        for (int p = 0; p < E / 2; ++p) store_pair(__fmul2_rn(v[p], r2), &raw[u][2 * p]);
        copy_bytes<E * (int)sizeof(T)>(Y + off_y[u], raw[u]);
      }
    }
  }
}

template <typename T, int E>
cudaError_t launch_rotate(const void* X, int64_t ldx, int64_t rows, int64_t K, int h, const signed char* signs, void* Y,
                          int64_t ldy, cudaStream_t st) {
  constexpr int kBytes = E * (int)sizeof(T);
  constexpr int U = kBytes >= 64 ? 1 : (kBytes >= 32 ? 2 : 4);
  const int64_t n_blocks = rows * (K / h);
  const int per_warp = 32 / (h / E);
  const int64_t passes = (n_blocks + per_warp - 1) / per_warp;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return cudaErrorInvalidDevice;
  const int64_t per_block = (int64_t)(kRotThreads / 32) * U;
  const int64_t want = (passes + per_block - 1) / per_block;
  const int64_t cap = (int64_t)sms * 8;                        // full occupancy; grid-stride beyond it
  const unsigned grid = (unsigned)(want < cap ? want : cap);
  const float inv = (float)(1.0 / std::sqrt((double)h));
  hadamard_rotate_kernel<T, E, U><<<grid, kRotThreads, 0, st>>>((const T*)X, ldx, n_blocks, (int)(K / h), h, signs, inv,
                                                                 (T*)Y, ldy);
  ++fmm_launch_counter();
  return cudaGetLastError();
}

// elements per lane: 16 bytes where the block is long enough, more once a block outgrows 32 lanes
template <typename T>
cudaError_t launch_rotate_t(const void* X, int64_t ldx, int64_t rows, int64_t K, int h, const signed char* signs, void* Y,
                            int64_t ldy, cudaStream_t st) {
  constexpr int kVec = 16 / (int)sizeof(T);          // 4 (fp32) or 8 (bf16)
  if (h == 2) return launch_rotate<T, 2>(X, ldx, rows, K, h, signs, Y, ldy, st);
  if (h == 4) return launch_rotate<T, 4>(X, ldx, rows, K, h, signs, Y, ldy, st);
  if (h < 128) return launch_rotate<T, kVec>(X, ldx, rows, K, h, signs, Y, ldy, st);
  // from 128 on, more elements per lane: every doubling trades a lane-exchange stage (a shuffle and an FMA per
  // element) for an in-register one (half a packed instruction per element) — the kernel is issue-bound
  // (32 elements per lane lose more to register pressure than they save: 2.8 against 3.6 TB/s at h = 512, bf16)
  if (h <= 32 * 2 * kVec) return launch_rotate<T, 2 * kVec>(X, ldx, rows, K, h, signs, Y, ldy, st);
  if (h <= 32 * 16) return launch_rotate<T, 16>(X, ldx, rows, K, h, signs, Y, ldy, st);
  return launch_rotate<T, 32>(X, ldx, rows, K, h, signs, Y, ldy, st);
}

}  // namespace

extern "C" fmm_status hadamard_rotate(int storage, const void* dX, int64_t ldx, int64_t rows, int64_t K, int h,
                                      const signed char* d_signs, void* dY, int64_t ldy, void* cuda_stream) {
  if (!dX || !dY) return FMM_ERR_ARG;
  if (storage != FMM_F32 && storage != FMM_BF16) return FMM_ERR_DTYPE;
  if (rows <= 0 || K <= 0 || K >= ((int64_t)1 << 31) || h < 2 || h > 1024 || (h & (h - 1)) != 0 || K % h != 0) return FMM_ERR_SHAPE;
  const int64_t eb = storage == FMM_F32 ? 4 : 2;
  if (ldx < K || ldy < K || (ldx * eb) % 16 != 0 || (ldy * eb) % 16 != 0) return FMM_ERR_SHAPE;
  if (((uintptr_t)dX | (uintptr_t)dY | (uintptr_t)d_signs) & 15u) return FMM_ERR_SHAPE;
  if (rows * (K / h) >= ((int64_t)1 << 40)) return FMM_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const cudaError_t e = storage == FMM_F32 ? launch_rotate_t<float>(dX, ldx, rows, K, h, d_signs, dY, ldy, st)
                                            : launch_rotate_t<__nv_bfloat16>(dX, ldx, rows, K, h, d_signs, dY, ldy, st);
  return e == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}
