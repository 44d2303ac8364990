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

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f32(float x, float* y) { *y = x; }
__device__ __forceinline__ void from_f32(float x, __nv_bfloat16* y) { *y = __float2bfloat16_rn(x); }

// E elements per lane, L = h / E lanes per h-block (a power of two <= 32), 32 / L blocks per warp pass.
template <typename T, int E>
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
  for (int64_t pass = warp0; pass < passes; pass += warps) {     // whole warps iterate together (shuffles below)
    const int64_t b = pass * per_warp + sub;
    const bool live = b < n_blocks;
    const int64_t row = live ? b / blocks_per_row : 0;
    const int col = live ? (int)(b - row * blocks_per_row) * h + l * E : 0;
    alignas(16) T raw[E];
    float v[E];
    if (live) {
      copy_bytes<E * (int)sizeof(T)>(raw, X + row * ldx + col);
#pragma unroll
      for (int j = 0; j < E; ++j) v[j] = to_f32(raw[j]);
      if (signs != nullptr) {
        alignas(16) signed char sg[E];
        copy_bytes<E>(sg, signs + col);
#pragma unroll
        for (int j = 0; j < E; ++j) v[j] = sg[j] < 0 ? -v[j] : v[j];
      }
    } else {
#pragma unroll
      for (int j = 0; j < E; ++j) v[j] = 0.0f;
    }
#pragma unroll
    for (int s = 1; s < E; s <<= 1) {
#pragma unroll
      for (int i = 0; i < E; ++i) {
        if ((i & s) == 0) {
          const float a = v[i], c = v[i + s];
          v[i] = __fadd_rn(a, c);
          v[i + s] = __fsub_rn(a, c);
        }
      }
    }
    for (int s = 1; s < L; s <<= 1) {
      const bool upper = (l & s) != 0;
#pragma unroll
      for (int j = 0; j < E; ++j) {
        const float o = __shfl_xor_sync(0xffffffffu, v[j], s);
        v[j] = upper ? __fsub_rn(o, v[j]) : __fadd_rn(v[j], o);
      }
    }
    if (live) {
#pragma unroll
      for (int j = 0; j < E; ++j) from_f32(__fmul_rn(v[j], inv_sqrt_h), &raw[j]);
      copy_bytes<E * (int)sizeof(T)>(Y + row * ldy + col, raw);
    }
  }
}

template <typename T, int E>
cudaError_t launch_rotate(const void* X, int64_t ldx, int64_t rows, int64_t K, int h, const signed char* signs, void* Y,
                          int64_t ldy, cudaStream_t st) {
  const int64_t n_blocks = rows * (K / h);
  const int per_warp = 32 / (h / E);
  const int64_t passes = (n_blocks + per_warp - 1) / per_warp;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return cudaErrorInvalidDevice;
  const int64_t want = (passes + kRotThreads / 32 - 1) / (kRotThreads / 32);
  const int64_t cap = (int64_t)sms * 16;                       // grid-stride beyond 16 blocks per SM
  const unsigned grid = (unsigned)(want < cap ? want : cap);
  const float inv = (float)(1.0 / std::sqrt((double)h));
  hadamard_rotate_kernel<T, E><<<grid, kRotThreads, 0, st>>>((const T*)X, ldx, n_blocks, (int)(K / h), h, signs, inv,
                                                              (T*)Y, ldy);
  ++fmm_launch_counter();
  return cudaGetLastError();
}

template <typename T>
cudaError_t launch_rotate_t(const void* X, int64_t ldx, int64_t rows, int64_t K, int h, const signed char* signs, void* Y,
                            int64_t ldy, cudaStream_t st) {
  if (h == 2) return launch_rotate<T, 2>(X, ldx, rows, K, h, signs, Y, ldy, st);
  if (h <= 128) return launch_rotate<T, 4>(X, ldx, rows, K, h, signs, Y, ldy, st);
  if (h == 256) return launch_rotate<T, 8>(X, ldx, rows, K, h, signs, Y, ldy, st);
  if (h == 512) return launch_rotate<T, 16>(X, ldx, rows, K, h, signs, Y, ldy, st);
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
