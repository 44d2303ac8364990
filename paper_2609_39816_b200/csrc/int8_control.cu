// The control of Section 4.2 that breaks condition (iii) of Proposition 1: scales on fine groups of h = call / k inner
// indices while a call of the algorithm spans `call` of them.  A block sum then mixes codes that carry different
// scales, cannot stay an integer, and is "rounded again with one scale, set by its largest magnitude": one scale per
// block sum and call, s = max|x| / b2 in fp32 (1 if all zero), codes = rint(x / s) — the quantiser's own rule with a
// second code bound b2 (a reading: the paper names neither).  The new codes are multiplied exactly, each product is
// rescaled (P * sA) * sB in fp32 and combined with w in fp32, ascending r within a call, calls ascending.
//
// This is a deliberately broken realisation, built to show what the certificate protects against (all 496 row pairs
// of the row-pair test move), not a fast path: plain CUDA-core kernels, one thread per element, every fp32 operation
// written with its rounding so that the result is the CPU restatement's bit for bit.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstring>
#include <vector>

#include "fmm_internal.h"
#include "kernels_stream.cuh"

namespace {

constexpr size_t kAlign = 256;
size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
template <typename T>
T* at(void* ws, size_t off) { return reinterpret_cast<T*>(static_cast<char*>(ws) + off); }

struct ControlLayout {
  size_t status, tabs, codesA, codesB, dA, dB, sumA, sumB, amax, total;
  int64_t calls, fine, bm, bn;
  int h;
};

// tabs: dense fp32 copies of U [R][m][k], V [R][k][n], W [R][m][n]
ControlLayout control_layout(const fmm_scheme& s, int64_t M, int64_t K, int64_t N, int call) {
  ControlLayout L{};
  L.h = call / s.k;
  L.calls = K / call; L.fine = K / L.h; L.bm = M / s.m; L.bn = N / s.n;
  size_t o = 0;
  L.status = o; o += align_up(sizeof(DeviceStatus));
  L.tabs = o; o += align_up((size_t)s.R * (s.m * s.k + s.k * s.n + s.m * s.n) * 4);
  L.codesA = o; o += align_up((size_t)M * K);
  L.codesB = o; o += align_up((size_t)N * K);
  L.dA = o; o += align_up((size_t)M * L.fine * 4);
  L.dB = o; o += align_up((size_t)N * L.fine * 4);
  L.sumA = o; o += align_up((size_t)L.calls * s.R * L.bm * L.h * 4);
  L.sumB = o; o += align_up((size_t)L.calls * s.R * L.bn * L.h * 4);
  L.amax = o; o += align_up((size_t)L.calls * s.R * 2 * 4);
  L.total = o;
  return L;
}

// fine-group quantiser: one thread per (row, fine group); d = max|x| / b in fp32 (1 if all zero), code = rint(x / d)
__global__ void __launch_bounds__(256)
fine_quantize_kernel(const float* __restrict__ X, int64_t ldx, int64_t rows, int64_t fine, int h, float b,
                     int8_t* __restrict__ codes, int64_t K, float* __restrict__ scales) {
  const int64_t id = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (id >= rows * fine) return;
  const int64_t row = id / fine, f = id - row * fine;
  const float* x = X + row * ldx + f * h;
  float amax = 0.0f;
  for (int t = 0; t < h; ++t) amax = fmaxf(amax, fabsf(x[t]));
  const float d = amax == 0.0f ? 1.0f : __fdiv_rn(amax, b);
  scales[id] = d;
  for (int t = 0; t < h; ++t) codes[row * K + f * h + t] = (int8_t)__float2int_rn(__fdiv_rn(x[t], d));
}

// block sums of the dequantised entries: one thread per (call, product, block row p, t).  coef: [R][gr][gc] with gc = k for
// A (cell (i, l)) and [R][k][n] read as cell (l, j) for B (b_side): the order of the chain is ascending (i, l) resp. (l, j).
__global__ void __launch_bounds__(256)
control_block_sum_kernel(const int8_t* __restrict__ codes, const float* __restrict__ scales, int64_t K, int64_t fine,
                         const float* __restrict__ coef, int R, int m_or_n, int k, int b_side, int64_t br, int h, int call,
                         int64_t calls, float* __restrict__ sums, unsigned* __restrict__ amax_bits) {
  const int64_t id = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const int64_t total = calls * R * br * h;
  if (id >= total) return;
  const int t = (int)(id % h);
  const int64_t p = (id / h) % br;
  const int r = (int)((id / (h * br)) % R);
  const int64_t q = id / ((int64_t)h * br * R);
  float sum = 0.0f;
  if (!b_side) {
    for (int i = 0; i < m_or_n; ++i)
      for (int l = 0; l < k; ++l) {
        const float u = coef[(r * m_or_n + i) * k + l];
        if (u == 0.0f) continue;
        const int64_t row = i * br + p, col = q * call + (int64_t)l * h + t;
        const float x = __fmul_rn((float)codes[row * K + col], scales[row * fine + col / h]);
        sum = __fmaf_rn(u, x, sum);
      }
  } else {
    for (int l = 0; l < k; ++l)
      for (int j = 0; j < m_or_n; ++j) {
        const float v = coef[(r * k + l) * m_or_n + j];
        if (v == 0.0f) continue;
        const int64_t row = j * br + p, col = q * call + (int64_t)l * h + t;
        const float x = __fmul_rn((float)codes[row * K + col], scales[row * fine + col / h]);
        sum = __fmaf_rn(v, x, sum);
      }
  }
  sums[id] = sum;
  const unsigned bits = __float_as_uint(fabsf(sum));     // non-negative floats order like their bit patterns
  if (bits != 0u && !(bits > 0x7f800000u)) atomicMax(&amax_bits[(q * R + r) * 2 + b_side], bits);
}

// the second rounding: one scale per block sum and call; the sums are replaced by their integer codes (as floats)
__global__ void __launch_bounds__(256)
control_requantize_kernel(float* __restrict__ sums, int64_t per_tensor, int64_t tensors, const unsigned* __restrict__ amax_bits,
                          int b_side, float b2) {
  const int64_t id = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (id >= per_tensor * tensors) return;
  const float amax = __uint_as_float(amax_bits[(id / per_tensor) * 2 + b_side]);
  const float s = amax == 0.0f ? 1.0f : __fdiv_rn(amax, b2);
  sums[id] = rintf(__fdiv_rn(sums[id], s));
}

// products and combination: one thread per position (p, c) of a block, all m x n output blocks of that position in
// registers; for every call and product: the exact integer product of the two code rows, (P * sA) * sB, and
// acc_ij = fma(w_ij, that, acc_ij), ascending r within a call, calls ascending; one rounding to the output dtype.
template <typename OutT>
__global__ void __launch_bounds__(128)
control_product_kernel(const float* __restrict__ codesA, const float* __restrict__ codesB, const unsigned* __restrict__ amax_bits,
                       const float* __restrict__ W, int R, int m, int n, int64_t bm, int64_t bn, int h, int64_t calls, float b2,
                       OutT* __restrict__ C, int64_t ldc) {
  const int64_t id = (int64_t)blockIdx.x * 128 + threadIdx.x;
  if (id >= bm * bn) return;
  const int64_t p = id / bn, c = id - p * bn;
  float acc[FMM_MAX_GRID * FMM_MAX_GRID];
#pragma unroll
  for (int x = 0; x < FMM_MAX_GRID * FMM_MAX_GRID; ++x) acc[x] = 0.0f;
  for (int64_t q = 0; q < calls; ++q)
    for (int r = 0; r < R; ++r) {
      const float* a = codesA + ((q * R + r) * bm + p) * h;
      const float* b = codesB + ((q * R + r) * bn + c) * h;
      long long prod = 0;
      for (int t = 0; t < h; ++t) prod += (long long)a[t] * (long long)b[t];
      const float amaxA = __uint_as_float(amax_bits[(q * R + r) * 2 + 0]), amaxB = __uint_as_float(amax_bits[(q * R + r) * 2 + 1]);
      const float sA = amaxA == 0.0f ? 1.0f : __fdiv_rn(amaxA, b2), sB = amaxB == 0.0f ? 1.0f : __fdiv_rn(amaxB, b2);
      const float scaled = __fmul_rn(__fmul_rn((float)prod, sA), sB);
#pragma unroll
      for (int i = 0; i < FMM_MAX_GRID; ++i)
#pragma unroll
        for (int j = 0; j < FMM_MAX_GRID; ++j)
          if (i < m && j < n) {
            const float w = W[(r * m + i) * n + j];
            if (w != 0.0f) acc[i * FMM_MAX_GRID + j] = __fmaf_rn(w, scaled, acc[i * FMM_MAX_GRID + j]);
          }
    }
#pragma unroll
  for (int i = 0; i < FMM_MAX_GRID; ++i)
#pragma unroll
    for (int j = 0; j < FMM_MAX_GRID; ++j)
      if (i < m && j < n) C[(i * bm + p) * ldc + j * bn + c] = (OutT)acc[i * FMM_MAX_GRID + j];
}

fmm_status control_shape_ok(const fmm_scheme* s, int64_t M, int64_t K, int64_t N, int call) {
  if (!s) return FMM_ERR_ARG;
  if (M <= 0 || K <= 0 || N <= 0 || call <= 0) return FMM_ERR_SHAPE;
  if (M % s->m || N % s->n || call % s->k || K % call) return FMM_ERR_SHAPE;
  if (M * K >= ((int64_t)1 << 31) || N * K >= ((int64_t)1 << 31)) return FMM_ERR_SHAPE;   // a control for tiles, not for layers
  return FMM_OK;
}

}  // namespace

extern "C" {

size_t int8_finegroup_control_workspace(const fmm_scheme* s, int64_t M, int64_t K, int64_t N, int call) {
  if (control_shape_ok(s, M, K, N, call) != FMM_OK) return 0;
  return control_layout(*s, M, K, N, call).total;
}

fmm_status int8_finegroup_control(const fmm_scheme* s, int code_bound, int second_bound, const float* d_A, int64_t lda,
                                  const float* d_B, int64_t ldb, int64_t M, int64_t K, int64_t N, int call, int output,
                                  void* d_C, int64_t ldc, void* d_ws, size_t ws_bytes, void* cuda_stream) {
  if (!d_A || !d_B || !d_C) return FMM_ERR_ARG;
  if (output != FMM_F32 && output != FMM_BF16) return FMM_ERR_DTYPE;
  if (code_bound < 1 || code_bound > 127 || second_bound < 1 || second_bound > 127) return FMM_ERR_ARG;
  fmm_status rc = control_shape_ok(s, M, K, N, call);
  if (rc != FMM_OK) return rc;
  if (lda < K || ldb < K || ldc < N) return FMM_ERR_SHAPE;
  const ControlLayout L = control_layout(*s, M, K, N, call);
  if (!d_ws || (reinterpret_cast<uintptr_t>(d_ws) & 255u) || ws_bytes < L.total) return FMM_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int R = s->R, m = s->m, k = s->k, n = s->n;
  // coefficients as fp32, the values every other path of the library uses
  std::vector<float> tabs((size_t)R * (m * k + k * n + m * n));
  float* hU = tabs.data(); float* hV = hU + (size_t)R * m * k; float* hW = hV + (size_t)R * k * n;
  for (size_t x = 0; x < (size_t)R * m * k; ++x) hU[x] = (float)s->U[x];
  for (size_t x = 0; x < (size_t)R * k * n; ++x) hV[x] = (float)s->V[x];
  for (size_t x = 0; x < (size_t)R * m * n; ++x) hW[x] = (float)s->W[x];
  float* dU = at<float>(d_ws, L.tabs); float* dV = dU + (size_t)R * m * k; float* dW = dV + (size_t)R * k * n;
  if (cudaMemcpyAsync(dU, tabs.data(), tabs.size() * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return FMM_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return FMM_ERR_CUDA;   // the host vector goes away when this call returns
  if (cudaMemsetAsync(at<char>(d_ws, L.status), 0, sizeof(DeviceStatus), st) != cudaSuccess) return FMM_ERR_CUDA;
  if (cudaMemsetAsync(at<char>(d_ws, L.amax), 0, (size_t)L.calls * R * 2 * 4, st) != cudaSuccess) return FMM_ERR_CUDA;
  auto blocks = [](int64_t items, int per) { return (unsigned)((items + per - 1) / per); };
  int8_t* cA = at<int8_t>(d_ws, L.codesA); int8_t* cB = at<int8_t>(d_ws, L.codesB);
  float* sA = at<float>(d_ws, L.dA); float* sB = at<float>(d_ws, L.dB);
  fine_quantize_kernel<<<blocks(M * L.fine, 256), 256, 0, st>>>(d_A, lda, M, L.fine, L.h, (float)code_bound, cA, K, sA);
  fine_quantize_kernel<<<blocks(N * L.fine, 256), 256, 0, st>>>(d_B, ldb, N, L.fine, L.h, (float)code_bound, cB, K, sB);
  float* sumA = at<float>(d_ws, L.sumA); float* sumB = at<float>(d_ws, L.sumB);
  unsigned* amax = at<unsigned>(d_ws, L.amax);
  control_block_sum_kernel<<<blocks(L.calls * R * L.bm * L.h, 256), 256, 0, st>>>(cA, sA, K, L.fine, dU, R, m, k, 0, L.bm, L.h, call,
                                                                                  L.calls, sumA, amax);
  control_block_sum_kernel<<<blocks(L.calls * R * L.bn * L.h, 256), 256, 0, st>>>(cB, sB, K, L.fine, dV, R, n, k, 1, L.bn, L.h, call,
                                                                                  L.calls, sumB, amax);
  control_requantize_kernel<<<blocks(L.calls * R * L.bm * L.h, 256), 256, 0, st>>>(sumA, L.bm * L.h, L.calls * R, amax, 0, (float)second_bound);
  control_requantize_kernel<<<blocks(L.calls * R * L.bn * L.h, 256), 256, 0, st>>>(sumB, L.bn * L.h, L.calls * R, amax, 1, (float)second_bound);
  if (output == FMM_F32)
    control_product_kernel<float><<<blocks(L.bm * L.bn, 128), 128, 0, st>>>(sumA, sumB, amax, dW, R, m, n, L.bm, L.bn, L.h, L.calls,
                                                                            (float)second_bound, (float*)d_C, ldc);
  else
    control_product_kernel<__nv_bfloat16><<<blocks(L.bm * L.bn, 128), 128, 0, st>>>(sumA, sumB, amax, dW, R, m, n, L.bm, L.bn, L.h,
                                                                                    L.calls, (float)second_bound, (__nv_bfloat16*)d_C, ldc);
  fmm_launch_counter() += 7;
  return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

}  // extern "C"
