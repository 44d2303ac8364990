// Certified realisation on bounded integer codes (Section 4.2, Proposition 1; quantisation specification of
// Appendix D): quantiser, the group-scaled int8 operator computed classically or by an algorithm <m,k,n;R> with
// integer coefficients called once per group of 128 inner indices, and the certificate check.
//
// Arithmetic: codes and block sums are integers of magnitude <= 127, exact in bf16; every product and every
// partial sum formed in a call is an integer below 2^24, exact in the fp32 accumulators of the tensor cores and
// of the decode.  The integer product of a group is therefore the exact one whatever the algorithm, and the
// rescale (P * d_A) * d_B, accumulated over ascending groups in fp32, gives the classical operator's bits.
//
// Data flow per call (all groups at once):
//   pack     int8 codes [rows][K]            -> bf16 cell matrix [(i, group, p)][(l, t)], t padded to 64
//   encode   block sums over the m x k grid  -> Ahat_r [group][bm][w]           (existing encode kernel)
//   products (r, group): Ahat_r[group] Bhat_r[group]^T -> fp32 [R][G][bm][bn]   (existing tcgen05 kernels)
//   decode   per group: P = sum_r w M_r, x = (P * d_A) * d_B, C += x; one cast at the end
#include <cuda_bf16.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <memory>
#include <vector>

#include "fmm_internal.h"
#include "kernels_stream.cuh"

namespace {

constexpr int kGroup = 128;           // inner indices that share a scale (Appendix D)
constexpr int kQuantThreads = 256;
constexpr int kDecThreads = 256;
constexpr size_t kAlign = 256;
constexpr int kSlabPadBytes = 256;    // spacing pad between consecutive slabs (avoids power-of-two strides)

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
template <typename T>
T* at(void* ws, size_t off) { return reinterpret_cast<T*>(static_cast<char*>(ws) + off); }

#define FMM_CUDA(x) do { if ((x) != cudaSuccess) return FMM_ERR_CUDA; } while (0)
#define FMM_TRY(x) do { fmm_status _s = (x); if (_s != FMM_OK) return _s; } while (0)

// ------------------------------------------------------------------------------------------
// Quantiser: one warp per (row, group).  d = max|x| / b in fp32 (1 for an all-zero group), code = x / d rounded
// to nearest even; IEEE division on both (the decision that fixes an integer is taken in fp32, as specified).
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void load4(const float* p, float v[4]) {
  const float4 x = *reinterpret_cast<const float4*>(p);
  v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* p, float v[4]) {
  const uint2 raw = *reinterpret_cast<const uint2*>(p);
  const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
  const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
  v[0] = __low2float(lo); v[1] = __high2float(lo); v[2] = __low2float(hi); v[3] = __high2float(hi);
}

template <typename SrcT>
__global__ void __launch_bounds__(kQuantThreads)
quantize_kernel(const SrcT* __restrict__ X, int64_t ldx, int64_t rows, int G, float b, int8_t* __restrict__ codes,
                float* __restrict__ scales) {
  const int lane = threadIdx.x & 31;
  const int64_t total = rows * G;
  for (int64_t id = (int64_t)blockIdx.x * (kQuantThreads / 32) + (threadIdx.x >> 5); id < total;
       id += (int64_t)gridDim.x * (kQuantThreads / 32)) {
    const int64_t row = id / G;
    const int g = (int)(id - row * G);
    float v[4];
    load4(X + row * ldx + (int64_t)g * kGroup + lane * 4, v);
    float amax = fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3])));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const float d = amax == 0.0f ? 1.0f : __fdiv_rn(amax, b);
    uint32_t packed = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int c = __float2int_rn(__fdiv_rn(v[e], d));
      packed |= ((uint32_t)c & 0xffu) << (8 * e);
    }
    *reinterpret_cast<uint32_t*>(codes + (row * G + g) * kGroup + lane * 4) = packed;
    if (lane == 0) scales[row * G + g] = d;
  }
}

// ------------------------------------------------------------------------------------------
// Pack: int8 codes [gr*br][K] -> bf16 matrix with rows (i, group, p) and columns (l, t), t in [0, w), zero for
// t >= h.  Block (i, l) of that matrix is the stack over groups of the [br x h] code blocks, so one encode pass
// and one grouped product launch serve every group.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
pack_kernel(const int8_t* __restrict__ codes, int64_t K, int64_t br, int G, int kk, int h, int w, int64_t nvec,
            __nv_bfloat16* __restrict__ Xq) {
  const int vpr = kk * w / 8;   // 16-byte vectors per packed row
  for (int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x; idx < nvec; idx += (int64_t)gridDim.x * 256) {
    const int64_t rowp = idx / vpr;
    const int col = (int)(idx - rowp * vpr) * 8;
    const int l = col / w, t = col - l * w;
    const int64_t i = rowp / (G * br);
    const int64_t rem = rowp - i * (G * br);
    const int64_t g = rem / br, p = rem - g * br;
    uint4 out = make_uint4(0u, 0u, 0u, 0u);
    if (t < h) {
      const uint2 raw = *reinterpret_cast<const uint2*>(codes + (i * br + p) * K + g * kGroup + l * h + t);
      uint32_t o[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t word = e < 2 ? raw.x : raw.y;
        const int c0 = (int)(int8_t)((word >> (16 * (e & 1))) & 0xffu);
        const int c1 = (int)(int8_t)((word >> (16 * (e & 1) + 8)) & 0xffu);
        const __nv_bfloat162 two = __floats2bfloat162_rn((float)c0, (float)c1);
        o[e] = *reinterpret_cast<const uint32_t*>(&two);
      }
      out = make_uint4(o[0], o[1], o[2], o[3]);
    }
    *reinterpret_cast<uint4*>(Xq + idx * 8) = out;
  }
}

// ------------------------------------------------------------------------------------------
// Grouped decode and rescale.  A block owns kPos position quads (4 consecutive columns of one row position of
// every C block); kSplit threads share a position and split the C blocks between them.  For every group in
// ascending order the R product vectors of the position are staged in shared memory, each thread forms its
// blocks' integer sums (exact in fp32), multiplies by d_A and then by d_B (two roundings, no fused
// multiply-add), and adds to its fp32 accumulators; one rounding to the output dtype after the last group.
// ------------------------------------------------------------------------------------------
struct GDecHead {
  int off[FMM_MAX_GRID * FMM_MAX_GRID + 1];
  int pad[3];
};

__device__ __forceinline__ void store4(__nv_bfloat16* p, float4 v) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  const __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 raw;
  raw.x = *reinterpret_cast<const uint32_t*>(&lo);
  raw.y = *reinterpret_cast<const uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = raw;
}
__device__ __forceinline__ void store4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }

template <typename OutT, int kSplit, int kStages, int kCells, bool kIntAcc>
__global__ void __launch_bounds__(kDecThreads)
decode_group_kernel(const float* __restrict__ prod, int64_t pstride, int G, const CoefTable* __restrict__ d_tab,
                    int R, const float* __restrict__ dAt, const float* __restrict__ dBt, int64_t Mtot, int64_t Ntot,
                    int n, int64_t bm, int64_t bn, OutT* __restrict__ C, int64_t ldc) {
  constexpr int kPos = kDecThreads / kSplit;   // kSplit * kCells >= number of C blocks
  constexpr int kSlab = kPos * 16;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  GDecHead& sm = *reinterpret_cast<GDecHead*>(smem_raw);
  const int ncell = d_tab->R;
  const int total = d_tab->off[ncell];
  int2* ent = reinterpret_cast<int2*>(smem_raw + sizeof(GDecHead));
  unsigned char* stage = smem_raw + ((sizeof(GDecHead) + (size_t)total * 8 + 15) / 16) * 16;
  const int stage_bytes = (R + 1) * kSlab;   // R product slabs and the all-zero padding slab

  const int tg = threadIdx.x / kPos;
  const int pq = threadIdx.x - tg * kPos;
  const int vec_per_row = (int)(bn >> 2);
  const int nvec = (int)bm * vec_per_row;
  const int idx = blockIdx.x * kPos + pq;
  const bool live = idx < nvec;
  const int p = live ? idx / vec_per_row : 0;
  const int q = live ? (idx - p * vec_per_row) << 2 : 0;
  unsigned char* my_stage = stage + pq * 16;
  const uint32_t dst0 = (uint32_t)__cvta_generic_to_shared(my_stage);
  const float* src = prod + (int64_t)p * bn + q;
  const int nbytes = live ? 16 : 0;   // 0 source bytes: the destination is zero-filled

  // the copies of group g land in ring slot g % kStages; kStages - 1 groups are in flight ahead of the reader
  auto issue = [&](int g) {
    if (g < G) {
      const uint32_t dst = dst0 + (uint32_t)((g % kStages) * stage_bytes);
      for (int r = tg; r < R; r += kSplit)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + r * kSlab),
                     "l"(src + ((int64_t)r * G + g) * pstride), "r"(nbytes) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");   // one (possibly empty) commit per step keeps the count uniform
  };
#pragma unroll
  for (int g = 0; g < kStages - 1; ++g) issue(g);

  for (int i = threadIdx.x; i <= ncell; i += kDecThreads) sm.off[i] = d_tab->off[i];
  for (int i = threadIdx.x; i < total; i += kDecThreads)
    ent[i] = make_int2(d_tab->cell[i] * kSlab, __float_as_int(d_tab->coef[i]));
  if (tg == 0)
#pragma unroll
    for (int b = 0; b < kStages; ++b)
      *reinterpret_cast<float4*>(my_stage + b * stage_bytes + R * kSlab) = make_float4(0.f, 0.f, 0.f, 0.f);

  float4 acc[kCells];
#pragma unroll
  for (int u = 0; u < kCells; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);

  for (int g = 0; g < G; ++g) {
    asm volatile("cp.async.wait_group %0;" ::"n"(kStages - 2) : "memory");   // this thread's copies of group g are done
    __syncthreads();            // everyone's are; and the slot read in the previous step is free again
    issue(g + kStages - 1);
    const unsigned char* cur = my_stage + (g % kStages) * stage_bytes;
#pragma unroll
    for (int u4 = 0; u4 < kCells; ++u4) {
      const int c = tg + u4 * kSplit;
      if (c >= ncell) break;
      float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
      const int e1 = sm.off[c + 1];
      if (kIntAcc) {
        // partial sums may pass 2^24 (each product is below it, the result is below it): add in int32
        int4 xi = make_int4(0, 0, 0, 0);
        for (int e = sm.off[c]; e < e1; ++e) {
          const int2 en = ent[e];
          const float4 v = *reinterpret_cast<const float4*>(cur + en.x);
          const int w = __float2int_rn(__int_as_float(en.y));
          xi.x += w * __float2int_rn(v.x); xi.y += w * __float2int_rn(v.y);
          xi.z += w * __float2int_rn(v.z); xi.w += w * __float2int_rn(v.w);
        }
        x = make_float4((float)xi.x, (float)xi.y, (float)xi.z, (float)xi.w);
      } else {
        for (int e = sm.off[c]; e < e1; e += 2) {   // lists are padded to an even number of entries
          const int4 two = *reinterpret_cast<const int4*>(&ent[e]);
          const float4 v0 = *reinterpret_cast<const float4*>(cur + two.x);
          const float4 v1 = *reinterpret_cast<const float4*>(cur + two.z);
          const float w0 = __int_as_float(two.y), w1 = __int_as_float(two.w);
          x.x = __fmaf_rn(w0, v0.x, x.x); x.y = __fmaf_rn(w0, v0.y, x.y);   // integers below 2^24: exact
          x.z = __fmaf_rn(w0, v0.z, x.z); x.w = __fmaf_rn(w0, v0.w, x.w);
          x.x = __fmaf_rn(w1, v1.x, x.x); x.y = __fmaf_rn(w1, v1.y, x.y);
          x.z = __fmaf_rn(w1, v1.z, x.z); x.w = __fmaf_rn(w1, v1.w, x.w);
        }
      }
      if (live) {
        const int i = c / n, j = c - i * n;
        const float da = dAt[(int64_t)g * Mtot + (int64_t)i * bm + p];
        const float4 db = *reinterpret_cast<const float4*>(dBt + (int64_t)g * Ntot + (int64_t)j * bn + q);
        acc[u4].x = __fadd_rn(acc[u4].x, __fmul_rn(__fmul_rn(x.x, da), db.x));
        acc[u4].y = __fadd_rn(acc[u4].y, __fmul_rn(__fmul_rn(x.y, da), db.y));
        acc[u4].z = __fadd_rn(acc[u4].z, __fmul_rn(__fmul_rn(x.z, da), db.z));
        acc[u4].w = __fadd_rn(acc[u4].w, __fmul_rn(__fmul_rn(x.w, da), db.w));
      }
    }
  }
  if (live) {
#pragma unroll
    for (int u4 = 0; u4 < kCells; ++u4) {
      const int c = tg + u4 * kSplit;
      if (c >= ncell) break;
      const int i = c / n, j = c - i * n;
      store4(C + ((int64_t)i * bm + p) * ldc + (int64_t)j * bn + q, acc[u4]);
    }
  }
}

// The classical operator needs no decode: one product per group.  A thread owns four consecutive outputs and walks
// the groups in ascending order, eight independent 16-byte loads in flight per step.
template <typename OutT>
__global__ void __launch_bounds__(256)
rescale_groups_kernel(const float* __restrict__ prod, int64_t pstride, int G, const float* __restrict__ dAt,
                      const float* __restrict__ dBt, int64_t M, int64_t N, OutT* __restrict__ C, int64_t ldc) {
  const int vec_per_row = (int)(N >> 2);
  const int64_t nvec = M * vec_per_row;
  const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (idx >= nvec) return;
  const int64_t p = idx / vec_per_row;
  const int64_t q = (idx - p * vec_per_row) << 2;
  const float* src = prod + p * N + q;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  constexpr int kU = 8;
  for (int g0 = 0; g0 < G; g0 += kU) {
    float4 v[kU], db[kU];
    float da[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int g = min(g0 + u, G - 1);   // the tail re-reads the last group; its result is not used
      v[u] = __ldcs(reinterpret_cast<const float4*>(src + (int64_t)g * pstride));
      db[u] = *reinterpret_cast<const float4*>(dBt + (int64_t)g * N + q);
      da[u] = dAt[(int64_t)g * M + p];
    }
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      if (g0 + u < G) {
        acc.x = __fadd_rn(acc.x, __fmul_rn(__fmul_rn(v[u].x, da[u]), db[u].x));
        acc.y = __fadd_rn(acc.y, __fmul_rn(__fmul_rn(v[u].y, da[u]), db[u].y));
        acc.z = __fadd_rn(acc.z, __fmul_rn(__fmul_rn(v[u].z, da[u]), db[u].z));
        acc.w = __fadd_rn(acc.w, __fmul_rn(__fmul_rn(v[u].w, da[u]), db[u].w));
      }
    }
  }
  store4(C + p * ldc + q, acc);
}

// scales [rows][G] -> [G][rows] (a few hundred KB: the decode reads one contiguous vector per group)
__global__ void __launch_bounds__(256) transpose_scales_kernel(const float* __restrict__ d, int64_t rows, int G,
                                                               float* __restrict__ dt) {
  const int64_t total = rows * G;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < total; i += (int64_t)gridDim.x * 256) {
    const int64_t g = i / rows, r = i - g * rows;
    dt[i] = d[r * G + g];
  }
}

// ------------------------------------------------------------------------------------------
// Block sums of int8 codes with the overflow split of Section 4.3: X = X0 + 256 R, R = floor((X + 128) / 256),
// X0 in [-128, 127].  One thread forms, for one (group, row position) and four consecutive inner indices t, the
// block sums of every product and writes them as bf16 (all values exact: |X0| <= 128, 256 |R| <= 512) into rows
// of 4h elements laid out so that ONE contraction over the row gives all four products of Eq. 2:
//   A side: [ A0 | 256 R_A | A0 | 256 R_A ]      B side: [ B0 | B0 | 256 R_B | 256 R_B ]
//   sum = A0 B0 + 256 R_A B0 + 256 A0 R_B + 256^2 R_A R_B = Ahat Bhat.
// The thread's codes are staged in shared memory ([cell][thread] words) so that the coefficient lists can index them.
// ------------------------------------------------------------------------------------------
constexpr int kSplitThreads = 128;

__global__ void __launch_bounds__(kSplitThreads)
encode_split_kernel(const int8_t* __restrict__ codes, int64_t K, int gc, int64_t br, int G, int h, int b_side,
                    const CoefTable* __restrict__ d_tab, __nv_bfloat16* __restrict__ out, int64_t rstride, int64_t nquad) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int R = d_tab->R, ncell = d_tab->ncell;
  const int total = d_tab->off[R];
  int* off = reinterpret_cast<int*>(smem_raw);                       // R + 1 list offsets
  int2* ent = reinterpret_cast<int2*>(smem_raw + ((size_t)(R + 1) * 4 + 15) / 16 * 16);
  uint32_t* stage = reinterpret_cast<uint32_t*>(reinterpret_cast<unsigned char*>(ent) + (size_t)total * 8);
  for (int i = threadIdx.x; i <= R; i += kSplitThreads) off[i] = d_tab->off[i];
  for (int i = threadIdx.x; i < total; i += kSplitThreads)
    ent[i] = make_int2(d_tab->cell[i], __float2int_rn(d_tab->coef[i]));
  stage[ncell * kSplitThreads + threadIdx.x] = 0u;                    // the padding cell
  const int64_t idx = (int64_t)blockIdx.x * kSplitThreads + threadIdx.x;
  const bool live = idx < nquad;
  const int qpr = h / 4;                                              // quads per (group, row position)
  const int64_t rowp = live ? idx / qpr : 0;                          // (group, p)
  const int t = live ? (int)(idx - rowp * qpr) * 4 : 0;
  const int64_t g = rowp / br, p = rowp - g * br;
  for (int c = 0; c < ncell; ++c) {
    const int gi = c / gc, gj = c - gi * gc;
    stage[c * kSplitThreads + threadIdx.x] =
        live ? *reinterpret_cast<const uint32_t*>(codes + ((int64_t)gi * br + p) * K + g * kGroup + gj * h + t) : 0u;
  }
  __syncthreads();
  if (!live) return;
  __nv_bfloat16* row = out + rowp * (4 * h) + t;
  for (int r = 0; r < R; ++r) {
    int s0 = 0, s1 = 0, s2 = 0, s3 = 0;
    for (int e = off[r]; e < off[r + 1]; ++e) {
      const int2 en = ent[e];
      const uint32_t wv = stage[en.x * kSplitThreads + threadIdx.x];
      s0 += en.y * (int)(int8_t)(wv & 0xffu);
      s1 += en.y * (int)(int8_t)((wv >> 8) & 0xffu);
      s2 += en.y * (int)(int8_t)((wv >> 16) & 0xffu);
      s3 += en.y * (int)(int8_t)(wv >> 24);
    }
    // arithmetic shift = floor division by 256 for either sign
    const int h0 = (s0 + 128) >> 8, h1 = (s1 + 128) >> 8, h2 = (s2 + 128) >> 8, h3 = (s3 + 128) >> 8;
    const __nv_bfloat162 lo01 = __floats2bfloat162_rn((float)(s0 - 256 * h0), (float)(s1 - 256 * h1));
    const __nv_bfloat162 lo23 = __floats2bfloat162_rn((float)(s2 - 256 * h2), (float)(s3 - 256 * h3));
    const __nv_bfloat162 hi01 = __floats2bfloat162_rn((float)(256 * h0), (float)(256 * h1));
    const __nv_bfloat162 hi23 = __floats2bfloat162_rn((float)(256 * h2), (float)(256 * h3));
    const uint2 lo = make_uint2(*reinterpret_cast<const uint32_t*>(&lo01), *reinterpret_cast<const uint32_t*>(&lo23));
    const uint2 hi = make_uint2(*reinterpret_cast<const uint32_t*>(&hi01), *reinterpret_cast<const uint32_t*>(&hi23));
    __nv_bfloat16* dst = row + (int64_t)r * rstride;
    *reinterpret_cast<uint2*>(dst) = lo;
    *reinterpret_cast<uint2*>(dst + h) = b_side ? lo : hi;
    *reinterpret_cast<uint2*>(dst + 2 * h) = b_side ? hi : lo;
    *reinterpret_cast<uint2*>(dst + 3 * h) = hi;
  }
}

cudaError_t launch_encode_split(const int8_t* codes, int64_t K, int gr, int gc, int64_t br, int G, int h, bool b_side,
                                const CoefTable* d_tab, const CoefTable* h_tab, __nv_bfloat16* out, int64_t rstride,
                                cudaStream_t st) {
  const int64_t nquad = (int64_t)G * br * (h / 4);
  const size_t smem = ((size_t)(h_tab->R + 1) * 4 + 15) / 16 * 16 + (size_t)h_tab->off[h_tab->R] * 8 +
                      (size_t)(gr * gc + 1) * kSplitThreads * 4;
  if (smem > 96 * 1024) return cudaErrorInvalidValue;
  static unsigned long long smem_ok = 0;
  cudaError_t e = fmm_allow_dynamic_smem(encode_split_kernel, 96 * 1024, &smem_ok);
  if (e != cudaSuccess) return e;
  const int64_t grid = (nquad + kSplitThreads - 1) / kSplitThreads;
  if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
  encode_split_kernel<<<(unsigned)grid, kSplitThreads, smem, st>>>(codes, K, gc, br, G, h, b_side ? 1 : 0, d_tab, out, rstride, nquad);
  ++fmm_launch_counter();
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Block sums of int8 codes as int8 (certificate (i): |sum| <= 127), packed for the one-kernel certified realisation:
// rows of 128 bytes that hold per = 128 / h products side by side, product r at byte (r % per) * h of row
// (group, p) of slab r / per.  One thread forms, for one (group, row position) and four consecutive inner indices t,
// the sums of every product (the same staging as encode_split_kernel).
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSplitThreads)
encode_codes_kernel(const int8_t* __restrict__ codes, int64_t K, int gc, int64_t br, int G, int h,
                    const CoefTable* __restrict__ d_tab, int8_t* __restrict__ out, int64_t nquad) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int R = d_tab->R, ncell = d_tab->ncell;
  const int total = d_tab->off[R];
  int* off = reinterpret_cast<int*>(smem_raw);
  int2* ent = reinterpret_cast<int2*>(smem_raw + ((size_t)(R + 1) * 4 + 15) / 16 * 16);
  uint32_t* stage = reinterpret_cast<uint32_t*>(reinterpret_cast<unsigned char*>(ent) + (size_t)total * 8);
  for (int i = threadIdx.x; i <= R; i += kSplitThreads) off[i] = d_tab->off[i];
  for (int i = threadIdx.x; i < total; i += kSplitThreads)
    ent[i] = make_int2(d_tab->cell[i], __float2int_rn(d_tab->coef[i]));
  stage[ncell * kSplitThreads + threadIdx.x] = 0u;                    // the padding cell
  const int64_t idx = (int64_t)blockIdx.x * kSplitThreads + threadIdx.x;
  const bool live = idx < nquad;
  const int qpr = h / 4;
  const int64_t rowp = live ? idx / qpr : 0;                          // (group, p)
  const int t = live ? (int)(idx - rowp * qpr) * 4 : 0;
  const int64_t g = rowp / br, p = rowp - g * br;
  for (int c = 0; c < ncell; ++c) {
    const int gi = c / gc, gj = c - gi * gc;
    stage[c * kSplitThreads + threadIdx.x] =
        live ? *reinterpret_cast<const uint32_t*>(codes + ((int64_t)gi * br + p) * K + g * kGroup + gj * h + t) : 0u;
  }
  __syncthreads();
  if (!live) return;
  const int per = kGroup / h;
  const int64_t slab = (int64_t)G * br * kGroup;                      // bytes of one slab of `per` products
  for (int r = 0; r < R; ++r) {
    int s0 = 0, s1 = 0, s2 = 0, s3 = 0;
    for (int e = off[r]; e < off[r + 1]; ++e) {
      const int2 en = ent[e];
      const uint32_t wv = stage[en.x * kSplitThreads + threadIdx.x];
      s0 += en.y * (int)(int8_t)(wv & 0xffu);
      s1 += en.y * (int)(int8_t)((wv >> 8) & 0xffu);
      s2 += en.y * (int)(int8_t)((wv >> 16) & 0xffu);
      s3 += en.y * (int)(int8_t)(wv >> 24);
    }
    const uint32_t packed = ((uint32_t)s0 & 0xffu) | (((uint32_t)s1 & 0xffu) << 8) | (((uint32_t)s2 & 0xffu) << 16) |
                            (((uint32_t)s3 & 0xffu) << 24);
    *reinterpret_cast<uint32_t*>(out + (r / per) * slab + rowp * kGroup + (r % per) * h + t) = packed;
  }
}

cudaError_t launch_encode_codes(const int8_t* codes, int64_t K, int gr, int gc, int64_t br, int G, int h,
                                const CoefTable* d_tab, const CoefTable* h_tab, int8_t* out, cudaStream_t st) {
  const int64_t nquad = (int64_t)G * br * (h / 4);
  const size_t smem = ((size_t)(h_tab->R + 1) * 4 + 15) / 16 * 16 + (size_t)h_tab->off[h_tab->R] * 8 +
                      (size_t)(gr * gc + 1) * kSplitThreads * 4;
  if (smem > 96 * 1024) return cudaErrorInvalidValue;
  static unsigned long long smem_ok = 0;
  cudaError_t e = fmm_allow_dynamic_smem(encode_codes_kernel, 96 * 1024, &smem_ok);
  if (e != cudaSuccess) return e;
  const int64_t grid = (nquad + kSplitThreads - 1) / kSplitThreads;
  if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
  encode_codes_kernel<<<(unsigned)grid, kSplitThreads, smem, st>>>(codes, K, gc, br, G, h, d_tab, out, nquad);
  ++fmm_launch_counter();
  return cudaGetLastError();
}

int padded_total(const CoefTable& t) { return t.off[t.R]; }

template <typename OutT, int kSplit, int kStages, int kCells, bool kIntAcc = false>
cudaError_t launch_decode_group_t(const float* prod, int64_t pstride, int G, const CoefTable* d_tab,
                                  const CoefTable* h_tab, int R, const float* dAt, const float* dBt, int m, int n,
                                  int64_t bm, int64_t bn, void* C, int64_t ldc, cudaStream_t st) {
  constexpr int kPos = kDecThreads / kSplit;
  const size_t smem = ((sizeof(GDecHead) + (size_t)padded_total(*h_tab) * 8 + 15) / 16) * 16 +
                      (size_t)kStages * (R + 1) * kPos * 16;
  const int64_t nvec = bm * (bn >> 2);
  if (nvec + kDecThreads >= (int64_t)1 << 31 || smem > 200 * 1024) return cudaErrorInvalidValue;
  if (m * n > kSplit * kCells) return cudaErrorInvalidValue;
  auto k = decode_group_kernel<OutT, kSplit, kStages, kCells, kIntAcc>;
  static unsigned long long smem_ok = 0;   // per template instantiation, one bit per device
  cudaError_t e = fmm_allow_dynamic_smem(k, 200 * 1024, &smem_ok);
  if (e != cudaSuccess) return e;
  const unsigned grid = (unsigned)((nvec + kPos - 1) / kPos);
  k<<<grid, kDecThreads, smem, st>>>(prod, pstride, G, d_tab, R, dAt, dBt, (int64_t)m * bm, (int64_t)n * bn, n, bm, bn,
                                     (OutT*)C, ldc);
  ++fmm_launch_counter();
  return cudaGetLastError();
}

// One C block and one product (the classical operator): the plain rescale kernel.  At most four C blocks and
// eight products: four threads share a position, four groups in flight; otherwise eight threads share a
// position (two C blocks each), two groups in flight.
template <typename OutT>
cudaError_t launch_decode_group_o(const float* prod, int64_t pstride, int G, const CoefTable* d_tab,
                                  const CoefTable* h_tab, int R, const float* dAt, const float* dBt, int m, int n,
                                  int64_t bm, int64_t bn, void* C, int64_t ldc, bool int_acc, cudaStream_t st) {
  if (int_acc) {
    if (m * n <= 4 && R <= 8)
      return launch_decode_group_t<OutT, 4, 4, 1, true>(prod, pstride, G, d_tab, h_tab, R, dAt, dBt, m, n, bm, bn, C, ldc, st);
    return launch_decode_group_t<OutT, 8, 2, 2, true>(prod, pstride, G, d_tab, h_tab, R, dAt, dBt, m, n, bm, bn, C, ldc, st);
  }
  if (m * n == 1 && R == 1) {
    const int64_t nvec = bm * (bn >> 2);
    rescale_groups_kernel<OutT><<<(unsigned)((nvec + 255) / 256), 256, 0, st>>>(prod, pstride, G, dAt, dBt, bm, bn, (OutT*)C, ldc);
    ++fmm_launch_counter();
    return cudaGetLastError();
  }
  if (m * n <= 4 && R <= 8)
    return launch_decode_group_t<OutT, 4, 4, 1>(prod, pstride, G, d_tab, h_tab, R, dAt, dBt, m, n, bm, bn, C, ldc, st);
  return launch_decode_group_t<OutT, 8, 2, 2>(prod, pstride, G, d_tab, h_tab, R, dAt, dBt, m, n, bm, bn, C, ldc, st);
}

cudaError_t launch_decode_group(int output, const float* prod, int64_t pstride, int G, const CoefTable* d_tab,
                                const CoefTable* h_tab, int R, const float* dAt, const float* dBt, int m, int n,
                                int64_t bm, int64_t bn, void* C, int64_t ldc, bool int_acc, cudaStream_t st) {
  if (output == FMM_F32)
    return launch_decode_group_o<float>(prod, pstride, G, d_tab, h_tab, R, dAt, dBt, m, n, bm, bn, C, ldc, int_acc, st);
  if (output == FMM_BF16)
    return launch_decode_group_o<__nv_bfloat16>(prod, pstride, G, d_tab, h_tab, R, dAt, dBt, m, n, bm, bn, C, ldc, int_acc, st);
  return cudaErrorInvalidValue;
}

int stream_blocks(int64_t items, int per_block) {
  int64_t g = (items + per_block - 1) / per_block;
  return (int)std::min<int64_t>(std::max<int64_t>(g, 1), 148 * 16);
}

// Workspace of one int8 product.
struct Int8Layout {
  size_t status, tabA, tabB, tabW, dAt, dBt, xqa, xqb, ahat, bhat, prod, total;
  int64_t sAhat, sBhat, sProd;   // element strides between products (Ahat/Bhat) and between (r, group) entries (prod)
  int G, h, w;
  bool trivial;
};

// Workspace of the one-kernel certified realisation
struct CertWs {
  size_t status, tabA, tabB, entries, pass_off, owned, dAt, dBt, ahat, bhat, total;
  size_t max_entries;
};

// the classical algorithm <1,1,1;1> as a scheme
struct TrivialScheme : fmm_scheme {
  TrivialScheme() {
    m = k = n = R = 1;
    U = {1.0}; V = {1.0}; W = {1.0};
  }
};

fmm_status int8_shape_ok(const fmm_scheme& s, int64_t M, int64_t K, int64_t N) {
  if (M <= 0 || K <= 0 || N <= 0 || K % kGroup) return FMM_ERR_SHAPE;
  if (M % s.m || N % s.n || kGroup % s.k) return FMM_ERR_SHAPE;
  const int h = kGroup / s.k;
  if (h != 32 && h != 64 && h != 128) return FMM_ERR_SHAPE;
  if ((N / s.n) % 8) return FMM_ERR_SHAPE;
  if (M * (K / kGroup) > 0x7fffffffLL / 2 || N * (K / kGroup) > 0x7fffffffLL / 2) return FMM_ERR_SHAPE;
  return FMM_OK;
}

CertWs cert_layout(const fmm_scheme& s, int64_t M, int64_t K, int64_t N) {
  CertWs L{};
  const int G = (int)(K / kGroup), h = kGroup / s.k, per = kGroup / h;
  const int64_t bm = M / s.m, bn = N / s.n;
  const int slabs = (s.R + per - 1) / per;
  L.max_entries = (size_t)s.R * s.m * s.n;
  size_t o = 0;
  L.status = o; o += align_up(sizeof(DeviceStatus));
  L.tabA = o; o += align_up(sizeof(CoefTable));
  L.tabB = o; o += align_up(sizeof(CoefTable));
  L.entries = o; o += align_up(L.max_entries * 8);
  L.pass_off = o; o += align_up((size_t)(FMM_MAX_R + 1) * FMM_MAX_GRID * FMM_MAX_GRID * 4);
  L.owned = o; o += align_up(FMM_MAX_GRID * FMM_MAX_GRID * 4);
  L.dAt = o; o += align_up((size_t)M * G * 4);
  L.dBt = o; o += align_up((size_t)N * G * 4);
  L.ahat = o; o += align_up((size_t)slabs * G * bm * kGroup + 128 * kGroup);   // + one tile of rows: boxes may read past the end
  L.bhat = o; o += align_up((size_t)slabs * G * bn * kGroup + 128 * kGroup);
  L.total = o;
  return L;
}

Int8Layout int8_layout(const fmm_scheme& s, int64_t M, int64_t K, int64_t N) {
  Int8Layout L;
  L.G = (int)(K / kGroup);
  L.h = kGroup / s.k;
  L.w = std::max(L.h, 64);
  L.trivial = s.m == 1 && s.k == 1 && s.n == 1 && s.R == 1;
  const int64_t bm = M / s.m, bn = N / s.n;
  size_t o = 0;
  L.status = o; o += align_up(sizeof(DeviceStatus));
  L.tabA = o; o += align_up(sizeof(CoefTable));
  L.tabB = o; o += align_up(sizeof(CoefTable));
  L.tabW = o; o += align_up(sizeof(CoefTable));
  L.dAt = o; o += align_up((size_t)M * L.G * 4);
  L.dBt = o; o += align_up((size_t)N * L.G * 4);
  L.xqa = o; o += align_up((size_t)M * L.G * s.k * L.w * 2);
  L.xqb = o; o += align_up((size_t)N * L.G * s.k * L.w * 2);
  L.sAhat = (int64_t)L.G * bm * L.w + kSlabPadBytes / 2;
  L.sBhat = (int64_t)L.G * bn * L.w + kSlabPadBytes / 2;
  L.sProd = bm * bn + kSlabPadBytes / 4;
  L.ahat = o; o += L.trivial ? 0 : align_up((size_t)s.R * L.sAhat * 2);
  L.bhat = o; o += L.trivial ? 0 : align_up((size_t)s.R * L.sBhat * 2);
  L.prod = o; o += align_up((size_t)s.R * L.G * L.sProd * 4);
  L.total = o;
  return L;
}

bool integer_coefficients(const fmm_scheme& s) {
  for (const std::vector<double>* v : {&s.U, &s.V, &s.W})
    for (double c : *v)
      if (c != std::rint(c)) return false;
  return true;
}

// Workspace of the corrected product: split block sums in rows of 4h, products, transposed scales.
struct CorrLayout {
  size_t status, tabA, tabB, tabW, dAt, dBt, ahat, bhat, prod, total;
  int64_t sAhat, sBhat, sProd;
  int G, h;
};

CorrLayout corr_layout(const fmm_scheme& s, int64_t M, int64_t K, int64_t N) {
  CorrLayout L;
  L.G = (int)(K / kGroup);
  L.h = kGroup / s.k;
  const int64_t bm = M / s.m, bn = N / s.n;
  size_t o = 0;
  L.status = o; o += align_up(sizeof(DeviceStatus));
  L.tabA = o; o += align_up(sizeof(CoefTable));
  L.tabB = o; o += align_up(sizeof(CoefTable));
  L.tabW = o; o += align_up(sizeof(CoefTable));
  L.dAt = o; o += align_up((size_t)M * L.G * 4);
  L.dBt = o; o += align_up((size_t)N * L.G * 4);
  L.sAhat = (int64_t)L.G * bm * 4 * L.h + kSlabPadBytes / 2;
  L.sBhat = (int64_t)L.G * bn * 4 * L.h + kSlabPadBytes / 2;
  L.sProd = bm * bn + kSlabPadBytes / 4;
  L.ahat = o; o += align_up((size_t)s.R * L.sAhat * 2);
  L.bhat = o; o += align_up((size_t)s.R * L.sBhat * 2);
  L.prod = o; o += align_up((size_t)s.R * L.G * L.sProd * 4);
  L.total = o;
  return L;
}

// The corrected computation's certificate (Appendix D) for this realisation: integer coefficients; block sums
// |X| <= L * 127 split as X0 + 256 R with |R| <= rmax; inside one rebuilt product the absolute values of all weighted
// terms add up to at most h (128 + 256 rmax)^2, which must stay below 2^24 (fp32 accumulators of the tensor cores);
// the combination adds at most L_W such products and must stay below 2^31 (int32 in the decode); the group's result
// is the classical product, at most 128 * 127^2 < 2^24, so its conversion to fp32 is exact.
bool corrected_certificate(const fmm_scheme& s, int h, double cert[4]) {
  double meta[8];
  if (scheme_info(&s, nullptr, meta) != FMM_OK) return false;
  const double sum_max = std::max(meta[0], meta[1]) * 127.0;
  const double rmax = std::floor((sum_max + 128.0) / 256.0);
  const double terms = (double)h * (128.0 + 256.0 * rmax) * (128.0 + 256.0 * rmax);
  const double comb = meta[2] * terms;
  if (cert) { cert[0] = sum_max; cert[1] = rmax; cert[2] = terms; cert[3] = comb; }
  return integer_coefficients(s) && terms < std::ldexp(1.0, 24) && comb < std::ldexp(1.0, 31) &&
         (int64_t)s.k * h == kGroup;
}

// Workspace of the fused classical operator: status word and the two transposed scale arrays.
struct FusedLayout { size_t status, dAt, dBt, total; };

FusedLayout fused_layout(int64_t M, int64_t K, int64_t N) {
  FusedLayout L;
  const size_t G = (size_t)(K / kGroup);
  size_t o = 0;
  L.status = o; o += align_up(sizeof(DeviceStatus));
  L.dAt = o; o += align_up((size_t)M * G * 4);
  L.dBt = o; o += align_up((size_t)N * G * 4);
  L.total = o;
  return L;
}

// The classical int8 operator in one tensor-core kernel (int8 MMAs, int32 accumulators, rescale in the epilogue).
fmm_status int8_classical_fused(const int8_t* d_cA, const float* d_dA, const int8_t* d_cB, const float* d_dB, int64_t M,
                                int64_t K, int64_t N, int output, void* d_C, int64_t ldc, void* d_ws, size_t ws_bytes,
                                cudaStream_t st) {
  const FusedLayout L = fused_layout(M, K, N);
  if (!d_ws || (reinterpret_cast<uintptr_t>(d_ws) & 255u) || ws_bytes < L.total) return FMM_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(d_cA) % 16) || (reinterpret_cast<uintptr_t>(d_cB) % 16)) return FMM_ERR_SHAPE;
  const int G = (int)(K / kGroup);
  FMM_CUDA(cudaMemsetAsync(at<char>(d_ws, L.status), 0, sizeof(DeviceStatus), st));
  {
    ProfScope ps(5, st);
    transpose_scales_kernel<<<stream_blocks(M * G, 256), 256, 0, st>>>(d_dA, M, G, at<float>(d_ws, L.dAt));
    ++fmm_launch_counter();
    transpose_scales_kernel<<<stream_blocks(N * G, 256), 256, 0, st>>>(d_dB, N, G, at<float>(d_ws, L.dBt));
    ++fmm_launch_counter();
    FMM_CUDA(cudaGetLastError());
  }
  ProfScope ps(4, st);
  return launch_int8_group_gemm(d_cA, d_cB, at<float>(d_ws, L.dAt), at<float>(d_ws, L.dBt), M, K, N, output, d_C, ldc,
                                at<DeviceStatus>(d_ws, L.status), st);
}

}  // namespace

extern "C" {

int scheme_certificate(const fmm_scheme* s, int bA, int bB, int h, int g, int acc_bits, double cert[4]) {
  TrivialScheme one;
  const fmm_scheme& sc = s ? *s : one;
  double meta[8];
  if (scheme_info(&sc, nullptr, meta) != FMM_OK) return 0;
  const double a = meta[0] * bA, b = meta[1] * bB;
  const double big = std::max(meta[2] * h * a * b, (double)g * bA * bB);
  const bool one_group = (int64_t)sc.k * h == g;
  if (cert) { cert[0] = a; cert[1] = b; cert[2] = big; cert[3] = one_group ? 1.0 : 0.0; }
  return integer_coefficients(sc) && a <= 127.0 && b <= 127.0 && big < std::ldexp(1.0, acc_bits) && one_group;
}

fmm_status int8_quantize(const void* d_X, int storage, int64_t rows, int64_t K, int64_t ldx, int code_bound,
                         int8_t* d_codes, float* d_scales, void* stream) {
  if (!d_X || !d_codes || !d_scales) return FMM_ERR_ARG;
  if (rows <= 0 || K <= 0 || K % kGroup || ldx < K) return FMM_ERR_SHAPE;
  if (code_bound < 1 || code_bound > 127) return FMM_ERR_ARG;
  if (storage != FMM_F32 && storage != FMM_BF16) return FMM_ERR_DTYPE;
  const int es = storage == FMM_F32 ? 4 : 2;
  if ((ldx * es) % (4 * es) || (reinterpret_cast<uintptr_t>(d_X) % (4 * es)) || (reinterpret_cast<uintptr_t>(d_codes) % 4))
    return FMM_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int G = (int)(K / kGroup);
  const int grid = stream_blocks(rows * G, kQuantThreads / 32);
  if (storage == FMM_F32)
    quantize_kernel<float><<<grid, kQuantThreads, 0, st>>>((const float*)d_X, ldx, rows, G, (float)code_bound, d_codes, d_scales);
  else
    quantize_kernel<__nv_bfloat16><<<grid, kQuantThreads, 0, st>>>((const __nv_bfloat16*)d_X, ldx, rows, G, (float)code_bound, d_codes, d_scales);
  ++fmm_launch_counter();
  return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

size_t int8_gemm_workspace(const fmm_scheme* s, int64_t M, int64_t K, int64_t N) {
  TrivialScheme one;
  const fmm_scheme& sc = s ? *s : one;
  if (int8_shape_ok(sc, M, K, N) != FMM_OK) return 0;
  if (!s) return fused_layout(M, K, N).total;
  return cert_layout(sc, M, K, N).total;
}

size_t int8_gemm_materialised_workspace(const fmm_scheme* s, int64_t M, int64_t K, int64_t N) {
  TrivialScheme one;
  const fmm_scheme& sc = s ? *s : one;
  if (int8_shape_ok(sc, M, K, N) != FMM_OK) return 0;
  return int8_layout(sc, M, K, N).total;
}

// The certified realisation in one kernel: block sums of the codes as int8 (two launches), scales transposed to
// group-major (two launches), then int8_certified_kernel.
static fmm_status int8_certified_one_kernel(const fmm_scheme& sc, const int8_t* d_cA, const float* d_dA, const int8_t* d_cB,
                                            const float* d_dB, int64_t M, int64_t K, int64_t N, int output, void* d_C,
                                            int64_t ldc, void* d_ws, size_t ws_bytes, cudaStream_t st) {
  const CertWs L = cert_layout(sc, M, K, N);
  if (!d_ws || (reinterpret_cast<uintptr_t>(d_ws) & 255u) || ws_bytes < L.total) return FMM_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(d_cA) % 4) || (reinterpret_cast<uintptr_t>(d_cB) % 4)) return FMM_ERR_SHAPE;
  const int64_t bm = M / sc.m, bn = N / sc.n;
  const int h = kGroup / sc.k, G = (int)(K / kGroup);
  FMM_CUDA(cudaMemsetAsync(at<char>(d_ws, L.status), 0, sizeof(DeviceStatus), st));
  std::unique_ptr<CoefTable> hA(new CoefTable), hB(new CoefTable);
  std::memset(hA.get(), 0, sizeof(CoefTable)); std::memset(hB.get(), 0, sizeof(CoefTable));
  fmm_build_tables(sc, hA.get(), hB.get(), nullptr);
  FMM_CUDA(cudaMemcpyAsync(at<char>(d_ws, L.tabA), hA.get(), sizeof(CoefTable), cudaMemcpyHostToDevice, st));
  FMM_CUDA(cudaMemcpyAsync(at<char>(d_ws, L.tabB), hB.get(), sizeof(CoefTable), cudaMemcpyHostToDevice, st));
  // Decode lists.  Every block of C is owned by one of four decode warps (per TMEM lane quarter); the blocks are dealt
  // out longest list first to the warp with the least work so far that still has a free slot.  The lists are then laid
  // out by (warp, pass of products, owned block, ascending r); an entry is (TMEM column of the product inside its
  // pass, integer w).
  const int blocks = sc.m * sc.n;
  int passes = 0, pass = 0;
  int8_certified_passes(sc.R, kGroup / h, &passes, &pass);
  const int kParts = int8_certified_decode_warps(), kOwn = FMM_MAX_GRID * FMM_MAX_GRID / kParts, kBN = int8_certified_tile_columns();
  std::vector<int> nnz(blocks, 0), order(blocks), owned(kParts * kOwn, -1), load(kParts, 0), used(kParts, 0);
  for (int d = 0; d < blocks; ++d)
    for (int r = 0; r < sc.R; ++r) nnz[d] += sc.W[(size_t)r * blocks + d] != 0.0;
  for (int d = 0; d < blocks; ++d) order[d] = d;
  std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return nnz[x] > nnz[y]; });
  for (int d : order) {
    int best = -1;
    for (int q = 0; q < kParts; ++q)
      if (used[q] < kOwn && (best < 0 || load[q] < load[best])) best = q;
    owned[best * kOwn + used[best]++] = d;
    load[best] += nnz[d];
  }
  std::vector<int2> ent;
  std::vector<int> poff;
  for (int q = 0; q < kParts; ++q)
    for (int ps = 0; ps < passes; ++ps)
      for (int b = 0; b < kOwn; ++b) {
        poff.push_back((int)ent.size());
        const int d = owned[q * kOwn + b];
        if (d < 0) continue;
        for (int r = ps * pass; r < (ps == passes - 1 ? sc.R : (ps + 1) * pass); ++r) {
          const double w = sc.W[(size_t)r * blocks + d];
          if (w != 0.0) ent.push_back(make_int2((r - ps * pass) * kBN, (int)std::lrint(w)));
        }
      }
  poff.push_back((int)ent.size());
  if (ent.size() > L.max_entries) return FMM_ERR_LIMIT;
  if (!ent.empty())
    FMM_CUDA(cudaMemcpyAsync(at<char>(d_ws, L.entries), ent.data(), ent.size() * sizeof(int2), cudaMemcpyHostToDevice, st));
  FMM_CUDA(cudaMemcpyAsync(at<char>(d_ws, L.pass_off), poff.data(), poff.size() * sizeof(int), cudaMemcpyHostToDevice, st));
  FMM_CUDA(cudaMemcpyAsync(at<char>(d_ws, L.owned), owned.data(), owned.size() * sizeof(int), cudaMemcpyHostToDevice, st));
  {
    ProfScope ps(0, st);
    FMM_CUDA(launch_encode_codes(d_cA, K, sc.m, sc.k, bm, G, h, at<CoefTable>(d_ws, L.tabA), hA.get(), at<int8_t>(d_ws, L.ahat), st));
    FMM_CUDA(launch_encode_codes(d_cB, K, sc.n, sc.k, bn, G, h, at<CoefTable>(d_ws, L.tabB), hB.get(), at<int8_t>(d_ws, L.bhat), st));
    transpose_scales_kernel<<<stream_blocks(M * G, 256), 256, 0, st>>>(d_dA, M, G, at<float>(d_ws, L.dAt));
    ++fmm_launch_counter();
    transpose_scales_kernel<<<stream_blocks(N * G, 256), 256, 0, st>>>(d_dB, N, G, at<float>(d_ws, L.dBt));
    ++fmm_launch_counter();
    FMM_CUDA(cudaGetLastError());
  }
  Int8CertArgs a{};
  a.Ahat = at<int8_t>(d_ws, L.ahat); a.Bhat = at<int8_t>(d_ws, L.bhat);
  a.m = sc.m; a.n = sc.n; a.R = sc.R; a.h = h; a.bm = bm; a.bn = bn; a.G = G; a.M = M; a.N = N;
  a.dAt = at<float>(d_ws, L.dAt); a.dBt = at<float>(d_ws, L.dBt);
  a.d_entries = at<int2>(d_ws, L.entries); a.d_pass_off = at<int>(d_ws, L.pass_off); a.d_owned = at<int>(d_ws, L.owned); a.n_entries = (int)ent.size();
  a.output = output; a.C = d_C; a.ldc = ldc; a.status = at<DeviceStatus>(d_ws, L.status);
  ProfScope ps(2, st);
  // the host tables were copied from pageable memory: those copies are complete when cudaMemcpyAsync returns
  return launch_int8_certified(a, st);
}

fmm_status int8_gemm(const fmm_scheme* s, int code_bound, const int8_t* d_cA, const float* d_dA, const int8_t* d_cB,
                     const float* d_dB, int64_t M, int64_t K, int64_t N, int output, void* d_C, int64_t ldc, void* d_ws,
                     size_t ws_bytes, void* stream) {
  if (!d_cA || !d_dA || !d_cB || !d_dB || !d_C) return FMM_ERR_ARG;
  if (output != FMM_F32 && output != FMM_BF16) return FMM_ERR_DTYPE;
  if (code_bound < 1 || code_bound > 127) return FMM_ERR_ARG;
  TrivialScheme one;
  const fmm_scheme& sc = s ? *s : one;
  FMM_TRY(int8_shape_ok(sc, M, K, N));
  const int eo = output == FMM_F32 ? 4 : 2;
  if (ldc < N || (ldc * eo) % 16 || (reinterpret_cast<uintptr_t>(d_C) % 16)) return FMM_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(d_cA) % 8) || (reinterpret_cast<uintptr_t>(d_cB) % 8)) return FMM_ERR_SHAPE;
  // Proposition 1 for this realisation: int8 block sums, integers exact in the fp32 accumulators (24 bits)
  if (!scheme_certificate(&sc, code_bound, code_bound, kGroup / sc.k, kGroup, 24, nullptr)) return FMM_ERR_CERTIFICATE;
  if (!s)   // the classical operator: one fused tensor-core kernel
    return int8_classical_fused(d_cA, d_dA, d_cB, d_dB, M, K, N, output, d_C, ldc, d_ws, ws_bytes, static_cast<cudaStream_t>(stream));
  return int8_certified_one_kernel(sc, d_cA, d_dA, d_cB, d_dB, M, K, N, output, d_C, ldc, d_ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

// The same operator with every per-group block product written to memory (pack, encode, grouped block products with
// bf16 operands and fp32 accumulators, grouped decode): the form the one-kernel realisation replaced, kept as an
// independent implementation to compare against and to time.
fmm_status int8_gemm_materialised(const fmm_scheme* s, int code_bound, const int8_t* d_cA, const float* d_dA, const int8_t* d_cB,
                                  const float* d_dB, int64_t M, int64_t K, int64_t N, int output, void* d_C, int64_t ldc,
                                  void* d_ws, size_t ws_bytes, void* stream) {
  if (!d_cA || !d_dA || !d_cB || !d_dB || !d_C) return FMM_ERR_ARG;
  if (output != FMM_F32 && output != FMM_BF16) return FMM_ERR_DTYPE;
  if (code_bound < 1 || code_bound > 127) return FMM_ERR_ARG;
  TrivialScheme one;
  const fmm_scheme& sc = s ? *s : one;
  FMM_TRY(int8_shape_ok(sc, M, K, N));
  const int eo = output == FMM_F32 ? 4 : 2;
  if (ldc < N || (ldc * eo) % 16 || (reinterpret_cast<uintptr_t>(d_C) % 16)) return FMM_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(d_cA) % 8) || (reinterpret_cast<uintptr_t>(d_cB) % 8)) return FMM_ERR_SHAPE;
  if (!scheme_certificate(&sc, code_bound, code_bound, kGroup / sc.k, kGroup, 24, nullptr)) return FMM_ERR_CERTIFICATE;
  const Int8Layout L = int8_layout(sc, M, K, N);
  if (!d_ws || (reinterpret_cast<uintptr_t>(d_ws) & 255u) || ws_bytes < L.total) return FMM_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t bm = M / sc.m, bn = N / sc.n;
  const int kw = sc.k * L.w;

  FMM_CUDA(cudaMemsetAsync(at<char>(d_ws, L.status), 0, sizeof(DeviceStatus), st));
  CoefTable *hA = new CoefTable, *hB = new CoefTable, *hW = new CoefTable;
  std::unique_ptr<CoefTable> ga(hA), gb(hB), gw(hW);
  std::memset(hA, 0, sizeof(CoefTable)); std::memset(hB, 0, sizeof(CoefTable)); std::memset(hW, 0, sizeof(CoefTable));
  fmm_build_tables(sc, hA, hB, hW);
  FMM_CUDA(cudaMemcpyAsync(at<char>(d_ws, L.tabW), hW, sizeof(CoefTable), cudaMemcpyHostToDevice, st));
  if (!L.trivial) {
    FMM_CUDA(cudaMemcpyAsync(at<char>(d_ws, L.tabA), hA, sizeof(CoefTable), cudaMemcpyHostToDevice, st));
    FMM_CUDA(cudaMemcpyAsync(at<char>(d_ws, L.tabB), hB, sizeof(CoefTable), cudaMemcpyHostToDevice, st));
  }
  {
    ProfScope ps(0, st);
    const int64_t nva = M * L.G * (kw / 8), nvb = N * L.G * (kw / 8);
    pack_kernel<<<stream_blocks(nva, 256 * 4), 256, 0, st>>>(d_cA, K, bm, L.G, sc.k, L.h, L.w, nva, at<__nv_bfloat16>(d_ws, L.xqa));
    ++fmm_launch_counter();
    pack_kernel<<<stream_blocks(nvb, 256 * 4), 256, 0, st>>>(d_cB, K, bn, L.G, sc.k, L.h, L.w, nvb, at<__nv_bfloat16>(d_ws, L.xqb));
    ++fmm_launch_counter();
    FMM_CUDA(cudaGetLastError());
    if (!L.trivial) {
      FMM_CUDA(launch_encode(FMM_BF16, FMM_BF16, at<char>(d_ws, L.xqa), kw, sc.m, sc.k, (int64_t)L.G * bm, L.w,
                             at<CoefTable>(d_ws, L.tabA), hA, at<char>(d_ws, L.ahat), L.sAhat, nullptr, nullptr, false, false, st));
      FMM_CUDA(launch_encode(FMM_BF16, FMM_BF16, at<char>(d_ws, L.xqb), kw, sc.n, sc.k, (int64_t)L.G * bn, L.w,
                             at<CoefTable>(d_ws, L.tabB), hB, at<char>(d_ws, L.bhat), L.sBhat, nullptr, nullptr, false, false, st));
    }
  }
  {
    BlockProductArgs g{};
    g.product = FMM_BF16;
    g.A = L.trivial ? at<char>(d_ws, L.xqa) : at<char>(d_ws, L.ahat); g.lda = L.w; g.a_batch = L.trivial ? 0 : L.sAhat;
    g.B = L.trivial ? at<char>(d_ws, L.xqb) : at<char>(d_ws, L.bhat); g.ldb = L.w; g.b_batch = L.trivial ? 0 : L.sBhat;
    g.rows_a = bm; g.rows_b = bn; g.kdim = L.w; g.batches = sc.R; g.groups = L.G;
    g.out = at<char>(d_ws, L.prod); g.ldo = bn; g.o_batch = L.sProd; g.out_mode = 0; g.output = FMM_F32;
    g.status = at<DeviceStatus>(d_ws, L.status);
    ProfScope ps(2, st);
    FMM_TRY(launch_block_products(g, st));
  }
  {
    ProfScope ps(3, st);
    transpose_scales_kernel<<<stream_blocks(M * L.G, 256), 256, 0, st>>>(d_dA, M, L.G, at<float>(d_ws, L.dAt));
    ++fmm_launch_counter();
    transpose_scales_kernel<<<stream_blocks(N * L.G, 256), 256, 0, st>>>(d_dB, N, L.G, at<float>(d_ws, L.dBt));
    ++fmm_launch_counter();
    FMM_CUDA(cudaGetLastError());
    FMM_CUDA(launch_decode_group(output, at<float>(d_ws, L.prod), L.sProd, L.G, at<CoefTable>(d_ws, L.tabW), hW, sc.R,
                                 at<float>(d_ws, L.dAt), at<float>(d_ws, L.dBt), sc.m, sc.n, bm, bn, d_C, ldc, false, st));
  }
  // the tables were copied from pageable host memory: the copies are complete when cudaMemcpyAsync returns
  return FMM_OK;
}

int scheme_certificate_corrected(const fmm_scheme* s, int h, double cert[4]) {
  if (!s) return 0;
  return corrected_certificate(*s, h, cert) ? 1 : 0;
}

size_t int8_gemm_corrected_workspace(const fmm_scheme* s, int64_t M, int64_t K, int64_t N) {
  if (!s || int8_shape_ok(*s, M, K, N) != FMM_OK) return 0;
  return corr_layout(*s, M, K, N).total;
}

fmm_status int8_gemm_corrected(const fmm_scheme* s, const int8_t* d_cA, const float* d_dA, const int8_t* d_cB,
                               const float* d_dB, int64_t M, int64_t K, int64_t N, int output, void* d_C, int64_t ldc,
                               void* d_ws, size_t ws_bytes, void* stream) {
  if (!s || !d_cA || !d_dA || !d_cB || !d_dB || !d_C) return FMM_ERR_ARG;
  if (output != FMM_F32 && output != FMM_BF16) return FMM_ERR_DTYPE;
  const fmm_scheme& sc = *s;
  FMM_TRY(int8_shape_ok(sc, M, K, N));
  const int eo = output == FMM_F32 ? 4 : 2;
  if (ldc < N || (ldc * eo) % 16 || (reinterpret_cast<uintptr_t>(d_C) % 16)) return FMM_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(d_cA) % 8) || (reinterpret_cast<uintptr_t>(d_cB) % 8)) return FMM_ERR_SHAPE;
  const CorrLayout L = corr_layout(sc, M, K, N);
  if (!corrected_certificate(sc, L.h, nullptr)) return FMM_ERR_CERTIFICATE;
  if (!d_ws || (reinterpret_cast<uintptr_t>(d_ws) & 255u) || ws_bytes < L.total) return FMM_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t bm = M / sc.m, bn = N / sc.n;

  FMM_CUDA(cudaMemsetAsync(at<char>(d_ws, L.status), 0, sizeof(DeviceStatus), st));
  std::unique_ptr<CoefTable> hA(new CoefTable), hB(new CoefTable), hW(new CoefTable);
  std::memset(hA.get(), 0, sizeof(CoefTable)); std::memset(hB.get(), 0, sizeof(CoefTable)); std::memset(hW.get(), 0, sizeof(CoefTable));
  fmm_build_tables(sc, hA.get(), hB.get(), hW.get());
  FMM_CUDA(cudaMemcpyAsync(at<char>(d_ws, L.tabA), hA.get(), sizeof(CoefTable), cudaMemcpyHostToDevice, st));
  FMM_CUDA(cudaMemcpyAsync(at<char>(d_ws, L.tabB), hB.get(), sizeof(CoefTable), cudaMemcpyHostToDevice, st));
  FMM_CUDA(cudaMemcpyAsync(at<char>(d_ws, L.tabW), hW.get(), sizeof(CoefTable), cudaMemcpyHostToDevice, st));
  {
    ProfScope ps(0, st);
    FMM_CUDA(launch_encode_split(d_cA, K, sc.m, sc.k, bm, L.G, L.h, false, at<CoefTable>(d_ws, L.tabA), hA.get(),
                                 at<__nv_bfloat16>(d_ws, L.ahat), L.sAhat, st));
    FMM_CUDA(launch_encode_split(d_cB, K, sc.n, sc.k, bn, L.G, L.h, true, at<CoefTable>(d_ws, L.tabB), hB.get(),
                                 at<__nv_bfloat16>(d_ws, L.bhat), L.sBhat, st));
  }
  {
    BlockProductArgs g{};
    g.product = FMM_BF16;
    g.A = at<char>(d_ws, L.ahat); g.lda = 4 * L.h; g.a_batch = L.sAhat;
    g.B = at<char>(d_ws, L.bhat); g.ldb = 4 * L.h; g.b_batch = L.sBhat;
    g.rows_a = bm; g.rows_b = bn; g.kdim = 4 * L.h; g.batches = sc.R; g.groups = L.G;
    g.out = at<char>(d_ws, L.prod); g.ldo = bn; g.o_batch = L.sProd; g.out_mode = 0; g.output = FMM_F32;
    g.status = at<DeviceStatus>(d_ws, L.status);
    ProfScope ps(2, st);
    FMM_TRY(launch_block_products(g, st));
  }
  {
    ProfScope ps(3, st);
    transpose_scales_kernel<<<stream_blocks(M * L.G, 256), 256, 0, st>>>(d_dA, M, L.G, at<float>(d_ws, L.dAt));
    ++fmm_launch_counter();
    transpose_scales_kernel<<<stream_blocks(N * L.G, 256), 256, 0, st>>>(d_dB, N, L.G, at<float>(d_ws, L.dBt));
    ++fmm_launch_counter();
    FMM_CUDA(cudaGetLastError());
    FMM_CUDA(launch_decode_group(output, at<float>(d_ws, L.prod), L.sProd, L.G, at<CoefTable>(d_ws, L.tabW), hW.get(), sc.R,
                                 at<float>(d_ws, L.dAt), at<float>(d_ws, L.dBt), sc.m, sc.n, bm, bn, d_C, ldc, true, st));
  }
  return FMM_OK;
}

}  // extern "C"
