// Bodies of the streaming passes (encode, decode, batch decode) as device functions, so that the same code runs as a
// kernel of its own (a CTA of 256 threads per block of the pass) and as a role inside the fused sweep kernel (eight warps
// beside the tensor-core roles of a block-product CTA).  Everything here has internal linkage.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include "kernels_stream.cuh"

namespace {

// ------------------------------------------------------------------------------------------
// small device helpers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void store4(__nv_bfloat16* p, float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 raw;
  raw.x = *reinterpret_cast<uint32_t*>(&lo);
  raw.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = raw;
}
__device__ __forceinline__ void store4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
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

// One group of 256 threads that works as a block of a streaming pass: a whole CTA (bar 0 = __syncthreads), or eight
// warps of a larger CTA that runs other roles beside them (a named barrier of their own).
struct StreamRole {
  int tid;       // thread index inside the group, 0..255 (group bases are multiples of 32: warps stay whole)
  int bid;       // index of this (virtual) block of the pass
  int nblocks;   // number of (virtual) blocks of the pass
  int bar;       // barrier id of the group
  __device__ __forceinline__ void sync() const {
    if (bar == 0) __syncthreads();
    else asm volatile("bar.sync %0, 256;" ::"r"(bar) : "memory");
  }
};

__device__ __forceinline__ double block_sum_double(const StreamRole role, double v, double* red /* >= 8 doubles smem */) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int warp = role.tid >> 5, lane = role.tid & 31;
  role.sync();
  if (lane == 0) red[warp] = v;
  role.sync();
  double tot = 0.0;
  if (role.tid == 0)
    for (int w = 0; w < 8; ++w) tot += red[w];
  return tot;  // valid in thread 0 of the group
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
// A block of 256 threads owns 64 "position vectors" (16 bytes = 8 bf16 or 4 fp32 consecutive
// inner-dimension elements of one block row).  Four threads share each position vector:
//   1. together they copy the raw 16-byte vectors of all grid cells at that position into shared memory with
//      cp.async ([cell][position], conflict free; slab `ncell` holds zeros), two stages deep, so the copies of
//      the next tile overlap the arithmetic and the stores of this one;
//   2. thread g of the four then forms the products r = g, g+4, g+8, ...: it walks the coefficient list
//      of r two entries per step (lists are padded to an even length with (zero slab, 0.0f) entries, which
//      add exactly nothing), an fp32 FMA chain in list order, two lanes per instruction (packed
//      fma.rn.f32x2: each lane is an ordinary IEEE fp32 FMA), and stores 16 / 8 bytes.
// ------------------------------------------------------------------------------------------
constexpr int kEncThreads = 256;
// kEncSplit threads share one position vector (4 for the 4 x 4 grids / 49 products; 1 when the scheme is small,
// where splitting would leave each thread almost nothing to do between barriers); kEncPos position vectors
// per block.
constexpr int kChunk = kTablePad;   // lists arrive padded to this multiple

struct EncSmemHead {
  int off[FMM_MAX_R + 1];   // in units of entries, multiples of kChunk
  int pad[3];
  float scale[FMM_MAX_R];
  float inv_scale[FMM_MAX_R];
  int use_mul[FMM_MAX_R];
  unsigned amax[FMM_MAX_R];
};  // followed by int2 ent[] {byte offset of the cell's slab, coefficient bits}, then the stage

template <typename SrcT> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int kElems = 4;
  static __device__ __forceinline__ void unpack(const uint4& raw, float2 (&v)[2]) {
    v[0] = make_float2(__uint_as_float(raw.x), __uint_as_float(raw.y));
    v[1] = make_float2(__uint_as_float(raw.z), __uint_as_float(raw.w));
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int kElems = 8;
  static __device__ __forceinline__ void unpack(const uint4& raw, float2 (&v)[4]) {
    v[0] = make_float2(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xFFFF0000u));
    v[1] = make_float2(__uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xFFFF0000u));
    v[2] = make_float2(__uint_as_float(raw.z << 16), __uint_as_float(raw.z & 0xFFFF0000u));
    v[3] = make_float2(__uint_as_float(raw.w << 16), __uint_as_float(raw.w & 0xFFFF0000u));
  }
};

// e4m3 source (the second level of a per-level rounding reads the first level's codes): 16 elements per vector
template <> struct Vec16<__nv_fp8_storage_t> {
  static constexpr int kElems = 16;
  static __device__ __forceinline__ float2 pair(unsigned short two) {
    const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)two, __NV_E4M3);
    return __half22float2(*reinterpret_cast<const __half2*>(&h));
  }
  static __device__ __forceinline__ void unpack(const uint4& raw, float2 (&v)[8]) {
    v[0] = pair((unsigned short)(raw.x & 0xFFFFu)); v[1] = pair((unsigned short)(raw.x >> 16));
    v[2] = pair((unsigned short)(raw.y & 0xFFFFu)); v[3] = pair((unsigned short)(raw.y >> 16));
    v[4] = pair((unsigned short)(raw.z & 0xFFFFu)); v[5] = pair((unsigned short)(raw.z >> 16));
    v[6] = pair((unsigned short)(raw.w & 0xFFFFu)); v[7] = pair((unsigned short)(raw.w >> 16));
  }
};

// `stream`: the outputs will have left L2 before they are read again, so store them evict-first (st.global.cs)
template <int NP> __device__ __forceinline__ void store_vec(__nv_bfloat16* p, const float2 (&a)[NP], bool stream) {
  uint32_t w[NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    __nv_bfloat162 b = __floats2bfloat162_rn(a[i].x, a[i].y);
    w[i] = *reinterpret_cast<uint32_t*>(&b);
  }
  if (NP == 4) {
    const uint4 v = make_uint4(w[0], w[1], w[2 % NP], w[3 % NP]);
    if (stream) __stcs(reinterpret_cast<uint4*>(p), v); else *reinterpret_cast<uint4*>(p) = v;
  } else {
    const uint2 v = make_uint2(w[0], w[1]);
    if (stream) __stcs(reinterpret_cast<uint2*>(p), v); else *reinterpret_cast<uint2*>(p) = v;
  }
}
// e4m3: round to nearest even, saturate to +-448 (NaN stays NaN)
template <int NP> __device__ __forceinline__ void store_vec(__nv_fp8_storage_t* p, const float2 (&a)[NP], bool stream) {
  uint32_t h[NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) h[i] = __nv_cvt_float2_to_fp8x2(a[i], __NV_SATFINITE, __NV_E4M3);
  if (NP == 8) {
    const uint4 v = make_uint4(h[0] | (h[1] << 16), h[2 % NP] | (h[3 % NP] << 16), h[4 % NP] | (h[5 % NP] << 16),
                               h[6 % NP] | (h[7 % NP] << 16));
    if (stream) __stcs(reinterpret_cast<uint4*>(p), v); else *reinterpret_cast<uint4*>(p) = v;
  } else if (NP == 4) {
    const uint2 v = make_uint2(h[0] | (h[1] << 16), h[2 % NP] | (h[3 % NP] << 16));
    if (stream) __stcs(reinterpret_cast<uint2*>(p), v); else *reinterpret_cast<uint2*>(p) = v;
  } else {
    const unsigned v = h[0] | (h[1] << 16);
    if (stream) __stcs(reinterpret_cast<unsigned*>(p), v); else *reinterpret_cast<unsigned*>(p) = v;
  }
}

// x / sc for values that are about to be rounded to e4m3, without eight IEEE divisions in the common case.  The exact
// schedule is code = rnd_e4m3(fl32(x / sc)).  q = x * fl32(1 / sc) lies within 1.5 * 2^-23 (relative) of fl32(x / sc); rounding
// to e4m3 is monotone, so if q (1 + 2^-21) and q (1 - 2^-21) round to the same code, so does fl32(x / sc), and q can stand
// in for it.  Otherwise (a value that close to a rounding boundary: a few in a million) the vector is divided exactly.
template <int NP>
__device__ __forceinline__ void divide_for_e4m3(float2 (&a)[NP], float sc) {
  const float r = __frcp_rn(sc);
  const float2 up = make_float2(1.0f + 4.76837158203125e-7f, 1.0f + 4.76837158203125e-7f);
  const float2 dn = make_float2(1.0f - 4.76837158203125e-7f, 1.0f - 4.76837158203125e-7f);
  float2 q[NP];
  bool same = true;
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    q[i] = __fmul2_rn(a[i], make_float2(r, r));
    const unsigned hi = __nv_cvt_float2_to_fp8x2(__fmul2_rn(q[i], up), __NV_SATFINITE, __NV_E4M3);
    const unsigned lo = __nv_cvt_float2_to_fp8x2(__fmul2_rn(q[i], dn), __NV_SATFINITE, __NV_E4M3);
    same = same && (hi == lo);
  }
  if (same) {
#pragma unroll
    for (int i = 0; i < NP; ++i) a[i] = q[i];
  } else {
#pragma unroll
    for (int i = 0; i < NP; ++i) { a[i].x = __fdiv_rn(a[i].x, sc); a[i].y = __fdiv_rn(a[i].y, sc); }
  }
}


// kM3: the model schedule (use_scale == 3) is compiled into its own instantiation so that the other modes carry none
// of its index arithmetic.
// kDense: a grid of four cells whose every product reads all four, in one cell order shared by all lists (what a general
// gauge on a 2 x 2 grid produces): the four source vectors are unpacked once per tile and every product is a four-term
// chain on registers — the same FMAs in the same order as the list walk.
template <typename SrcT, typename DstT, bool kAmaxOnly, int kEncSplit, bool kM3, bool kDense = false>
__device__ __forceinline__ void encode_body(const StreamRole role, unsigned char* smem_raw, const EncodeJob& job_a,
                                             const EncodeJob& job_b, int use_scale) {
  const bool second = role.bid >= job_a.blocks;
  const int bid = role.bid - (second ? job_a.blocks : 0);
  const SrcT* __restrict__ X = static_cast<const SrcT*>(second ? job_b.X : job_a.X);
  const int64_t ldx = second ? job_b.ldx : job_a.ldx;
  const int gc = second ? job_b.gc : job_a.gc;
  const int64_t br = second ? job_b.br : job_a.br, bc = second ? job_b.bc : job_a.bc;
  const CoefTable* __restrict__ d_tab = second ? job_b.tab : job_a.tab;
  DstT* __restrict__ out = static_cast<DstT*>(second ? job_b.out : job_a.out);
  unsigned* __restrict__ amax_bits = second ? job_b.amax_bits : job_a.amax_bits;
  float* __restrict__ scale_out = second ? job_b.scale_out : job_a.scale_out;
  const int tiles_per_block = second ? job_b.tiles_per_block : job_a.tiles_per_block;
  const int64_t rstride = second ? job_b.rstride : job_a.rstride;
  const int stream_out = second ? job_b.stream_out : job_a.stream_out;
  const int scale_rows = second ? job_b.scale_rows : job_a.scale_rows;
  const int bf16_first = second ? job_b.bf16_first : job_a.bf16_first;
  const float* __restrict__ pre_scale = second ? job_b.pre_scale : job_a.pre_scale;
  constexpr int VE = Vec16<SrcT>::kElems;
  constexpr int kEncPos = kEncThreads / kEncSplit;
  constexpr int kCellsPerThread = 16 / kEncSplit; // grids have at most 16 cells
  constexpr int NP = VE / 2;                     // float2 pairs per vector
  constexpr int kSlab = kEncPos * 16;            // bytes of one cell's slab: the raw 16-byte vectors of a tile
  EncSmemHead& sm = *reinterpret_cast<EncSmemHead*>(smem_raw);
  const int R = d_tab->R, ncell = d_tab->ncell;
  const int total = d_tab->off[R];               // lists arrive padded to multiples of kChunk
  int2* ent = reinterpret_cast<int2*>(smem_raw + sizeof(EncSmemHead));
  // two stages of (ncell + 1) slabs: the copies of tile it+1 land in one while tile it is read from the other
  unsigned char* stage = smem_raw + ((sizeof(EncSmemHead) + (size_t)total * 8 + 15) / 16) * 16;
  const int kStageBytes = (ncell + 1) * kSlab;

  for (int i = role.tid; i <= R; i += kEncThreads) sm.off[i] = d_tab->off[i];
  for (int i = role.tid; i < total; i += kEncThreads)
    ent[i] = make_int2(d_tab->cell[i] * kSlab, __float_as_int(d_tab->coef[i]));
  if (role.tid < R) {
    float s = 1.0f;
    if (!kAmaxOnly && use_scale == 1) s = pow2_scale_448(__uint_as_float(amax_bits[role.tid]));
    sm.scale[role.tid] = s;
    const float inv = 1.0f / s;
    sm.use_mul[role.tid] = (isfinite(inv) && inv * s == 1.0f && fabsf(inv) >= 1.17549435e-38f);
    sm.inv_scale[role.tid] = inv;
    sm.amax[role.tid] = 0u;
    if (!kAmaxOnly && use_scale == 1 && bid == 0 && scale_out)
      scale_out[role.tid] = pre_scale ? s * pre_scale[0] : s;   // powers of two: the product is exact
  }

  const int g = role.tid / kEncPos;           // which share of the cells / products this thread handles
  const int pv = role.tid - g * kEncPos;      // position vector inside the tile
  const int vec_per_row = (int)(bc / VE);        // 32-bit index arithmetic: br * bc / VE < 2^31 (checked by the host)
  const int nvec = (int)br * vec_per_row;
  // element offset of each grid cell this thread stages (cells g, g+kEncSplit, ...), computed once
  int64_t cell_base[kCellsPerThread];
#pragma unroll
  for (int u = 0; u < kCellsPerThread; ++u) {
    const int c = g + u * kEncSplit;
    const int gi = c / gc, gj = c - gi * gc;
    cell_base[u] = (int64_t)gi * br * ldx + (int64_t)gj * bc;
  }
  if (g == 0) {   // the all-zero slab behind the data slabs, in both stages
    *reinterpret_cast<uint4*>(stage + ncell * kSlab + pv * 16) = make_uint4(0u, 0u, 0u, 0u);
    *reinterpret_cast<uint4*>(stage + kStageBytes + ncell * kSlab + pv * 16) = make_uint4(0u, 0u, 0u, 0u);
  }
  const uint32_t stage_u32 = (uint32_t)__cvta_generic_to_shared(stage) + pv * 16;

  // asynchronous copies of this thread's cells of tile `it` into stage `it & 1` (16 bytes each, L2 only)
  auto issue_copies = [&](int it) {
    if (it < tiles_per_block) {
      const int idx = (bid * tiles_per_block + it) * kEncPos + pv;
      const bool live = idx < nvec;
      const int p = live ? idx / vec_per_row : 0;
      const int t = live ? (idx - p * vec_per_row) * VE : 0;
      const SrcT* src = X + (int64_t)p * ldx + t;
      const uint32_t dst = stage_u32 + (it & 1) * kStageBytes;
      const int nbytes = live ? 16 : 0;          // 0 source bytes: the destination is zero-filled
#pragma unroll
      for (int u = 0; u < kCellsPerThread; ++u) {
        const int c = g + u * kEncSplit;
        if (c < ncell)
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + c * kSlab), "l"(src + cell_base[u]),
                       "r"(nbytes) : "memory");
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  issue_copies(0);

  for (int it = 0; it < tiles_per_block; ++it) {
    const int idx = (bid * tiles_per_block + it) * kEncPos + pv;
    const bool live = idx < nvec;
    const int p = live ? idx / vec_per_row : 0;
    const int t = live ? (idx - p * vec_per_row) * VE : 0;
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    role.sync();        // tile it has landed for every thread, and everyone is done reading tile it-1's stage
    issue_copies(it + 1);   // overlaps the arithmetic and the stores below
    const unsigned char* my_stage = stage + (it & 1) * kStageBytes + pv * 16;

    DstT* dst = out + (int64_t)p * bc + t;
    const int m3_gk = (int)((bc + 127) >> 7);                                   // used by the model schedule only
    const int64_t m3_row_groups = scale_rows == 1 ? br : (br + 127) >> 7;       // scale_rows is 1 or 128
    const int64_t m3_row_group = scale_rows == 1 ? p : p >> 7;
    // one product at a time, its list walked two entries per step (lists are padded to an even length with
    // (zero slab, 0.0f) entries, which add exactly nothing); the four accumulator pairs are independent chains
    float2 src[kDense ? 4 : 1][NP];
    if constexpr (kDense) {     // slab offsets of the list's four entries are the same for every product: take product 0's
#pragma unroll
      for (int c = 0; c < 4; ++c) Vec16<SrcT>::unpack(*reinterpret_cast<const uint4*>(my_stage + ent[c].x), src[c]);
    }
    for (int r = g; r < R; r += kEncSplit) {
      float2 acc[NP];
#pragma unroll
      for (int i = 0; i < NP; ++i) acc[i] = make_float2(0.0f, 0.0f);
      const int eend = sm.off[r + 1];
      if constexpr (kDense) {
        const int4 p0 = *reinterpret_cast<const int4*>(&ent[4 * r]);
        const int4 p1 = *reinterpret_cast<const int4*>(&ent[4 * r + 2]);
        const float cf[4] = {__int_as_float(p0.y), __int_as_float(p0.w), __int_as_float(p1.y), __int_as_float(p1.w)};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
#pragma unroll
          for (int i = 0; i < NP; ++i) acc[i] = __ffma2_rn(make_float2(cf[c], cf[c]), src[c][i], acc[i]);
        }
      } else
      for (int e = sm.off[r]; e < eend; e += 2) {
        const int4 pair = *reinterpret_cast<const int4*>(&ent[e]);
        const uint4 raw0 = *reinterpret_cast<const uint4*>(my_stage + pair.x);
        const uint4 raw1 = *reinterpret_cast<const uint4*>(my_stage + pair.z);
        float2 v[NP];
        const float c0 = __int_as_float(pair.y), c1 = __int_as_float(pair.w);
        Vec16<SrcT>::unpack(raw0, v);
#pragma unroll
        for (int i = 0; i < NP; ++i) acc[i] = __ffma2_rn(make_float2(c0, c0), v[i], acc[i]);
        Vec16<SrcT>::unpack(raw1, v);
#pragma unroll
        for (int i = 0; i < NP; ++i) acc[i] = __ffma2_rn(make_float2(c1, c1), v[i], acc[i]);
      }
      // model schedule (use_scale 3): one scale per 128 consecutive entries of a row, shared by scale_rows rows
      int64_t sidx3 = 0;
      if constexpr (kM3) sidx3 = ((int64_t)r * m3_row_groups + m3_row_group) * m3_gk + (t >> 7);
      if (kM3 && bf16_first) {
#pragma unroll
        for (int i = 0; i < NP; ++i) {
          acc[i].x = __bfloat162float(__float2bfloat16_rn(acc[i].x));
          acc[i].y = __bfloat162float(__float2bfloat16_rn(acc[i].y));
        }
      }
      if (kAmaxOnly) {
        float a = 0.0f;
#pragma unroll
        for (int i = 0; i < NP; ++i) a = fmaxf(a, fmaxf(fabsf(acc[i].x), fabsf(acc[i].y)));   // fmaxf drops NaN
        if (kM3) {
          constexpr int kLanesPerGroup = 128 / VE;   // 16 (bf16 source) or 32 (fp32 source) lanes cover one 128-group
          if ((vec_per_row & 31) == 0) {             // a warp's 32 consecutive vectors lie in one row
            const unsigned mask = kLanesPerGroup == 32 ? 0xffffffffu : (0xffffu << (role.tid & 16));
            const unsigned wmax = __reduce_max_sync(mask, live ? __float_as_uint(a) : 0u);
            if ((role.tid & (kLanesPerGroup - 1)) == 0 && wmax != 0u) atomicMax(&amax_bits[sidx3], wmax);
          } else if (live && a > 0.0f) {
            atomicMax(&amax_bits[sidx3], __float_as_uint(a));
          }
        } else if (use_scale == 2) {
          // one scale per row of the block sum: largest magnitude of row p of product r
          if ((vec_per_row & 31) == 0) {       // a warp's 32 consecutive vectors lie in one row
            const unsigned wmax = __reduce_max_sync(0xffffffffu, live ? __float_as_uint(a) : 0u);
            if ((role.tid & 31) == 0 && wmax != 0u) atomicMax(&amax_bits[(int64_t)r * br + p], wmax);
          } else if (live && a > 0.0f) {
            atomicMax(&amax_bits[(int64_t)r * br + p], __float_as_uint(a));
          }
        } else {
          // non-negative floats order like their bit patterns: one warp-wide integer max
          const unsigned wmax = __reduce_max_sync(0xffffffffu, __float_as_uint(a));
          if ((role.tid & 31) == 0 && wmax != 0u) atomicMax(&sm.amax[r], wmax);
        }
      } else if (live) {
        if (kM3) {
          const float amax = __uint_as_float(amax_bits[sidx3]);
          const float sc = amax > 0.0f ? __fdiv_rn(amax, 448.0f) : 1.0f;
          if constexpr (sizeof(DstT) == 1) {
            divide_for_e4m3<NP>(acc, sc);
          } else {
#pragma unroll
            for (int i = 0; i < NP; ++i) { acc[i].x = __fdiv_rn(acc[i].x, sc); acc[i].y = __fdiv_rn(acc[i].y, sc); }
          }
          if ((t & 127) == 0 && (p & (scale_rows - 1)) == 0 && scale_out) scale_out[sidx3] = sc;
        } else if (use_scale == 2) {
          // scale = max|x| / 448 in fp32 (1 for an all-zero row), code = x / scale in fp32, then one rounding
          const float amax = __uint_as_float(amax_bits[(int64_t)r * br + p]);
          const float sc = amax > 0.0f ? __fdiv_rn(amax, 448.0f) : 1.0f;
          if constexpr (sizeof(DstT) == 1) {
            divide_for_e4m3<NP>(acc, sc);
          } else {
#pragma unroll
            for (int i = 0; i < NP; ++i) { acc[i].x = __fdiv_rn(acc[i].x, sc); acc[i].y = __fdiv_rn(acc[i].y, sc); }
          }
          if (t == 0 && scale_out) scale_out[(int64_t)r * br + p] = sc;
        } else if (use_scale) {
          if (sm.use_mul[r]) {
            const float inv = sm.inv_scale[r];
#pragma unroll
            for (int i = 0; i < NP; ++i) { acc[i].x *= inv; acc[i].y *= inv; }
          } else {
            const float sc = sm.scale[r];
#pragma unroll
            for (int i = 0; i < NP; ++i) { acc[i].x = __fdiv_rn(acc[i].x, sc); acc[i].y = __fdiv_rn(acc[i].y, sc); }
          }
        }
        store_vec<NP>(dst + r * rstride, acc, stream_out != 0);
      }
    }
  }
  if (kAmaxOnly && use_scale == 1) {
    role.sync();
    if (role.tid < R && sm.amax[role.tid] != 0u) atomicMax(&amax_bits[role.tid], sm.amax[role.tid]);
  }
}

// ------------------------------------------------------------------------------------------
// decode: C_ij = rnd_O( sum_r w_{r,ij} sA_r sB_r M_r ), ascending r, fp32 FMA chain; optional error
// reduction sum (rnd_O(c) - C*)^2 per block (fp32 per thread -> fp64 shuffle tree -> one fp64 partial
// per block).  A block of 256 threads owns 64 "position quads" (4 consecutive columns of one block
// position).  Four threads share each quad:
//   1. together they copy the R product vectors of that position straight into shared memory with
//      cp.async ([r][position], slab R holds zeros) — thread g copies r = g, g+4, ...;
//   2. thread g then forms the output cells c = g, g+4, ...: it walks the cell's (r, w) list (cell-major
//      table, ascending r, padded to a multiple of 4 with (zero slab, 0.0f) entries) in registers, two
//      lanes per packed fma.rn.f32x2, rounds, stores, and accumulates its share of the error.
// ------------------------------------------------------------------------------------------
constexpr int kDecThreads = 256;   // kDecSplit threads share one position quad (4, or 1 for small schemes)

struct DecSmemHead {
  int off[kMaxCells + 1];   // entries, multiples of kChunk
  int pad[3];
  double red[kDecThreads / 32];
};  // followed by int2 ent[] {byte offset of product r's slab, scaled coefficient bits}, then the stage

// four consecutive products of one row, staged as 16 bytes (fp32) or 8 bytes (bf16)
__device__ __forceinline__ float4 staged_quad(const unsigned char* p, const float*) {
  return *reinterpret_cast<const float4*>(p);
}
__device__ __forceinline__ float4 staged_quad(const unsigned char* p, const __nv_bfloat16*) {
  const uint2 raw = *reinterpret_cast<const uint2*>(p);
  const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
  const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
  return make_float4(__low2float(lo), __high2float(lo), __low2float(hi), __high2float(hi));
}

template <typename OutT, bool kStore, bool kErr, int kDecSplit, typename ProdT>
__device__ __forceinline__ void decode_body(const StreamRole role, unsigned char* smem_raw, const ProdT* __restrict__ prod, const CoefTable* __restrict__ d_tab, int R,
              const float* __restrict__ sA, const float* __restrict__ sB, int n, int64_t bm, int64_t bn,
              OutT* __restrict__ C, int64_t ldc, const float* __restrict__ cstar32, int64_t ldcs,
              double* __restrict__ partials, int tiles_per_block, int64_t rstride, int gauges) {
  // gauges > 1 (error reduction only): the table describes `gauges` equivalent algorithms at once; list c belongs to
  // C block c / gauges of algorithm c % gauges, and every algorithm gets its own error sum.  gauges divides kDecSplit,
  // so a thread's lists (c = g, g + kDecSplit, ...) all belong to one algorithm.
  constexpr int kDecPos = kDecThreads / kDecSplit;
  constexpr int kCellsPerThread = 16 / kDecSplit;
  constexpr int kVecBytes = 4 * (int)sizeof(ProdT);   // one position quad of products: 16 bytes (fp32) or 8 (bf16)
  constexpr int kSlab = kDecPos * kVecBytes;
  DecSmemHead& sm = *reinterpret_cast<DecSmemHead*>(smem_raw);
  const int ncell = d_tab->R;                  // number of lists = number of C blocks
  const int total = d_tab->off[ncell];         // lists arrive padded to multiples of kChunk
  int2* ent = reinterpret_cast<int2*>(smem_raw + sizeof(DecSmemHead));
  unsigned char* stage = smem_raw + ((sizeof(DecSmemHead) + (size_t)total * 8 + 15) / 16) * 16;

  const int g = role.tid / kDecPos;
  const int pq = role.tid - g * kDecPos;
  const int vec_per_row = (int)(bn >> 2);      // 32-bit index arithmetic: bm * bn / 4 < 2^31 (checked by the host)
  const int nvec = (int)bm * vec_per_row;
  unsigned char* my_stage = stage + pq * kVecBytes;
  const uint32_t dst0 = (uint32_t)__cvta_generic_to_shared(my_stage);
  // element offsets of the output cells this thread forms (cells g, g+4, ...), computed once
  int64_t out_base[kCellsPerThread], cs_base[kCellsPerThread];
#pragma unroll
  for (int u = 0; u < kCellsPerThread; ++u) {
    const int c = (g + u * kDecSplit) / gauges;   // the C block this list feeds
    const int i = c / n, j = c - i * n;
    out_base[u] = (int64_t)i * bm * ldc + (int64_t)j * bn;
    cs_base[u] = (int64_t)i * bm * ldcs + (int64_t)j * bn;
  }

  // one algorithm per thread group: the reference values of C block g are staged once per position by thread group g
  // and read by all groups, instead of every algorithm loading them again
  const bool stage_cs = kErr && kDecSplit > 1 && gauges == kDecSplit;
  unsigned char* cs_stage = stage + (size_t)(R + 1) * kSlab + pq * 16;
  const bool cs_mine = stage_cs && g * gauges < ncell;
  const int64_t cs_src = (int64_t)(g / n) * bm * ldcs + (int64_t)(g % n) * bn;

  float err = 0.0f;
  for (int it = 0; it < tiles_per_block; ++it) {
    const int idx = (role.bid * tiles_per_block + it) * kDecPos + pq;
    const bool live = idx < nvec;
    const int p = live ? idx / vec_per_row : 0;
    const int q = live ? (idx - p * vec_per_row) << 2 : 0;
    if (it > 0) role.sync();               // previous tile's readers are done with the stage
    {
      const ProdT* src = prod + (int64_t)p * bn + q;
      const int nbytes = live ? kVecBytes : 0;  // 0 source bytes -> the destination bytes are zero-filled
      for (int r = g; r < R; r += kDecSplit) {
        if (kVecBytes == 16)
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst0 + r * kSlab), "l"(src + r * rstride),
                       "r"(nbytes) : "memory");
        else
          asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst0 + r * kSlab), "l"(src + r * rstride),
                       "r"(nbytes) : "memory");
      }
      if (kErr && cs_mine)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(cs_stage + g * (kDecPos * 16))),
                     "l"(cstar32 + cs_src + (int64_t)p * ldcs + q), "r"(live ? 16 : 0) : "memory");
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    if (it == 0) {                             // table set-up overlaps the first tile's copies
      if (g == 0) {
        if (kVecBytes == 16) *reinterpret_cast<float4*>(my_stage + R * kSlab) = make_float4(0.f, 0.f, 0.f, 0.f);
        else *reinterpret_cast<uint2*>(my_stage + R * kSlab) = make_uint2(0u, 0u);
      }
      for (int i = role.tid; i <= ncell; i += kDecThreads) sm.off[i] = d_tab->off[i];
      for (int i = role.tid; i < total; i += kDecThreads) {
        const int r = d_tab->cell[i];
        float w = d_tab->coef[i];
        if (sA != nullptr && r < R) w *= sA[r] * sB[r];   // power-of-two scales fold exactly into the coefficient
        ent[i] = make_int2(r * kSlab, __float_as_int(w));
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    role.sync();

#pragma unroll
    for (int u4 = 0; u4 < kCellsPerThread; ++u4) {   // ncell <= 16
      const int c = g + u4 * kDecSplit;
      if (c >= ncell) break;
      float2 x0 = make_float2(0.f, 0.f), x1 = make_float2(0.f, 0.f);
      const int e1 = sm.off[c + 1];
      for (int e = sm.off[c]; e < e1; e += kChunk) {
        int2 en[kChunk];
        float4 v[kChunk];
#pragma unroll
        for (int u = 0; u < kChunk; u += 2) {
          const int4 two = *reinterpret_cast<const int4*>(&ent[e + u]);
          en[u] = make_int2(two.x, two.y);
          en[u + 1] = make_int2(two.z, two.w);
        }
#pragma unroll
        for (int u = 0; u < kChunk; ++u) v[u] = staged_quad(my_stage + en[u].x, (const ProdT*)nullptr);
#pragma unroll
        for (int u = 0; u < kChunk; ++u) {
          const float w = __int_as_float(en[u].y);
          const float2 ww = make_float2(w, w);
          x0 = __ffma2_rn(ww, make_float2(v[u].x, v[u].y), x0);
          x1 = __ffma2_rn(ww, make_float2(v[u].z, v[u].w), x1);
        }
      }
      if (live) {
        const float4 x = make_float4(x0.x, x0.y, x1.x, x1.y);
        if (kStore) store4(C + out_base[u4] + (int64_t)p * ldc + q, x);
        if (kErr) {
          const float4 cs = stage_cs ? *reinterpret_cast<const float4*>(cs_stage + u4 * (kDecPos * 16))
                                     : __ldcs(reinterpret_cast<const float4*>(cstar32 + cs_base[u4] + (int64_t)p * ldcs + q));
          const float d0 = round_out(x.x, (OutT*)nullptr) - cs.x, d1 = round_out(x.y, (OutT*)nullptr) - cs.y;
          const float d2 = round_out(x.z, (OutT*)nullptr) - cs.z, d3 = round_out(x.w, (OutT*)nullptr) - cs.w;
          err = __fmaf_rn(d0, d0, err); err = __fmaf_rn(d1, d1, err);
          err = __fmaf_rn(d2, d2, err); err = __fmaf_rn(d3, d3, err);
        }
      }
    }
  }
  if (kErr) {
    if (gauges == 1) {
      const double tot = block_sum_double(role, (double)err, sm.red);
      if (role.tid == 0) partials[role.bid] = tot;
    } else {
      // one sum per algorithm: warps with the same (g % gauges); partials laid out [algorithm][block]
      double v = (double)err;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      const int warp = role.tid >> 5;
      role.sync();
      if ((role.tid & 31) == 0) sm.red[warp] = v;
      role.sync();
      if (role.tid < gauges) {
        double tot = 0.0;
        for (int w = 0; w < kDecThreads / 32; ++w)
          if (((w * 32) / kDecPos) % gauges == (int)role.tid) tot += sm.red[w];
        partials[(size_t)role.tid * role.nblocks + role.bid] = tot;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// reductions
// ------------------------------------------------------------------------------------------
// Error-only decode of a batch of four or eight gauge-equivalent algorithms with at most kBatchR products and four output
// cells each (one level on a 2 x 2 grid).  Thread group g (two warps, or one for eight algorithms) owns algorithm g: a thread keeps the
// algorithm's products of its position quad in registers — 16-byte loads straight from the product buffers, all
// issued before the first use — and forms every output cell as the same fp32 FMA chain in ascending r that the list
// walk of decode_kernel performs (coefficients from a dense [algorithm][cell][r] copy of the table in shared memory;
// absent entries are skipped, not multiplied).  The reference values of a position are staged once for the four
// algorithms, two tiles deep.  The table is the merged one of the batch: list c * kGauges + g holds cell c of algorithm g,
// its products numbered g * RB .. g * RB + RB - 1.
// ------------------------------------------------------------------------------------------
constexpr int kBatchR = 8;

// shared memory of one group running decode_batch_body
template <int kGauges>
struct __align__(16) DecBatchSmem {
  float4 cs_stage[2][4][kDecThreads / kGauges];
  float Wd[kGauges][4][kBatchR];
  double red[kDecThreads / 32];
};

template <typename OutT, typename ProdT, int kGauges>
__device__ __forceinline__ void decode_batch_body(const StreamRole role, DecBatchSmem<kGauges>& sm, const ProdT* __restrict__ prod, const CoefTable* __restrict__ d_tab, int RB,
                    const float* __restrict__ sA, const float* __restrict__ sB, int n, int64_t bm, int64_t bn,
                    const float* __restrict__ cstar32, int64_t ldcs, double* __restrict__ partials,
                    int tiles_per_block, int64_t rstride) {
  constexpr int kPos = kDecThreads / kGauges;          // 64 positions for four algorithms, 32 for eight
  auto& Wd = sm.Wd;
  auto& cs_stage = sm.cs_stage;
  double* red = sm.red;
  const int cells = d_tab->R / kGauges;           // output cells per algorithm (<= 4)
  const int Rtot = RB * kGauges;
  for (int i = role.tid; i < kGauges * 4 * kBatchR; i += kDecThreads) (&Wd[0][0][0])[i] = 0.0f;
  role.sync();
  {
    const int total = d_tab->off[d_tab->R];
    for (int i = role.tid; i < total; i += kDecThreads) {
      const int r = d_tab->cell[i];
      if (r >= Rtot) continue;                     // padding entry
      int c = 0;                                   // the list this entry belongs to
      while (d_tab->off[c + 1] <= i) ++c;
      float w = d_tab->coef[i];
      if (sA != nullptr) w *= sA[r] * sB[r];       // power-of-two scales fold exactly into the coefficient
      const int g2 = c % kGauges;
      Wd[g2][c / kGauges][r - g2 * RB] = w;
    }
  }
  const int g = role.tid / kPos;
  const int pq = role.tid - g * kPos;
  const int vec_per_row = (int)(bn >> 2);
  const int nvec = (int)bm * vec_per_row;
  const bool cs_mine = g < cells;
  const int64_t cs_src = (int64_t)(g / n) * bm * ldcs + (int64_t)(g % n) * bn;
  const uint32_t cs_dst = (uint32_t)__cvta_generic_to_shared(&cs_stage[0][g][pq]);
  constexpr uint32_t kCsBuf = 4 * kPos * 16;
  auto issue_cs = [&](int it) {
    if (it < tiles_per_block && cs_mine) {
      const int idx = (role.bid * tiles_per_block + it) * kPos + pq;
      const bool live = idx < nvec;
      const int p = live ? idx / vec_per_row : 0;
      const int q = live ? (idx - p * vec_per_row) << 2 : 0;
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(cs_dst + (it & 1) * kCsBuf),
                   "l"(cstar32 + cs_src + (int64_t)p * ldcs + q), "r"(live ? 16 : 0) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  issue_cs(0);
  float err = 0.0f;
  const ProdT* my_prod = prod + (int64_t)g * RB * rstride;
  for (int it = 0; it < tiles_per_block; ++it) {
    const int idx = (role.bid * tiles_per_block + it) * kPos + pq;
    const bool live = idx < nvec;
    const int p = live ? idx / vec_per_row : 0;
    const int q = live ? (idx - p * vec_per_row) << 2 : 0;
    float4 v[kBatchR];
#pragma unroll
    for (int r = 0; r < kBatchR; ++r) {
      v[r] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (r < RB && live) {
        const ProdT* src = my_prod + (int64_t)r * rstride + (int64_t)p * bn + q;
        if constexpr (sizeof(ProdT) == 4) {
          v[r] = __ldcs(reinterpret_cast<const float4*>(src));
        } else {
          const uint2 raw = __ldcs(reinterpret_cast<const uint2*>(src));
          v[r] = staged_quad(reinterpret_cast<const unsigned char*>(&raw), (const ProdT*)nullptr);
        }
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    role.sync();          // tile it's reference values have landed; everyone is done reading the other buffer
    issue_cs(it + 1);
    if (live) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        if (c < cells) {
          float2 x0 = make_float2(0.f, 0.f), x1 = make_float2(0.f, 0.f);
#pragma unroll
          for (int r = 0; r < kBatchR; ++r) {
            const float w = Wd[g][c][r];
            if (w != 0.0f) {                       // warp-uniform: absent entries are skipped, as in the list walk
              const float2 ww = make_float2(w, w);
              x0 = __ffma2_rn(ww, make_float2(v[r].x, v[r].y), x0);
              x1 = __ffma2_rn(ww, make_float2(v[r].z, v[r].w), x1);
            }
          }
          const float4 cs = cs_stage[it & 1][c][pq];
          const float d0 = round_out(x0.x, (OutT*)nullptr) - cs.x, d1 = round_out(x0.y, (OutT*)nullptr) - cs.y;
          const float d2 = round_out(x1.x, (OutT*)nullptr) - cs.z, d3 = round_out(x1.y, (OutT*)nullptr) - cs.w;
          err = __fmaf_rn(d0, d0, err); err = __fmaf_rn(d1, d1, err);
          err = __fmaf_rn(d2, d2, err); err = __fmaf_rn(d3, d3, err);
        }
      }
    }
  }
  // one sum per algorithm; partials laid out [algorithm][block]
  double sv = (double)err;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sv += __shfl_xor_sync(0xffffffffu, sv, o);
  const int warp = role.tid >> 5;
  role.sync();
  if ((role.tid & 31) == 0) red[warp] = sv;
  role.sync();
  if (role.tid < kGauges) {
    double tot = 0.0;
    for (int w = 0; w < kDecThreads / 32; ++w)
      if ((w * 32) / kPos == (int)role.tid) tot += red[w];
    partials[(size_t)role.tid * role.nblocks + role.bid] = tot;
  }
}

}  // namespace
