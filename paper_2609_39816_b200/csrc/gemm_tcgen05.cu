// Batched block products M_r = Ahat_r * Bhat_r^T on Blackwell tensor cores (sm_100a).
//
// One persistent CTA per SM walks a static list of (product r, row tile, column tile).
//   warp 0        : TMA producer  — cp.async.bulk.tensor loads of a 128 x BK tile of Ahat_r and a
//                   BN x BK tile of Bhat_r (both K-major, 128-byte swizzle) into a shared-memory ring;
//   warp 1        : allocates TMEM, then one lane issues tcgen05.mma (M=128, N=BN, K=32 bytes) into one
//                   of two fp32 accumulator buffers in TMEM, and tcgen05.commit releases ring stages /
//                   publishes the finished accumulator through mbarriers;
//   warps 2..5    : epilogue — tcgen05.ld the accumulator (each warp its own 32-lane quadrant),
//                   store fp32 products (or the rounded, scaled result) to global memory, and hand the
//                   TMEM buffer back.
// Double-buffered TMEM lets the epilogue of tile i overlap the main loop of tile i+1.
// Every mbarrier wait is bounded: after ~2 s without progress a role raises the CTA's abort flag,
// records FMM_ERR_TIMEOUT in the device status word, lets its outstanding copies land (bounded),
// and the CTA frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "kernels_stream.cuh"
#include "stream_bodies.cuh"

namespace {

constexpr int BM = 128;             // rows of A per tile = UMMA M
constexpr int BKB = 128;            // bytes of the inner dimension per ring stage (one swizzle span)
constexpr int UMMA_KB = 32;         // bytes of the inner dimension per tcgen05.mma
constexpr int kNumThreads = 192;    // 6 warps
constexpr unsigned long long kDefaultWaitLimitNs = 2000000000ull;   // 2 s

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// one lane of a converged warp, chosen by the hardware: lets the whole warp run a role's loop with warp-uniform control
// flow (so that loop state and descriptors can live in uniform registers) while a single lane issues
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred != 0;
}

__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait.  Returns false when the CTA is aborting (this wait or another one gave up).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int where,
                                          DeviceStatus* status, unsigned long long limit_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_timer_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 0u) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t0 > limit_ns) {
        *abort_flag = 1;
        if (status != nullptr) {
          atomicExch(&status->code, (int)FMM_ERR_TIMEOUT);
          atomicExch(&status->where, where);
        }
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

template <bool kFp8>
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  if (kFp8) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}

__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile stored as rows of 128 bytes with the 128-byte
// swizzle (what TMA writes with CU_TENSOR_MAP_SWIZZLE_128B): start address (>>4), leading byte offset
// (unused for this layout, 1), stride byte offset = 8 rows * 128 B = 1024 (>>4), descriptor version 1,
// layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Instruction descriptor: fp32 accumulator, A and B formats (kind::f16: 1 = bf16; kind::f8f6f4: 0 = e4m3),
// both operands K-major, N >> 3 at bit 17, M >> 4 at bit 24.
__host__ __device__ constexpr uint32_t make_idesc(bool fp8, int n) {
  return (1u << 4) | ((fp8 ? 0u : 1u) << 7) | ((fp8 ? 0u : 1u) << 10) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(BM >> 4) << 24);
}

// 32-byte store: one full L2 sector per thread (16-byte stores touch half a sector each and double the
// sector writes L2 sees).
__device__ __forceinline__ void st_global_256(void* p, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t a4, uint32_t a5, uint32_t a6, uint32_t a7) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(a0), "r"(a1), "r"(a2),
               "r"(a3), "r"(a4), "r"(a5), "r"(a6), "r"(a7) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&b2);
}

// Store up to 32 consecutive columns of one accumulator row (fp32 products, or the scaled and rounded result).
// `wide` = the destination row is 32-byte aligned.
__device__ __forceinline__ void store_row_chunk(void* out, long long off, int ncols, const uint32_t (&v)[32],
                                                int out_mode, int out_bf16, float alpha, bool wide) {
  if (out_mode == 1 && out_bf16) {
    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(out) + off;
    if (ncols == 32) {
      uint32_t w[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) w[j] = pack_bf16(__uint_as_float(v[2 * j]) * alpha, __uint_as_float(v[2 * j + 1]) * alpha);
      if (wide) {
        st_global_256(dst, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
        st_global_256(dst + 16, w[8], w[9], w[10], w[11], w[12], w[13], w[14], w[15]);
      } else {
#pragma unroll
        for (int j = 0; j < 16; j += 4) *reinterpret_cast<uint4*>(dst + 2 * j) = make_uint4(w[j], w[j + 1], w[j + 2], w[j + 3]);
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (j < ncols) dst[j] = __float2bfloat16_rn(__uint_as_float(v[j]) * alpha);
    }
    return;
  }
  float* dst = reinterpret_cast<float*>(out) + off;
  const float a = out_mode == 1 ? alpha : 1.0f;   // fp32 products are stored unscaled (x * 1.0f is exact)
  if (ncols == 32) {
    uint32_t w[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) w[j] = __float_as_uint(__uint_as_float(v[j]) * a);
    if (wide) {
#pragma unroll
      for (int j = 0; j < 32; j += 8) st_global_256(dst + j, w[j], w[j + 1], w[j + 2], w[j + 3], w[j + 4], w[j + 5], w[j + 6], w[j + 7]);
    } else {
#pragma unroll
      for (int j = 0; j < 32; j += 4) *reinterpret_cast<uint4*>(dst + j) = make_uint4(w[j], w[j + 1], w[j + 2], w[j + 3]);
    }
  } else {
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (j < ncols) dst[j] = __uint_as_float(v[j]) * a;
  }
}

template <int BN>
struct SmemLayout {
  static constexpr int kStages = (BN == 256) ? 4 : 6;
  static constexpr int kABytes = BM * BKB;
  static constexpr int kBBytes = BN * BKB;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kBarBytes = 256;
  static constexpr int kTotal = kStages * kStageBytes + kBarBytes + 1024;  // + alignment slack
};

// acc -> (acc * row factor) * column factor for the 32 columns starting at col0 (columns come in multiples of 4)
__device__ __forceinline__ void apply_row_col_scale(uint32_t (&v)[32], float rs, const float* __restrict__ cs, int ncols) {
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    if (4 * q < ncols) {
      const float4 c = *reinterpret_cast<const float4*>(cs + 4 * q);
      v[4 * q + 0] = __float_as_uint(__fmul_rn(__fmul_rn(__uint_as_float(v[4 * q + 0]), rs), c.x));
      v[4 * q + 1] = __float_as_uint(__fmul_rn(__fmul_rn(__uint_as_float(v[4 * q + 1]), rs), c.y));
      v[4 * q + 2] = __float_as_uint(__fmul_rn(__fmul_rn(__uint_as_float(v[4 * q + 2]), rs), c.z));
      v[4 * q + 3] = __float_as_uint(__fmul_rn(__fmul_rn(__uint_as_float(v[4 * q + 3]), rs), c.w));
    }
  }
}

struct TileParams {
  int rows_a, rows_b;       // extents of one batch entry
  int kbytes;               // inner extent in bytes
  int elem_bytes;           // 2 (bf16) or 1 (e4m3)
  int batches;
  int groups;               // row groups per batch entry: product (r, g) pairs rows [g*rows_a, +rows_a) with [g*rows_b, +rows_b)
  int tiles_m, tiles_n;
  long long ldo, o_batch;   // output strides in elements
  int out_mode;             // 0: fp32 products; 1: scaled + rounded result
  int out_bf16;             // out_mode 1: 1 -> bf16, 0 -> fp32
  int wide;                 // every output row starts on a 32-byte boundary
  const float* row_scale;   // optional factors of the accumulator: per output row and per output column
  const float* col_scale;
  long long rs_batch, cs_batch;
  int selftest_no_producer; // failure-reporting self-test: the TMA producer issues nothing
  unsigned long long wait_limit_ns;   // bound of every mbarrier wait
};

template <int BN, bool kFp8>
__global__ void __launch_bounds__(kNumThreads, 1)
block_products_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                      void* __restrict__ out, const float* __restrict__ sA, const float* __restrict__ sB,
                      TileParams tp, DeviceStatus* status) {
  grid_launch_dependents();   // the decode may set up while this grid drains; it waits before reading the products
  using L = SmemLayout<BN>;
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment of the swizzled tiles
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - raw_addr);
  unsigned char* bar_mem = smem + L::kStages * L::kStageBytes;
  // barrier block: full[kStages], empty[kStages], tmem_full[2], tmem_empty[2], drain, tmem base, abort flag
  const uint32_t bar_base = smem_u32(bar_mem);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (L::kStages + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * L::kStages + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * L::kStages + 2 + b); };
  const uint32_t drain_bar = bar_base + 8u * (2 * L::kStages + 4);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_mem + 8 * (2 * L::kStages + 5));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_mem + 8 * (2 * L::kStages + 5) + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr uint32_t kTmemCols = 2 * BN;  // two accumulator buffers (256 or 512 columns)

  if (threadIdx.x == 0) {
    for (int s = 0; s < L::kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 4); }
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {  // TMEM allocation (whole warp), address lands in shared memory
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  grid_dependency_wait();     // operands and scales come from the previous kernel of the stream

  const int num_kb = (tp.kbytes + BKB - 1) / BKB;
  const int tiles_per_batch = tp.tiles_m * tp.tiles_n;
  const int total_tiles = tiles_per_batch * tp.batches * tp.groups;
  const int kelems_per_stage = BKB / tp.elem_bytes;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0 && !tp.selftest_no_producer) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int bb = tile / tiles_per_batch;
        const int rem = tile - bb * tiles_per_batch;
        const int r = bb / tp.groups, g = bb - r * tp.groups;
        const int tm = rem / tp.tiles_n, tn = rem - tm * tp.tiles_n;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, 0x01, status, tp.wait_limit_ns);
          if (!ok) break;
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          const uint32_t sb = sa + L::kABytes;
          mbar_arrive_expect_tx(full_bar(stage), (uint32_t)L::kStageBytes);
          tma_load_3d(sa, &map_a, full_bar(stage), kb * kelems_per_stage, g * tp.rows_a + tm * BM, r);
          tma_load_3d(sb, &map_b, full_bar(stage), kb * kelems_per_stage, g * tp.rows_b + tn * BN, r);
          if (++stage == L::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // let copies that were already issued land before the CTA's shared memory goes away:
        // the most recent fill of every stage completes phase (fills-1)&1 of its full barrier.
        for (int s = 0; s < L::kStages; ++s) {
          const uint32_t last_parity = (s < stage) ? phase : (phase ^ 1u);
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(full_bar(s), last_parity)) {
            if (global_timer_ns() - t0 > 20000000ull) break;  // 20 ms
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(kFp8, BN);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, 0x12, status, tp.wait_limit_ns);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = mbar_wait(full_bar(stage), phase, abort_flag, 0x11, status, tp.wait_limit_ns);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          const uint64_t da = make_smem_desc(sa);
          const uint64_t db = make_smem_desc(sa + L::kABytes);
#pragma unroll
          for (int k = 0; k < BKB / UMMA_KB; ++k) {
            // advance both descriptors by 32 bytes along K inside the swizzle span (address field is >>4)
            tc_mma<kFp8>(d_tmem, da + (uint64_t)(k * (UMMA_KB >> 4)), db + (uint64_t)(k * (UMMA_KB >> 4)), idesc,
                         (kb | k) != 0 ? 1u : 0u);
          }
          tc_commit(empty_bar(stage));  // stage reusable once these MMAs have read it
          if (++stage == L::kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(tfull_bar(acc));  // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) {  // wait (bounded) for MMAs in flight before TMEM is freed
        tc_commit(drain_bar);
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(drain_bar, 0)) {
          if (global_timer_ns() - t0 > 20000000ull) break;
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;  // TMEM lanes [32*quad, 32*quad+32) are the ones this warp may read
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    float alpha = 1.0f;
    if (tp.out_mode == 1 && sA != nullptr && sB != nullptr) alpha = sA[0] * sB[0];
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int r = tile / tiles_per_batch;     // index of the (batch, group) product
      const int rem = tile - r * tiles_per_batch;
      const int tm = rem / tp.tiles_n, tn = rem - tm * tp.tiles_n;
      ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, 0x23, status, tp.wait_limit_ns);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row = tm * BM + quad * 32 + lane;
      const bool row_ok = row < tp.rows_a;
      const long long row_off = (long long)r * tp.o_batch + (long long)row * tp.ldo;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t v[32];
        const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN + c * 32);
        tc_ld32(taddr, v);
        tc_wait_ld();
        const int col0 = tn * BN + c * 32;
        if (row_ok && col0 < tp.rows_b) {
          if (tp.row_scale != nullptr)
            apply_row_col_scale(v, tp.row_scale[(long long)r * tp.rs_batch + row],
                                tp.col_scale + (long long)r * tp.cs_batch + col0, min(32, tp.rows_b - col0));
          store_row_chunk(out, row_off + col0, min(32, tp.rows_b - col0), v, tp.out_mode, tp.out_bf16, alpha, tp.wide != 0);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------- CTA-pair kernel (cta_group::2)
// Two CTAs of a cluster (consecutive SMs) own one 256 x 256 output tile.  Each CTA loads its own 128 rows
// of Ahat_r and HALF of the Bhat_r tile (128 of the 256 rows), so the pair moves 2/3 of the bytes two
// independent 128 x 256 tiles would pull through L2.  The even CTA (leader) issues tcgen05.mma with
// M = 256 for both; the accumulator rows [128*rank, 128*rank + 128) live in each CTA's own TMEM.
//   - TMA loads of both CTAs complete on the LEADER's "full" barrier (cp.async.bulk.tensor ... .cta_group::2,
//     barrier address with the CTA-rank bit cleared); the leader alone arms it with the pair's byte count;
//   - tcgen05.commit.cta_group::2 with a two-CTA mask releases the ring stage in both CTAs and publishes the
//     accumulator to both epilogues;
//   - the epilogue warps of both CTAs hand the accumulator buffer back on the leader's barrier.
constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu;   // clears the CTA-rank bit of a shared::cluster address

__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t leader_bar, int c0,
                                                 int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(leader_bar)
      : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .b16 m;\n\tmov.b16 m, 3;\n\t"
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n\t}"
      ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}
template <bool kFp8>
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
  if (kFp8) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

struct PairLayout {
  static constexpr int BN = 256;                 // columns of the pair's tile
  static constexpr int kStages = 6;
  static constexpr int kABytes = BM * BKB;       // this CTA's 128 rows of A
  static constexpr int kBBytes = (BN / 2) * BKB; // this CTA's half of the B tile
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kBarBytes = 256;
  static constexpr int kTotal = kStages * kStageBytes + kBarBytes + 1024;
};

// The three roles of one CTA of a pair (producer warp 0, MMA warp 1, epilogue warps 2..5), given the CTA's ring,
// barrier block and TMEM base.  `warp` is the warp's index among those six.
struct PairCtx {
  unsigned char* smem;        // 1024-byte aligned ring
  uint32_t bar_base;          // shared-memory address of the barrier block behind it
  volatile int* abort_flag;
  uint32_t tmem_base;
  uint32_t rank;              // CTA rank in the pair (0 = leader)
};

template <bool kFp8>
__device__ __forceinline__ void pair_roles(const int warp, const int lane, const PairCtx& cx, const CUtensorMap& map_a,
                                           const CUtensorMap& map_b, void* __restrict__ out, const float* __restrict__ sA,
                                           const float* __restrict__ sB, const TileParams& tp, DeviceStatus* status) {
  using L = PairLayout;
  constexpr int BN = L::BN;
  unsigned char* smem = cx.smem;
  const uint32_t bar_base = cx.bar_base;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };                       // used in the leader only
  auto empty_bar = [&](int s) { return bar_base + 8u * (L::kStages + s); };       // one per CTA
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * L::kStages + b); };   // one per CTA
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * L::kStages + 2 + b); };  // used in the leader only
  const uint32_t drain_bar = bar_base + 8u * (2 * L::kStages + 4);
  volatile int* abort_flag = cx.abort_flag;
  const uint32_t tmem_base = cx.tmem_base;
  const uint32_t rank = cx.rank;
  const bool leader = rank == 0;
  const int num_kb = (tp.kbytes + BKB - 1) / BKB;
  const int tiles_m = (tp.rows_a + 2 * BM - 1) / (2 * BM);
  const int tiles_n = (tp.rows_b + BN - 1) / BN;
  const int tiles_per_batch = tiles_m * tiles_n;
  const int total_tiles = tiles_per_batch * tp.batches * tp.groups;
  const int kelems_per_stage = BKB / tp.elem_bytes;
  const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair_id; tile < total_tiles && ok; tile += num_pairs) {
        const int bb = tile / tiles_per_batch;
        const int rem = tile - bb * tiles_per_batch;
        const int r = bb / tp.groups, g = bb - r * tp.groups;
        const int tm = rem / tiles_n, tn = rem - tm * tiles_n;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, 0x01, status, tp.wait_limit_ns);
          if (!ok) break;
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          const uint32_t sb = sa + L::kABytes;
          const uint32_t lead_full = full_bar(stage) & kPeerBitMask;
          if (leader) mbar_arrive_expect_tx(full_bar(stage), 2u * (uint32_t)L::kStageBytes);
          tma_load_3d_pair(sa, &map_a, lead_full, kb * kelems_per_stage, g * tp.rows_a + tm * 2 * BM + (int)rank * BM, r);
          tma_load_3d_pair(sb, &map_b, lead_full, kb * kelems_per_stage, g * tp.rows_b + tn * BN + (int)rank * (BN / 2), r);
          if (++stage == L::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok && leader) {
        // Let copies that were already issued land before shared memory goes away.  The copies of BOTH CTAs complete
        // on the leader's full barriers, so the leader waits (bounded) for the most recent fill of every stage; its
        // partner cannot leave before the leader does (the cluster barrier at the end of the kernel), so the partner's
        // shared memory outlives its own copies too.  A fill the partner never issued leaves its barrier incomplete:
        // that wait runs into its bound.
        for (int s = 0; s < L::kStages; ++s) {
          const uint32_t last_parity = (s < stage) ? phase : (phase ^ 1u);
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(full_bar(s), last_parity)) {
            if (global_timer_ns() - t0 > 20000000ull) break;  // 20 ms
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    // all 32 lanes run the loop with warp-uniform control flow; one elected lane issues the MMAs and the commits
    if (leader) {
      // M = 256 across the pair, N = 256
      constexpr uint32_t idesc = (1u << 4) | ((kFp8 ? 0u : 1u) << 7) | ((kFp8 ? 0u : 1u) << 10) |
                                 ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = pair_id; tile < total_tiles && ok; tile += num_pairs) {
        ok = __all_sync(0xffffffffu, mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, 0x12, status, tp.wait_limit_ns));
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = __all_sync(0xffffffffu, mbar_wait(full_bar(stage), phase, abort_flag, 0x11, status, tp.wait_limit_ns));
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          const uint64_t da = make_smem_desc(sa);
          const uint64_t db = make_smem_desc(sa + L::kABytes);
          if (elect_one()) {
#pragma unroll
            for (int k = 0; k < BKB / UMMA_KB; ++k)
              tc_mma_pair<kFp8>(d_tmem, da + (uint64_t)(k * (UMMA_KB >> 4)), db + (uint64_t)(k * (UMMA_KB >> 4)), idesc,
                                (kb | k) != 0 ? 1u : 0u);
            tc_commit_pair(empty_bar(stage));   // frees this stage in both CTAs
          }
          __syncwarp();
          if (++stage == L::kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (elect_one()) tc_commit_pair(tfull_bar(acc));       // accumulator complete, visible to both epilogues
        __syncwarp();
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok && lane == 0) {
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(drain_bar)
                     : "memory");
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(drain_bar, 0)) {
          if (global_timer_ns() - t0 > 20000000ull) break;
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5 of both CTAs)
    const int quad = warp & 3;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    float alpha = 1.0f;
    if (tp.out_mode == 1 && sA != nullptr && sB != nullptr) alpha = sA[0] * sB[0];
    for (int tile = pair_id; tile < total_tiles && ok; tile += num_pairs) {
      const int r = tile / tiles_per_batch;
      const int rem = tile - r * tiles_per_batch;
      const int tm = rem / tiles_n, tn = rem - tm * tiles_n;
      ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, 0x23, status, tp.wait_limit_ns);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row = tm * 2 * BM + (int)rank * BM + quad * 32 + lane;
      const bool row_ok = row < tp.rows_a;
      const long long row_off = (long long)r * tp.o_batch + (long long)row * tp.ldo;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t v[32];
        const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN + c * 32);
        tc_ld32(taddr, v);
        tc_wait_ld();
        const int col0 = tn * BN + c * 32;
        if (row_ok && col0 < tp.rows_b) {
          if (tp.row_scale != nullptr)
            apply_row_col_scale(v, tp.row_scale[(long long)r * tp.rs_batch + row],
                                tp.col_scale + (long long)r * tp.cs_batch + col0, min(32, tp.rows_b - col0));
          store_row_chunk(out, row_off + col0, min(32, tp.rows_b - col0), v, tp.out_mode, tp.out_bf16, alpha, tp.wide != 0);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(tempty_bar(acc) & kPeerBitMask);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

}

// Set-up shared by every kernel that runs the pair roles: barrier block, TMEM allocation (warp 1 of the CTA), and the
// CTA- and cluster-wide barriers that make them visible.  Every thread of the CTA calls it, and pair_teardown at the end.
__device__ __forceinline__ PairCtx pair_setup(unsigned char* smem_raw, const int warp) {
  using L = PairLayout;
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - raw_addr);
  unsigned char* bar_mem = smem + L::kStages * L::kStageBytes;
  const uint32_t bar_base = smem_u32(bar_mem);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_mem + 8 * (2 * L::kStages + 5));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_mem + 8 * (2 * L::kStages + 5) + 8);
  constexpr uint32_t kTmemCols = 2 * L::BN;     // two accumulator buffers of 256 columns
  if (threadIdx.x == 0) {
    for (int st = 0; st < L::kStages; ++st) {
      mbar_init(bar_base + 8u * st, 1);                       // full (used in the leader only)
      mbar_init(bar_base + 8u * (L::kStages + st), 1);        // empty
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_base + 8u * (2 * L::kStages + b), 1);     // accumulator full
      mbar_init(bar_base + 8u * (2 * L::kStages + 2 + b), 8); // accumulator empty: four epilogue warps of each CTA
    }
    mbar_init(bar_base + 8u * (2 * L::kStages + 4), 1);       // drain
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // both CTAs' barriers are initialised before anything signals across the pair
  tc_fence_after();
  return PairCtx{smem, bar_base, abort_flag, *tmem_slot, cluster_ctarank()};
}

__device__ __forceinline__ void pair_teardown(const PairCtx& cx, const int warp) {
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // neither CTA frees TMEM / leaves while its partner may still touch it
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(cx.tmem_base), "r"(2 * PairLayout::BN) : "memory");
  }
}

template <bool kFp8>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kNumThreads, 1)
block_products_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                           void* __restrict__ out, const float* __restrict__ sA, const float* __restrict__ sB,
                           TileParams tp, DeviceStatus* status) {
  grid_launch_dependents();   // the decode may set up while this grid drains; it waits before reading the products
  extern __shared__ unsigned char smem_raw[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const PairCtx cx = pair_setup(smem_raw, warp);
  grid_dependency_wait();     // operands and scales come from the previous kernel of the stream
  pair_roles<kFp8>(warp, lane, cx, map_a, map_b, out, sA, sB, tp, status);
  pair_teardown(cx, warp);
}

// ---------------------------------------------------------------- fused sweep kernel
// One launch of a gauge sweep's pipeline: the block products of batch c on the tensor cores (the pair roles above,
// warps 0..5) and, beside them in the same CTAs, groups of eight warps that run the streaming passes of the neighbouring
// batches — first the error-only decode of batch c-1 (its products were written by the previous launch), then the
// encode of batch c+1 (its block sums are read by the next launch).  The three passes touch disjoint buffers, so no
// CTA waits for another inside the launch; all dependencies are launch-to-launch in stream order.  Why: each pass alone
// leaves most of the machine idle (the products use the tensor pipe and a sixth of the warp slots, the streaming passes
// are bound by issue slots and memory latency at 0.65-0.72 of the HBM peak), and as separate kernels they cannot share
// an SM, because a product CTA holds nearly all of its shared memory.
// A streaming group is a virtual block of the pass: group g of CTA b is block b * kGroups + g of gridDim.x * kGroups.
struct FusedStreamArgs {
  // error-only batch decode of the previous batch (dec_gauges = 0: none).  Arguments as decode_batch_kernel's.
  int dec_gauges;               // 4 or 8 algorithms in the batch
  const float* prod; const CoefTable* tab_w; int RB; int n; long long bm, bn;
  const float* cstar32; long long ldcs; double* partials; int dec_tiles_per_block; long long prod_stride;
  // encode of the next batch (enc_dense < 0: none)
  int enc_dense;                // 1: register-chain variant (every product reads the four cells in one order)
  EncodeJob ja, jb;
};

template <int kGroups> struct FusedLayout {
  static constexpr int kThreads = kNumThreads + 256 * kGroups;
  static constexpr int kGroupBytes = 14 * 1024;   // one streaming group: the larger of its decode and encode needs
  static constexpr int kTotal = PairLayout::kTotal + kGroups * kGroupBytes;
};

template <typename OutT, int kGroups>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(FusedLayout<kGroups>::kThreads, 1)
fused_sweep_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                   void* __restrict__ out, TileParams tp, DeviceStatus* status, const FusedStreamArgs fa) {
  grid_launch_dependents();
  extern __shared__ unsigned char smem_raw[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const PairCtx cx = pair_setup(smem_raw, warp);
  grid_dependency_wait();     // everything this launch reads was written by earlier work of the stream
  if (warp < kNumThreads / 32) {
    if (tp.batches > 0) pair_roles<false>(warp, lane, cx, map_a, map_b, out, nullptr, nullptr, tp, status);
  } else {
    const int grp = (warp - kNumThreads / 32) >> 3;
    unsigned char* gsm = smem_raw + PairLayout::kTotal + grp * FusedLayout<kGroups>::kGroupBytes;
    const StreamRole role{(int)threadIdx.x - kNumThreads - grp * 256, (int)blockIdx.x * kGroups + grp, (int)gridDim.x * kGroups,
                          1 + grp};
    if (fa.dec_gauges == 8)
      decode_batch_body<OutT, float, 8>(role, *reinterpret_cast<DecBatchSmem<8>*>(gsm), fa.prod, fa.tab_w, fa.RB, nullptr, nullptr,
                                        fa.n, fa.bm, fa.bn, fa.cstar32, fa.ldcs, fa.partials, fa.dec_tiles_per_block, fa.prod_stride);
    else if (fa.dec_gauges == 4)
      decode_batch_body<OutT, float, 4>(role, *reinterpret_cast<DecBatchSmem<4>*>(gsm), fa.prod, fa.tab_w, fa.RB, nullptr, nullptr,
                                        fa.n, fa.bm, fa.bn, fa.cstar32, fa.ldcs, fa.partials, fa.dec_tiles_per_block, fa.prod_stride);
    if (fa.enc_dense >= 0 && role.bid < fa.ja.blocks + fa.jb.blocks) {
      role.sync();            // the group is done with the decode's shared memory
      if (fa.enc_dense)
        encode_body<__nv_bfloat16, __nv_bfloat16, false, 4, false, true>(role, gsm, fa.ja, fa.jb, 0);
      else
        encode_body<__nv_bfloat16, __nv_bfloat16, false, 4, false, false>(role, gsm, fa.ja, fa.jb, 0);
    }
  }
  pair_teardown(cx, warp);
}

// ---------------------------------------------------------------- host side
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// K-major operand [batches][rows][kdim] -> 3-D map, box {128 bytes of K, box_rows, 1}, 128-byte swizzle.
bool make_operand_map(CUtensorMap* map, bool fp8, const void* ptr, int64_t rows, int64_t kdim, int64_t ld,
                      int64_t batch_stride, int batches, int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  const int es = fp8 ? 1 : 2;
  cuuint64_t dims[3] = {(cuuint64_t)kdim, (cuuint64_t)rows, (cuuint64_t)batches};
  cuuint64_t strides[2] = {(cuuint64_t)(ld * es), (cuuint64_t)((batches > 1 ? batch_stride : rows * ld) * es)};
  cuuint32_t box[3] = {(cuuint32_t)(BKB / es), (cuuint32_t)box_rows, 1u};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  CUresult rc = fn(map, fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
                   const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS;
}

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n = 0;
  }
  return n;
}

// 1 when every output row (and batch) starts on a 32-byte boundary
int rows_32b_aligned(const BlockProductArgs& a) {
  const int es = (a.out_mode == 1 && a.output == FMM_BF16) ? 2 : 4;
  return (reinterpret_cast<uintptr_t>(a.out) % 32 == 0) && ((a.ldo * es) % 32 == 0) && ((a.o_batch * es) % 32 == 0);
}

template <int BN, bool kFp8>
fmm_status launch_t(const BlockProductArgs& a, cudaStream_t st) {
  using L = SmemLayout<BN>;
  CUtensorMap ma, mb;
  const int groups = a.groups > 1 ? a.groups : 1;
  if (!make_operand_map(&ma, kFp8, a.A, a.rows_a * groups, a.kdim, a.lda, a.a_batch, a.batches, BM)) return FMM_ERR_CUDA;
  if (!make_operand_map(&mb, kFp8, a.B, a.rows_b * groups, a.kdim, a.ldb, a.b_batch, a.batches, BN)) return FMM_ERR_CUDA;
  TileParams tp;
  tp.rows_a = (int)a.rows_a; tp.rows_b = (int)a.rows_b;
  tp.elem_bytes = kFp8 ? 1 : 2;
  tp.kbytes = (int)a.kdim * tp.elem_bytes;
  tp.batches = a.batches;
  tp.groups = groups;
  tp.tiles_m = (int)((a.rows_a + BM - 1) / BM);
  tp.tiles_n = (int)((a.rows_b + BN - 1) / BN);
  tp.ldo = a.ldo; tp.o_batch = a.o_batch;
  tp.out_mode = a.out_mode; tp.out_bf16 = (a.output == FMM_BF16);
  tp.wide = rows_32b_aligned(a);
  tp.row_scale = a.row_scale; tp.col_scale = a.col_scale; tp.rs_batch = a.rs_batch; tp.cs_batch = a.cs_batch;
  tp.selftest_no_producer = a.selftest_no_producer;
  tp.wait_limit_ns = a.wait_limit_ns ? a.wait_limit_ns : kDefaultWaitLimitNs;
  const long long total = (long long)tp.tiles_m * tp.tiles_n * tp.batches * tp.groups;
  if (total <= 0) return FMM_OK;
  const int sms = sm_count();
  if (sms <= 0) return FMM_ERR_CUDA;
  const int grid = (int)(total < sms ? total : sms);
  auto k = block_products_kernel<BN, kFp8>;
  static unsigned long long smem_ok = 0;   // per template instantiation, one bit per device
  if (fmm_allow_dynamic_smem(k, L::kTotal, &smem_ok) != cudaSuccess) return FMM_ERR_CUDA;
  if (launch_dependent(k, dim3(grid), dim3(kNumThreads), (size_t)L::kTotal, st, ma, mb, a.out, a.sA, a.sB, tp, a.status) != cudaSuccess)
    return FMM_ERR_CUDA;
  ++fmm_launch_counter();
  return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

template <bool kFp8>
fmm_status launch_pair(const BlockProductArgs& a, cudaStream_t st) {
  using L = PairLayout;
  CUtensorMap ma, mb;
  const int groups = a.groups > 1 ? a.groups : 1;
  if (!make_operand_map(&ma, kFp8, a.A, a.rows_a * groups, a.kdim, a.lda, a.a_batch, a.batches, BM)) return FMM_ERR_CUDA;
  if (!make_operand_map(&mb, kFp8, a.B, a.rows_b * groups, a.kdim, a.ldb, a.b_batch, a.batches, L::BN / 2)) return FMM_ERR_CUDA;
  TileParams tp;
  tp.rows_a = (int)a.rows_a; tp.rows_b = (int)a.rows_b;
  tp.elem_bytes = kFp8 ? 1 : 2;
  tp.kbytes = (int)a.kdim * tp.elem_bytes;
  tp.batches = a.batches;
  tp.groups = groups;
  tp.tiles_m = (int)((a.rows_a + 2 * BM - 1) / (2 * BM));
  tp.tiles_n = (int)((a.rows_b + L::BN - 1) / L::BN);
  tp.ldo = a.ldo; tp.o_batch = a.o_batch;
  tp.out_mode = a.out_mode; tp.out_bf16 = (a.output == FMM_BF16);
  tp.wide = rows_32b_aligned(a);
  tp.row_scale = a.row_scale; tp.col_scale = a.col_scale; tp.rs_batch = a.rs_batch; tp.cs_batch = a.cs_batch;
  tp.selftest_no_producer = a.selftest_no_producer;
  tp.wait_limit_ns = a.wait_limit_ns ? a.wait_limit_ns : kDefaultWaitLimitNs;
  const long long total = (long long)tp.tiles_m * tp.tiles_n * tp.batches * tp.groups;
  if (total <= 0) return FMM_OK;
  const int sms = sm_count();
  if (sms < 2) return FMM_ERR_CUDA;
  const long long pairs = std::min<long long>(total, sms / 2);
  auto k = block_products_pair_kernel<kFp8>;
  static unsigned long long smem_ok = 0;
  if (fmm_allow_dynamic_smem(k, L::kTotal, &smem_ok) != cudaSuccess) return FMM_ERR_CUDA;
  if (launch_dependent(k, dim3((unsigned)(2 * pairs)), dim3(kNumThreads), (size_t)L::kTotal, st, ma, mb, a.out, a.sA, a.sB, tp, a.status) != cudaSuccess)
    return FMM_ERR_CUDA;
  ++fmm_launch_counter();
  return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

template <typename OutT, int kGroups>
fmm_status launch_fused_t(const FusedSweepArgs& f, cudaStream_t st) {
  using F = FusedLayout<kGroups>;
  const BlockProductArgs& a = f.products;
  CUtensorMap ma, mb;
  TileParams tp{};
  const int sms = sm_count();
  if (sms < 2) return FMM_ERR_CUDA;
  long long pairs = sms / 2;
  if (f.have_products) {
    if (!make_operand_map(&ma, false, a.A, a.rows_a, a.kdim, a.lda, a.a_batch, a.batches, BM)) return FMM_ERR_CUDA;
    if (!make_operand_map(&mb, false, a.B, a.rows_b, a.kdim, a.ldb, a.b_batch, a.batches, PairLayout::BN / 2)) return FMM_ERR_CUDA;
    tp.rows_a = (int)a.rows_a; tp.rows_b = (int)a.rows_b;
    tp.elem_bytes = 2;
    tp.kbytes = (int)a.kdim * 2;
    tp.batches = a.batches;
    tp.groups = 1;
    tp.tiles_m = (int)((a.rows_a + 2 * BM - 1) / (2 * BM));
    tp.tiles_n = (int)((a.rows_b + PairLayout::BN - 1) / PairLayout::BN);
    tp.ldo = a.ldo; tp.o_batch = a.o_batch;
    tp.out_mode = 0; tp.out_bf16 = 0;
    tp.wide = rows_32b_aligned(a);
    tp.wait_limit_ns = kDefaultWaitLimitNs;
  } else {
    std::memset(&ma, 0, sizeof(ma)); std::memset(&mb, 0, sizeof(mb));
    tp.batches = 0;             // the tensor-core roles do nothing in this launch
    tp.wait_limit_ns = kDefaultWaitLimitNs;
  }
  FusedStreamArgs fa{};
  fa.dec_gauges = f.dec_gauges;
  fa.prod = f.dec_prod; fa.tab_w = f.dec_tab; fa.RB = f.dec_RB; fa.n = f.n; fa.bm = f.bm; fa.bn = f.bn;
  fa.cstar32 = f.cstar32; fa.ldcs = (long long)f.n * f.bn; fa.partials = f.partials; fa.prod_stride = f.dec_prod_stride;
  const int nblocks = (int)(2 * pairs) * kGroups;
  if (f.dec_gauges) {
    const long long pos = 256 / f.dec_gauges;
    const long long tiles = (f.bm * (f.bn >> 2) + pos - 1) / pos;
    fa.dec_tiles_per_block = (int)((tiles + nblocks - 1) / nblocks);
  }
  fa.enc_dense = -1;
  if (f.have_encode) {
    size_t smem = 0; int dense = 0;
    if (!fmm_encode_jobs_for_blocks(f.enc_a, f.enc_b, nblocks, &fa.ja, &fa.jb, &smem, &dense)) return FMM_ERR_SHAPE;
    if (smem > (size_t)F::kGroupBytes) return FMM_ERR_SHAPE;
    fa.enc_dense = dense;
  }
  static_assert(sizeof(DecBatchSmem<4>) <= F::kGroupBytes && sizeof(DecBatchSmem<8>) <= F::kGroupBytes, "group shared memory");
  auto k = fused_sweep_kernel<OutT, kGroups>;
  static unsigned long long smem_ok = 0;
  if (fmm_allow_dynamic_smem(k, F::kTotal, &smem_ok) != cudaSuccess) return FMM_ERR_CUDA;
  if (launch_dependent(k, dim3((unsigned)(2 * pairs)), dim3(F::kThreads), (size_t)F::kTotal, st, ma, mb, a.out, tp, a.status, fa) != cudaSuccess)
    return FMM_ERR_CUDA;
  ++fmm_launch_counter();
  return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}


// ---------------------------------------------------------------- group-scaled int8 GEMM
// The classical int8 operator of the quantisation specification (Appendix D) as one kernel:
//     C[t][j] = rnd_O( sum over groups g, ascending, of (float(P_g[t][j]) * dA[t][g]) * dB[j][g] ),
//     P_g = exact integer product of the int8 codes of group g (128 inner indices).
// One CTA owns a 128 x 128 output tile.  Warp 0 streams, per group, the 128 x 128-byte code tiles of A and B (one
// 128-byte swizzle span = one group) through a shared-memory ring; one lane of warp 1 issues four tcgen05.mma
// kind::i8 (K = 32 each) per group into one of two int32 accumulator buffers in TMEM, a FRESH accumulator per group;
// warps 2-5 read the finished group's accumulator, convert it exactly to fp32, apply the two scales with two separate
// roundings, and add to 128 fp32 accumulators per thread (one output row each); after the last group one rounding to
// the output dtype.  The MMA of group g+1 overlaps the rescale of group g.
struct Int8Layout {
  static constexpr int BN = 128;
  static constexpr int kStages = 4;
  static constexpr int kABytes = BM * BKB;
  static constexpr int kBBytes = BN * BKB;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kBarBytes = 256;
  static constexpr int kMaxGroupsStaged = 64;                 // column scales of a tile staged in shared memory up to this many groups
  static constexpr int kScaleBytes = kMaxGroupsStaged * BN * 4;
  static constexpr int kTotal = kStages * kStageBytes + kBarBytes + kScaleBytes + 1024;
};

struct Int8Params {
  int M, N, G;                  // rows of A, rows of B (= output columns), groups of 128 along K
  int tiles_m, tiles_n;
  long long ldc;
  int out_bf16;
  int wide;                     // every output row starts on a 32-byte boundary
  const float* dAt;             // [G][M] row scales, group-major
  const float* dBt;             // [G][N] column scales, group-major
  unsigned long long wait_limit_ns;
};

__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// Packed fp32 pairs (__fmul2_rn, __fadd2_rn): each lane one IEEE operation.  Measured on this toolchain: a packed
// multiply followed by a packed add IS merged into a packed fused multiply-add, even when both are written with an
// explicit rounding mode, so the accumulation that must round twice (product, then sum) uses scalar __fadd_rn; the
// packed forms are used only where merging is impossible (multiply after multiply) or harmless (an exact subtraction).
constexpr int kInt8Threads = 576;   // 18 warps: TMA, MMA, and 16 rescale warps (four per TMEM lane quarter, 32 columns each)

__global__ void __launch_bounds__(kInt8Threads, 1)
int8_group_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                       void* __restrict__ out, Int8Params p, DeviceStatus* status) {
  using L = Int8Layout;
  constexpr int BN = L::BN;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - raw_addr);
  unsigned char* bar_mem = smem + L::kStages * L::kStageBytes;
  const uint32_t bar_base = smem_u32(bar_mem);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (L::kStages + s); };
  constexpr int kAcc = 4;   // accumulator buffers: all 512 TMEM columns, so the MMAs run up to three groups ahead of the rescale
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * L::kStages + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * L::kStages + kAcc + b); };
  const uint32_t drain_bar = bar_base + 8u * (2 * L::kStages + 2 * kAcc);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_mem + 8 * (2 * L::kStages + 2 * kAcc + 1));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_mem + 8 * (2 * L::kStages + 2 * kAcc + 1) + 8);
  float* scale_sm = reinterpret_cast<float*>(bar_mem + L::kBarBytes);   // [group][BN] column scales of the current tile
  const uint32_t sfull_bar = bar_base + 8u * (2 * L::kStages + 2 * kAcc + 3);   // the tile's scales are staged (16 warps arrive)
  const uint32_t sempty_bar = bar_base + 8u * (2 * L::kStages + 2 * kAcc + 4);  // the tile's scales are no longer read

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr uint32_t kTmemCols = kAcc * BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < L::kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < kAcc; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 16); }
    mbar_init(drain_bar, 1);
    mbar_init(sfull_bar, 16); mbar_init(sempty_bar, 16);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int total_tiles = p.tiles_m * p.tiles_n;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int tm = tile / p.tiles_n, tn = tile - tm * p.tiles_n;
        for (int g = 0; g < p.G; ++g) {
          ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, 0x41, status, p.wait_limit_ns);
          if (!ok) break;
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          mbar_arrive_expect_tx(full_bar(stage), (uint32_t)L::kStageBytes);
          tma_load_3d(sa, &map_a, full_bar(stage), g * BKB, tm * BM, 0);
          tma_load_3d(sa + L::kABytes, &map_b, full_bar(stage), g * BKB, tn * BN, 0);
          if (++stage == L::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        for (int s = 0; s < L::kStages; ++s) {
          const uint32_t last_parity = (s < stage) ? phase : (phase ^ 1u);
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(full_bar(s), last_parity)) {
            if (global_timer_ns() - t0 > 20000000ull) break;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer: one fresh accumulator per group
    if (lane == 0) {
      // int32 accumulator (c format 2), signed 8-bit A and B (format 1), K-major, N >> 3, M >> 4
      constexpr uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        for (int g = 0; g < p.G; ++g) {
          ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, 0x52, status, p.wait_limit_ns);
          if (!ok) break;
          ok = mbar_wait(full_bar(stage), phase, abort_flag, 0x51, status, p.wait_limit_ns);
          if (!ok) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          const uint64_t da = make_smem_desc(sa);
          const uint64_t db = make_smem_desc(sa + L::kABytes);
#pragma unroll
          for (int k = 0; k < BKB / UMMA_KB; ++k)
            tc_mma_i8(d_tmem, da + (uint64_t)(k * (UMMA_KB >> 4)), db + (uint64_t)(k * (UMMA_KB >> 4)), idesc, k != 0 ? 1u : 0u);
          tc_commit(empty_bar(stage));
          tc_commit(tfull_bar(acc));
          if (++stage == L::kStages) { stage = 0; phase ^= 1u; }
          if (++acc == kAcc) { acc = 0; acc_phase ^= 1u; }
        }
      }
      if (!ok) {
        tc_commit(drain_bar);
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(drain_bar, 0)) {
          if (global_timer_ns() - t0 > 20000000ull) break;
        }
      }
    }
  } else {
    // ------------------------------------------------------------ rescale and accumulate (warps 2..17)
    const int quad = warp & 3;             // TMEM lanes [32*quad, 32*quad+32) are the ones this warp may read
    const int part = (warp - 2) >> 2;      // which 32 of the tile's 128 columns
    constexpr int PN = 32;
    int acc = 0;
    uint32_t acc_phase = 0;
    uint32_t scale_phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int tm = tile / p.tiles_n, tn = tile - tm * p.tiles_n;
      const int row = tm * BM + quad * 32 + lane;
      const bool row_ok = row < p.M;
      const int col_base = tn * BN + part * PN;
      float2 sum[PN / 2];
#pragma unroll
      for (int j = 0; j < PN / 2; ++j) sum[j] = make_float2(0.0f, 0.0f);
      // column scales of this tile: [group][128] into shared memory (zero beyond N), by the 512 rescale threads
      const bool staged = p.G <= L::kMaxGroupsStaged;
      if (staged) {
        // bounded waits on mbarriers, not a named barrier: a warp that gives up elsewhere must not strand the others
        ok = mbar_wait(sempty_bar, scale_phase ^ 1u, abort_flag, 0x64, status, p.wait_limit_ns);   // previous tile's readers are done
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const int et = threadIdx.x - 64;                  // 0 .. 511
        for (int i = et; i < p.G * (BN / 4); i += 512) {
          const int g = i / (BN / 4), c4 = (i - g * (BN / 4)) * 4;
          const int col = tn * BN + c4;
          const float4 val = col < p.N ? *reinterpret_cast<const float4*>(p.dBt + (long long)g * p.N + col) : make_float4(0.f, 0.f, 0.f, 0.f);
          *reinterpret_cast<float4*>(scale_sm + g * BN + c4) = val;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(sfull_bar);            // release: this warp's share is written
        ok = mbar_wait(sfull_bar, scale_phase, abort_flag, 0x65, status, p.wait_limit_ns);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      float da_next = row_ok ? p.dAt[row] : 0.0f;
      for (int g = 0; g < p.G; ++g) {
        // the row scale does not depend on the products: the next group's is fetched a step ahead
        const float da = da_next;
        if (g + 1 < p.G) da_next = row_ok ? p.dAt[(long long)(g + 1) * p.M + row] : 0.0f;
        const float* dbp = staged ? scale_sm + g * BN + part * PN : p.dBt + (long long)g * p.N + col_base;
        ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, 0x63, status, p.wait_limit_ns);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        uint32_t v[32];
        tc_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN + part * PN), v);
        tc_wait_ld();
        // the accumulator is in registers: hand the buffer back before the arithmetic
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(acc));
        if (++acc == kAcc) { acc = 0; acc_phase ^= 1u; }
        const float2 da2 = make_float2(da, da);
        const float2 neg_magic = make_float2(-12582912.0f, -12582912.0f);
#pragma unroll
        for (int q4 = 0; q4 < PN / 4; ++q4) {
          // exact int -> float for |P| < 2^22 (a group product is at most 128 * 127^2): add the integer to the bits
          // of 1.5 * 2^23, subtract that constant (exact).  Then two separately rounded multiplications and a
          // separately rounded addition, as the specification orders them.
          float2 p0 = make_float2(__uint_as_float(v[q4 * 4 + 0] + 0x4B400000u), __uint_as_float(v[q4 * 4 + 1] + 0x4B400000u));
          float2 p1 = make_float2(__uint_as_float(v[q4 * 4 + 2] + 0x4B400000u), __uint_as_float(v[q4 * 4 + 3] + 0x4B400000u));
          p0 = __fadd2_rn(p0, neg_magic); p1 = __fadd2_rn(p1, neg_magic);
          p0 = __fmul2_rn(p0, da2); p1 = __fmul2_rn(p1, da2);
          const float4 db = (staged || col_base + q4 * 4 < p.N) ? *reinterpret_cast<const float4*>(dbp + q4 * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
          p0 = __fmul2_rn(p0, make_float2(db.x, db.y)); p1 = __fmul2_rn(p1, make_float2(db.z, db.w));
          sum[q4 * 2].x = __fadd_rn(sum[q4 * 2].x, p0.x); sum[q4 * 2].y = __fadd_rn(sum[q4 * 2].y, p0.y);
          sum[q4 * 2 + 1].x = __fadd_rn(sum[q4 * 2 + 1].x, p1.x); sum[q4 * 2 + 1].y = __fadd_rn(sum[q4 * 2 + 1].y, p1.y);
        }
      }
      if (!ok) break;
      if (staged) {                                        // this warp no longer reads the tile's scales
        __syncwarp();
        if (lane == 0) mbar_arrive(sempty_bar);
        scale_phase ^= 1u;
      }
      if (row_ok && col_base < p.N) {
        uint32_t w[32];
#pragma unroll
        for (int j = 0; j < PN / 2; ++j) { w[2 * j] = __float_as_uint(sum[j].x); w[2 * j + 1] = __float_as_uint(sum[j].y); }
        store_row_chunk(out, (long long)row * p.ldc + col_base, min(32, p.N - col_base), w, 1, p.out_bf16, 1.0f, p.wide != 0);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------- group-scaled fp8 GEMM (model schedule)
// Batched block products under the model schedule of Appendix B.1: e4m3 codes of A with one scale per row and per
// 128 inner indices, e4m3 codes of B with one scale per 128 x 128 block.  As in the int8 kernel every 128-group gets a
// fresh fp32 accumulator in TMEM (four kind::f8f6f4 MMAs of K = 32); the epilogue multiplies the finished group by
// s_A[row][g] * s_B[column block][g] and adds it to its fp32 running sums (one fused multiply-add per element and group);
// after the last group one rounding to the output dtype (bf16 when the product kernel "returns each product in bf16").
// One CTA per 128 x 128 tile of one product, so a tile's columns lie in one 128-column scale block.
struct Fp8GroupParams {
  int rows_a, rows_b, G, batches;   // extents of one product, 128-groups along K, number of products
  int tiles_m, tiles_n;
  long long ldo, o_batch;           // output strides in elements
  int out_bf16, wide;
  const float* sA; long long sa_batch;   // [batch][rows_a][G]
  const float* sB; long long sb_batch;   // [batch][ceil(rows_b / 128)][G]
  unsigned long long wait_limit_ns;
};

__global__ void __launch_bounds__(kInt8Threads, 1)
fp8_group_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                      void* __restrict__ out, Fp8GroupParams p, DeviceStatus* status) {
  grid_launch_dependents();
  using L = Int8Layout;             // same tile, ring and barrier block (the scale staging area is unused here)
  constexpr int BN = L::BN;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - raw_addr);
  unsigned char* bar_mem = smem + L::kStages * L::kStageBytes;
  const uint32_t bar_base = smem_u32(bar_mem);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (L::kStages + s); };
  // four accumulator buffers (all 512 TMEM columns): the MMAs of the next three groups run while the rescale warps wait
  // for the tcgen05.ld of a finished one — that latency, not the arithmetic, sets the pace of this kernel
  constexpr int kAcc = 4;
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * L::kStages + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * L::kStages + kAcc + b); };
  const uint32_t drain_bar = bar_base + 8u * (2 * L::kStages + 2 * kAcc);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_mem + 8 * (2 * L::kStages + 2 * kAcc + 1));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_mem + 8 * (2 * L::kStages + 2 * kAcc + 1) + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr uint32_t kTmemCols = kAcc * BN;
  if (threadIdx.x == 0) {
    for (int s = 0; s < L::kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < kAcc; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 16); }
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  grid_dependency_wait();           // codes and scales come from the previous kernel of the stream

  const int tiles_per_batch = p.tiles_m * p.tiles_n;
  const int total_tiles = tiles_per_batch * p.batches;
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int r = tile / tiles_per_batch;
        const int rem = tile - r * tiles_per_batch;
        const int tm = rem / p.tiles_n, tn = rem - tm * p.tiles_n;
        for (int g = 0; g < p.G; ++g) {
          ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, 0x71, status, p.wait_limit_ns);
          if (!ok) break;
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          mbar_arrive_expect_tx(full_bar(stage), (uint32_t)L::kStageBytes);
          tma_load_3d(sa, &map_a, full_bar(stage), g * BKB, tm * BM, r);
          tma_load_3d(sa + L::kABytes, &map_b, full_bar(stage), g * BKB, tn * BN, r);
          if (++stage == L::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        for (int s = 0; s < L::kStages; ++s) {
          const uint32_t last_parity = (s < stage) ? phase : (phase ^ 1u);
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(full_bar(s), last_parity)) {
            if (global_timer_ns() - t0 > 20000000ull) break;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer: one fresh accumulator per group
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(true, BN);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        for (int g = 0; g < p.G; ++g) {
          ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, 0x82, status, p.wait_limit_ns);
          if (!ok) break;
          ok = mbar_wait(full_bar(stage), phase, abort_flag, 0x81, status, p.wait_limit_ns);
          if (!ok) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          const uint64_t da = make_smem_desc(sa);
          const uint64_t db = make_smem_desc(sa + L::kABytes);
#pragma unroll
          for (int k = 0; k < BKB / UMMA_KB; ++k)
            tc_mma<true>(d_tmem, da + (uint64_t)(k * (UMMA_KB >> 4)), db + (uint64_t)(k * (UMMA_KB >> 4)), idesc, k != 0 ? 1u : 0u);
          tc_commit(empty_bar(stage));
          tc_commit(tfull_bar(acc));
          if (++stage == L::kStages) { stage = 0; phase ^= 1u; }
          if (++acc == kAcc) { acc = 0; acc_phase ^= 1u; }
        }
      }
      if (!ok) {
        tc_commit(drain_bar);
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(drain_bar, 0)) {
          if (global_timer_ns() - t0 > 20000000ull) break;
        }
      }
    }
  } else {
    // ------------------------------------------------------------ scale and accumulate (warps 2..17)
    const int quad = warp & 3;
    const int part = (warp - 2) >> 2;
    constexpr int PN = 32;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int r = tile / tiles_per_batch;
      const int rem = tile - r * tiles_per_batch;
      const int tm = rem / p.tiles_n, tn = rem - tm * p.tiles_n;
      const int row = tm * BM + quad * 32 + lane;
      const bool row_ok = row < p.rows_a;
      const int col_base = tn * BN + part * PN;
      const float* sa_row = p.sA + (long long)r * p.sa_batch + (long long)(row_ok ? row : 0) * p.G;
      const float* sb_blk = p.sB + (long long)r * p.sb_batch + (long long)tn * p.G;   // BN = 128 = one scale block of columns
      float2 sum[PN / 2];
#pragma unroll
      for (int j = 0; j < PN / 2; ++j) sum[j] = make_float2(0.0f, 0.0f);
      // the scales do not depend on the products: they are fetched two groups ahead of their use
      float s_next = row_ok ? sa_row[0] * sb_blk[0] : 0.0f;
      float s_next2 = (row_ok && p.G > 1) ? sa_row[1] * sb_blk[1] : 0.0f;
      for (int g = 0; g < p.G; ++g) {
        const float sc = s_next;
        s_next = s_next2;
        if (g + 2 < p.G) s_next2 = row_ok ? sa_row[g + 2] * sb_blk[g + 2] : 0.0f;
        ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, 0x93, status, p.wait_limit_ns);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        uint32_t v[32];
        tc_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN + part * PN), v);
        tc_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(acc));
        if (++acc == kAcc) { acc = 0; acc_phase ^= 1u; }
        const float2 sc2 = make_float2(sc, sc);
#pragma unroll
        for (int j = 0; j < PN / 2; ++j)      // one fused multiply-add per element, two elements per instruction
          sum[j] = __ffma2_rn(make_float2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])), sc2, sum[j]);
      }
      if (!ok) break;
      if (row_ok && col_base < p.rows_b) {
        uint32_t w[32];
#pragma unroll
        for (int j = 0; j < PN / 2; ++j) { w[2 * j] = __float_as_uint(sum[j].x); w[2 * j + 1] = __float_as_uint(sum[j].y); }
        store_row_chunk(out, (long long)r * p.o_batch + (long long)row * p.ldo + col_base, min(32, p.rows_b - col_base), w, 1,
                        p.out_bf16, 1.0f, p.wide != 0);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

#include "int8_certified.inc"

}  // namespace

fmm_status launch_fp8_group_gemm(const Fp8GroupArgs& a, cudaStream_t st) {
  using L = Int8Layout;
  if (a.rows_a > 0x7fffffff || a.rows_b > 0x7fffffff || a.kdim <= 0 || a.kdim > 0x3fffffff) return FMM_ERR_SHAPE;
  CUtensorMap ma, mb;
  if (!make_operand_map(&ma, true, a.A, a.rows_a, a.kdim, a.lda, a.a_batch, a.batches, BM)) return FMM_ERR_CUDA;
  if (!make_operand_map(&mb, true, a.B, a.rows_b, a.kdim, a.ldb, a.b_batch, a.batches, L::BN)) return FMM_ERR_CUDA;
  Fp8GroupParams p;
  p.rows_a = (int)a.rows_a; p.rows_b = (int)a.rows_b; p.G = (int)((a.kdim + BKB - 1) / BKB); p.batches = a.batches;   // a ragged last group is zero-filled by the copies
  p.tiles_m = (int)((a.rows_a + BM - 1) / BM);
  p.tiles_n = (int)((a.rows_b + L::BN - 1) / L::BN);
  p.ldo = a.ldo; p.o_batch = a.o_batch; p.out_bf16 = a.output == FMM_BF16;
  const int es = p.out_bf16 ? 2 : 4;
  p.wide = (reinterpret_cast<uintptr_t>(a.out) % 32 == 0) && ((a.ldo * es) % 32 == 0) && ((a.o_batch * es) % 32 == 0);
  p.sA = a.sA; p.sa_batch = a.rows_a * p.G;
  p.sB = a.sB; p.sb_batch = (long long)p.tiles_n * p.G;
  p.wait_limit_ns = kDefaultWaitLimitNs;
  const long long total = (long long)p.tiles_m * p.tiles_n * p.batches;
  if (total <= 0) return FMM_OK;
  const int sms = sm_count();
  if (sms <= 0) return FMM_ERR_CUDA;
  const int grid = (int)(total < sms ? total : sms);
  static unsigned long long smem_ok = 0;
  if (fmm_allow_dynamic_smem(fp8_group_gemm_kernel, L::kTotal, &smem_ok) != cudaSuccess) return FMM_ERR_CUDA;
  if (launch_dependent(fp8_group_gemm_kernel, dim3(grid), dim3(kInt8Threads), (size_t)L::kTotal, st, ma, mb, a.out, p, a.status) != cudaSuccess)
    return FMM_ERR_CUDA;
  ++fmm_launch_counter();
  return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

fmm_status launch_int8_group_gemm(const int8_t* cA, const int8_t* cB, const float* dAt, const float* dBt, int64_t M,
                                  int64_t K, int64_t N, int output, void* C, int64_t ldc, DeviceStatus* status, cudaStream_t st) {
  using L = Int8Layout;
  if (M > 0x7fffffff || N > 0x7fffffff || K % BKB || K / BKB > 0x7fffffff) return FMM_ERR_SHAPE;
  CUtensorMap ma, mb;
  if (!make_operand_map(&ma, true, cA, M, K, K, 0, 1, BM)) return FMM_ERR_CUDA;
  if (!make_operand_map(&mb, true, cB, N, K, K, 0, 1, L::BN)) return FMM_ERR_CUDA;
  Int8Params p;
  p.M = (int)M; p.N = (int)N; p.G = (int)(K / BKB);
  p.tiles_m = (int)((M + BM - 1) / BM);
  p.tiles_n = (int)((N + L::BN - 1) / L::BN);
  p.ldc = ldc; p.out_bf16 = output == FMM_BF16;
  const int es = p.out_bf16 ? 2 : 4;
  p.wide = (reinterpret_cast<uintptr_t>(C) % 32 == 0) && ((ldc * es) % 32 == 0);
  p.dAt = dAt; p.dBt = dBt;
  p.wait_limit_ns = kDefaultWaitLimitNs;
  const long long total = (long long)p.tiles_m * p.tiles_n;
  if (total <= 0) return FMM_OK;
  const int sms = sm_count();
  if (sms <= 0) return FMM_ERR_CUDA;
  const int grid = (int)(total < sms ? total : sms);
  static unsigned long long smem_ok = 0;
  if (fmm_allow_dynamic_smem(int8_group_gemm_kernel, L::kTotal, &smem_ok) != cudaSuccess) return FMM_ERR_CUDA;
  int8_group_gemm_kernel<<<grid, kInt8Threads, L::kTotal, st>>>(ma, mb, C, p, status);
  ++fmm_launch_counter();
  return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

fmm_status launch_int8_certified(const Int8CertArgs& a, cudaStream_t st) {
  using L = CertLayout;
  if (a.h != 32 && a.h != 64 && a.h != 128) return FMM_ERR_SHAPE;
  if (a.m * a.n > L::kMaxBlocks || a.R > FMM_MAX_R || a.n_entries > L::kMaxEntries) return FMM_ERR_LIMIT;
  if (a.bm * a.G > 0x7fffffff || a.bn * a.G > 0x7fffffff || a.M > 0x7fffffff || a.N > 0x7fffffff) return FMM_ERR_SHAPE;
  const int per = BKB / a.h;
  const int row_stages = (a.R + per - 1) / per;
  CUtensorMap ma, mb;
  if (!make_operand_map(&ma, true, a.Ahat, a.bm * a.G, BKB, BKB, a.bm * a.G * BKB, row_stages, BM)) return FMM_ERR_CUDA;
  if (!make_operand_map(&mb, true, a.Bhat, a.bn * a.G, BKB, BKB, a.bn * a.G * BKB, row_stages, L::BN)) return FMM_ERR_CUDA;
  CertParams p{};
  p.M = (int)a.M; p.N = (int)a.N; p.m = a.m; p.n = a.n; p.bm = (int)a.bm; p.bn = (int)a.bn;
  p.G = a.G; p.R = a.R; p.h = a.h; p.per = per; p.ksteps = a.h / UMMA_KB;
  int8_certified_passes(a.R, per, &p.passes, &p.pass_len);
  p.tiles_m = (int)((a.bm + BM - 1) / BM);
  p.tiles_n = (int)((a.bn + L::BN - 1) / L::BN);
  p.ldc = a.ldc; p.out_bf16 = a.output == FMM_BF16;
  p.dAt = a.dAt; p.dBt = a.dBt;
  p.entries = a.d_entries; p.pass_off = a.d_pass_off; p.owned = a.d_owned; p.n_entries = a.n_entries;
  p.wait_limit_ns = kDefaultWaitLimitNs;
  const long long total = (long long)p.tiles_m * p.tiles_n;
  if (total <= 0) return FMM_OK;
  const int sms = sm_count();
  if (sms <= 0) return FMM_ERR_CUDA;
  const int grid = (int)(total < sms ? total : sms);
  static unsigned long long smem_ok = 0;
  if (fmm_allow_dynamic_smem(int8_certified_kernel, L::kTotal, &smem_ok) != cudaSuccess) return FMM_ERR_CUDA;
  int8_certified_kernel<<<grid, kCertThreads, L::kTotal, st>>>(ma, mb, a.C, p, a.status);
  ++fmm_launch_counter();
  return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

int int8_certified_tile_columns() { return CertLayout::BN; }
int int8_certified_decode_warps() { return CertLayout::kParts; }

// The R products of a group go through TMEM in ceil(R / kPass) passes of equal length (a multiple of the products per
// ring stage), the last one taking the remainder, when that fits a buffer; otherwise in passes of kPass.
void int8_certified_passes(int R, int per, int* passes, int* pass_len) {
  const int n = (R + CertLayout::kPass - 1) / CertLayout::kPass;
  int len = R / n / per * per;
  if (len == 0 || R - len * (n - 1) > CertLayout::kPass) len = CertLayout::kPass;
  *passes = n;
  *pass_len = len;
}

fmm_status launch_block_products(const BlockProductArgs& a, cudaStream_t st) {
  if (a.rows_a > 0x7fffffff || a.rows_b > 0x7fffffff || a.kdim > 0x3fffffff) return FMM_ERR_SHAPE;
  const bool fp8 = (a.product == FMM_E4M3);
  if (!fp8 && a.product != FMM_BF16) return FMM_ERR_DTYPE;
  // large problems: CTA pairs on 256 x 256 tiles (less L2 traffic per flop)
  if (a.rows_a > 128 && a.rows_b > 128 && !a.selftest_no_producer)
    return fp8 ? launch_pair<true>(a, st) : launch_pair<false>(a, st);
  // narrow problems use the 128-column tile (less padding, more tiles in flight)
  const bool narrow = a.rows_b <= 128;
  if (fp8) return narrow ? launch_t<128, true>(a, st) : launch_t<256, true>(a, st);
  return narrow ? launch_t<128, false>(a, st) : launch_t<256, false>(a, st);
}

int fused_sweep_blocks(int groups) { return (sm_count() / 2) * 2 * groups; }

fmm_status launch_fused_sweep(const FusedSweepArgs& f, cudaStream_t st) {
  if (f.output != FMM_F32 && f.output != FMM_BF16) return FMM_ERR_DTYPE;
  if (f.dec_gauges != 0 && f.dec_gauges != 4 && f.dec_gauges != 8) return FMM_ERR_ARG;
  if (f.groups == 1)
    return f.output == FMM_F32 ? launch_fused_t<float, 1>(f, st) : launch_fused_t<__nv_bfloat16, 1>(f, st);
  if (f.groups == 2)
    return f.output == FMM_F32 ? launch_fused_t<float, 2>(f, st) : launch_fused_t<__nv_bfloat16, 2>(f, st);
  return FMM_ERR_ARG;
}
