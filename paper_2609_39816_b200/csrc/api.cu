// C-ABI entry points that run on the device: scheme_gemm, classical_gemm, exact_gemm_f64,
// error_frobenius, error_sweep.  Host code only validates, lays out the workspace and enqueues
// kernels on the caller's stream.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "kernels_stream.cuh"

// ---------------------------------------------------------------- phase timing
namespace {
struct ProfRec { int kind; cudaEvent_t a, b; };
bool g_prof_on = false;
std::vector<ProfRec> g_prof;
}  // namespace

ProfScope::ProfScope(int kind, cudaStream_t s) : slot(-1), st(s) {
  if (!g_prof_on) return;
  ProfRec r{kind, nullptr, nullptr};
  if (cudaEventCreate(&r.a) != cudaSuccess) return;
  if (cudaEventCreate(&r.b) != cudaSuccess) { cudaEventDestroy(r.a); return; }
  cudaEventRecord(r.a, st);
  g_prof.push_back(r);
  slot = (int)g_prof.size() - 1;
}
ProfScope::~ProfScope() {
  if (slot >= 0) cudaEventRecord(g_prof[slot].b, st);
}

// ---------------------------------------------------------------- side stream for concurrent passes
// The streaming passes leave most of the machine idle (they are latency-bound), so independent ones run side
// by side: work is forked from the caller's stream onto one library-owned stream and joined back with events.
// Nothing here synchronises the host.  One side stream and a ring of events per device, created on first use
// (device calls of this library are therefore not safe to issue from several host threads at once).
namespace {
constexpr int kMaxDev = 64, kEventRing = 64;
struct SideStream {
  cudaStream_t stream = nullptr;    // general side stream (encode B beside encode A)
  cudaStream_t stream2 = nullptr;   // second side stream (decode stage of a pipelined sweep)
  cudaEvent_t ev[kEventRing] = {};
  int next = 0;
};
SideStream g_side[kMaxDev];

SideStream* side_stream() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return nullptr;
  SideStream& s = g_side[dev];
  if (s.stream == nullptr) {
    if (cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithFlags(&s.stream2, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    for (int i = 0; i < kEventRing; ++i)
      if (cudaEventCreateWithFlags(&s.ev[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
  }
  return &s;
}
// record a fresh event of the ring on `from` (an event handed out stays untouched for kEventRing - 1 more records)
cudaEvent_t record_event(SideStream* s, cudaStream_t from) {
  cudaEvent_t e = s->ev[s->next];
  s->next = (s->next + 1) % kEventRing;
  return cudaEventRecord(e, from) == cudaSuccess ? e : nullptr;
}
// `to` waits for everything enqueued on `from` so far
bool stream_wait(SideStream* s, cudaStream_t from, cudaStream_t to) {
  cudaEvent_t e = s->ev[s->next];
  s->next = (s->next + 1) % kEventRing;
  return cudaEventRecord(e, from) == cudaSuccess && cudaStreamWaitEvent(to, e, 0) == cudaSuccess;
}
}  // namespace

namespace {

inline size_t align_up(size_t x, size_t a = kPackedAlign) { return (x + a - 1) / a * a; }
inline int esize(int dt) { return dt == FMM_F32 ? 4 : dt == FMM_BF16 ? 2 : 1; }

constexpr int kMaxStreamPartials = 148 * 8;
constexpr int kSlabPadBytes = 256;

// Workspace of one scheme GEMM.  Everything is an offset from the workspace base.
struct GemmLayout {
  size_t status, tabA, tabB, tabW, amaxA, amaxB, sA, sB, partials, bt, ahat, bhat, prod, total;
  int64_t sAhat, sBhat, sProd;   // elements between consecutive products (block size + padding)
  int n_partials;
  // FMM_FLAG_ROUND_PER_LEVEL: the outer level's rounded block sums (R1 tensors per operand), its tables, amax words
  // and scales, and the inner level's tables
  size_t lvl_tab_outer, lvl_tab_inner, lvl_amax, lvl_scale, lvl_a, lvl_b;
  int64_t sLvlA, sLvlB;
};

// codes_ok: operands may already be e4m3 codes (classical_gemm on pre-quantised operands, read in place)
fmm_status check_desc(const fmm_gemm_desc* d, int m, int k, int n, bool codes_ok = false) {
  if (!d) return FMM_ERR_ARG;
  if (d->M <= 0 || d->K <= 0 || d->N <= 0) return FMM_ERR_SHAPE;
  const bool codes = codes_ok && d->storage == FMM_E4M3 && d->product == FMM_E4M3 && d->scale_mode == 0 && d->b_is_weight_layout;
  if (d->storage != FMM_F32 && d->storage != FMM_BF16 && !codes) return FMM_ERR_DTYPE;
  if (d->product != FMM_BF16 && d->product != FMM_E4M3) return FMM_ERR_DTYPE;
  if (d->output != FMM_F32 && d->output != FMM_BF16) return FMM_ERR_DTYPE;
  if (d->scale_mode != 0 && !(d->scale_mode >= 1 && d->scale_mode <= 3 && d->product == FMM_E4M3)) return FMM_ERR_DTYPE;
  if (d->M % m || d->K % k || d->N % n) return FMM_ERR_SHAPE;
  if ((d->K / k) % 16 || (d->N / n) % 8) return FMM_ERR_SHAPE;
  const int es = esize(d->storage), eo = esize(d->output);
  const int64_t min_ldb = d->b_is_weight_layout ? d->K : d->N;
  if (d->lda < d->K || d->ldb < min_ldb || d->ldc < d->N) return FMM_ERR_SHAPE;
  if ((d->lda * es) % 16 || (d->ldb * es) % 16 || (d->ldc * eo) % 16) return FMM_ERR_SHAPE;
  // the streaming kernels index the positions of one block in 32 bits (16-byte vectors of the source / of fp32
  // products), and the tensor maps take 32-bit extents: reject anything beyond, before any launch
  const int64_t bm = d->M / m, bk = d->K / k, bn = d->N / n;
  const int64_t limit = ((int64_t)1 << 31) - 4096;
  if (bm * (bk / (16 / es)) >= limit || bn * (bk / (16 / es)) >= limit || bm * (bn / 4) >= limit) return FMM_ERR_SHAPE;
  if (bm >= limit || bn >= limit || bk >= ((int64_t)1 << 30)) return FMM_ERR_SHAPE;
  return FMM_OK;
}

// Number of amax / scale words of one operand: rows x inner extent of one block sum, R of them.
size_t scale_words(int mode, int R, int64_t rows, int64_t inner, bool b_side) {
  if (mode == 2) return (size_t)R * rows;
  if (mode == 3) return (size_t)R * (b_side ? (rows + 127) / 128 : rows) * ((inner + 127) / 128);
  return FMM_MAX_R;
}

GemmLayout gemm_layout(int m, int k, int n, int R, const fmm_gemm_desc* d, const fmm_scheme* nested = nullptr) {
  GemmLayout L{};
  const int64_t bm = d->M / m, bk = d->K / k, bn = d->N / n;
  const int ep = esize(d->product), es = esize(d->storage);
  size_t o = 0;
  L.status = o; o += align_up(sizeof(DeviceStatus));
  L.tabA = o; o += align_up(sizeof(CoefTable));
  L.tabB = o; o += align_up(sizeof(CoefTable));
  L.tabW = o; o += align_up(sizeof(CoefTable));
  // scale_mode 2 keeps one amax / scale per row of every block sum: [R][bm] and [R][bn]
  const size_t nsa = scale_words(d->scale_mode, R, bm, bk, false), nsb = scale_words(d->scale_mode, R, bn, bk, true);
  L.amaxA = o; o += align_up(nsa * 4);
  L.amaxB = o; o += align_up(nsb * 4);
  L.sA = o; o += align_up(nsa * 4);
  L.sB = o; o += align_up(nsb * 4);
  L.n_partials = std::max(decode_grid(bm, bn), kMaxStreamPartials);
  L.partials = o; o += align_up((size_t)L.n_partials * 8 * 8);   // up to eight algorithms' error sums per decode launch
  L.bt = o; o += d->b_is_weight_layout ? 0 : align_up((size_t)d->N * d->K * es);
  // Consecutive products are spaced by the block size plus 256 bytes: block sizes are often powers of two, and
  // R streams written (or read) at the same offset of power-of-two-spaced slabs land on the same memory
  // channels (measured on B200: 37.6 us vs 28.3 us for the traffic of one encode pass).
  L.sAhat = bm * bk + kSlabPadBytes / ep;
  L.sBhat = bn * bk + kSlabPadBytes / ep;
  L.sProd = bm * bn + kSlabPadBytes / 4;
  L.ahat = o; o += align_up((size_t)R * L.sAhat * ep);
  L.bhat = o; o += align_up((size_t)R * L.sBhat * ep);
  L.prod = o; o += align_up((size_t)R * L.sProd * ((d->flags & FMM_FLAG_PRODUCTS_BF16) ? 2 : 4));
  if ((d->flags & FMM_FLAG_ROUND_PER_LEVEL) && nested && nested->outer && nested->inner) {
    const fmm_scheme& so = *nested->outer;
    L.lvl_tab_outer = o; o += 2 * align_up(sizeof(CoefTable));
    L.lvl_tab_inner = o; o += 2 * align_up(sizeof(CoefTable));
    L.lvl_amax = o; o += align_up(2 * FMM_MAX_R * 4);
    L.lvl_scale = o; o += align_up(2 * FMM_MAX_R * 4);
    L.sLvlA = (d->M / so.m) * (d->K / so.k) + kSlabPadBytes / ep;
    L.sLvlB = (d->N / so.n) * (d->K / so.k) + kSlabPadBytes / ep;
    L.lvl_a = o; o += align_up((size_t)so.R * L.sLvlA * ep);
    L.lvl_b = o; o += align_up((size_t)so.R * L.sLvlB * ep);
  }
  L.total = o;
  return L;
}

template <typename T>
T* at(void* ws, size_t off) { return reinterpret_cast<T*>(static_cast<char*>(ws) + off); }

#define FMM_CUDA(x) do { if ((x) != cudaSuccess) return FMM_ERR_CUDA; } while (0)
#define FMM_TRY(x) do { fmm_status _s = (x); if (_s != FMM_OK) return _s; } while (0)

// Encode one operand: optional amax pass, then block sums -> product dtype.
fmm_status encode_operand(const fmm_gemm_desc* d, const void* X, int64_t ldx, int gr, int gc, int64_t br, int64_t bc,
                          const CoefTable* d_tab, const CoefTable* h_tab, void* hat, int64_t hat_stride, unsigned* amax,
                          float* scale, bool b_side, cudaStream_t st) {
  const int mode = d->scale_mode;   // 0 none, 1 per encoded tensor, 2 per row of it, 3 model schedule (128-groups)
  const EncodeOperand o{X, ldx, gr, gc, br, bc, d_tab, h_tab, hat, hat_stride, amax, scale, b_side ? 128 : 1, b_side ? 1 : 0};
  if (mode != 0) {
    FMM_CUDA(cudaMemsetAsync(amax, 0, scale_words(mode, h_tab->R, br, bc, b_side) * 4, st));
    FMM_CUDA(launch_encode_pair(d->storage, d->product, o, nullptr, true, mode, st));
  }
  FMM_CUDA(launch_encode_pair(d->storage, d->product, o, nullptr, false, mode, st));
  return FMM_OK;
}

// The classical control's operand: the whole matrix as one block with coefficient 1.
fmm_status quantize_operand(const fmm_gemm_desc* d, const void* X, int64_t ldx, int64_t rows, int64_t cols, void* hat,
                            unsigned* amax, float* scale, bool b_side, cudaStream_t st) {
  const int mode = d->scale_mode;
  const int srows = b_side ? 128 : 1, bf16_first = b_side ? 1 : 0;   // model schedule only
  if (mode != 0) {
    FMM_CUDA(cudaMemsetAsync(amax, 0, scale_words(mode, 1, rows, cols, b_side) * 4, st));
    FMM_CUDA(launch_quantize_plain(d->storage, d->product, X, ldx, rows, cols, hat, amax, scale, true, mode, srows, bf16_first, st));
  }
  FMM_CUDA(launch_quantize_plain(d->storage, d->product, X, ldx, rows, cols, hat, amax, scale, false, mode, srows, bf16_first, st));
  return FMM_OK;
}

// One scheme applied to one operand pair inside one workspace: the pieces every stage needs.
struct SchemeRun {
  const fmm_scheme* s;
  const fmm_gemm_desc* d;
  GemmLayout L;
  void* ws;
  const CoefTable *hA, *hB, *hW;   // host tables (list lengths size the kernels' shared memory)
  const CoefTable *dA, *dB, *dW;   // device copies
  float* sA() const { return d->scale_mode != 0 ? at<float>(ws, L.sA) : nullptr; }
  float* sB() const { return d->scale_mode != 0 ? at<float>(ws, L.sB) : nullptr; }
};

fmm_status stage_encode_a(const SchemeRun& r, const void* A, cudaStream_t st) {
  const fmm_scheme* s = r.s;
  ProfScope ps(0, st);
  return encode_operand(r.d, A, r.d->lda, s->m, s->k, r.d->M / s->m, r.d->K / s->k, r.dA, r.hA, at<char>(r.ws, r.L.ahat),
                        r.L.sAhat, at<unsigned>(r.ws, r.L.amaxA), r.sA(), false, st);
}
fmm_status stage_encode_b(const SchemeRun& r, const void* Bk, int64_t ldbk, cudaStream_t st) {
  const fmm_scheme* s = r.s;
  ProfScope ps(1, st);
  return encode_operand(r.d, Bk, ldbk, s->n, s->k, r.d->N / s->n, r.d->K / s->k, r.dB, r.hB, at<char>(r.ws, r.L.bhat),
                        r.L.sBhat, at<unsigned>(r.ws, r.L.amaxB), r.sB(), true, st);
}
// Both operands in one launch per pass (amax pass if scaled, then the encode pass), on one stream.
fmm_status stage_encode_pair(const SchemeRun& r, const void* A, const void* Bk, int64_t ldbk, cudaStream_t st) {
  const fmm_scheme* s = r.s;
  const fmm_gemm_desc* d = r.d;
  const int64_t bm = d->M / s->m, bk = d->K / s->k, bn = d->N / s->n;
  const EncodeOperand oa{A, d->lda, s->m, s->k, bm, bk, r.dA, r.hA, at<char>(r.ws, r.L.ahat), r.L.sAhat,
                         at<unsigned>(r.ws, r.L.amaxA), r.sA(), 1, 0};
  const EncodeOperand ob{Bk, ldbk, s->n, s->k, bn, bk, r.dB, r.hB, at<char>(r.ws, r.L.bhat), r.L.sBhat,
                         at<unsigned>(r.ws, r.L.amaxB), r.sB(), 128, 1};
  ProfScope ps(0, st);
  const int mode = d->scale_mode;
  if (mode != 0) {
    // amaxA and amaxB are neighbours in the workspace: one memset clears both
    FMM_CUDA(cudaMemsetAsync(at<char>(r.ws, r.L.amaxA), 0, r.L.sA - r.L.amaxA, st));
    FMM_CUDA(launch_encode_pair(d->storage, d->product, oa, &ob, true, mode, st));
  }
  FMM_CUDA(launch_encode_pair(d->storage, d->product, oa, &ob, false, mode, st));
  return FMM_OK;
}

// Block sums rounded at every level of a nested algorithm (FMM_FLAG_ROUND_PER_LEVEL): the outer factor's block sums
// of the operand are scaled, rounded to the product dtype and kept as R1 tensors; for each of them the inner factor's
// block sums are formed of those rounded values and rounded again into products r1 * R2 .. r1 * R2 + R2 - 1.  With one
// scale per encoded tensor the inner pass works in units of the outer scale and writes the product of the two.
fmm_status stage_encode_per_level(const SchemeRun& r, const void* X, int64_t ldx, bool b_side, cudaStream_t st) {
  const fmm_scheme& so = *r.s->outer;
  const fmm_scheme& si = *r.s->inner;
  const fmm_gemm_desc* d = r.d;
  const int mode = d->scale_mode;
  const int gr1 = b_side ? so.n : so.m, gc1 = so.k, gr2 = b_side ? si.n : si.m, gc2 = si.k;
  const int64_t Br = (b_side ? d->N : d->M) / gr1, Bc = d->K / gc1;      // outer blocks
  const int64_t br = Br / gr2, bc = Bc / gc2;                            // inner blocks
  const int which = b_side ? 1 : 0;
  const size_t tstride = align_up(sizeof(CoefTable));
  const CoefTable* h_out = fmm_packed_table(so, which);
  const CoefTable* h_in = fmm_packed_table(si, which);
  const CoefTable* d_out = at<CoefTable>(r.ws, r.L.lvl_tab_outer + which * tstride);
  const CoefTable* d_in = at<CoefTable>(r.ws, r.L.lvl_tab_inner + which * tstride);
  FMM_CUDA(cudaMemcpyAsync(const_cast<CoefTable*>(d_out), h_out, sizeof(CoefTable), cudaMemcpyHostToDevice, st));
  FMM_CUDA(cudaMemcpyAsync(const_cast<CoefTable*>(d_in), h_in, sizeof(CoefTable), cudaMemcpyHostToDevice, st));
  unsigned* amax1 = at<unsigned>(r.ws, r.L.lvl_amax) + which * FMM_MAX_R;
  float* scale1 = at<float>(r.ws, r.L.lvl_scale) + which * FMM_MAX_R;
  const int ep = esize(d->product);
  char* lvl = at<char>(r.ws, b_side ? r.L.lvl_b : r.L.lvl_a);
  const int64_t lvl_stride = b_side ? r.L.sLvlB : r.L.sLvlA;
  ProfScope ps(b_side ? 1 : 0, st);
  // outer level
  const EncodeOperand o1{X, ldx, gr1, gc1, Br, Bc, d_out, h_out, lvl, lvl_stride, amax1, mode ? scale1 : nullptr, 1, 0, nullptr};
  if (mode != 0) {
    FMM_CUDA(cudaMemsetAsync(amax1, 0, FMM_MAX_R * 4, st));
    FMM_CUDA(launch_encode_pair(d->storage, d->product, o1, nullptr, true, mode, st));
  }
  FMM_CUDA(launch_encode_pair(d->storage, d->product, o1, nullptr, false, mode, st));
  // inner level, one outer product at a time: its source is the rounded outer block sum (product dtype)
  char* hat = at<char>(r.ws, b_side ? r.L.bhat : r.L.ahat);
  const int64_t hat_stride = b_side ? r.L.sBhat : r.L.sAhat;
  unsigned* amax2 = at<unsigned>(r.ws, b_side ? r.L.amaxB : r.L.amaxA);
  float* scale2 = b_side ? r.sB() : r.sA();
  if (mode != 0) FMM_CUDA(cudaMemsetAsync(amax2, 0, FMM_MAX_R * 4, st));
  for (int r1 = 0; r1 < so.R; ++r1) {
    const EncodeOperand o2{lvl + (size_t)r1 * lvl_stride * ep, Bc, gr2, gc2, br, bc, d_in, h_in,
                           hat + (size_t)r1 * si.R * hat_stride * ep, hat_stride, amax2 + r1 * si.R,
                           mode ? scale2 + r1 * si.R : nullptr, 1, 0, mode ? scale1 + r1 : nullptr};
    if (mode != 0) FMM_CUDA(launch_encode_pair(d->product, d->product, o2, nullptr, true, mode, st));
    FMM_CUDA(launch_encode_pair(d->product, d->product, o2, nullptr, false, mode, st));
  }
  return FMM_OK;
}

fmm_status stage_products(const SchemeRun& r, cudaStream_t st) {
  const fmm_scheme* s = r.s;
  const int64_t bm = r.d->M / s->m, bk = r.d->K / s->k, bn = r.d->N / s->n;
  if (r.d->scale_mode == 3) {   // model schedule: every 128-group of inner indices is scaled on its own inside the product kernel
    Fp8GroupArgs g{};
    g.A = at<char>(r.ws, r.L.ahat); g.lda = bk; g.a_batch = r.L.sAhat;
    g.B = at<char>(r.ws, r.L.bhat); g.ldb = bk; g.b_batch = r.L.sBhat;
    g.rows_a = bm; g.rows_b = bn; g.kdim = bk; g.batches = s->R;
    g.out = at<char>(r.ws, r.L.prod); g.ldo = bn; g.o_batch = r.L.sProd;
    g.output = (r.d->flags & FMM_FLAG_PRODUCTS_BF16) ? FMM_BF16 : FMM_F32;
    g.sA = r.sA(); g.sB = r.sB();
    g.status = at<DeviceStatus>(r.ws, r.L.status);
    ProfScope ps(2, st);
    return launch_fp8_group_gemm(g, st);
  }
  BlockProductArgs g{};
  g.product = r.d->product;
  g.A = at<char>(r.ws, r.L.ahat); g.lda = bk; g.a_batch = r.L.sAhat;
  g.B = at<char>(r.ws, r.L.bhat); g.ldb = bk; g.b_batch = r.L.sBhat;
  g.rows_a = bm; g.rows_b = bn; g.kdim = bk; g.batches = s->R;
  g.out = at<char>(r.ws, r.L.prod); g.ldo = bn; g.o_batch = r.L.sProd; g.out_mode = 0; g.output = FMM_F32;
  if (r.d->flags & FMM_FLAG_PRODUCTS_BF16) { g.out_mode = 1; g.output = FMM_BF16; }   // one rounding of each product
  if (r.d->scale_mode == 2) {   // row / column scales are folded into the stored products
    g.row_scale = r.sA(); g.rs_batch = bm;
    g.col_scale = r.sB(); g.cs_batch = bn;
  }
  g.status = at<DeviceStatus>(r.ws, r.L.status);
  ProfScope ps(2, st);
  return launch_block_products(g, st);
}
// If C is null the result is not stored; if cstar32 is given the squared error is reduced into err_out[0].
fmm_status stage_decode(const SchemeRun& r, void* C, const float* cstar32, double* err_out, cudaStream_t st, int gauges = 1) {
  const fmm_scheme* s = r.s;
  ProfScope ps(3, st);
  int np = 0;
  const bool per_product = r.d->scale_mode == 1;   // mode 2: the products already carry their scales
  FMM_CUDA(launch_decode(r.d->output, at<char>(r.ws, r.L.prod), (r.d->flags & FMM_FLAG_PRODUCTS_BF16) ? FMM_BF16 : FMM_F32,
                         r.L.sProd, r.dW, r.hW, s->R, per_product ? r.sA() : nullptr,
                         per_product ? r.sB() : nullptr, s->m, s->n,
                         r.d->M / s->m, r.d->N / s->n, C, r.d->ldc, cstar32, at<double>(r.ws, r.L.partials), &np, st, gauges));
  if (cstar32 && err_out) FMM_CUDA(launch_sum_partials(at<double>(r.ws, r.L.partials), np, err_out, st, gauges));
  return FMM_OK;
}

// The whole path on the caller's stream (encode B runs beside encode A on the side stream).  Host tables are
// uploaded into the workspace unless device copies are passed in.
fmm_status run_scheme(const fmm_scheme* s, const fmm_gemm_desc* d, const GemmLayout& L, const CoefTable* hA,
                      const CoefTable* hB, const CoefTable* hW, const CoefTable* dA_tab, const CoefTable* dB_tab,
                      const CoefTable* dW_tab, const void* A, const void* Bsrc_kmajor, int64_t ldb_kmajor, void* C,
                      const float* cstar32, double* err_out, void* ws, bool skip_b, cudaStream_t st) {
  if (!dA_tab) {
    FMM_CUDA(cudaMemcpyAsync(at<char>(ws, L.tabA), hA, sizeof(CoefTable), cudaMemcpyHostToDevice, st));
    dA_tab = at<CoefTable>(ws, L.tabA);
  }
  if (!dB_tab) {
    if (!skip_b) FMM_CUDA(cudaMemcpyAsync(at<char>(ws, L.tabB), hB, sizeof(CoefTable), cudaMemcpyHostToDevice, st));
    dB_tab = at<CoefTable>(ws, L.tabB);
  }
  if (!dW_tab) {
    FMM_CUDA(cudaMemcpyAsync(at<char>(ws, L.tabW), hW, sizeof(CoefTable), cudaMemcpyHostToDevice, st));
    dW_tab = at<CoefTable>(ws, L.tabW);
  }
  const SchemeRun r{s, d, L, ws, hA, hB, hW, dA_tab, dB_tab, dW_tab};
  // encode A and encode B side by side: one launch whose blocks split between the two operands (they share nothing)
  if (d->flags & FMM_FLAG_ROUND_PER_LEVEL) {
    FMM_TRY(stage_encode_per_level(r, A, d->lda, false, st));
    if (!skip_b) FMM_TRY(stage_encode_per_level(r, Bsrc_kmajor, ldb_kmajor, true, st));
  } else if (skip_b) {
    FMM_TRY(stage_encode_a(r, A, st));
  } else {
    FMM_TRY(stage_encode_pair(r, A, Bsrc_kmajor, ldb_kmajor, st));
  }
  FMM_TRY(stage_products(r, st));
  return stage_decode(r, C, cstar32, err_out, st);
}

// B as a K-major matrix [N x K]: in place for the weight layout, else transposed into the workspace.
fmm_status kmajor_b(const fmm_gemm_desc* d, const void* B, void* ws, size_t bt_off, const void** out, int64_t* ld,
                    bool skip, cudaStream_t st) {
  if (d->b_is_weight_layout) { *out = B; *ld = d->ldb; return FMM_OK; }
  void* bt = at<char>(ws, bt_off);
  ProfScope ps(1, st);
  if (!skip) FMM_CUDA(launch_transpose(esize(d->storage), B, d->ldb, d->K, d->N, bt, st));
  *out = bt; *ld = d->K;
  return FMM_OK;
}

// FMM_FLAG_ROUND_PER_LEVEL needs a handle that remembers its factors, scale mode 0 or 1, and inner blocks the 16-byte
// vectors of the product dtype tile (a multiple of 16 inner indices per inner block already holds)
fmm_status check_per_level(const fmm_scheme* s, const fmm_gemm_desc* d) {
  if (!(d->flags & FMM_FLAG_ROUND_PER_LEVEL)) return FMM_OK;
  if (!s->outer || !s->inner) return FMM_ERR_ARG;
  if (d->scale_mode != 0 && d->scale_mode != 1) return FMM_ERR_DTYPE;
  return FMM_OK;
}

fmm_status check_ws(const void* ws, size_t have, size_t need) {
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) || have < need) return FMM_ERR_WORKSPACE;
  return FMM_OK;
}

// Workspace of the classical product.
struct ClassicalLayout { size_t status, tab, amaxA, amaxB, sA, sB, bt, ahat, bhat, total; bool direct; };

ClassicalLayout classical_layout(const fmm_gemm_desc* d) {
  ClassicalLayout L;
  const int ep = esize(d->product), es = esize(d->storage);
  L.direct = d->storage == d->product && d->scale_mode == 0;   // bf16, or e4m3 codes: the operands are read in place
  size_t o = 0;
  L.status = o; o += align_up(sizeof(DeviceStatus));
  L.tab = o; o += align_up(sizeof(CoefTable));
  const size_t nsa = scale_words(d->scale_mode, 1, d->M, d->K, false), nsb = scale_words(d->scale_mode, 1, d->N, d->K, true);
  L.amaxA = o; o += align_up(nsa * 4);
  L.amaxB = o; o += align_up(nsb * 4);
  L.sA = o; o += align_up(nsa * 4);
  L.sB = o; o += align_up(nsb * 4);
  L.bt = o; o += d->b_is_weight_layout ? 0 : align_up((size_t)d->N * d->K * es);
  L.ahat = o; o += L.direct ? 0 : align_up((size_t)d->M * d->K * ep);
  L.bhat = o; o += L.direct ? 0 : align_up((size_t)d->N * d->K * ep);
  L.total = o;
  return L;
}

fmm_status run_classical(const fmm_gemm_desc* d, const ClassicalLayout& L, const void* A, const void* B, void* C,
                         void* ws, cudaStream_t st) {
  const void* bk_ptr; int64_t bk_ld;
  FMM_TRY(kmajor_b(d, B, ws, L.bt, &bk_ptr, &bk_ld, false, st));
  BlockProductArgs g{};
  g.product = d->product;
  g.rows_a = d->M; g.rows_b = d->N; g.kdim = d->K; g.batches = 1;
  g.out = C; g.ldo = d->ldc; g.o_batch = 0; g.out_mode = 1; g.output = d->output;
  g.status = at<DeviceStatus>(ws, L.status);
  if (L.direct) {
    g.A = A; g.lda = d->lda; g.a_batch = 0;
    g.B = bk_ptr; g.ldb = bk_ld; g.b_batch = 0;
  } else {
    const bool scaled = d->scale_mode != 0;
    float* sA = scaled ? at<float>(ws, L.sA) : nullptr;
    float* sB = scaled ? at<float>(ws, L.sB) : nullptr;
    ProfScope pe(5, st);
    FMM_TRY(quantize_operand(d, A, d->lda, d->M, d->K, at<char>(ws, L.ahat), at<unsigned>(ws, L.amaxA), sA, false, st));
    FMM_TRY(quantize_operand(d, bk_ptr, bk_ld, d->N, d->K, at<char>(ws, L.bhat), at<unsigned>(ws, L.amaxB), sB, true, st));
    g.A = at<char>(ws, L.ahat); g.lda = d->K; g.a_batch = 0;
    g.B = at<char>(ws, L.bhat); g.ldb = d->K; g.b_batch = 0;
    if (d->scale_mode == 3) {
      Fp8GroupArgs q{};
      q.A = g.A; q.lda = d->K; q.a_batch = 0; q.B = g.B; q.ldb = d->K; q.b_batch = 0;
      q.rows_a = d->M; q.rows_b = d->N; q.kdim = d->K; q.batches = 1;
      q.out = C; q.ldo = d->ldc; q.o_batch = 0; q.output = d->output;
      q.sA = sA; q.sB = sB; q.status = g.status;
      ProfScope ps(4, st);
      return launch_fp8_group_gemm(q, st);
    }
    if (d->scale_mode == 2) { g.row_scale = sA; g.col_scale = sB; g.rs_batch = 0; g.cs_batch = 0; }
    else { g.sA = sA; g.sB = sB; }
  }
  ProfScope ps(4, st);
  return launch_block_products(g, st);
}

// Workspace of a sweep: the GEMM layout plus reference copies, classical result, tables and sums.
// Gauge batching in the sweep.  Equivalent algorithms share their operands, so several of them can run as ONE set of
// launches: the encode reads A and B once for all of them, the block products fill the machine with more tiles, the
// decode walks the positions once.  `kb` algorithms become one table set with kb * R products; the decode table keeps
// their C blocks apart (list c feeds block c / kb of algorithm c % kb).  Limits: kb * R <= FMM_MAX_R products,
// kb * m * n <= 16 decode lists, kb in {1, 2, 4} (it must divide the decode's thread split); eight algorithms of at
// most 8 products and 4 output cells each also fit (32 lists: the register-resident batch decode takes them).
int sweep_batch(const fmm_scheme* s) {
  constexpr int cap = 8;
  if (cap >= 8 && 8 * s->R <= FMM_MAX_R && s->R <= 8 && s->m * s->n <= 4) return 8;
  for (int kb = 4; kb > 1; kb /= 2)
    if (kb <= cap && kb * s->R <= FMM_MAX_R && kb * s->m * s->n <= 16) return kb;
  return 1;
}

// Merge the tables of kb algorithms (tabs[3*i .. 3*i+2] = encode A, encode B, decode of algorithm i).  Returns false if the
// merged lists do not fit a table.
bool merge_tables(const CoefTable* tabs, int kb, int R, CoefTable* mA, CoefTable* mB, CoefTable* mW) {
  for (int which = 0; which < 2; ++which) {
    CoefTable* out = which == 0 ? mA : mB;
    std::memset(out, 0, sizeof(CoefTable));
    out->ncell = tabs[which].ncell;
    int n = 0, lists = 0;
    for (int i = 0; i < kb; ++i) {
      const CoefTable& t = tabs[3 * i + which];
      for (int r = 0; r < t.R; ++r) {
        out->off[lists++] = n;
        for (int e = t.off[r]; e < t.off[r + 1]; ++e) {
          if (n >= kMaxNnz) return false;
          out->cell[n] = t.cell[e]; out->coef[n] = t.coef[e]; ++n;
        }
      }
    }
    out->off[lists] = n;
    out->R = lists;
  }
  std::memset(mW, 0, sizeof(CoefTable));
  const int cells = tabs[2].R;
  mW->ncell = kb * R;                       // the padding slab sits behind all kb * R products
  int n = 0, lists = 0;
  for (int c = 0; c < cells; ++c)
    for (int i = 0; i < kb; ++i) {
      const CoefTable& t = tabs[3 * i + 2];
      mW->off[lists++] = n;
      for (int e = t.off[c]; e < t.off[c + 1]; ++e) {
        if (n >= kMaxNnz) return false;
        mW->cell[n] = t.cell[e] == t.ncell ? kb * R : t.cell[e] + i * R;
        mW->coef[n] = t.coef[e]; ++n;
      }
    }
  mW->off[lists] = n;
  mW->R = lists;
  return true;
}

struct SweepLayout {
  GemmLayout g; ClassicalLayout c;
  size_t gemm, gemm2, classical, cstar, cstar32, ccl, tables, sums, fpart, total;   // two GEMM workspaces: gauges are pipelined
};
constexpr int kFusedPartialsPerGauge = 512;   // room for the streaming blocks of a fused launch (2 per SM)

SweepLayout sweep_layout(const fmm_scheme* s, const fmm_gemm_desc* d, int G) {
  SweepLayout L;
  L.g = gemm_layout(s->m, s->k, s->n, s->R * sweep_batch(s), d);   // room for a whole batch of algorithms
  L.c = classical_layout(d);
  size_t o = 0;
  L.gemm = o; o += align_up(L.g.total);
  L.gemm2 = o; o += align_up(L.g.total);
  L.classical = o; o += align_up(L.c.total);
  L.cstar = o; o += align_up((size_t)d->M * d->N * 8);
  L.cstar32 = o; o += align_up((size_t)d->M * d->N * 4);
  L.ccl = o; o += align_up((size_t)d->M * d->N * esize(d->output));
  L.tables = o; o += align_up((size_t)G * 3 * sizeof(CoefTable));
  L.sums = o; o += align_up((size_t)(G + 8) * 8);
  L.fpart = o; o += align_up((size_t)G * kFusedPartialsPerGauge * 8);
  L.total = o;
  return L;
}

}  // namespace

extern "C" {

int64_t fmm_launch_count(void) { return fmm_launch_counter(); }

void fmm_profile_enable(int on) { g_prof_on = on != 0; }

fmm_status fmm_profile_collect(double ms[8], int64_t count[8]) {
  if (!ms || !count) return FMM_ERR_ARG;
  for (int i = 0; i < 8; ++i) { ms[i] = 0.0; count[i] = 0; }
  fmm_status rc = FMM_OK;
  for (ProfRec& r : g_prof) {
    float t = 0.f;
    if (cudaEventSynchronize(r.b) != cudaSuccess || cudaEventElapsedTime(&t, r.a, r.b) != cudaSuccess) rc = FMM_ERR_CUDA;
    if (r.kind >= 0 && r.kind < 8) { ms[r.kind] += t; count[r.kind] += 1; }
    cudaEventDestroy(r.a); cudaEventDestroy(r.b);
  }
  g_prof.clear();
  return rc;
}

size_t scheme_gemm_workspace(const fmm_scheme* s, const fmm_gemm_desc* d) {
  if (!s || check_desc(d, s->m, s->k, s->n) != FMM_OK || check_per_level(s, d) != FMM_OK) return 0;
  return gemm_layout(s->m, s->k, s->n, s->R, d, s).total;
}

fmm_status scheme_gemm_workspace_layout(const fmm_scheme* s, const fmm_gemm_desc* d, size_t off[8]) {
  if (!s || !off) return FMM_ERR_ARG;
  FMM_TRY(check_desc(d, s->m, s->k, s->n));
  FMM_TRY(check_per_level(s, d));
  const GemmLayout L = gemm_layout(s->m, s->k, s->n, s->R, d, s);
  off[0] = L.ahat; off[1] = L.bhat; off[2] = L.prod; off[3] = L.sA; off[4] = L.sB;
  off[5] = (size_t)L.sAhat; off[6] = (size_t)L.sBhat; off[7] = (size_t)L.sProd;
  return FMM_OK;
}

fmm_status scheme_gemm(const fmm_scheme* s, const fmm_gemm_desc* d, const void* dA, const void* dB, void* dC,
                       void* d_ws, size_t ws_bytes, void* cuda_stream) {
  if (!s || !d || !dA || !dB || !dC) return FMM_ERR_ARG;
  FMM_TRY(check_desc(d, s->m, s->k, s->n));
  FMM_TRY(check_per_level(s, d));
  const GemmLayout L = gemm_layout(s->m, s->k, s->n, s->R, d, s);
  FMM_TRY(check_ws(d_ws, ws_bytes, L.total));
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const bool skip_b = (d->flags & FMM_FLAG_REUSE_BHAT) != 0;
  // one copy brings a zeroed status block and the three kernel tables (cached in the handle) to the head of the
  // workspace, whose layout they mirror
  const std::vector<unsigned char>& packed = fmm_packed_tables(*s);
  if (L.status != 0 || L.tabA != kPackedStatusBytes || L.tabB != L.tabA + fmm_packed_table_stride() ||
      L.tabW != L.tabB + fmm_packed_table_stride() || sizeof(DeviceStatus) > kPackedStatusBytes)
    return FMM_ERR_CUDA;
  FMM_CUDA(cudaMemcpyAsync(d_ws, packed.data(), packed.size(), cudaMemcpyHostToDevice, st));
  const void* bk_ptr; int64_t bk_ld;
  FMM_TRY(kmajor_b(d, dB, d_ws, L.bt, &bk_ptr, &bk_ld, skip_b, st));
  return run_scheme(s, d, L, fmm_packed_table(*s, 0), fmm_packed_table(*s, 1), fmm_packed_table(*s, 2),
                    at<CoefTable>(d_ws, L.tabA), at<CoefTable>(d_ws, L.tabB), at<CoefTable>(d_ws, L.tabW), dA, bk_ptr, bk_ld, dC,
                    nullptr, nullptr, d_ws, skip_b, st);
}

fmm_status scheme_joint_round_weights(const fmm_scheme* s, const fmm_gemm_desc* d, const void* dB, int max_sweeps,
                                      void* d_ws, size_t ws_bytes, void* cuda_stream) {
  if (!s || !d || !dB || max_sweeps < 0) return FMM_ERR_ARG;
  FMM_TRY(check_desc(d, s->m, s->k, s->n));
  if (d->scale_mode != 3 || d->product != FMM_E4M3) return FMM_ERR_DTYPE;
  const GemmLayout L = gemm_layout(s->m, s->k, s->n, s->R, d);
  FMM_TRY(check_ws(d_ws, ws_bytes, L.total));
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const std::vector<unsigned char>& packed = fmm_packed_tables(*s);
  if (L.status != 0 || L.tabA != kPackedStatusBytes || L.tabB != L.tabA + fmm_packed_table_stride() ||
      L.tabW != L.tabB + fmm_packed_table_stride() || sizeof(DeviceStatus) > kPackedStatusBytes)
    return FMM_ERR_CUDA;
  FMM_CUDA(cudaMemcpyAsync(d_ws, packed.data(), packed.size(), cudaMemcpyHostToDevice, st));
  const void* bk_ptr; int64_t bk_ld;
  FMM_TRY(kmajor_b(d, dB, d_ws, L.bt, &bk_ptr, &bk_ld, false, st));
  // H_rs = <w_r, w_s> <u_r, u_s>, fp64 on the host, rounded to fp32; parked in the product buffer, which nothing uses yet
  const int R = s->R, mk = s->m * s->k, mn = s->m * s->n;
  std::vector<float> H((size_t)R * R);
  for (int r = 0; r < R; ++r)
    for (int q = 0; q < R; ++q) {
      double uu = 0.0, ww = 0.0;
      for (int x = 0; x < mk; ++x) uu += s->U[(size_t)r * mk + x] * s->U[(size_t)q * mk + x];
      for (int x = 0; x < mn; ++x) ww += s->W[(size_t)r * mn + x] * s->W[(size_t)q * mn + x];
      H[(size_t)r * R + q] = (float)(ww * uu);
    }
  float* d_H = at<float>(d_ws, L.prod);
  if (L.total - L.prod < H.size() * sizeof(float)) return FMM_ERR_SHAPE;   // blocks of a few elements only
  FMM_CUDA(cudaMemcpyAsync(d_H, H.data(), H.size() * sizeof(float), cudaMemcpyHostToDevice, st));   // pageable: staged before it returns
  const int64_t bn = d->N / s->n, bk = d->K / s->k;
  const CoefTable* hB = fmm_packed_table(*s, 1);
  const CoefTable* dB_tab = at<CoefTable>(d_ws, L.tabB);
  unsigned* amax = at<unsigned>(d_ws, L.amaxB);
  float* sB = at<float>(d_ws, L.sB);
  // the model schedule's amax pass over the bf16 block sums, then the search in place of the plain encode pass
  const EncodeOperand ob{bk_ptr, bk_ld, s->n, s->k, bn, bk, dB_tab, hB, at<char>(d_ws, L.bhat), L.sBhat, amax, sB, 128, 1};
  FMM_CUDA(cudaMemsetAsync(amax, 0, scale_words(3, R, bn, bk, true) * 4, st));
  FMM_CUDA(launch_encode_pair(d->storage, d->product, ob, nullptr, true, 3, st));
  FMM_CUDA(launch_joint_round(d->storage, bk_ptr, bk_ld, s->n, s->k, bn, bk, dB_tab, d_H, amax, sB, at<char>(d_ws, L.bhat),
                              L.sBhat, max_sweeps, st));
  return FMM_OK;
}

// ---- scheme_gemm on operands in HOST memory: copies in, the whole path, copy out, all on one stream
namespace {
struct HostLayout { size_t a, b, c, ws, total; fmm_gemm_desc dev; };
HostLayout host_layout(const fmm_scheme* s, const fmm_gemm_desc* d) {
  HostLayout L;
  L.dev = *d;                      // the device copies are dense
  L.dev.lda = d->K;
  L.dev.ldb = d->b_is_weight_layout ? d->K : d->N;
  L.dev.ldc = d->N;
  const size_t es = (size_t)esize(d->storage), eo = (size_t)esize(d->output);
  size_t o = 0;
  L.a = o; o += align_up((size_t)d->M * d->K * es);
  L.b = o; o += align_up((size_t)d->K * d->N * es);
  L.c = o; o += align_up((size_t)d->M * d->N * eo);
  L.ws = o; o += gemm_layout(s->m, s->k, s->n, s->R, &L.dev, s).total;
  L.total = o;
  return L;
}
}  // namespace

size_t scheme_gemm_host_workspace(const fmm_scheme* s, const fmm_gemm_desc* d) {
  if (!s || check_desc(d, s->m, s->k, s->n) != FMM_OK) return 0;
  return host_layout(s, d).total;
}

fmm_status scheme_gemm_host(const fmm_scheme* s, const fmm_gemm_desc* d, const void* hA, const void* hB, void* hC,
                            void* d_ws, size_t ws_bytes, void* cuda_stream) {
  if (!s || !d || !hA || !hC) return FMM_ERR_ARG;
  const bool reuse_b = (d->flags & FMM_FLAG_REUSE_BHAT) != 0;
  if (!hB && !reuse_b) return FMM_ERR_ARG;
  FMM_TRY(check_desc(d, s->m, s->k, s->n));
  const HostLayout L = host_layout(s, d);
  FMM_TRY(check_ws(d_ws, ws_bytes, L.total));
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t es = (size_t)esize(d->storage), eo = (size_t)esize(d->output);
  char* ws = static_cast<char*>(d_ws);
  FMM_CUDA(cudaMemcpy2DAsync(ws + L.a, (size_t)d->K * es, hA, (size_t)d->lda * es, (size_t)d->K * es, (size_t)d->M,
                             cudaMemcpyHostToDevice, st));
  if (!reuse_b) {
    const size_t rows = d->b_is_weight_layout ? d->N : d->K, cols = d->b_is_weight_layout ? d->K : d->N;
    FMM_CUDA(cudaMemcpy2DAsync(ws + L.b, cols * es, hB, (size_t)d->ldb * es, cols * es, rows, cudaMemcpyHostToDevice, st));
  }
  FMM_TRY(scheme_gemm(s, &L.dev, ws + L.a, ws + L.b, ws + L.c, ws + L.ws, ws_bytes - L.ws, cuda_stream));
  FMM_CUDA(cudaMemcpy2DAsync(hC, (size_t)d->ldc * eo, ws + L.c, (size_t)d->N * eo, (size_t)d->N * eo, (size_t)d->M,
                             cudaMemcpyDeviceToHost, st));
  return FMM_OK;
}

fmm_status fmm_device_status(const void* d_ws, void* cuda_stream);
fmm_status scheme_gemm_host_status(const fmm_scheme* s, const fmm_gemm_desc* d, const void* d_ws, void* cuda_stream) {
  if (!s || !d_ws) return FMM_ERR_ARG;
  FMM_TRY(check_desc(d, s->m, s->k, s->n));
  return fmm_device_status(static_cast<const char*>(d_ws) + host_layout(s, d).ws, cuda_stream);
}

fmm_status fmm_device_status(const void* d_ws, void* cuda_stream) {
  if (!d_ws) return FMM_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DeviceStatus h;
  FMM_CUDA(cudaMemcpyAsync(&h, d_ws, sizeof(h), cudaMemcpyDeviceToHost, st));
  FMM_CUDA(cudaStreamSynchronize(st));
  return h.code == 0 ? FMM_OK : FMM_ERR_TIMEOUT;
}

size_t classical_gemm_workspace(const fmm_gemm_desc* d) {
  if (check_desc(d, 1, 1, 1, true) != FMM_OK) return 0;
  return classical_layout(d).total;
}

fmm_status classical_gemm(const fmm_gemm_desc* d, const void* dA, const void* dB, void* dC, void* d_ws,
                          size_t ws_bytes, void* cuda_stream) {
  if (!d || !dA || !dB || !dC) return FMM_ERR_ARG;
  FMM_TRY(check_desc(d, 1, 1, 1, true));
  const ClassicalLayout L = classical_layout(d);
  FMM_TRY(check_ws(d_ws, ws_bytes, L.total));
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  FMM_CUDA(cudaMemsetAsync(at<char>(d_ws, L.status), 0, sizeof(DeviceStatus), st));
  return run_classical(d, L, dA, dB, dC, d_ws, st);
}

fmm_status exact_gemm_f64(const fmm_gemm_desc* d, const void* dA, const void* dB, double* dCstar, void* cuda_stream) {
  if (!d || !dA || !dB || !dCstar) return FMM_ERR_ARG;
  if (d->M <= 0 || d->K <= 0 || d->N <= 0) return FMM_ERR_SHAPE;
  if (d->storage != FMM_F32 && d->storage != FMM_BF16) return FMM_ERR_DTYPE;
  FMM_CUDA(launch_exact_f64(d->storage, dA, d->lda, dB, d->ldb, d->b_is_weight_layout, d->M, d->K, d->N, dCstar,
                            static_cast<cudaStream_t>(cuda_stream)));
  return FMM_OK;
}

fmm_status fmm_selftest_timeout(void* d_ws, size_t ws_bytes, unsigned wait_ms, void* cuda_stream) {
  // one 128 x 128 x 64 bf16 tile, one block; operands and output live in the workspace
  const size_t need = 1024 + 2 * (128 * 64 * 2) + 128 * 128 * 4;
  FMM_TRY(check_ws(d_ws, ws_bytes, need));
  if (wait_ms == 0 || wait_ms > 2000) return FMM_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  FMM_CUDA(cudaMemsetAsync(d_ws, 0, need, st));
  BlockProductArgs g{};
  g.product = FMM_BF16;
  g.A = at<char>(d_ws, 1024); g.lda = 64; g.a_batch = 0;
  g.B = at<char>(d_ws, 1024 + 128 * 64 * 2); g.ldb = 64; g.b_batch = 0;
  g.rows_a = 128; g.rows_b = 128; g.kdim = 64; g.batches = 1;
  g.out = at<char>(d_ws, 1024 + 2 * 128 * 64 * 2); g.ldo = 128; g.o_batch = 0; g.out_mode = 0; g.output = FMM_F32;
  g.status = at<DeviceStatus>(d_ws, 0);
  g.selftest_no_producer = 1;
  g.wait_limit_ns = (unsigned long long)wait_ms * 1000000ull;
  return launch_block_products(g, st);
}

size_t error_frobenius_workspace(void) { return align_up((size_t)kMaxStreamPartials * 8 * 2); }

fmm_status error_frobenius(const fmm_gemm_desc* d, const void* dC, const double* dCstar, double* d_out, void* d_ws,
                           size_t ws_bytes, void* cuda_stream) {
  if (!d || !dC || !dCstar || !d_out) return FMM_ERR_ARG;
  if (d->M <= 0 || d->N <= 0 || d->ldc < d->N) return FMM_ERR_SHAPE;
  if (d->output != FMM_F32 && d->output != FMM_BF16) return FMM_ERR_DTYPE;
  FMM_TRY(check_ws(d_ws, ws_bytes, error_frobenius_workspace()));
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  double* pe = at<double>(d_ws, 0);
  double* pr = pe + kMaxStreamPartials;
  int np = 0;
  FMM_CUDA(launch_frob_err(d->output, dC, d->ldc, dCstar, d->M, d->N, pe, pr, &np, st));
  FMM_CUDA(launch_sum_partials(pe, np, d_out, st));
  FMM_CUDA(launch_sum_partials(pr, np, d_out + 1, st));
  return FMM_OK;
}

size_t error_sweep_workspace(const fmm_scheme* base, const fmm_gemm_desc* d, int G) {
  if (!base || G < 1 || check_desc(d, base->m, base->k, base->n) != FMM_OK) return 0;
  return sweep_layout(base, d, G).total;
}

fmm_status error_sweep(const fmm_scheme* base, int level, int G, const double* P, const double* Q, const double* S,
                       const fmm_gemm_desc* d, const void* dA, const void* dB, const double* dCstar, double* h_ratios,
                       fmm_sweep_summary* out, void* d_ws, size_t ws_bytes, void* cuda_stream) {
  if (!base || !P || !Q || !S || !d || !dA || !dB || !out || G < 1) return FMM_ERR_ARG;
  if (level != 0 && level != 1) return FMM_ERR_ARG;
  if (level == 1 && (!base->outer || !base->inner)) return FMM_ERR_ARG;
  FMM_TRY(check_desc(d, base->m, base->k, base->n));
  if (d->flags & FMM_FLAG_ROUND_PER_LEVEL) return FMM_ERR_ARG;   // the sweep runs the flat operator
  const SweepLayout L = sweep_layout(base, d, G);
  FMM_TRY(check_ws(d_ws, ws_bytes, L.total));
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const fmm_scheme* grid = level == 1 ? base->outer.get() : base;
  const int gm = grid->m, gk = grid->k, gn = grid->n;
  // every gauge matrix is checked before the first launch: a singular one returns with nothing enqueued
  for (int g = 0; g < G; ++g)
    if (!fmm_gauge_invertible(gm, gk, gn, P + (size_t)g * gm * gm, Q + (size_t)g * gk * gk, S + (size_t)g * gn * gn))
      return FMM_ERR_SINGULAR;

  // 1. gauge-transformed coefficient tables: built on the host, merged per batch of algorithms and uploaded in groups
  //    of kTableGroup gauges while the device works on the groups before (the first launch waits for one group only)
  constexpr int kTableGroup = 32;
  std::vector<CoefTable> single((size_t)G * 3);
  std::memset(single.data(), 0, single.size() * sizeof(CoefTable));
  struct Chunk { int g0, count; };
  std::vector<Chunk> chunks;
  std::vector<CoefTable> tabs;          // three tables per chunk
  tabs.reserve((size_t)G * 3);          // never reallocates: launches keep pointers into it
  const int kb = sweep_batch(base);
  int next_gauge = 0;
  char* ws = static_cast<char*>(d_ws);
  void* gws = ws + L.gemm;
  void* cws = ws + L.classical;
  CoefTable* d_tabs = at<CoefTable>(ws, L.tables);
  double* sums = at<double>(ws, L.sums);  // [0]=n*, [1]=e_cl, [2]=scratch, [8..8+G) = e_g
  auto build_group = [&](cudaStream_t up) -> fmm_status {
    const int g_end = std::min(G, next_gauge + kTableGroup);
    for (int g = next_gauge; g < g_end; ++g) {
      fmm_scheme* gs = nullptr;
      FMM_TRY(fmm_gauge_core(*base, level, P + (size_t)g * gm * gm, Q + (size_t)g * gk * gk, S + (size_t)g * gn * gn, 0.0, &gs));
      fmm_build_tables(*gs, &single[3 * g], &single[3 * g + 1], &single[3 * g + 2]);
      scheme_free(gs);
    }
    const size_t first = chunks.size();
    int g = next_gauge;
    while (g < g_end) {
      int kc = kb;
      while (kc > g_end - g) kc /= 2;   // 8, 4, 2 or 1 algorithms
      CoefTable mA, mB, mW;
      while (kc > 1 && !merge_tables(&single[3 * g], kc, base->R, &mA, &mB, &mW)) kc /= 2;   // lists too long: smaller batch
      if (kc == 1) { mA = single[3 * g]; mB = single[3 * g + 1]; mW = single[3 * g + 2]; }
      tabs.push_back(mA); tabs.push_back(mB); tabs.push_back(mW);
      chunks.push_back({g, kc});
      g += kc;
    }
    next_gauge = g_end;
    FMM_CUDA(cudaMemcpyAsync(d_tabs + 3 * first, tabs.data() + 3 * first, (tabs.size() - 3 * first) * sizeof(CoefTable),
                             cudaMemcpyHostToDevice, up));
    return FMM_OK;
  };
  FMM_CUDA(cudaMemsetAsync(at<char>(gws, L.g.status), 0, sizeof(DeviceStatus), st));
  FMM_CUDA(cudaMemsetAsync(at<char>(cws, L.c.status), 0, sizeof(DeviceStatus), st));

  // 2. fp64 reference, its fp32 copy and its squared norm
  const double* cstar = dCstar;
  if (!cstar) {
    double* mine = at<double>(ws, L.cstar);
    FMM_CUDA(launch_exact_f64(d->storage, dA, d->lda, dB, d->ldb, d->b_is_weight_layout, d->M, d->K, d->N, mine, st));
    cstar = mine;
  }
  float* cstar32 = at<float>(ws, L.cstar32);
  double* part = at<double>(gws, L.g.partials);
  int np = 0;
  FMM_CUDA(launch_cstar_prepare(cstar, d->M * d->N, cstar32, part, &np, st));
  FMM_CUDA(launch_sum_partials(part, np, sums + 0, st));

  // 3. classical product at the same dtypes and its error
  fmm_gemm_desc dcl = *d;
  dcl.ldc = d->N;
  void* ccl = at<char>(ws, L.ccl);
  FMM_TRY(run_classical(&dcl, L.c, dA, dB, ccl, cws, st));
  FMM_CUDA(launch_frob_err(d->output, ccl, d->N, cstar, d->M, d->N, part, nullptr, &np, st));
  FMM_CUDA(launch_sum_partials(part, np, sums + 1, st));

  // 4. the sweep: per gauge encode A, encode B, R products, decode + error reduction.
  // The three stages stress different parts of the machine (memory system, tensor cores + L2, memory system),
  // so consecutive gauges are software-pipelined over three streams with two workspaces:
  //   encode(g+1)  ||  products(g)  ||  decode(g-1).
  const void* bk_ptr; int64_t bk_ld;
  FMM_TRY(kmajor_b(d, dB, gws, L.g.bt, &bk_ptr, &bk_ld, false, st));
  void* gws2 = ws + L.gemm2;
  FMM_CUDA(cudaMemsetAsync(at<char>(gws2, L.g.status), 0, sizeof(DeviceStatus), st));
  // with phase timing on, or when the caller asks for it, the stages run back to back on the caller's stream
  const bool serial = g_prof_on || (d->flags & FMM_FLAG_SWEEP_SERIAL) != 0;
  SideStream* side = serial ? nullptr : side_stream();
  fmm_scheme batched;                   // dimensions only: a batch of kc algorithms looks like one with kc * R products
  batched.m = base->m; batched.k = base->k; batched.n = base->n;
  fmm_status loop_rc = FMM_OK;
  // Fused pipeline (unless FMM_FLAG_SWEEP_UNFUSED; bf16 storage and products, no scales, batches of four or eight one-level
  // algorithms): ONE launch per batch runs its block products together with the decode of the batch before and the
  // encode of the batch after, in the same CTAs (launch_fused_sweep), on the caller's stream; the pipeline starts with a
  // plain encode and ends with a decode-only launch.  Batches of one or two algorithms at the end of the list take the
  // ordinary path below.  Measured on B200: the three passes do overlap inside the launch, and the chip answers by
  // lowering its clock (the board's power limit: tensor cores and the memory system cannot both run flat out), so the
  // gain over the passes one after another is a few per cent (512 gauges of config 3: 42-43 ms against 44-46 ms after
  // idle, 45.4 against 46.8-47.9 ms sustained), not the sum of the hidden passes.
  size_t first_plain_chunk = 0;
  const int kFusedGroups = 2;
  const int64_t bm_ = d->M / base->m, bn_ = d->N / base->n, bk_ = d->K / base->k;
  const bool fused_ok = !(d->flags & FMM_FLAG_SWEEP_UNFUSED) && !serial && kb >= 4 && d->storage == FMM_BF16 && d->product == FMM_BF16 && d->scale_mode == 0 &&
                        !(d->flags & FMM_FLAG_PRODUCTS_BF16) && base->m * base->k <= 4 && base->n * base->k <= 4 &&
                        base->m * base->n <= 4 && bm_ > 128 && bn_ > 128 &&
                        fused_sweep_blocks(kFusedGroups) <= kFusedPartialsPerGauge && fused_sweep_blocks(kFusedGroups) >= 2 &&
                        (int64_t)4 * base->R * ((bm_ + 255) / 256) * ((bn_ + 255) / 256) >= fused_sweep_blocks(1) / 2;
  if (fused_ok) {
    const int nblk = fused_sweep_blocks(kFusedGroups);
    double* fpart = at<double>(ws, L.fpart);
    auto chunk_ready = [&](size_t c) -> fmm_status {   // tables of chunk c built and uploaded (in groups, ahead of use)
      while (c >= chunks.size() && next_gauge < G) FMM_TRY(build_group(st));
      return FMM_OK;
    };
    auto run_of = [&](size_t c, int b) {
      batched.R = base->R * chunks[c].count;
      return SchemeRun{&batched, d, L.g, b ? gws2 : gws, &tabs[3 * c], &tabs[3 * c + 1], &tabs[3 * c + 2],
                       d_tabs + 3 * c, d_tabs + 3 * c + 1, d_tabs + 3 * c + 2};
    };
    auto fusable = [&](size_t c) { return c < chunks.size() && chunks[c].count >= 4; };
    loop_rc = chunk_ready(0);
    size_t nf = 0;                     // fused chunks so far: chunk i lives in buffer i & 1
    if (loop_rc == FMM_OK && fusable(0)) {
      const SchemeRun r0 = run_of(0, 0);
      loop_rc = stage_encode_pair(r0, dA, bk_ptr, bk_ld, st);
      for (size_t c = 0; loop_rc == FMM_OK; ++c) {
        if ((loop_rc = chunk_ready(c + 1)) != FMM_OK) break;
        const int b = (int)(c & 1);
        const bool more = fusable(c + 1);
        FusedSweepArgs f{};
        f.groups = kFusedGroups; f.output = d->output;
        f.n = base->n; f.bm = bm_; f.bn = bn_; f.cstar32 = cstar32;
        {  // products of chunk c
          const SchemeRun r = run_of(c, b);
          BlockProductArgs& g = f.products;
          g.product = FMM_BF16;
          g.A = at<char>(r.ws, L.g.ahat); g.lda = bk_; g.a_batch = L.g.sAhat;
          g.B = at<char>(r.ws, L.g.bhat); g.ldb = bk_; g.b_batch = L.g.sBhat;
          g.rows_a = bm_; g.rows_b = bn_; g.kdim = bk_; g.batches = base->R * chunks[c].count;
          g.out = at<char>(r.ws, L.g.prod); g.ldo = bn_; g.o_batch = L.g.sProd; g.out_mode = 0; g.output = FMM_F32;
          g.status = at<DeviceStatus>(r.ws, L.g.status);
          f.have_products = 1;
        }
        if (c > 0) {  // decode of chunk c-1 out of the other buffer
          const SchemeRun rp = run_of(c - 1, b ^ 1);
          f.dec_gauges = chunks[c - 1].count;
          f.dec_prod = at<float>(rp.ws, L.g.prod); f.dec_prod_stride = L.g.sProd; f.dec_tab = rp.dW; f.dec_RB = base->R;
          f.partials = fpart + (size_t)chunks[c - 1].g0 * nblk;
        }
        if (more) {   // encode of chunk c+1 into the other buffer (its last reader was the previous launch)
          const SchemeRun rn = run_of(c + 1, b ^ 1);
          f.have_encode = 1;
          f.enc_a = EncodeOperand{dA, d->lda, base->m, base->k, bm_, bk_, rn.dA, rn.hA, at<char>(rn.ws, L.g.ahat), L.g.sAhat,
                                  nullptr, nullptr, 1, 0, nullptr};
          f.enc_b = EncodeOperand{bk_ptr, bk_ld, base->n, base->k, bn_, bk_, rn.dB, rn.hB, at<char>(rn.ws, L.g.bhat), L.g.sBhat,
                                  nullptr, nullptr, 128, 1, nullptr};
        }
        {
          ProfScope ps(2, st);
          loop_rc = launch_fused_sweep(f, st);
        }
        nf = c + 1;
        if (!more) break;
      }
      if (loop_rc == FMM_OK && nf > 0) {   // tail of the pipeline: decode of the last fused chunk, then all its sums
        const size_t c = nf - 1;
        FusedSweepArgs f{};
        f.groups = kFusedGroups; f.output = d->output;
        f.n = base->n; f.bm = bm_; f.bn = bn_; f.cstar32 = cstar32;
        const SchemeRun rp = run_of(c, (int)(c & 1));
        f.products.status = at<DeviceStatus>(rp.ws, L.g.status);
        f.dec_gauges = chunks[c].count;
        f.dec_prod = at<float>(rp.ws, L.g.prod); f.dec_prod_stride = L.g.sProd; f.dec_tab = rp.dW; f.dec_RB = base->R;
        f.partials = fpart + (size_t)chunks[c].g0 * nblk;
        loop_rc = launch_fused_sweep(f, st);
        const int gauges_done = chunks[c].g0 + chunks[c].count;
        if (loop_rc == FMM_OK && launch_sum_partials(fpart, nblk, sums + 8, st, gauges_done) != cudaSuccess) loop_rc = FMM_ERR_CUDA;
      }
      first_plain_chunk = nf;
    }
  }
  if (loop_rc != FMM_OK) return loop_rc;    // everything so far ran on the caller's stream
  if (side == nullptr) {
    for (size_t c = first_plain_chunk; loop_rc == FMM_OK; ++c) {
      if (c == chunks.size()) {
        if (next_gauge >= G) break;
        if ((loop_rc = build_group(st)) != FMM_OK) break;
      }
      batched.R = base->R * chunks[c].count;
      const SchemeRun r{&batched, d, L.g, gws, &tabs[3 * c], &tabs[3 * c + 1], &tabs[3 * c + 2],
                        d_tabs + 3 * c, d_tabs + 3 * c + 1, d_tabs + 3 * c + 2};
      if ((loop_rc = stage_encode_pair(r, dA, bk_ptr, bk_ld, st)) != FMM_OK) break;
      if ((loop_rc = stage_products(r, st)) != FMM_OK) break;
      loop_rc = stage_decode(r, nullptr, cstar32, sums + 8 + chunks[c].g0, st, chunks[c].count);
    }
  } else {
    cudaStream_t sE = side->stream, sG = st, sD = side->stream2;
    if (!stream_wait(side, st, sE) || !stream_wait(side, st, sD)) return FMM_ERR_CUDA;   // nothing of the sweep is enqueued yet
    if (sG != st && !stream_wait(side, st, sG)) return FMM_ERR_CUDA;
    cudaEvent_t evG[2] = {nullptr, nullptr}, evD[2] = {nullptr, nullptr};
    // One step of the pipeline; any failure leaves the loop through the joins below, so that the caller's stream is
    // ordered behind everything that was enqueued on the library's streams (the caller owns the workspace they use).
    auto step = [&](size_t c) -> fmm_status {
      const int b = (int)(c & 1);
      batched.R = base->R * chunks[c].count;
      const SchemeRun r{&batched, d, L.g, b ? gws2 : gws, &tabs[3 * c], &tabs[3 * c + 1], &tabs[3 * c + 2],
                        d_tabs + 3 * c, d_tabs + 3 * c + 1, d_tabs + 3 * c + 2};
      // encode: the products of batch c-2 must have finished reading this buffer's Ahat / Bhat.  With one scale per
      // encoded tensor (mode 1) the decode of batch c-2 still reads this buffer's scales, which the encode rewrites:
      // then the encode waits for that decode too (the other modes fold their scales into the products).
      if (evG[b] && cudaStreamWaitEvent(sE, evG[b], 0) != cudaSuccess) return FMM_ERR_CUDA;
      if (d->scale_mode == 1 && evD[b] && cudaStreamWaitEvent(sE, evD[b], 0) != cudaSuccess) return FMM_ERR_CUDA;
      // Large operands: two launches, not the paired one — beside the products and decode of the neighbouring batches
      // the two smaller kernels pack better.  Small operands are launch-bound: one paired launch.
      const bool small_operands = (d->M + d->N) * d->K * (int64_t)esize(d->storage) < ((int64_t)16 << 20);
      if (small_operands) {
        FMM_TRY(stage_encode_pair(r, dA, bk_ptr, bk_ld, sE));
      } else {
        FMM_TRY(stage_encode_b(r, bk_ptr, bk_ld, sE));
        FMM_TRY(stage_encode_a(r, dA, sE));
      }
      cudaEvent_t evE = record_event(side, sE);
      // products: need this batch's encode, and the decode of batch c-2 must be done with this product buffer
      if (!evE || cudaStreamWaitEvent(sG, evE, 0) != cudaSuccess) return FMM_ERR_CUDA;
      if (evD[b] && cudaStreamWaitEvent(sG, evD[b], 0) != cudaSuccess) return FMM_ERR_CUDA;
      FMM_TRY(stage_products(r, sG));
      evG[b] = record_event(side, sG);
      // decode + error reduction, one sum per algorithm of the batch
      if (!evG[b] || cudaStreamWaitEvent(sD, evG[b], 0) != cudaSuccess) return FMM_ERR_CUDA;
      FMM_TRY(stage_decode(r, nullptr, cstar32, sums + 8 + chunks[c].g0, sD, chunks[c].count));
      evD[b] = record_event(side, sD);
      return evD[b] ? FMM_OK : FMM_ERR_CUDA;
    };
    for (size_t c = first_plain_chunk; loop_rc == FMM_OK; ++c) {
      if (c == chunks.size()) {
        if (next_gauge >= G) break;
        // the encode stream reads the tables first; products and decode follow it
        if ((loop_rc = build_group(sE)) != FMM_OK) break;
      }
      loop_rc = step(c);
    }
    // join: the caller's stream continues after everything enqueued on the library's streams
    bool joined = stream_wait(side, sD, st) && stream_wait(side, sE, st);
    if (sG != st) joined = stream_wait(side, sG, st) && joined;
    if (!joined) {   // last resort: nothing may still run on streams the caller cannot see
      cudaStreamSynchronize(sE); cudaStreamSynchronize(sD); cudaStreamSynchronize(sG);
      if (loop_rc == FMM_OK) loop_rc = FMM_ERR_CUDA;
    }
  }
  if (loop_rc != FMM_OK) return loop_rc;

  // 5. results to the host
  std::vector<double> h((size_t)G + 8);
  DeviceStatus hs_g, hs_g2, hs_c;
  FMM_CUDA(cudaMemcpyAsync(h.data(), sums, h.size() * 8, cudaMemcpyDeviceToHost, st));
  FMM_CUDA(cudaMemcpyAsync(&hs_g, at<char>(gws, L.g.status), sizeof(DeviceStatus), cudaMemcpyDeviceToHost, st));
  FMM_CUDA(cudaMemcpyAsync(&hs_g2, at<char>(ws + L.gemm2, L.g.status), sizeof(DeviceStatus), cudaMemcpyDeviceToHost, st));
  FMM_CUDA(cudaMemcpyAsync(&hs_c, at<char>(cws, L.c.status), sizeof(DeviceStatus), cudaMemcpyDeviceToHost, st));
  FMM_CUDA(cudaStreamSynchronize(st));
  if (hs_g.code != 0 || hs_g2.code != 0 || hs_c.code != 0) return FMM_ERR_TIMEOUT;

  const double nref = h[0], ecl = h[1];
  std::vector<double> rho(G);
  for (int g = 0; g < G; ++g) {
    const double eg = h[8 + g];
    rho[g] = (ecl == 0.0) ? (eg == 0.0 ? 1.0 : INFINITY) : std::sqrt(eg / ecl);
  }
  if (h_ratios) std::copy(rho.begin(), rho.end(), h_ratios);
  // NaN in the operands propagates into the ratios; a summary over a set that contains NaN is NaN (ordering NaN
  // with operator< is undefined), the count of ratios above 2 is taken over the comparable ones
  const bool any_nan = std::any_of(rho.begin(), rho.end(), [](double x) { return std::isnan(x); });
  if (any_nan) {
    out->min = out->max = out->median = out->spread = NAN;
  } else {
    std::vector<double> sorted = rho;
    std::sort(sorted.begin(), sorted.end());
    out->min = sorted.front();
    out->max = sorted.back();
    out->median = sorted[G / 2];  // upper of the two middle values when G is even
    out->spread = sorted.front() > 0 ? sorted.back() / sorted.front() : INFINITY;
  }
  out->count_gt2 = (int64_t)std::count_if(rho.begin(), rho.end(), [](double x) { return x > 2.0; });
  out->G = G;
  out->e_classical_rel = nref > 0 ? std::sqrt(ecl / nref) : 0.0;
  out->norm_ref = std::sqrt(nref);
  return FMM_OK;
}

}  // extern "C"
