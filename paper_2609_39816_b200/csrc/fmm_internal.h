// Internal declarations shared by the translation units of libfmm_b200 (not installed).
#pragma once
#include <cstdint>
#include <memory>
#include <mutex>
#include <vector>

#include "fmm_b200.h"

constexpr int kMaxCells = FMM_MAX_GRID * FMM_MAX_GRID;  // blocks in one operand grid
constexpr int kMaxNnz = FMM_MAX_R * kMaxCells;          // entries in one table (padding included)
constexpr int kTablePad = 2;                            // every list is padded to a multiple of this

struct CoefTable;

struct fmm_scheme {
  int m = 0, k = 0, n = 0, R = 0;
  std::vector<double> U, V, W;                 // [R][m][k], [R][k][n], [R][m][n]
  std::unique_ptr<fmm_scheme> outer, inner;    // factors, when built by scheme_kron
  // Kernel tables of this scheme, built once on first use (a handle's coefficients never change): a zeroed
  // device-status block followed by the encode-A, encode-B and decode tables, laid out exactly as the head of a
  // scheme_gemm workspace so that one copy uploads all of it.
  mutable std::once_flag tables_once;
  mutable std::vector<unsigned char> packed_tables;
};

// Offsets inside fmm_scheme::packed_tables (and inside the head of a scheme_gemm workspace).
constexpr size_t kPackedAlign = 1024;           // alignment of every region of a workspace
constexpr size_t kPackedStatusBytes = 1024;     // the status block's slot (the block itself is 256 bytes)
size_t fmm_packed_table_stride();              // sizeof(CoefTable) rounded up to kPackedAlign
const std::vector<unsigned char>& fmm_packed_tables(const fmm_scheme& s);
const CoefTable* fmm_packed_table(const fmm_scheme& s, int which);   // 0: A, 1: B, 2: W (host copies)

// Sparse coefficient table as the kernels read it: R lists of (slab, coefficient) pairs in the order in
// which they are to be accumulated, each list padded to a multiple of kTablePad with (ncell, 0.0f).
// Encode tables: one list per product, slab = flat index of a block in the SOURCE matrix's grid as stored
// in memory, ncell = number of blocks.  Decode table: one list per C block (cell-major), slab = product
// index r (ascending), ncell = number of products.
struct CoefTable {
  int32_t R;       // number of lists
  int32_t ncell;   // number of data slabs; index ncell is the all-zero padding slab
  int32_t off[FMM_MAX_R + 1];
  int32_t cell[kMaxNnz];
  float coef[kMaxNnz];
};

// host helpers (scheme_host.cpp)
// tA: cells of A's m x k grid; tB: cells of B^T's n x k grid (B is always read K-major), entries in
// ascending (l,j) order of V; tW: cell-major decode table (R field = m*n lists, `cell` = product index r,
// ascending).  Any pointer may be null.
void fmm_build_tables(const fmm_scheme& s, CoefTable* tA, CoefTable* tB, CoefTable* tW);
// true when P (m x m), Q (k x k) and S (n x n) can all be inverted (the test gauge_apply / fmm_gauge_core apply)
bool fmm_gauge_invertible(int m, int k, int n, const double* P, const double* Q, const double* S);
fmm_status fmm_gauge_core(const fmm_scheme& in, int level, const double* P, const double* Q, const double* S,
                          double cond_limit, fmm_scheme** out);
