// Internal declarations shared by the translation units of libfmm_b200 (not installed).
#pragma once
#include <cstdint>
#include <memory>
#include <vector>

#include "fmm_b200.h"

constexpr int kMaxCells = FMM_MAX_GRID * FMM_MAX_GRID;  // blocks in one operand grid
constexpr int kMaxNnz = FMM_MAX_R * kMaxCells;          // entries in one table (padding included)
constexpr int kTablePad = 2;                            // every list is padded to a multiple of this

struct fmm_scheme {
  int m = 0, k = 0, n = 0, R = 0;
  std::vector<double> U, V, W;                 // [R][m][k], [R][k][n], [R][m][n]
  std::unique_ptr<fmm_scheme> outer, inner;    // factors, when built by scheme_kron
};

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
fmm_status fmm_gauge_core(const fmm_scheme& in, int level, const double* P, const double* Q, const double* S,
                          double cond_limit, fmm_scheme** out);
