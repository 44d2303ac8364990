// Internal declarations shared by the translation units of libfmm_b200 (not installed).
#pragma once
#include <cstdint>
#include <memory>
#include <vector>

#include "fmm_b200.h"

constexpr int kMaxCells = FMM_MAX_GRID * FMM_MAX_GRID;  // blocks in one operand grid
constexpr int kMaxNnz = FMM_MAX_R * kMaxCells;          // nonzero coefficients in one table

struct fmm_scheme {
  int m = 0, k = 0, n = 0, R = 0;
  std::vector<double> U, V, W;                 // [R][m][k], [R][k][n], [R][m][n]
  std::unique_ptr<fmm_scheme> outer, inner;    // factors, when built by scheme_kron
};

// Sparse coefficient table as the kernels read it: for each product r the nonzero
// (cell, coefficient) pairs, in the order in which they are to be accumulated.
// For the encode tables `cell` is the flat index of a block in the SOURCE matrix's
// grid as stored in memory; for the decode table it is the flat index i*n+j of a C block.
struct CoefTable {
  int32_t R;
  int32_t ncell;
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
