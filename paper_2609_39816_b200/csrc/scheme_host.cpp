// Host side of the library: scheme handles, nesting, gauge transforms, criteria.
// Pure fp64 host code; needs no GPU.  (Section 2.1: coefficients and sign variants;
// Section 4.2: L_A, L_B, L_W; Appendix B.1: Phi, Q, E.)
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

#include "fmm_internal.h"

namespace {

inline double& at3(std::vector<double>& a, int r, int i, int j, int d1, int d2) { return a[(size_t)(r * d1 + i) * d2 + j]; }
inline double at3(const std::vector<double>& a, int r, int i, int j, int d1, int d2) { return a[(size_t)(r * d1 + i) * d2 + j]; }

double max_abs(const std::vector<double>& a) {
  double m = 0;
  for (double x : a) m = std::max(m, std::fabs(x));
  return m;
}

// Largest residual of sum_r u_{r,il} v_{r,l'j} w_{r,i'j'} - [i=i'][l=l'][j=j'].
double brent_residual(const fmm_scheme& s) {
  double worst = 0;
  const int m = s.m, k = s.k, n = s.n;
  for (int i = 0; i < m; ++i)
    for (int l = 0; l < k; ++l)
      for (int l2 = 0; l2 < k; ++l2)
        for (int j = 0; j < n; ++j)
          for (int i2 = 0; i2 < m; ++i2)
            for (int j2 = 0; j2 < n; ++j2) {
              double acc = 0;
              for (int r = 0; r < s.R; ++r)
                acc += at3(s.U, r, i, l, m, k) * at3(s.V, r, l2, j, k, n) * at3(s.W, r, i2, j2, m, n);
              const double want = (i == i2 && l == l2 && j == j2) ? 1.0 : 0.0;
              worst = std::max(worst, std::fabs(acc - want));
            }
  return worst;
}

bool dims_ok(int m, int k, int n, int R) {
  return m >= 1 && k >= 1 && n >= 1 && R >= 1 && m <= FMM_MAX_GRID && k <= FMM_MAX_GRID && n <= FMM_MAX_GRID &&
         R <= FMM_MAX_R;
}

std::unique_ptr<fmm_scheme> clone(const fmm_scheme& s) {
  std::unique_ptr<fmm_scheme> c(new fmm_scheme);
  c->m = s.m; c->k = s.k; c->n = s.n; c->R = s.R;
  c->U = s.U; c->V = s.V; c->W = s.W;
  if (s.outer) c->outer = clone(*s.outer);
  if (s.inner) c->inner = clone(*s.inner);
  return c;
}

// LU with partial pivoting on a d x d matrix (d <= 4): inverse, or false if singular.
bool invert(int d, const double* X, double* Xi) {
  double a[FMM_MAX_GRID][2 * FMM_MAX_GRID];
  for (int i = 0; i < d; ++i)
    for (int j = 0; j < d; ++j) { a[i][j] = X[i * d + j]; a[i][d + j] = (i == j); }
  for (int c = 0; c < d; ++c) {
    int p = c;
    for (int i = c + 1; i < d; ++i) if (std::fabs(a[i][c]) > std::fabs(a[p][c])) p = i;
    if (a[p][c] == 0.0 || !std::isfinite(a[p][c])) return false;
    if (p != c) for (int j = 0; j < 2 * d; ++j) std::swap(a[c][j], a[p][j]);
    const double inv = 1.0 / a[c][c];
    for (int j = 0; j < 2 * d; ++j) a[c][j] *= inv;
    for (int i = 0; i < d; ++i) {
      if (i == c || a[i][c] == 0.0) continue;
      const double f = a[i][c];
      for (int j = 0; j < 2 * d; ++j) a[i][j] -= f * a[c][j];
    }
  }
  for (int i = 0; i < d; ++i) for (int j = 0; j < d; ++j) Xi[i * d + j] = a[i][d + j];
  return true;
}

// 2-norm condition number: sqrt(lambda_max / lambda_min) of X^T X by cyclic Jacobi.
double cond2(int d, const double* X) {
  double g[FMM_MAX_GRID][FMM_MAX_GRID];
  for (int i = 0; i < d; ++i)
    for (int j = 0; j < d; ++j) {
      double s = 0;
      for (int t = 0; t < d; ++t) s += X[t * d + i] * X[t * d + j];
      g[i][j] = s;
    }
  for (int sweep = 0; sweep < 64; ++sweep) {
    double off = 0;
    for (int i = 0; i < d; ++i) for (int j = i + 1; j < d; ++j) off += g[i][j] * g[i][j];
    if (off < 1e-300) break;
    for (int p = 0; p < d; ++p)
      for (int q = p + 1; q < d; ++q) {
        if (g[p][q] == 0.0) continue;
        const double theta = (g[q][q] - g[p][p]) / (2.0 * g[p][q]);
        const double t = (theta >= 0 ? 1.0 : -1.0) / (std::fabs(theta) + std::sqrt(theta * theta + 1.0));
        const double c = 1.0 / std::sqrt(t * t + 1.0), sn = t * c;
        for (int x = 0; x < d; ++x) {  // columns
          const double gp = g[x][p], gq = g[x][q];
          g[x][p] = c * gp - sn * gq; g[x][q] = sn * gp + c * gq;
        }
        for (int x = 0; x < d; ++x) {  // rows
          const double gp = g[p][x], gq = g[q][x];
          g[p][x] = c * gp - sn * gq; g[q][x] = sn * gp + c * gq;
        }
      }
  }
  double lo = g[0][0], hi = g[0][0];
  for (int i = 1; i < d; ++i) { lo = std::min(lo, g[i][i]); hi = std::max(hi, g[i][i]); }
  if (!(lo > 0)) return INFINITY;
  return std::sqrt(hi / lo);
}

// out = gauge of a flat scheme s by P (m x m), Q (k x k), S (n x n).
fmm_status gauge_flat(const fmm_scheme& s, const double* P, const double* Q, const double* S, double cond_limit,
                      fmm_scheme* out) {
  const int m = s.m, k = s.k, n = s.n;
  double Pi[16], Qi[16], Si[16];
  if (!invert(m, P, Pi) || !invert(k, Q, Qi) || !invert(n, S, Si)) return FMM_ERR_SINGULAR;
  if (cond_limit > 0 && (cond2(m, P) > cond_limit || cond2(k, Q) > cond_limit || cond2(n, S) > cond_limit))
    return FMM_ERR_SINGULAR;
  out->m = m; out->k = k; out->n = n; out->R = s.R;
  out->U.assign(s.U.size(), 0.0); out->V.assign(s.V.size(), 0.0); out->W.assign(s.W.size(), 0.0);
  for (int r = 0; r < s.R; ++r) {
    for (int a = 0; a < m; ++a)      // U'_r = P^T U_r Q^-T
      for (int b = 0; b < k; ++b) {
        double acc = 0;
        for (int i = 0; i < m; ++i) for (int l = 0; l < k; ++l) acc += P[i * m + a] * at3(s.U, r, i, l, m, k) * Qi[b * k + l];
        at3(out->U, r, a, b, m, k) = acc;
      }
    for (int a = 0; a < k; ++a)      // V'_r = Q^T V_r S^-T
      for (int b = 0; b < n; ++b) {
        double acc = 0;
        for (int l = 0; l < k; ++l) for (int j = 0; j < n; ++j) acc += Q[l * k + a] * at3(s.V, r, l, j, k, n) * Si[b * n + j];
        at3(out->V, r, a, b, k, n) = acc;
      }
    for (int a = 0; a < m; ++a)      // W'_r = P^-1 W_r S
      for (int b = 0; b < n; ++b) {
        double acc = 0;
        for (int i = 0; i < m; ++i) for (int j = 0; j < n; ++j) acc += Pi[a * m + i] * at3(s.W, r, i, j, m, n) * S[j * n + b];
        at3(out->W, r, a, b, m, n) = acc;
      }
  }
  return FMM_OK;
}

void kron_into(const fmm_scheme& o, const fmm_scheme& in, fmm_scheme* out) {
  const int m = o.m * in.m, k = o.k * in.k, n = o.n * in.n, R = o.R * in.R;
  out->m = m; out->k = k; out->n = n; out->R = R;
  out->U.assign((size_t)R * m * k, 0.0); out->V.assign((size_t)R * k * n, 0.0); out->W.assign((size_t)R * m * n, 0.0);
  for (int r1 = 0; r1 < o.R; ++r1)
    for (int r2 = 0; r2 < in.R; ++r2) {
      const int r = r1 * in.R + r2;
      for (int I = 0; I < o.m; ++I) for (int i = 0; i < in.m; ++i)
        for (int L = 0; L < o.k; ++L) for (int l = 0; l < in.k; ++l)
          at3(out->U, r, I * in.m + i, L * in.k + l, m, k) = at3(o.U, r1, I, L, o.m, o.k) * at3(in.U, r2, i, l, in.m, in.k);
      for (int L = 0; L < o.k; ++L) for (int l = 0; l < in.k; ++l)
        for (int J = 0; J < o.n; ++J) for (int j = 0; j < in.n; ++j)
          at3(out->V, r, L * in.k + l, J * in.n + j, k, n) = at3(o.V, r1, L, J, o.k, o.n) * at3(in.V, r2, l, j, in.k, in.n);
      for (int I = 0; I < o.m; ++I) for (int i = 0; i < in.m; ++i)
        for (int J = 0; J < o.n; ++J) for (int j = 0; j < in.n; ++j)
          at3(out->W, r, I * in.m + i, J * in.n + j, m, n) = at3(o.W, r1, I, J, o.m, o.n) * at3(in.W, r2, i, j, in.m, in.n);
    }
}

void fill_strassen(fmm_scheme* s) {
  // Seven products and four outputs of the paper's Appendix A.1 table (0-based block indices):
  //   M1=(A00+A11)(B00+B11) M2=(A10+A11)B00 M3=A00(B01-B11) M4=A11(B10-B00)
  //   M5=(A00+A01)B11 M6=(A10-A00)(B00+B01) M7=(A01-A11)(B10+B11)
  //   C00=M1+M4-M5+M7 C01=M3+M5 C10=M2+M4 C11=M1-M2+M3+M6
  static const signed char u[7][4] = {{1, 0, 0, 1}, {0, 0, 1, 1}, {1, 0, 0, 0}, {0, 0, 0, 1}, {1, 1, 0, 0}, {-1, 0, 1, 0}, {0, 1, 0, -1}};
  static const signed char v[7][4] = {{1, 0, 0, 1}, {1, 0, 0, 0}, {0, 1, 0, -1}, {-1, 0, 1, 0}, {0, 0, 0, 1}, {1, 1, 0, 0}, {0, 0, 1, 1}};
  static const signed char w[7][4] = {{1, 0, 0, 1}, {0, 0, 1, -1}, {0, 1, 0, 1}, {1, 0, 1, 0}, {-1, 1, 0, 0}, {0, 0, 0, 1}, {1, 0, 0, 0}};
  s->m = s->k = s->n = 2; s->R = 7;
  s->U.resize(28); s->V.resize(28); s->W.resize(28);
  for (int r = 0; r < 7; ++r)
    for (int x = 0; x < 4; ++x) { s->U[r * 4 + x] = u[r][x]; s->V[r * 4 + x] = v[r][x]; s->W[r * 4 + x] = w[r][x]; }
}

void fill_classical(fmm_scheme* s, int m, int k, int n) {
  s->m = m; s->k = k; s->n = n; s->R = m * k * n;
  s->U.assign((size_t)s->R * m * k, 0.0); s->V.assign((size_t)s->R * k * n, 0.0); s->W.assign((size_t)s->R * m * n, 0.0);
  int r = 0;
  for (int i = 0; i < m; ++i) for (int l = 0; l < k; ++l) for (int j = 0; j < n; ++j, ++r) {
    at3(s->U, r, i, l, m, k) = 1; at3(s->V, r, l, j, k, n) = 1; at3(s->W, r, i, j, m, n) = 1;
  }
}

}  // namespace

// Lists are padded to a multiple of kTablePad entries with (pad slab, 0.0f): the kernels walk them in
// fixed chunks, and a padding entry multiplies a slab of zeros by zero, which adds exactly nothing.
namespace {
struct ListBuilder {
  CoefTable* t;
  int c = 0, lists = 0;
  ListBuilder(CoefTable* tab, int nlists, int nslabs) : t(tab) { t->R = nlists; t->ncell = nslabs; t->off[0] = 0; }
  void add(int slab, float f) { if (f != 0.0f) { t->cell[c] = slab; t->coef[c] = f; ++c; } }
  void close() {
    while (c % kTablePad) { t->cell[c] = t->ncell; t->coef[c] = 0.0f; ++c; }
    t->off[++lists] = c;
  }
};
}  // namespace

void fmm_build_tables(const fmm_scheme& s, CoefTable* tA, CoefTable* tB, CoefTable* tW) {
  const int m = s.m, k = s.k, n = s.n;
  if (tA) {
    ListBuilder b(tA, s.R, m * k);
    for (int r = 0; r < s.R; ++r) {
      for (int i = 0; i < m; ++i) for (int l = 0; l < k; ++l) b.add(i * k + l, (float)at3(s.U, r, i, l, m, k));
      b.close();
    }
  }
  if (tB) {  // source is B^T stored [N x K]: block (l,j) of B is cell j*k + l; order ascending (l,j)
    ListBuilder b(tB, s.R, n * k);
    for (int r = 0; r < s.R; ++r) {
      for (int l = 0; l < k; ++l) for (int j = 0; j < n; ++j) b.add(j * k + l, (float)at3(s.V, r, l, j, k, n));
      b.close();
    }
  }
  if (tW) {  // cell-major: list x = i*n+j holds the (r, w_{r,ij}) pairs feeding C block (i,j), ascending r
    ListBuilder b(tW, m * n, s.R);
    for (int i = 0; i < m; ++i) for (int j = 0; j < n; ++j) {
      for (int r = 0; r < s.R; ++r) b.add(r, (float)at3(s.W, r, i, j, m, n));
      b.close();
    }
  }
}

size_t fmm_packed_table_stride() { return (sizeof(CoefTable) + kPackedAlign - 1) / kPackedAlign * kPackedAlign; }

const std::vector<unsigned char>& fmm_packed_tables(const fmm_scheme& s) {
  std::call_once(s.tables_once, [&s] {
    const size_t stride = fmm_packed_table_stride();
    s.packed_tables.assign(kPackedStatusBytes + 3 * stride, 0);
    CoefTable* t = reinterpret_cast<CoefTable*>(s.packed_tables.data() + kPackedStatusBytes);
    auto tab = [&](int w) { return reinterpret_cast<CoefTable*>(reinterpret_cast<unsigned char*>(t) + w * stride); };
    fmm_build_tables(s, tab(0), tab(1), tab(2));
  });
  return s.packed_tables;
}

const CoefTable* fmm_packed_table(const fmm_scheme& s, int which) {
  return reinterpret_cast<const CoefTable*>(fmm_packed_tables(s).data() + kPackedStatusBytes + which * fmm_packed_table_stride());
}

bool fmm_gauge_invertible(int m, int k, int n, const double* P, const double* Q, const double* S) {
  double inv[FMM_MAX_GRID * FMM_MAX_GRID];
  if (m < 1 || k < 1 || n < 1 || m > FMM_MAX_GRID || k > FMM_MAX_GRID || n > FMM_MAX_GRID) return false;
  return invert(m, P, inv) && invert(k, Q, inv) && invert(n, S, inv);
}

fmm_status fmm_gauge_core(const fmm_scheme& in, int level, const double* P, const double* Q, const double* S,
                          double cond_limit, fmm_scheme** out) {
  std::unique_ptr<fmm_scheme> res(new (std::nothrow) fmm_scheme);
  if (!res) return FMM_ERR_ARG;
  if (level == 0) {
    fmm_status st = gauge_flat(in, P, Q, S, cond_limit, res.get());
    if (st != FMM_OK) return st;
  } else if (level == 1) {
    if (!in.outer || !in.inner) return FMM_ERR_ARG;
    std::unique_ptr<fmm_scheme> go(new fmm_scheme);
    fmm_status st = gauge_flat(*in.outer, P, Q, S, cond_limit, go.get());
    if (st != FMM_OK) return st;
    kron_into(*go, *in.inner, res.get());
    res->outer = std::move(go);
    res->inner = clone(*in.inner);
  } else {
    return FMM_ERR_ARG;
  }
  *out = res.release();
  return FMM_OK;
}

extern "C" {

fmm_status scheme_load(int m, int k, int n, int R, const double* U, const double* V, const double* W,
                       double brent_tol, fmm_scheme** out) {
  if (!U || !V || !W || !out) return FMM_ERR_ARG;
  if (m < 1 || k < 1 || n < 1 || R < 1) return FMM_ERR_ARG;
  if (!dims_ok(m, k, n, R)) return FMM_ERR_LIMIT;
  std::unique_ptr<fmm_scheme> s(new (std::nothrow) fmm_scheme);
  if (!s) return FMM_ERR_ARG;
  s->m = m; s->k = k; s->n = n; s->R = R;
  s->U.assign(U, U + (size_t)R * m * k);
  s->V.assign(V, V + (size_t)R * k * n);
  s->W.assign(W, W + (size_t)R * m * n);
  for (const auto* vec : {&s->U, &s->V, &s->W})
    for (double x : *vec) if (!std::isfinite(x)) return FMM_ERR_ARG;
  const double tol = (brent_tol > 0 ? brent_tol : 1e-12) *
                     std::max(1.0, R * max_abs(s->U) * max_abs(s->V) * max_abs(s->W));
  if (!(brent_residual(*s) <= tol)) return FMM_ERR_BRENT;
  *out = s.release();
  return FMM_OK;
}

fmm_status scheme_builtin(const char* name, fmm_scheme** out) {
  if (!name || !out) return FMM_ERR_ARG;
  std::unique_ptr<fmm_scheme> s(new (std::nothrow) fmm_scheme);
  if (!s) return FMM_ERR_ARG;
  if (!std::strcmp(name, "strassen222")) {
    fill_strassen(s.get());
  } else if (!std::strcmp(name, "strassen444")) {
    std::unique_ptr<fmm_scheme> a(new fmm_scheme), b(new fmm_scheme);
    fill_strassen(a.get()); fill_strassen(b.get());
    kron_into(*a, *b, s.get());
    s->outer = std::move(a); s->inner = std::move(b);
  } else if (!std::strcmp(name, "classical111")) {
    fill_classical(s.get(), 1, 1, 1);
  } else if (!std::strcmp(name, "classical222")) {
    fill_classical(s.get(), 2, 2, 2);
  } else {
    return FMM_ERR_ARG;
  }
  *out = s.release();
  return FMM_OK;
}

fmm_status scheme_kron(const fmm_scheme* outer, const fmm_scheme* inner, fmm_scheme** out) {
  if (!outer || !inner || !out) return FMM_ERR_ARG;
  if (!dims_ok(outer->m * inner->m, outer->k * inner->k, outer->n * inner->n, outer->R * inner->R)) return FMM_ERR_LIMIT;
  std::unique_ptr<fmm_scheme> s(new (std::nothrow) fmm_scheme);
  if (!s) return FMM_ERR_ARG;
  kron_into(*outer, *inner, s.get());
  s->outer = clone(*outer);
  s->inner = clone(*inner);
  s->outer->outer.reset(); s->outer->inner.reset();
  s->inner->outer.reset(); s->inner->inner.reset();
  *out = s.release();
  return FMM_OK;
}

fmm_status scheme_permute_products(const fmm_scheme* in, const int* perm, fmm_scheme** out) {
  if (!in || !perm || !out) return FMM_ERR_ARG;
  const int R = in->R, m = in->m, k = in->k, n = in->n;
  std::vector<char> seen(R, 0);
  for (int r = 0; r < R; ++r) {
    if (perm[r] < 0 || perm[r] >= R || seen[perm[r]]) return FMM_ERR_ARG;
    seen[perm[r]] = 1;
  }
  std::unique_ptr<fmm_scheme> s(new (std::nothrow) fmm_scheme);
  if (!s) return FMM_ERR_ARG;
  s->m = m; s->k = k; s->n = n; s->R = R;
  s->U.resize(in->U.size()); s->V.resize(in->V.size()); s->W.resize(in->W.size());
  for (int r = 0; r < R; ++r) {   // product r of the result is product perm[r] of the input
    std::copy_n(in->U.begin() + (size_t)perm[r] * m * k, (size_t)m * k, s->U.begin() + (size_t)r * m * k);
    std::copy_n(in->V.begin() + (size_t)perm[r] * k * n, (size_t)k * n, s->V.begin() + (size_t)r * k * n);
    std::copy_n(in->W.begin() + (size_t)perm[r] * m * n, (size_t)m * n, s->W.begin() + (size_t)r * m * n);
  }
  *out = s.release();
  return FMM_OK;
}

fmm_status gauge_apply(const fmm_scheme* in, int level, const double* P, const double* Q, const double* S,
                       double cond_limit, fmm_scheme** out) {
  if (!in || !P || !Q || !S || !out) return FMM_ERR_ARG;
  return fmm_gauge_core(*in, level, P, Q, S, cond_limit, out);
}

fmm_status scheme_info(const fmm_scheme* s, int dims[4], double meta[8]) {
  if (!s) return FMM_ERR_ARG;
  if (dims) { dims[0] = s->m; dims[1] = s->k; dims[2] = s->n; dims[3] = s->R; }
  if (meta) {
    const int m = s->m, k = s->k, n = s->n, R = s->R;
    std::vector<double> a1(R, 0.0), b1(R, 0.0), al(R, 0.0), be(R, 0.0);
    double LA = 0, LB = 0, LW = 0, Phi = 0, nnz = 0, mx = 0, Qc = 0, Ec = 0;
    for (int r = 0; r < R; ++r) {
      double u2 = 0, v2 = 0, w2 = 0;
      for (int x = 0; x < m * k; ++x) { const double c = s->U[(size_t)r * m * k + x]; a1[r] += std::fabs(c); u2 += c * c; if (c != 0) { al[r] += 1; nnz += 1; } }
      for (int x = 0; x < k * n; ++x) { const double c = s->V[(size_t)r * k * n + x]; b1[r] += std::fabs(c); v2 += c * c; if (c != 0) { be[r] += 1; nnz += 1; } }
      for (int x = 0; x < m * n; ++x) { const double c = s->W[(size_t)r * m * n + x]; w2 += c * c; if (c != 0) nnz += 1; }
      LA = std::max(LA, a1[r]); LB = std::max(LB, b1[r]);
      Phi += u2 * v2 * w2;
    }
    mx = std::max({max_abs(s->U), max_abs(s->V), max_abs(s->W)});
    for (int x = 0; x < m * n; ++x) {
      double lw = 0, gamma = 0, ab = 0, e = 0;
      for (int r = 0; r < R; ++r) {
        const double c = s->W[(size_t)r * m * n + x];
        lw += std::fabs(c); e += a1[r] * b1[r] * std::fabs(c);
        if (c != 0) { gamma += 1; ab = std::max(ab, al[r] + be[r]); }
      }
      LW = std::max(LW, lw); Qc = std::max(Qc, gamma + ab); Ec = std::max(Ec, e);
    }
    meta[0] = LA; meta[1] = LB; meta[2] = LW; meta[3] = Phi; meta[4] = nnz; meta[5] = mx; meta[6] = Qc; meta[7] = Ec;
  }
  return FMM_OK;
}

fmm_status scheme_coefficients(const fmm_scheme* s, double* U, double* V, double* W) {
  if (!s) return FMM_ERR_ARG;
  if (U) std::copy(s->U.begin(), s->U.end(), U);
  if (V) std::copy(s->V.begin(), s->V.end(), V);
  if (W) std::copy(s->W.begin(), s->W.end(), W);
  return FMM_OK;
}

void scheme_free(fmm_scheme* s) { delete s; }

const char* fmm_status_string(fmm_status st) {
  switch (st) {
    case FMM_OK: return "ok";
    case FMM_ERR_ARG: return "bad argument";
    case FMM_ERR_SHAPE: return "shape or alignment not supported";
    case FMM_ERR_BRENT: return "coefficients violate the Brent equations";
    case FMM_ERR_SINGULAR: return "gauge matrix singular or ill-conditioned";
    case FMM_ERR_DTYPE: return "dtype combination not supported";
    case FMM_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case FMM_ERR_CUDA: return "CUDA call failed";
    case FMM_ERR_TIMEOUT: return "device-side wait timed out";
    case FMM_ERR_LIMIT: return "scheme exceeds table limits";
    case FMM_ERR_CERTIFICATE: return "exactness certificate does not hold";
  }
  return "unknown status";
}

}  // extern "C"
