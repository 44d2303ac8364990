"""Python face of the CPU oracle: ctypes over ``fmm_oracle.c`` plus the few host-side
definitions that are clearer in numpy (the printed Strassen table, the sign-variant
formula as printed, the summary statistics).

TEST INFRASTRUCTURE ONLY — see the header of ``fmm_oracle.c``.  Nothing here imports
the CUDA library; the library never imports this.

Citations are to the paper's sections / equations / tables.
"""
from __future__ import annotations

import ctypes as C
import math
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fmm_oracle.c")
_SO = os.path.join(_HERE, "libfmm_oracle.so")

F32, BF16, E4M3, F64 = 0, 1, 2, 3
_FMT = {"f32": F32, "fp32": F32, "bf16": BF16, "e4m3": E4M3, "f64": F64, "fp64": F64}

__all__ = [
    "F32", "BF16", "E4M3", "F64", "Scheme", "build", "num_threads", "set_num_threads", "round_to", "strassen",
    "classical_scheme", "kron", "gauge", "sign_variant", "sign_variants", "brent_residual",
    "criteria", "scheme_gemm", "scheme_gemm_per_level", "classical_gemm", "exact_gemm", "fro_err", "rel_error",
    "error_ratio", "summary", "quantize_rows", "int8_classical", "int8_certified", "int8_corrected", "int8_finegroup_control", "certificate",
    "hadamard_matrix", "hadamard_rotate", "row_pow2_scales", "joint_round_weights", "scheme_gemm_weights",
]


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, no FP contraction)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O3", "-march=x86-64-v3", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-shared", "-fPIC", "-std=c11", "-o", _SO, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


_lib = None


def _L():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        dp = C.POINTER(C.c_double)
        i64 = C.c_int64
        lib.orc_num_threads.restype = C.c_int
        lib.orc_set_num_threads.argtypes = [C.c_int]
        lib.orc_round.restype = C.c_double
        lib.orc_round.argtypes = [C.c_double, C.c_int]
        lib.orc_round_array.argtypes = [dp, dp, i64, C.c_int]
        lib.orc_brent_max_residual.restype = C.c_double
        lib.orc_brent_max_residual.argtypes = [C.c_int] * 4 + [dp] * 3
        lib.orc_kron.argtypes = [C.c_int] * 4 + [dp] * 3 + [C.c_int] * 4 + [dp] * 3 + [dp] * 3
        lib.orc_gauge.restype = C.c_int
        lib.orc_gauge.argtypes = [C.c_int] * 4 + [dp] * 9
        lib.orc_criteria.argtypes = [C.c_int] * 4 + [dp] * 4
        lib.orc_scheme_gemm.restype = C.c_int
        lib.orc_scheme_gemm.argtypes = ([C.c_int] * 4 + [dp] * 3 + [i64] * 3 + [dp] * 2 +
                                        [C.c_int] * 3 + [dp] * 6 + [C.c_int])
        lib.orc_scheme_gemm_sum.restype = C.c_int
        lib.orc_scheme_gemm_sum.argtypes = ([C.c_int] * 4 + [dp] * 3 + [i64] * 3 + [dp] * 2 +
                                            [C.c_int] * 3 + [dp] * 6 + [C.c_int] * 2)
        lib.orc_scheme_gemm_per_level.restype = C.c_int
        lib.orc_scheme_gemm_per_level.argtypes = ([C.c_int] * 4 + [dp] * 3 + [C.c_int] * 4 + [dp] * 3 + [i64] * 3 +
                                                  [dp] * 2 + [C.c_int] * 4 + [dp] * 6)
        lib.orc_classical_gemm.restype = C.c_int
        lib.orc_classical_gemm.argtypes = [i64] * 3 + [dp] * 2 + [C.c_int] * 3 + [dp]
        lib.orc_exact_gemm.argtypes = [i64] * 3 + [dp] * 3
        lib.orc_fro_err.argtypes = [dp, dp, i64, dp]
        lib.orc_quantize_rows.argtypes = [dp, i64, i64, C.c_int, C.c_int, dp, dp]
        lib.orc_int8_classical.argtypes = [dp] * 4 + [i64] * 3 + [C.c_int] * 2 + [dp] * 2
        lib.orc_int8_certified.restype = C.c_int
        lib.orc_int8_certified.argtypes = ([C.c_int] * 4 + [dp] * 3 + [dp] * 4 + [i64] * 3 + [C.c_int] * 2 + [dp] * 3)
        lib.orc_int8_corrected.restype = C.c_int
        lib.orc_int8_corrected.argtypes = ([C.c_int] * 4 + [dp] * 3 + [dp] * 4 + [i64] * 3 + [C.c_int] * 2 + [dp] * 3)
        lib.orc_scheme_gemm_weights.restype = C.c_int
        lib.orc_scheme_gemm_weights.argtypes = ([C.c_int] * 4 + [dp] * 3 + [i64] * 3 + [dp] * 2 + [C.c_int] * 2 +
                                                [dp] * 2 + [C.c_int] + [dp] * 2)
        lib.orc_joint_round.restype = C.c_int
        lib.orc_joint_round.argtypes = [C.c_int] * 4 + [dp] * 3 + [i64] * 2 + [dp] + [C.c_int] + [dp] * 3
        lib.orc_int8_finegroup_control.restype = C.c_int
        lib.orc_int8_finegroup_control.argtypes = [C.c_int] * 4 + [dp] * 3 + [dp] * 4 + [i64] * 3 + [C.c_int] * 3 + [dp]
        lib.orc_certificate.restype = C.c_int
        lib.orc_certificate.argtypes = [C.c_int] * 4 + [dp] * 3 + [C.c_int] * 5 + [dp]
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.POINTER(C.c_double))


def _d(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _fmt(f):
    return _FMT[f] if isinstance(f, str) else int(f)


def num_threads() -> int:
    return int(_L().orc_num_threads())


def set_num_threads(n: int) -> None:
    """Threads of the oracle's OpenMP loops (results do not depend on it)."""
    _L().orc_set_num_threads(int(n))


def round_to(x, fmt):
    """Round real value(s) to a storage format (round to nearest even; e4m3 saturates)."""
    x = _d(x)
    y = np.empty_like(x)
    _L().orc_round_array(_p(x), _p(y), x.size, _fmt(fmt))
    return y


@dataclass(frozen=True)
class Scheme:
    """Coefficients of Eq. 1: U[R,m,k], V[R,k,n], W[R,m,n] (w indexed by the C block it feeds)."""
    U: np.ndarray
    V: np.ndarray
    W: np.ndarray

    @property
    def dims(self):
        R, m, k = self.U.shape
        return m, k, self.V.shape[2], R


def strassen() -> Scheme:
    """Strassen's <2,2,2;7>, typed from the product table of Appendix A.1:
    M1=(A11+A22)(B11+B22), M2=(A21+A22)B11, M3=A11(B12-B22), M4=A22(B21-B11),
    M5=(A11+A12)B22, M6=(A21-A11)(B11+B12), M7=(A12-A22)(B21+B22);
    C11=M1+M4-M5+M7, C12=M3+M5, C21=M2+M4, C22=M1-M2+M3+M6."""
    U = np.zeros((7, 2, 2)); V = np.zeros((7, 2, 2)); W = np.zeros((7, 2, 2))
    a = {(1, 1): (0, 0), (1, 2): (0, 1), (2, 1): (1, 0), (2, 2): (1, 1)}
    prods = [
        ([(1, 1, 1), (2, 2, 1)], [(1, 1, 1), (2, 2, 1)]),
        ([(2, 1, 1), (2, 2, 1)], [(1, 1, 1)]),
        ([(1, 1, 1)], [(1, 2, 1), (2, 2, -1)]),
        ([(2, 2, 1)], [(2, 1, 1), (1, 1, -1)]),
        ([(1, 1, 1), (1, 2, 1)], [(2, 2, 1)]),
        ([(2, 1, 1), (1, 1, -1)], [(1, 1, 1), (1, 2, 1)]),
        ([(1, 2, 1), (2, 2, -1)], [(2, 1, 1), (2, 2, 1)]),
    ]
    for r, (ua, vb) in enumerate(prods):
        for (i, l, s) in ua:
            U[(r,) + a[(i, l)]] = s
        for (l, j, s) in vb:
            V[(r,) + a[(l, j)]] = s
    outs = {(1, 1): [(1, 1), (4, 1), (5, -1), (7, 1)], (1, 2): [(3, 1), (5, 1)],
            (2, 1): [(2, 1), (4, 1)], (2, 2): [(1, 1), (2, -1), (3, 1), (6, 1)]}
    for ij, terms in outs.items():
        for (r, s) in terms:
            W[(r - 1,) + a[ij]] = s
    return Scheme(U, V, W)


def classical_scheme(m: int, k: int, n: int) -> Scheme:
    """The classical algorithm as a scheme: R = mkn products A_il B_lj (Section 2.1)."""
    R = m * k * n
    U = np.zeros((R, m, k)); V = np.zeros((R, k, n)); W = np.zeros((R, m, n))
    r = 0
    for i in range(m):
        for l in range(k):
            for j in range(n):
                U[r, i, l] = 1; V[r, l, j] = 1; W[r, i, j] = 1
                r += 1
    return Scheme(U, V, W)


def kron(outer: Scheme, inner: Scheme) -> Scheme:
    """Nested algorithm (outer applied to blocks multiplied by inner); contiguous blocks."""
    m1, k1, n1, R1 = outer.dims
    m2, k2, n2, R2 = inner.dims
    U = np.zeros((R1 * R2, m1 * m2, k1 * k2)); V = np.zeros((R1 * R2, k1 * k2, n1 * n2))
    W = np.zeros((R1 * R2, m1 * m2, n1 * n2))
    _L().orc_kron(m1, k1, n1, R1, _p(_d(outer.U)), _p(_d(outer.V)), _p(_d(outer.W)),
                  m2, k2, n2, R2, _p(_d(inner.U)), _p(_d(inner.V)), _p(_d(inner.W)),
                  _p(U), _p(V), _p(W))
    return Scheme(U, V, W)


def gauge(s: Scheme, P, Q, S) -> Scheme:
    """General gauge: U'_r = P^T U_r Q^-T, V'_r = Q^T V_r S^-T, W'_r = P^-1 W_r S."""
    m, k, n, R = s.dims
    U = np.empty_like(_d(s.U)); V = np.empty_like(_d(s.V)); W = np.empty_like(_d(s.W))
    rc = _L().orc_gauge(m, k, n, R, _p(_d(s.U)), _p(_d(s.V)), _p(_d(s.W)),
                        _p(_d(P)), _p(_d(Q)), _p(_d(S)), _p(U), _p(V), _p(W))
    if rc:
        raise ValueError("singular gauge matrix")
    return Scheme(U, V, W)


def sign_variant(s: Scheme, d, e, f) -> Scheme:
    """Sign variant exactly as Section 2.1 prints it: d_i e_l u, e_l f_j v, d_i f_j w."""
    d = np.asarray(d, float); e = np.asarray(e, float); f = np.asarray(f, float)
    U = s.U * d[None, :, None] * e[None, None, :]
    V = s.V * e[None, :, None] * f[None, None, :]
    W = s.W * d[None, :, None] * f[None, None, :]
    return Scheme(U, V, W)


def sign_variants(m: int, k: int, n: int):
    """All (d, e, f) with d_1 = e_1 = f_1 = 1 (Section 2.1): 2^(m-1) 2^(k-1) 2^(n-1) triples."""
    out = []
    for a in range(2 ** (m - 1)):
        d = [1.0] + [(-1.0 if (a >> b) & 1 else 1.0) for b in range(m - 1)]
        for bb in range(2 ** (k - 1)):
            e = [1.0] + [(-1.0 if (bb >> b) & 1 else 1.0) for b in range(k - 1)]
            for c in range(2 ** (n - 1)):
                f = [1.0] + [(-1.0 if (c >> b) & 1 else 1.0) for b in range(n - 1)]
                out.append((np.array(d), np.array(e), np.array(f)))
    return out


def brent_residual(s: Scheme) -> float:
    m, k, n, R = s.dims
    return float(_L().orc_brent_max_residual(m, k, n, R, _p(_d(s.U)), _p(_d(s.V)), _p(_d(s.W))))


def criteria(s: Scheme) -> dict:
    m, k, n, R = s.dims
    meta = np.zeros(8)
    _L().orc_criteria(m, k, n, R, _p(_d(s.U)), _p(_d(s.V)), _p(_d(s.W)), _p(meta))
    keys = ["L_A", "L_B", "L_W", "Phi", "nnz", "maxabs", "Q", "E"]
    return dict(zip(keys, meta.tolist()))


_SUM = {"f32chain": 0, "f64": 1}


def scheme_gemm(s: Scheme, A, B, pd="bf16", od="f32", scale_mode: int = 0, parts: bool = False, md="f64",
                sum: str = "f32chain"):
    """Apply the algorithm with block sums rounded to ``pd``; returns C (values of ``od``).  ``md``: dtype each
    product is rounded to before the combination ("f64": none; "bf16": the paper's model schedule).
    ``sum``: how a block sum is formed before its one rounding — "f64": the definition (fp64 sum of the products
    coefficient x entry); "f32chain": an fp32 fused-multiply-add chain in ascending block order, the reading under
    which quantised codes can be compared bit for bit with fp32 hardware.
    With ``parts`` also returns dict(Ahat, Bhat, sA, sB, M); ``parts="scales"`` fills only sA and sB."""
    m, k, n, R = s.dims
    A = _d(A); B = _d(B)
    M, K = A.shape
    K2, N = B.shape
    assert K == K2
    Cm = np.empty((M, N))
    Ah = Bh = sA = sB = Mr = None
    if parts:
        bm, bk, bn = M // m, K // k, N // n
        if parts != "scales":      # "scales": only the scale arrays (full-size problems, where the rest is gigabytes)
            Ah = np.empty((R, bm, bk)); Bh = np.empty((R, bk, bn)); Mr = np.empty((R, bm, bn))
        G3, CB3 = -(-bk // 128), -(-bn // 128)
        sA = np.empty({2: (R, bm), 3: (R, bm, G3)}.get(scale_mode, (R,)))
        sB = np.empty({2: (R, bn), 3: (R, CB3, G3)}.get(scale_mode, (R,)))
    rc = _L().orc_scheme_gemm_sum(m, k, n, R, _p(_d(s.U)), _p(_d(s.V)), _p(_d(s.W)), M, K, N, _p(A), _p(B),
                                  _fmt(pd), _fmt(od), int(scale_mode), _p(Cm), _p(Ah), _p(Bh), _p(sA),
                                  _p(sB), _p(Mr), _fmt(md), _SUM[sum])
    if rc:
        raise ValueError("matrix dimensions are not divisible by the block grid")
    if parts:
        return Cm, dict(Ahat=Ah, Bhat=Bh, sA=sA, sB=sB, M=Mr)
    return Cm


def scheme_gemm_per_level(outer: Scheme, inner: Scheme, A, B, pd="bf16", od="f32", scale_mode: int = 0,
                          parts: bool = False, sum: str = "f32chain"):
    """The nested algorithm outer (x) inner with the block sums rounded at EVERY level: the outer level's block
    sums are rounded to ``pd``, the inner level's block sums are formed of those rounded values and rounded again
    (Section 1, "applied to its own blocks", taken literally).  ``kron(outer, inner)`` through ``scheme_gemm`` is
    the flat reading (one rounding of each of the R1 R2 block sums).  scale_mode 0 or 1."""
    m1, k1, n1, R1 = outer.dims
    m2, k2, n2, R2 = inner.dims
    m, k, n, R = m1 * m2, k1 * k2, n1 * n2, R1 * R2
    A = _d(A); B = _d(B)
    M, K = A.shape
    K2, N = B.shape
    assert K == K2
    Cm = np.empty((M, N))
    Ah = Bh = sA = sB = Mr = None
    if parts:
        bm, bk, bn = M // m, K // k, N // n
        Ah = np.empty((R, bm, bk)); Bh = np.empty((R, bk, bn)); Mr = np.empty((R, bm, bn))
        sA = np.empty((R,)); sB = np.empty((R,))
    rc = _L().orc_scheme_gemm_per_level(m1, k1, n1, R1, _p(_d(outer.U)), _p(_d(outer.V)), _p(_d(outer.W)),
                                        m2, k2, n2, R2, _p(_d(inner.U)), _p(_d(inner.V)), _p(_d(inner.W)),
                                        M, K, N, _p(A), _p(B), _fmt(pd), _fmt(od), int(scale_mode), _SUM[sum],
                                        _p(Cm), _p(Ah), _p(Bh), _p(sA), _p(sB), _p(Mr))
    if rc:
        raise ValueError("dimensions not divisible by the block grid, or unsupported scale mode")
    if parts:
        return Cm, dict(Ahat=Ah, Bhat=Bh, sA=sA, sB=sB, M=Mr)
    return Cm


def classical_gemm(A, B, pd="bf16", od="f32", scale_mode: int = 0):
    A = _d(A); B = _d(B)
    M, K = A.shape
    N = B.shape[1]
    Cm = np.empty((M, N))
    _L().orc_classical_gemm(M, K, N, _p(A), _p(B), _fmt(pd), _fmt(od), int(scale_mode), _p(Cm))
    return Cm


def exact_gemm(A, B):
    A = _d(A); B = _d(B)
    M, K = A.shape
    N = B.shape[1]
    Cm = np.empty((M, N))
    _L().orc_exact_gemm(M, K, N, _p(A), _p(B), _p(Cm))
    return Cm


def fro_err(Cm, Cs):
    """(sum (C-C*)^2, sum C*^2) in fp64."""
    Cm = _d(Cm); Cs = _d(Cs)
    out = np.zeros(2)
    _L().orc_fro_err(_p(Cm), _p(Cs), Cm.size, _p(out))
    return float(out[0]), float(out[1])


def rel_error(Cm, Cs) -> float:
    """Relative error in the Frobenius norm against the float64 reference (Appendix B.1)."""
    e, s = fro_err(Cm, Cs)
    return math.sqrt(e / s) if s > 0 else (0.0 if e == 0 else math.inf)


def error_ratio(E_scheme: float, E_classical: float) -> float:
    """Error-amplification ratio rho = E_scheme / E_classical; 1 if both vanish, inf if only
    the classical error vanishes."""
    if E_classical == 0.0:
        return 1.0 if E_scheme == 0.0 else math.inf
    return E_scheme / E_classical


def summary(ratios) -> dict:
    """Smallest, median (upper of the two middle values when the count is even, Table 3
    caption), largest, spread = largest/smallest, and the number of ratios above 2.  A set that holds NaN has no
    order: its smallest, median, largest and spread are NaN; the count is over the comparable ratios."""
    r = np.asarray(ratios, dtype=np.float64)
    if np.isnan(r).any():
        return dict(min=math.nan, median=math.nan, max=math.nan, spread=math.nan,
                    count_gt2=int(np.sum(r[~np.isnan(r)] > 2.0)), G=int(r.size))
    r = np.sort(r)
    G = r.size
    return dict(min=float(r[0]), median=float(r[G // 2]), max=float(r[-1]),
                spread=float(r[-1] / r[0]) if r[0] > 0 else math.inf,
                count_gt2=int(np.sum(r > 2.0)), G=int(G))


# ---------------------------------------------------------------- certified int8 realisation (Section 4.2)
def quantize_rows(X, b: int, g: int = 128):
    """Appendix D quantiser: per row and per group of g inner indices, d = max|x|/b in fp32 (1 if all zero),
    codes = x/d rounded to nearest even, no clipping.  Returns (codes, scales[rows, K/g])."""
    X = _d(X)
    rows, K = X.shape
    assert K % g == 0
    codes = np.empty((rows, K)); scales = np.empty((rows, K // g))
    _L().orc_quantize_rows(_p(X), rows, K, g, b, _p(codes), _p(scales))
    return codes, scales


def int8_classical(cA, dA, cB, dB, g: int = 128, od="bf16", products: bool = False):
    """Classical int8 operator: exact group products, (P*dA)*dB in fp32, ascending groups, one cast to `od`.
    cA [M,K], cB [N,K] (one row per output column)."""
    cA = _d(cA); cB = _d(cB); dA = _d(dA); dB = _d(dB)
    M, K = cA.shape
    N = cB.shape[0]
    out = np.empty((M, N))
    P = np.empty((K // g, M, N)) if products else None
    _L().orc_int8_classical(_p(cA), _p(dA), _p(cB), _p(dB), M, K, N, g, _fmt(od), _p(out), _p(P))
    return (out, P) if products else out


def int8_certified(s: "Scheme", cA, dA, cB, dB, g: int = 128, od="bf16", products: bool = False):
    """The same operator with each group's integer product computed by the algorithm `s` (one call per group).
    Returns (out, maxabs[3]) or (out, maxabs, P)."""
    m, k, n, R = s.dims
    cA = _d(cA); cB = _d(cB); dA = _d(dA); dB = _d(dB)
    M, K = cA.shape
    N = cB.shape[0]
    out = np.empty((M, N)); mx = np.zeros(3)
    P = np.empty((K // g, M, N)) if products else None
    rc = _L().orc_int8_certified(m, k, n, R, _p(_d(s.U)), _p(_d(s.V)), _p(_d(s.W)), _p(cA), _p(dA), _p(cB), _p(dB),
                                 M, K, N, g, _fmt(od), _p(out), _p(P), _p(mx))
    if rc:
        raise ValueError("shape does not divide, or coefficients are not integers")
    return (out, mx, P) if products else (out, mx)


def int8_finegroup_control(s: "Scheme", cA, dA, cB, dB, call: int = 128, b2: int = 127, od="bf16"):
    """The control of Section 4.2 that breaks condition (iii): scales on fine groups of call / k inner indices (dA
    [M, K / (call / k)], dB likewise) under calls of `call`; every mixed block sum is formed of dequantised values and
    rounded again with ONE scale max|x| / b2 per block sum and call.  cA [M, K], cB [N, K] codes.  Returns [M, N]."""
    m, k, n, R = s.dims
    cA = _d(cA); cB = _d(cB); dA = _d(dA); dB = _d(dB)
    M, K = cA.shape
    N = cB.shape[0]
    out = np.empty((M, N))
    rc = _L().orc_int8_finegroup_control(m, k, n, R, _p(_d(s.U)), _p(_d(s.V)), _p(_d(s.W)), _p(cA), _p(dA), _p(cB), _p(dB),
                                         M, K, N, int(call), int(b2), _fmt(od), _p(out))
    if rc:
        raise ValueError("shape does not fit the call")
    return out


def certificate(s: "Scheme", bA: int, bB: int, h: int, g: int, acc_bits: int = 31):
    """Proposition 1 from coefficients, tiling and specification.  Returns (holds, dict)."""
    m, k, n, R = s.dims
    c = np.zeros(4)
    ok = _L().orc_certificate(m, k, n, R, _p(_d(s.U)), _p(_d(s.V)), _p(_d(s.W)), bA, bB, h, g, acc_bits, _p(c))
    return bool(ok), dict(LAbA=c[0], LBbB=c[1], largest=c[2], one_group=bool(c[3]))


def int8_corrected(s: "Scheme", cA, dA, cB, dB, g: int = 128, od="bf16", products: bool = False):
    """Section 4.3: the algorithm `s` per group with every block sum split as X0 + 256 R (X0 in int8) and each block
    product rebuilt from the four products of Eq. 2.  Returns (out, maxabs[5]) or (out, maxabs, P); maxabs =
    [excess of X0 over the int8 range, max |R|, largest sum of |terms| inside a rebuilt product, largest partial sum
    of the combination, largest |block sum|]."""
    m, k, n, R = s.dims
    cA = _d(cA); cB = _d(cB); dA = _d(dA); dB = _d(dB)
    M, K = cA.shape
    N = cB.shape[0]
    out = np.empty((M, N)); mx = np.zeros(5)
    P = np.empty((K // g, M, N)) if products else None
    rc = _L().orc_int8_corrected(m, k, n, R, _p(_d(s.U)), _p(_d(s.V)), _p(_d(s.W)), _p(cA), _p(dA), _p(cB), _p(dB),
                                 M, K, N, g, _fmt(od), _p(out), _p(P), _p(mx))
    if rc:
        raise ValueError("shape does not divide, or coefficients are not integers")
    return (out, mx, P) if products else (out, mx)


# ---------------------------------------------------------------------------- rotation pre-pass (Appendix B, "A rotation ...")
def hadamard_matrix(h: int) -> np.ndarray:
    """Sylvester's Hadamard matrix of order h (a power of two): H[i, j] = (-1)^popcount(i & j), entries +-1."""
    if h < 1 or h & (h - 1):
        raise ValueError("order must be a power of two")
    i = np.arange(h)
    bits = i[:, None] & i[None, :]
    par = np.zeros((h, h), dtype=np.int64)
    while bits.any():
        par ^= bits & 1
        bits >>= 1
    return (1 - 2 * par).astype(np.float64)


def hadamard_rotate(X, signs, h: int, fmt="f64") -> np.ndarray:
    """Randomised Hadamard rotation along the inner dimension (Appendix B: A -> A H, B -> H^T B with H orthogonal).

    X is [rows, K] with the inner dimension last (for B that is its transpose, so one routine serves both operands);
    H = diag(signs) . blockdiag(H_h, ..., H_h) / sqrt(h) with K a multiple of h.  Computed in fp64 from the
    definition, then rounded once to ``fmt`` (the storage type the rotated operand is kept in).
    """
    X = np.asarray(X, dtype=np.float64)
    K = X.shape[1]
    signs = np.asarray(signs, dtype=np.float64)
    if K % h or signs.shape != (K,) or not np.all(np.abs(signs) == 1.0):
        raise ValueError("K must be a multiple of h and signs must be K entries of +-1")
    Hh = hadamard_matrix(h)
    Y = np.empty_like(X)
    for b in range(K // h):
        sl = slice(b * h, (b + 1) * h)
        Y[:, sl] = ((X[:, sl] * signs[sl]) @ Hh) / math.sqrt(h)     # +-1 sums first: exact cancellations stay exact
    return round_to(Y, fmt)


# ---------------------------------------------------------------------------- the repair rules (Appendix C)
def row_pow2_scales(A) -> np.ndarray:
    """d_t = 2^ceil(log2(max(RMS(x_t), 1e-3))) for every row x_t of A, the RMS over the full row (Appendix C, "The
    repair rules").  The row is divided by d_t before the block sums and its output row multiplied by d_t after the
    combination; both are exact, d_t being a power of two."""
    A = _d(A)
    rms = np.sqrt(np.mean(A * A, axis=1))
    out = np.empty(A.shape[0])
    for t, v in enumerate(np.maximum(rms, 1e-3)):
        f, e = math.frexp(float(v))            # v = f 2^e, f in [0.5, 1)
        out[t] = math.ldexp(1.0, e - 1 if f == 0.5 else e)
    return out


def joint_round_weights(s: Scheme, B, max_sweeps: int = 12):
    """Joint rounding of the weight's block sums under the model schedule (Appendix C, "The repair rules"): returns
    (codes [R, bk, bn], scales [R, ceil(bn/128), ceil(bk/128)], dict(objective_before, objective_after, moved, sweeps))."""
    m, k, n, R = s.dims
    B = _d(B)
    K, N = B.shape
    bk, bn = K // k, N // n
    Bq = np.empty((R, bk, bn)); sB = np.empty((R, -(-bn // 128), -(-bk // 128))); st = np.zeros(4)
    rc = _L().orc_joint_round(m, k, n, R, _p(_d(s.U)), _p(_d(s.V)), _p(_d(s.W)), K, N, _p(B), int(max_sweeps),
                              _p(Bq), _p(sB), _p(st))
    if rc:
        raise ValueError("matrix dimensions are not divisible by the block grid")
    return Bq, sB, dict(objective_before=st[0], objective_after=st[1], moved=int(st[2]), sweeps=int(st[3]))


def scheme_gemm_weights(s: Scheme, A, B, Bq, sB, od="bf16", md="bf16", products: bool = False):
    """The model schedule (scale_mode 3, e4m3) with the weight side given as codes and scales (joint_round_weights)."""
    m, k, n, R = s.dims
    A = _d(A); B = _d(B)
    M, K = A.shape
    N = B.shape[1]
    Cm = np.empty((M, N))
    Mr = np.empty((R, M // m, N // n)) if products else None
    rc = _L().orc_scheme_gemm_weights(m, k, n, R, _p(_d(s.U)), _p(_d(s.V)), _p(_d(s.W)), M, K, N, _p(A), _p(B),
                                      _fmt("e4m3"), _fmt(od), _p(Cm), _p(Mr), _fmt(md), _p(_d(Bq)), _p(_d(sB)))
    if rc:
        raise ValueError("matrix dimensions are not divisible by the block grid")
    return (Cm, Mr) if products else Cm
