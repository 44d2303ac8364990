"""ctypes binding with the same names as the C ABI declared in ``include/fmm_b200.h``.

Only marshalling happens here: torch tensors are reduced to ``data_ptr()`` and the current CUDA
stream to its handle.  The shared library is loaded at import; if it is missing the import fails
loudly (build it with ``python -m paper_2609_39816_b200._build`` or ``__graft_entry__.build()``).
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from ._build import LIB_PATH

F32, BF16, E4M3 = 0, 1, 2
FLAG_REUSE_BHAT = 1
FLAG_PRODUCTS_BF16 = 2
FLAG_SWEEP_SERIAL = 4
FLAG_ROUND_PER_LEVEL = 8
FLAG_SWEEP_UNFUSED = 16
_DT = {"f32": F32, "fp32": F32, "bf16": BF16, "e4m3": E4M3}

EXPORTED_SYMBOLS = [
    "scheme_load", "scheme_builtin", "scheme_kron", "scheme_permute_products", "gauge_apply", "scheme_info", "scheme_coefficients",
    "scheme_free", "scheme_gemm_workspace", "scheme_gemm_workspace_layout", "scheme_gemm", "fmm_device_status",
    "scheme_gemm_host_workspace", "scheme_gemm_host", "scheme_gemm_host_status",
    "fmm_selftest_timeout", "classical_gemm_workspace",
    "classical_gemm", "exact_gemm_f64", "error_frobenius_workspace", "error_frobenius", "error_frobenius_noalloc",
    "error_frobenius_noalloc_max_elements", "scheme_certificate", "int8_quantize", "int8_gemm_workspace", "int8_gemm",
    "int8_gemm_materialised_workspace", "int8_gemm_materialised",
    "scheme_certificate_corrected", "int8_gemm_corrected_workspace", "int8_gemm_corrected",
    "int8_finegroup_control_workspace", "int8_finegroup_control", "hadamard_rotate", "row_pow2_scale", "row_unscale",
    "scheme_joint_round_weights",
    "error_sweep_workspace", "error_sweep", "fmm_status_string", "fmm_launch_count", "fmm_profile_enable",
    "fmm_profile_collect",
]


class FmmError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: fmm_status {code} ({_status_string(code)})")
        self.code = code


class GemmDesc(C.Structure):
    _fields_ = [("M", C.c_int64), ("K", C.c_int64), ("N", C.c_int64), ("lda", C.c_int64), ("ldb", C.c_int64),
                ("ldc", C.c_int64), ("storage", C.c_int32), ("product", C.c_int32), ("output", C.c_int32),
                ("b_is_weight_layout", C.c_int32), ("scale_mode", C.c_int32), ("flags", C.c_int32)]

    @staticmethod
    def make(M, K, N, storage, product, output, weight_layout=False, scale_mode=0, flags=0, lda=None, ldb=None,
             ldc=None):
        d = GemmDesc()
        d.M, d.K, d.N = M, K, N
        d.lda = K if lda is None else lda
        d.ldb = (K if weight_layout else N) if ldb is None else ldb
        d.ldc = N if ldc is None else ldc
        d.storage = _DT[storage] if isinstance(storage, str) else storage
        d.product = _DT[product] if isinstance(product, str) else product
        d.output = _DT[output] if isinstance(output, str) else output
        d.b_is_weight_layout = int(bool(weight_layout))
        d.scale_mode = scale_mode
        d.flags = flags
        return d


class SweepSummary(C.Structure):
    _fields_ = [("min", C.c_double), ("median", C.c_double), ("max", C.c_double), ("spread", C.c_double),
                ("count_gt2", C.c_int64), ("G", C.c_int64), ("e_classical_rel", C.c_double),
                ("norm_ref", C.c_double)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build the CUDA library first (there is no CPU fallback)")
_lib = C.CDLL(LIB_PATH)
_vp, _dp, _sz = C.c_void_p, C.POINTER(C.c_double), C.c_size_t
_lib.scheme_load.argtypes = [C.c_int] * 4 + [_dp] * 3 + [C.c_double, C.POINTER(_vp)]
_lib.scheme_builtin.argtypes = [C.c_char_p, C.POINTER(_vp)]
_lib.scheme_kron.argtypes = [_vp, _vp, C.POINTER(_vp)]
_lib.scheme_permute_products.argtypes = [_vp, C.POINTER(C.c_int), C.POINTER(_vp)]
_lib.gauge_apply.argtypes = [_vp, C.c_int, _dp, _dp, _dp, C.c_double, C.POINTER(_vp)]
_lib.scheme_info.argtypes = [_vp, C.POINTER(C.c_int), _dp]
_lib.scheme_coefficients.argtypes = [_vp, _dp, _dp, _dp]
_lib.scheme_free.argtypes = [_vp]
_lib.scheme_free.restype = None
_lib.scheme_gemm_workspace.argtypes = [_vp, C.POINTER(GemmDesc)]
_lib.scheme_gemm_workspace.restype = _sz
_lib.scheme_gemm_workspace_layout.argtypes = [_vp, C.POINTER(GemmDesc), C.POINTER(_sz)]
_lib.scheme_gemm.argtypes = [_vp, C.POINTER(GemmDesc), _vp, _vp, _vp, _vp, _sz, _vp]
_lib.scheme_gemm_host_workspace.argtypes = [_vp, C.POINTER(GemmDesc)]
_lib.scheme_gemm_host_workspace.restype = _sz
_lib.scheme_gemm_host.argtypes = [_vp, C.POINTER(GemmDesc), _vp, _vp, _vp, _vp, _sz, _vp]
_lib.scheme_gemm_host_status.argtypes = [_vp, C.POINTER(GemmDesc), _vp, _vp]
_lib.fmm_device_status.argtypes = [_vp, _vp]
_lib.fmm_selftest_timeout.argtypes = [_vp, _sz, C.c_uint, _vp]
_lib.classical_gemm_workspace.argtypes = [C.POINTER(GemmDesc)]
_lib.classical_gemm_workspace.restype = _sz
_lib.classical_gemm.argtypes = [C.POINTER(GemmDesc), _vp, _vp, _vp, _vp, _sz, _vp]
_lib.exact_gemm_f64.argtypes = [C.POINTER(GemmDesc), _vp, _vp, _vp, _vp]
_lib.error_frobenius_workspace.argtypes = []
_lib.error_frobenius_workspace.restype = _sz
_lib.error_frobenius.argtypes = [C.POINTER(GemmDesc), _vp, _vp, _vp, _vp, _sz, _vp]
_lib.error_frobenius_noalloc.argtypes = [C.POINTER(GemmDesc), _vp, _vp, _vp, _vp]
_lib.error_frobenius_noalloc_max_elements.restype = C.c_int64
_lib.scheme_certificate.argtypes = [_vp] + [C.c_int] * 5 + [_dp]
_lib.scheme_certificate.restype = C.c_int
_lib.hadamard_rotate.argtypes = [C.c_int, _vp, C.c_int64, C.c_int64, C.c_int64, C.c_int, _vp, _vp, C.c_int64, _vp]
_lib.row_pow2_scale.argtypes = [C.c_int, _vp, C.c_int64, C.c_int64, C.c_int64, _vp, _vp, C.c_int64, _vp]
_lib.row_unscale.argtypes = [C.c_int, _vp, C.c_int64, C.c_int64, C.c_int64, _vp, _vp]
_lib.scheme_joint_round_weights.argtypes = [_vp, C.POINTER(GemmDesc), _vp, C.c_int, _vp, _sz, _vp]
_lib.int8_quantize.argtypes = [_vp, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_int, _vp, _vp, _vp]
_lib.int8_gemm_workspace.argtypes = [_vp, C.c_int64, C.c_int64, C.c_int64]
_lib.int8_gemm_workspace.restype = _sz
_lib.int8_gemm_materialised_workspace.argtypes = [_vp, C.c_int64, C.c_int64, C.c_int64]
_lib.int8_gemm_materialised_workspace.restype = _sz
_lib.int8_gemm_materialised.argtypes = [_vp, C.c_int, _vp, _vp, _vp, _vp, C.c_int64, C.c_int64, C.c_int64, C.c_int, _vp, C.c_int64,
                                        _vp, _sz, _vp]
_lib.int8_gemm.argtypes = [_vp, C.c_int, _vp, _vp, _vp, _vp, C.c_int64, C.c_int64, C.c_int64, C.c_int, _vp, C.c_int64,
                           _vp, _sz, _vp]
_lib.scheme_certificate_corrected.argtypes = [_vp, C.c_int, _dp]
_lib.scheme_certificate_corrected.restype = C.c_int
_lib.int8_gemm_corrected_workspace.argtypes = [_vp, C.c_int64, C.c_int64, C.c_int64]
_lib.int8_gemm_corrected_workspace.restype = _sz
_lib.int8_gemm_corrected.argtypes = [_vp, _vp, _vp, _vp, _vp, C.c_int64, C.c_int64, C.c_int64, C.c_int, _vp, C.c_int64,
                                     _vp, _sz, _vp]
_lib.int8_finegroup_control_workspace.argtypes = [_vp, C.c_int64, C.c_int64, C.c_int64, C.c_int]
_lib.int8_finegroup_control_workspace.restype = _sz
_lib.int8_finegroup_control.argtypes = [_vp, C.c_int, C.c_int, _vp, C.c_int64, _vp, C.c_int64, C.c_int64, C.c_int64, C.c_int64,
                                        C.c_int, C.c_int, _vp, C.c_int64, _vp, _sz, _vp]
_lib.error_sweep_workspace.argtypes = [_vp, C.POINTER(GemmDesc), C.c_int]
_lib.error_sweep_workspace.restype = _sz
_lib.error_sweep.argtypes = [_vp, C.c_int, C.c_int, _dp, _dp, _dp, C.POINTER(GemmDesc), _vp, _vp, _vp, _dp,
                             C.POINTER(SweepSummary), _vp, _sz, _vp]
_lib.fmm_status_string.argtypes = [C.c_int]
_lib.fmm_status_string.restype = C.c_char_p
_lib.fmm_launch_count.restype = C.c_int64
_lib.fmm_profile_enable.argtypes = [C.c_int]
_lib.fmm_profile_enable.restype = None
_lib.fmm_profile_collect.argtypes = [_dp, C.POINTER(C.c_int64)]


def lib_path() -> str:
    return LIB_PATH


def _status_string(code: int) -> str:
    return _lib.fmm_status_string(code).decode()


def _check(code: int, what: str):
    if code != 0:
        raise FmmError(code, what)


def _dbl(a):
    a = np.ascontiguousarray(np.asarray(a, dtype=np.float64))
    return a, a.ctypes.data_as(_dp)


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t):
    return C.c_void_p(0 if t is None else t.data_ptr())


class Scheme:
    """Owning wrapper of an ``fmm_scheme*``."""

    def __init__(self, handle):
        self._h = handle

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h and _lib is not None:      # at interpreter shutdown the module's globals may already be gone
            _lib.scheme_free(h)

    @property
    def handle(self):
        return self._h

    @property
    def dims(self):
        d = (C.c_int * 4)()
        _check(_lib.scheme_info(self._h, d, None), "scheme_info")
        return tuple(d)

    @property
    def info(self) -> dict:
        meta = np.zeros(8)
        _check(_lib.scheme_info(self._h, None, meta.ctypes.data_as(_dp)), "scheme_info")
        return dict(zip(["L_A", "L_B", "L_W", "Phi", "nnz", "maxabs", "Q", "E"], meta.tolist()))

    def coefficients(self):
        m, k, n, R = self.dims
        U, V, W = np.empty((R, m, k)), np.empty((R, k, n)), np.empty((R, m, n))
        _check(_lib.scheme_coefficients(self._h, U.ctypes.data_as(_dp), V.ctypes.data_as(_dp),
                                        W.ctypes.data_as(_dp)), "scheme_coefficients")
        return U, V, W


def scheme_load(U, V, W, brent_tol: float = 0.0) -> Scheme:
    U, pu = _dbl(U); V, pv = _dbl(V); W, pw = _dbl(W)
    R, m, k = U.shape
    n = V.shape[2]
    if V.shape != (R, k, n) or W.shape != (R, m, n):
        raise ValueError("coefficient arrays must be U[R,m,k], V[R,k,n], W[R,m,n]")
    h = _vp()
    _check(_lib.scheme_load(m, k, n, R, pu, pv, pw, brent_tol, C.byref(h)), "scheme_load")
    return Scheme(h)


def scheme_builtin(name: str) -> Scheme:
    h = _vp()
    _check(_lib.scheme_builtin(name.encode(), C.byref(h)), "scheme_builtin")
    return Scheme(h)


def scheme_kron(outer: Scheme, inner: Scheme) -> Scheme:
    h = _vp()
    _check(_lib.scheme_kron(outer.handle, inner.handle, C.byref(h)), "scheme_kron")
    return Scheme(h)


def scheme_permute_products(s: Scheme, perm) -> Scheme:
    """The same algorithm with product r taken from product perm[r] (changes only the order of the decode's sums)."""
    perm = [int(x) for x in perm]
    arr = (C.c_int * len(perm))(*perm)
    if len(perm) != s.dims[3]:
        raise ValueError("perm must have R entries")
    h = _vp()
    _check(_lib.scheme_permute_products(s.handle, arr, C.byref(h)), "scheme_permute_products")
    return Scheme(h)


def gauge_apply(s: Scheme, P, Q, S, level: int = 0, cond_limit: float = 0.0) -> Scheme:
    _, pp = _dbl(P); _, pq = _dbl(Q); _, ps = _dbl(S)
    h = _vp()
    _check(_lib.gauge_apply(s.handle, level, pp, pq, ps, cond_limit, C.byref(h)), "gauge_apply")
    return Scheme(h)


def scheme_gemm_workspace(s: Scheme, d: GemmDesc) -> int:
    return int(_lib.scheme_gemm_workspace(s.handle, C.byref(d)))


def scheme_gemm_workspace_layout(s: Scheme, d: GemmDesc) -> dict:
    off = (_sz * 8)()
    _check(_lib.scheme_gemm_workspace_layout(s.handle, C.byref(d), off), "scheme_gemm_workspace_layout")
    return dict(zip(["Ahat", "Bhat", "M", "sA", "sB", "stride_Ahat", "stride_Bhat", "stride_M"], [int(x) for x in off]))


def classical_gemm_workspace(d: GemmDesc) -> int:
    return int(_lib.classical_gemm_workspace(C.byref(d)))


def error_sweep_workspace(s: Scheme, d: GemmDesc, G: int) -> int:
    return int(_lib.error_sweep_workspace(s.handle, C.byref(d), G))


def scheme_gemm(s: Scheme, d: GemmDesc, A, B, Cout, ws) -> None:
    _check(_lib.scheme_gemm(s.handle, C.byref(d), _ptr(A), _ptr(B), _ptr(Cout), _ptr(ws),
                            ws.numel() * ws.element_size(), _stream()), "scheme_gemm")


def scheme_gemm_host_workspace(s: Scheme, d: GemmDesc) -> int:
    return int(_lib.scheme_gemm_host_workspace(s.handle, C.byref(d)))


def scheme_gemm_host(s: Scheme, d: GemmDesc, A_host, B_host, C_host, ws) -> None:
    """scheme_gemm on HOST tensors (pinned for asynchronous copies): copies in, the path, copy out, on the current
    stream; C_host is valid after the stream has been synchronised.  B_host may be None with FLAG_REUSE_BHAT."""
    _check(_lib.scheme_gemm_host(s.handle, C.byref(d), _ptr(A_host), _ptr(B_host) if B_host is not None else None,
                                 _ptr(C_host), _ptr(ws), ws.numel() * ws.element_size(), _stream()), "scheme_gemm_host")


def scheme_gemm_host_status(s: Scheme, d: GemmDesc, ws) -> None:
    _check(_lib.scheme_gemm_host_status(s.handle, C.byref(d), _ptr(ws), _stream()), "scheme_gemm_host_status")


def classical_gemm(d: GemmDesc, A, B, Cout, ws) -> None:
    _check(_lib.classical_gemm(C.byref(d), _ptr(A), _ptr(B), _ptr(Cout), _ptr(ws),
                               ws.numel() * ws.element_size(), _stream()), "classical_gemm")


def exact_gemm_f64(d: GemmDesc, A, B, Cstar) -> None:
    _check(_lib.exact_gemm_f64(C.byref(d), _ptr(A), _ptr(B), _ptr(Cstar), _stream()), "exact_gemm_f64")


def error_frobenius(d: GemmDesc, Cmat, Cstar, out2, ws) -> None:
    _check(_lib.error_frobenius(C.byref(d), _ptr(Cmat), _ptr(Cstar), _ptr(out2), _ptr(ws),
                                ws.numel() * ws.element_size(), _stream()), "error_frobenius")


def error_frobenius_noalloc(d: GemmDesc, Cmat, Cstar, out2) -> None:
    """error_frobenius for callers that may not allocate: no workspace argument; the partial sums live in
    a fixed array inside the library.  Raises FmmError (FMM_ERR_LIMIT) above
    error_frobenius_noalloc_max_elements() elements.  Calls that overlap on the GPU race on that array."""
    _check(_lib.error_frobenius_noalloc(C.byref(d), _ptr(Cmat), _ptr(Cstar), _ptr(out2), _stream()),
           "error_frobenius_noalloc")


def error_frobenius_noalloc_max_elements() -> int:
    return int(_lib.error_frobenius_noalloc_max_elements())


def scheme_certificate(s, bA: int, bB: int, h: int, g: int = 128, acc_bits: int = 31):
    """Proposition 1 for scheme `s` (None: classical).  Returns (holds, dict of the bounded quantities)."""
    c = np.zeros(4)
    ok = _lib.scheme_certificate(s.handle if s is not None else None, bA, bB, h, g, acc_bits, c.ctypes.data_as(_dp))
    return bool(ok), dict(LAbA=c[0], LBbB=c[1], largest=c[2], one_group=bool(c[3]))


def int8_quantize(X, code_bound: int, codes, scales) -> None:
    """X [rows, K] fp32/bf16 (K % 128 == 0) -> codes int8 [rows, K], scales fp32 [rows, K/128]."""
    import torch
    rows, K = X.shape
    st = F32 if X.dtype == torch.float32 else BF16
    _check(_lib.int8_quantize(_ptr(X), st, rows, K, X.stride(0), code_bound, _ptr(codes), _ptr(scales), _stream()),
           "int8_quantize")


def hadamard_rotate(X, signs, h: int, out=None):
    """Y = (X * signs) . blockdiag(H_h) / sqrt(h) along the last (contiguous) dimension; X [rows, K] fp32/bf16 on the
    device, signs int8 [K] on the device (or None), out defaults to a new tensor (pass X to rotate in place)."""
    import torch
    rows, K = X.shape
    if out is None:
        out = torch.empty_like(X)
    st = F32 if X.dtype == torch.float32 else BF16
    _check(_lib.hadamard_rotate(st, _ptr(X), X.stride(0), rows, K, h, _ptr(signs) if signs is not None else None,
                                _ptr(out), out.stride(0), _stream()), "hadamard_rotate")
    return out


def row_pow2_scale(X, out=None):
    """(X / d, d) with d[t] = 2^ceil(log2(max(RMS(X[t]), 1e-3))); X [rows, K] fp32/bf16 on the device."""
    import torch
    rows, K = X.shape
    if out is None:
        out = torch.empty_like(X)
    d = torch.empty(rows, dtype=torch.float32, device=X.device)
    st = F32 if X.dtype == torch.float32 else BF16
    _check(_lib.row_pow2_scale(st, _ptr(X), X.stride(0), rows, K, _ptr(d), _ptr(out), out.stride(0), _stream()),
           "row_pow2_scale")
    return out, d


def row_unscale(Cmat, d) -> None:
    """C[t, :] *= d[t] in place."""
    import torch
    rows, N = Cmat.shape
    out = F32 if Cmat.dtype == torch.float32 else BF16
    _check(_lib.row_unscale(out, _ptr(Cmat), Cmat.stride(0), rows, N, _ptr(d), _stream()), "row_unscale")


def scheme_joint_round_weights(s, d, B, ws, max_sweeps: int = 12) -> None:
    """Fill the workspace's weight side with jointly rounded codes; follow with scheme_gemm(..., flags |= FLAG_REUSE_BHAT)."""
    _check(_lib.scheme_joint_round_weights(s.handle, C.byref(d), _ptr(B), int(max_sweeps), _ptr(ws),
                                           ws.numel() * ws.element_size(), _stream()), "scheme_joint_round_weights")


def int8_gemm_workspace(s, M: int, K: int, N: int) -> int:
    return int(_lib.int8_gemm_workspace(s.handle if s is not None else None, M, K, N))


def int8_gemm(s, code_bound: int, cA, dA, cB, dB, Cmat, ws) -> None:
    """The group-scaled int8 operator; s None -> classical integer products, else one call of s per group."""
    import torch
    M, K = cA.shape
    N = cB.shape[0]
    out = F32 if Cmat.dtype == torch.float32 else BF16
    _check(_lib.int8_gemm(s.handle if s is not None else None, code_bound, _ptr(cA), _ptr(dA), _ptr(cB), _ptr(dB), M, K, N,
                          out, _ptr(Cmat), Cmat.stride(0), _ptr(ws), ws.numel() * ws.element_size(), _stream()),
           "int8_gemm")


def int8_gemm_materialised_workspace(s, M: int, K: int, N: int) -> int:
    return int(_lib.int8_gemm_materialised_workspace(s.handle if s is not None else None, M, K, N))


def int8_gemm_materialised(s, code_bound: int, cA, dA, cB, dB, Cmat, ws) -> None:
    """The same operator as int8_gemm through the pipeline that writes every per-group block product to memory."""
    import torch
    M, K = cA.shape
    N = cB.shape[0]
    out = F32 if Cmat.dtype == torch.float32 else BF16
    _check(_lib.int8_gemm_materialised(s.handle if s is not None else None, code_bound, _ptr(cA), _ptr(dA), _ptr(cB), _ptr(dB),
                                       M, K, N, out, _ptr(Cmat), Cmat.stride(0), _ptr(ws), ws.numel() * ws.element_size(),
                                       _stream()), "int8_gemm_materialised")


def scheme_certificate_corrected(s, h: int):
    """Certificate of the overflow-corrected computation (Section 4.3).  Returns (holds, dict)."""
    c = np.zeros(4)
    ok = _lib.scheme_certificate_corrected(s.handle, h, c.ctypes.data_as(_dp))
    return bool(ok), dict(block_sum_max=c[0], r_max=c[1], product_terms=c[2], combination=c[3])


def int8_gemm_corrected_workspace(s, M: int, K: int, N: int) -> int:
    return int(_lib.int8_gemm_corrected_workspace(s.handle, M, K, N))


def int8_gemm_corrected(s, cA, dA, cB, dB, Cmat, ws) -> None:
    """The int8 operator at code bound 127 computed by `s` per group with the overflow correction of Eq. 2."""
    import torch
    M, K = cA.shape
    N = cB.shape[0]
    out = F32 if Cmat.dtype == torch.float32 else BF16
    _check(_lib.int8_gemm_corrected(s.handle, _ptr(cA), _ptr(dA), _ptr(cB), _ptr(dB), M, K, N, out, _ptr(Cmat),
                                    Cmat.stride(0), _ptr(ws), ws.numel() * ws.element_size(), _stream()),
           "int8_gemm_corrected")


def int8_finegroup_control_workspace(s, M: int, K: int, N: int, call: int = 128) -> int:
    return int(_lib.int8_finegroup_control_workspace(s.handle, M, K, N, call))


def int8_finegroup_control(s, A, B, Cmat, ws, code_bound: int = 31, second_bound: int = 127, call: int = 128) -> None:
    """The control that breaks condition (iii): fine-group scales (call / k indices) under calls of `call` indices, every
    mixed block sum rounded again with one scale.  A [M, K], B [N, K]: fp32 CUDA tensors; Cmat [M, N] fp32 or bf16."""
    import torch
    M, K = A.shape
    N = B.shape[0]
    out = F32 if Cmat.dtype == torch.float32 else BF16
    _check(_lib.int8_finegroup_control(s.handle, code_bound, second_bound, _ptr(A), A.stride(0), _ptr(B), B.stride(0), M, K, N,
                                       call, out, _ptr(Cmat), Cmat.stride(0), _ptr(ws), ws.numel() * ws.element_size(),
                                       _stream()), "int8_finegroup_control")


def error_sweep(base: Scheme, level: int, P, Q, S, d: GemmDesc, A, B, ws, Cstar=None):
    """Returns (ratios[G] as numpy fp64, summary dict)."""
    P, pp = _dbl(P); Q, pq = _dbl(Q); S, ps = _dbl(S)
    G = P.shape[0]
    ratios = np.empty(G)
    summ = SweepSummary()
    _check(_lib.error_sweep(base.handle, level, G, pp, pq, ps, C.byref(d), _ptr(A), _ptr(B), _ptr(Cstar),
                            ratios.ctypes.data_as(_dp), C.byref(summ), _ptr(ws), ws.numel() * ws.element_size(),
                            _stream()), "error_sweep")
    return ratios, summ.as_dict()


def device_status(ws) -> None:
    _check(_lib.fmm_device_status(_ptr(ws), _stream()), "fmm_device_status")


def selftest_timeout(ws, wait_ms: int = 50) -> None:
    """Enqueue the failure-reporting self-test (one block whose wait must expire); follow with device_status(ws),
    which then raises FmmError with code 8 (FMM_ERR_TIMEOUT)."""
    _check(_lib.fmm_selftest_timeout(_ptr(ws), ws.numel() * ws.element_size(), wait_ms, _stream()),
           "fmm_selftest_timeout")


def launch_count() -> int:
    return int(_lib.fmm_launch_count())


PHASES = ["encode_a", "encode_b", "products", "decode", "classical_products", "other"]


def profile_enable(on: bool) -> None:
    _lib.fmm_profile_enable(int(on))


def profile_collect() -> dict:
    """{phase: (total milliseconds, number of bracketed regions)} since the last collect."""
    ms = np.zeros(8)
    cnt = (C.c_int64 * 8)()
    _check(_lib.fmm_profile_collect(ms.ctypes.data_as(_dp), cnt), "fmm_profile_collect")
    return {name: (float(ms[i]), int(cnt[i])) for i, name in enumerate(PHASES)}
