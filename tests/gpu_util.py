"""Helpers shared by the GPU parity tests: move seeded inputs to the device, call the library through
its C-ABI binding, and fetch results (and the per-step intermediates) back as fp64 numpy arrays."""
import numpy as np
import torch

import oracle
from fmm_inputs import generators as gen

_TD = {"f32": torch.float32, "bf16": torch.bfloat16}


def fmm():
    import paper_2609_39816_b200 as lib
    return lib


def oracle_scheme(name):
    s1 = oracle.strassen()
    return {"strassen222": s1, "strassen444": oracle.kron(s1, s1)}[name]


def storage_pair(x64, dtype):
    """fp64 array -> (cuda tensor in storage dtype, fp64 numpy of the stored values)."""
    t, v = gen.to_storage(x64, dtype)
    return t.cuda(), v


def workspace(nbytes):
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device="cuda")


def run_scheme_gemm(s, A_t, B_t, S, Pd, O, weight_layout=False, scale_mode=0, flags=0, ws=None, parts=False):
    """A_t [M,K]; B_t [K,N] (or [N,K] with weight_layout).  Returns C as fp64 numpy (+ parts dict)."""
    lib = fmm()
    M, K = A_t.shape
    N = B_t.shape[0] if weight_layout else B_t.shape[1]
    d = lib.GemmDesc.make(M, K, N, S, Pd, O, weight_layout=weight_layout, scale_mode=scale_mode, flags=flags)
    need = lib.scheme_gemm_workspace(s, d)
    assert need > 0, "descriptor rejected"
    if ws is None:
        ws = workspace(need)
    C = torch.empty((M, N), dtype=_TD[O], device="cuda")
    lib.scheme_gemm(s, d, A_t, B_t, C, ws)
    lib.device_status(ws)
    out = C.to(torch.float64).cpu().numpy()
    if not parts:
        return out
    off = lib.scheme_gemm_workspace_layout(s, d)
    m, k, n, R = s.dims
    bm, bk, bn = M // m, K // k, N // n

    def grab(o, stride, rows, cols, dt):
        """R blocks [rows, cols] of dtype dt, `stride` elements apart, starting at byte offset o."""
        es = torch.empty((), dtype=dt).element_size()
        flat = ws[o:o + R * stride * es].view(dt).view(R, stride)[:, :rows * cols]
        return flat.to(torch.float64).cpu().numpy().reshape(R, rows, cols)

    pdt = torch.bfloat16 if Pd == "bf16" else torch.float8_e4m3fn
    p = dict(
        Ahat=grab(off["Ahat"], off["stride_Ahat"], bm, bk, pdt),
        BhatT=grab(off["Bhat"], off["stride_Bhat"], bn, bk, pdt),
        M=grab(off["M"], off["stride_M"], bm, bn, torch.bfloat16 if flags & 2 else torch.float32),
    )
    if scale_mode == 1:
        p["sA"] = ws[off["sA"]:off["sA"] + 4 * R].view(torch.float32).to(torch.float64).cpu().numpy()
        p["sB"] = ws[off["sB"]:off["sB"] + 4 * R].view(torch.float32).to(torch.float64).cpu().numpy()
    elif scale_mode == 3:     # model schedule: [R][bm][G] and [R][ceil(bn/128)][G]
        G3, CB3 = -(-bk // 128), -(-bn // 128)
        p["sA"] = ws[off["sA"]:off["sA"] + 4 * R * bm * G3].view(torch.float32).to(torch.float64).cpu().numpy().reshape(R, bm, G3)
        p["sB"] = ws[off["sB"]:off["sB"] + 4 * R * CB3 * G3].view(torch.float32).to(torch.float64).cpu().numpy().reshape(R, CB3, G3)
    elif scale_mode == 2:     # one scale per row of each block sum of A / per column of each block sum of B
        p["sA"] = ws[off["sA"]:off["sA"] + 4 * R * bm].view(torch.float32).to(torch.float64).cpu().numpy().reshape(R, bm)
        p["sB"] = ws[off["sB"]:off["sB"] + 4 * R * bn].view(torch.float32).to(torch.float64).cpu().numpy().reshape(R, bn)
    return out, p, ws


def run_classical(A_t, B_t, S, Pd, O, weight_layout=False, scale_mode=0):
    lib = fmm()
    M, K = A_t.shape
    N = B_t.shape[0] if weight_layout else B_t.shape[1]
    d = lib.GemmDesc.make(M, K, N, S, Pd, O, weight_layout=weight_layout, scale_mode=scale_mode)
    ws = workspace(lib.classical_gemm_workspace(d))
    C = torch.empty((M, N), dtype=_TD[O], device="cuda")
    lib.classical_gemm(d, A_t, B_t, C, ws)
    lib.device_status(ws)
    return C.to(torch.float64).cpu().numpy()


def run_exact(A_t, B_t, S, weight_layout=False):
    lib = fmm()
    M, K = A_t.shape
    N = B_t.shape[0] if weight_layout else B_t.shape[1]
    d = lib.GemmDesc.make(M, K, N, S, "bf16", "f32", weight_layout=weight_layout)
    Cs = torch.empty((M, N), dtype=torch.float64, device="cuda")
    lib.exact_gemm_f64(d, A_t, B_t, Cs)
    torch.cuda.synchronize()
    return Cs


def rel_fro(a, b):
    nb = np.linalg.norm(b)
    return np.linalg.norm(a - b) / nb if nb > 0 else np.linalg.norm(a - b)


def subsample_problem(A64, B64, m, k, n, rows, cols):
    """Rows `rows` of every block row of A and columns `cols` of every block column of B.  Because a
    scheme acts position-wise on blocks, the scheme product of the sub-problem equals the full
    product restricted to those rows and columns (valid when no per-tensor scale is used)."""
    M, K = A64.shape
    N = B64.shape[1]
    bm, bn = M // m, N // n
    ridx = np.concatenate([i * bm + np.asarray(rows) for i in range(m)])
    cidx = np.concatenate([j * bn + np.asarray(cols) for j in range(n)])
    return A64[ridx], B64[:, cidx], ridx, cidx
