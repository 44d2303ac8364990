"""GPU parity of the two repair rules (Appendix C, "The repair rules") against the oracle, through the C ABI: the
row scales and the scaled rows bit for bit; the jointly rounded weight codes and their scales bit for bit (both
sides take every decision of the search in fp32, in the same order); the product that uses them within the
tolerances of the plain model schedule; and the first repaired algorithm end to end (one Strassen and one classical
level, both rules)."""
import numpy as np
import pytest
import torch

import oracle
from fmm_inputs import generators as gen
import gpu_util as gu

pytestmark = pytest.mark.gpu

TOL_FRO = 1e-3


@pytest.fixture(scope="module")
def lib():
    return gu.fmm()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_row_scale_and_unscale_are_exact(lib, dtype):
    rows, K, ld = 77, 200, 208
    X = gen.normal(1, 0, (rows, K)) * np.exp2(gen.uniform(1, 1, (rows, 1), -12, 12))
    X[3] = 1.0; X[4] = 0.0; X[5] = 0.5; X[6] = 1e-4; X[7] = 3.0; X[8] = 0.0; X[8, 0] = 8.0 * np.sqrt(K / 64.0)
    Xt, X64 = gu.storage_pair(X, dtype)
    Xp = torch.zeros((rows, ld), dtype=Xt.dtype, device="cuda"); Xp[:, :K] = Xt
    Y, d = lib.row_pow2_scale(Xp[:, :K])
    want_d = oracle.row_pow2_scales(X64)
    assert np.array_equal(d.double().cpu().numpy(), want_d)
    assert want_d[3] == 1.0 and want_d[4] == 2.0 ** -9 and want_d[5] == 0.5 and want_d[6] == 2.0 ** -9 and want_d[7] == 4.0
    assert np.array_equal(Y.double().cpu().numpy(), X64 / want_d[:, None])
    Cm = Y.clone()
    lib.row_unscale(Cm, d)
    assert np.array_equal(Cm.double().cpu().numpy(), X64)
    lib.row_pow2_scale(Xp[:, :K], out=Xp[:, :K])                   # in place
    assert torch.equal(Xp[:, :K], Y)


@pytest.mark.parametrize("dtype,rows,K", [("bf16", 5, 100), ("bf16", 9, 11008), ("f32", 7, 8192), ("f32", 3, 50), ("bf16", 1, 8)])
def test_row_scale_paths_for_short_long_and_unaligned_rows(lib, dtype, rows, K):
    """Rows that are not a whole number of 16-byte vectors (scalar path), rows longer than the register-resident
    limit (two passes over memory), and a single short row."""
    X = gen.normal(2, K, (rows, K)) * np.exp2(gen.uniform(2, K + 1, (rows, 1), -6, 6))
    Xt, X64 = gu.storage_pair(X, dtype)
    Y, d = lib.row_pow2_scale(Xt)
    want_d = oracle.row_pow2_scales(X64)
    assert np.array_equal(d.double().cpu().numpy(), want_d)
    assert np.array_equal(Y.double().cpu().numpy(), X64 / want_d[:, None])
    lib.row_unscale(Y, d)
    assert np.array_equal(Y.double().cpu().numpy(), X64)


def _schemes(lib, name):
    st, cl = lib.scheme_builtin("strassen222"), lib.scheme_builtin("classical222")
    ost, ocl = oracle.strassen(), oracle.classical_scheme(2, 2, 2)
    if name == "strassen222":
        return st, ost
    if name == "strassen444":
        return lib.scheme_builtin("strassen444"), oracle.kron(ost, ost)
    return lib.scheme_kron(st, cl), oracle.kron(ost, ocl)            # the first repaired algorithm's nesting


@pytest.mark.parametrize("name,M,K,N,S,wl", [
    ("strassen222", 64, 512, 640, "bf16", True),      # 2 groups, bn = 320: three column blocks, the last ragged
    ("strassen444", 64, 832, 512, "bf16", False),     # bk = 208: a ragged second group; B given K x N
    ("hybrid", 128, 512, 1088, "bf16", True),         # R = 56, bn = 272
    ("strassen222", 64, 256, 256, "f32", True),       # fp32 weights: block sums rounded to bf16 first
])
def test_joint_rounding_matches_the_oracle_bit_for_bit(lib, name, M, K, N, S, wl):
    s, so = _schemes(lib, name)
    A = gen.activations_outlier(7, 1, M, K, frac=0.01, factor=50.0)
    B = gen.weights(7, 2, K, N)
    At, A64 = gu.storage_pair(A, S)
    Bt_kn, B64 = gu.storage_pair(B, S)
    Bt = Bt_kn.T.contiguous() if wl else Bt_kn
    d = lib.GemmDesc.make(M, K, N, S, "e4m3", "bf16", weight_layout=wl, scale_mode=3)
    ws = gu.workspace(lib.scheme_gemm_workspace(s, d))
    Bq, sB, st = oracle.joint_round_weights(so, B64)
    assert st["moved"] > 0
    for sweeps, want in ((0, oracle.joint_round_weights(so, B64, max_sweeps=0)[0]), (12, Bq)):
        lib.scheme_joint_round_weights(s, d, Bt, ws, max_sweeps=sweeps)
        C, p, _ = gu.run_scheme_gemm(s, At, Bt, S, "e4m3", "bf16", weight_layout=wl, scale_mode=3,
                                     flags=lib.FLAG_REUSE_BHAT, ws=ws, parts=True)
        assert np.array_equal(p["BhatT"], want.transpose(0, 2, 1))
        assert np.array_equal(p["sB"], sB)
    Co, Mo = oracle.scheme_gemm_weights(so, A64, B64, Bq, sB, od="bf16", md="f64", products=True)
    assert gu.rel_fro(p["M"], Mo) <= 1e-5
    assert gu.rel_fro(C, Co) <= TOL_FRO
    # zero sweeps are the plain schedule: the same product as scheme_gemm without the search
    lib.scheme_joint_round_weights(s, d, Bt, ws, max_sweeps=0)
    C0 = gu.run_scheme_gemm(s, At, Bt, S, "e4m3", "bf16", weight_layout=wl, scale_mode=3, flags=lib.FLAG_REUSE_BHAT, ws=ws)
    C1 = gu.run_scheme_gemm(s, At, Bt, S, "e4m3", "bf16", weight_layout=wl, scale_mode=3)
    assert np.array_equal(C0, C1)


def test_joint_rounding_needs_the_model_schedule(lib):
    s = lib.scheme_builtin("strassen222")
    B = torch.zeros((256, 256), dtype=torch.bfloat16, device="cuda")
    for pd, mode in (("bf16", 0), ("e4m3", 1), ("e4m3", 2)):
        d = lib.GemmDesc.make(64, 256, 256, "bf16", pd, "bf16", weight_layout=True, scale_mode=mode)
        ws = gu.workspace(lib.scheme_gemm_workspace(s, d))
        with pytest.raises(lib.FmmError):
            lib.scheme_joint_round_weights(s, d, B, ws)


def test_first_repaired_algorithm_end_to_end(lib):
    """One Strassen and one classical level, row scale, jointly rounded weights, products returned in bf16: the
    device pipeline against the oracle's; and the row rule's point — a token row scaled by a power of two leaves every
    other output row's bits alone."""
    s, so = _schemes(lib, "hybrid")
    M, K, N = 256, 512, 512
    A = gen.normal(9, 1, (M, K)); A[37] *= 300.0; A[130] *= 2.0 ** -6          # token rows of very different norms
    At, A64 = gu.storage_pair(A, "bf16")
    Bt_kn, B64 = gu.storage_pair(gen.weights(9, 2, K, N), "bf16")
    Bt = Bt_kn.T.contiguous()
    d = lib.GemmDesc.make(M, K, N, "bf16", "e4m3", "bf16", weight_layout=True, scale_mode=3,
                          flags=lib.FLAG_REUSE_BHAT | lib.FLAG_PRODUCTS_BF16)
    ws = gu.workspace(lib.scheme_gemm_workspace(s, d))
    lib.scheme_joint_round_weights(s, d, Bt, ws)

    def device(Ain):
        As, dt = lib.row_pow2_scale(Ain)
        Cm = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        lib.scheme_gemm(s, d, As, Bt, Cm, ws)
        lib.device_status(ws)
        lib.row_unscale(Cm, dt)
        return Cm.double().cpu().numpy()

    C = device(At)
    dq = oracle.row_pow2_scales(A64)
    Bq, sB, _ = oracle.joint_round_weights(so, B64)
    Co = oracle.scheme_gemm_weights(so, A64 / dq[:, None], B64, Bq, sB, od="bf16", md="bf16") * dq[:, None]
    assert gu.rel_fro(C, Co) <= TOL_FRO
    Cs = A64 @ B64
    plain = gu.run_scheme_gemm(s, At, Bt, "bf16", "e4m3", "bf16", weight_layout=True, scale_mode=3, flags=lib.FLAG_PRODUCTS_BF16)
    rows = [37 + 128]                 # the row the loud row is added to: same offset in the other outer (Strassen) block
    err = lambda X: np.linalg.norm((X - Cs)[rows]) / np.linalg.norm(Cs[rows])
    assert err(C) < 0.5 * err(plain)
    A2 = At.clone(); A2[37] *= 16.0
    C2 = device(A2)
    keep = [t for t in range(M) if t != 37]
    assert np.array_equal(C2[keep], C[keep]) and np.array_equal(C2[37], C[37] * 16.0)
