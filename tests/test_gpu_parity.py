"""Parity of the CUDA path (called through the C ABI) against the CPU oracle, element by element on
the same seeded inputs.

Bars: bit-exact for integer-valued inputs and for the encoded operands (quantised codes);
relative Frobenius difference <= 1e-3 for floating-point results; error-amplification ratios within
2 % relative of the oracle's.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from fmm_inputs import generators as gen

import gpu_util as gu

pytestmark = pytest.mark.gpu

TOL_FRO = 1e-3
TOL_RATIO = 0.02


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__
    __graft_entry__.build()
    return gu.fmm()


def _inputs(seed, M, K, N, S, kind="normal", bound=None):
    if kind == "int":
        A, B = gen.integer_matrix(seed, 1, (M, K), bound), gen.integer_matrix(seed, 2, (K, N), bound)
    elif kind == "llm":
        A, B = gen.activations_outlier(seed, 1, M, K, frac=0.01, factor=100.0), gen.weights(seed, 2, K, N)
    elif kind in ("u01", "upm1"):
        lo = 0.0 if kind == "u01" else -1.0
        A, B = gen.uniform(seed, 1, (M, K), lo, 1.0), gen.uniform(seed, 2, (K, N), lo, 1.0)
    elif kind == "t3":
        A = gen.activations_outlier(seed, 1, M, K, dist="t3", frac=0.001, factor=300.0, at_least=1)
        B = gen.weights(seed, 2, K, N)
    else:
        A, B = gen.normal(seed, 1, (M, K)), gen.normal(seed, 2, (K, N))
    At, A64 = gu.storage_pair(A, S)
    Bt, B64 = gu.storage_pair(B, S)
    return At, Bt, A64, B64


# ---------------------------------------------------------------------------- per-step parity
@pytest.mark.parametrize("scheme,M,K,N,S,Pd,O,kind,scale", [
    ("strassen222", 256, 256, 256, "f32", "bf16", "f32", "normal", 0),      # config 1 shape
    ("strassen444", 384, 320, 288, "bf16", "bf16", "f32", "llm", 0),        # ragged tiles in M, K and N
    ("strassen444", 1024, 1024, 2048, "bf16", "bf16", "bf16", "llm", 0),    # several tiles per product
    ("strassen222", 640, 1088, 528, "bf16", "bf16", "bf16", "normal", 0),   # bn = 264: 256-tile + ragged tail
    ("strassen444", 512, 1024, 512, "bf16", "e4m3", "bf16", "t3", 1),       # fp8 with per-tensor scales
    ("strassen222", 256, 2240, 272, "bf16", "e4m3", "f32", "llm", 1),       # fp8, K tail inside a stage
    ("strassen444", 64, 64, 32, "f32", "bf16", "f32", "normal", 0),         # smallest legal blocks
    ("strassen444", 256, 11008, 512, "bf16", "e4m3", "bf16", "t3", 1),      # config-4 down-projection K: K/4 = 2752 = 21.5 stages
    ("strassen444", 128, 128, 128, "f32", "e4m3", "f32", "u01", 2),         # the ensemble's shape: row / column scales
    ("strassen444", 512, 1024, 544, "bf16", "e4m3", "bf16", "t3", 2),       # row / column scales, several tiles, CTA pairs
    ("strassen222", 200, 2240, 272, "bf16", "e4m3", "f32", "llm", 2),       # rows of 280 vectors: per-thread amax path
    ("strassen444", 512, 1024, 512, "bf16", "e4m3", "f32", "t3", 3),        # model schedule: 2 groups, one 128-column block
    ("strassen444", 256, 2048, 1088, "bf16", "e4m3", "bf16", "llm", 3),     # 4 groups, bn = 272: three column blocks, ragged
    ("strassen222", 384, 768, 528, "f32", "e4m3", "f32", "llm", 3),         # fp32 source (weights rounded to bf16 first), 3 groups
    ("strassen444", 128, 11008, 512, "bf16", "e4m3", "f32", "t3", 3),       # K/4 = 2752 = 21.5 groups: ragged last group
])
def test_every_step_matches_oracle(lib, scheme, M, K, N, S, Pd, O, kind, scale):
    At, Bt, A64, B64 = _inputs(3, M, K, N, S, kind)
    s, so = lib.scheme_builtin(scheme), gu.oracle_scheme(scheme)
    C, p, _ = gu.run_scheme_gemm(s, At, Bt, S, Pd, O, scale_mode=scale, parts=True)
    Co, po = oracle.scheme_gemm(so, A64, B64, pd=Pd, od=O, scale_mode=scale, parts=True)
    # encode A / encode B: quantised codes, decided in fp32 on both sides -> bit-exact
    assert np.array_equal(p["Ahat"], po["Ahat"])
    assert np.array_equal(p["BhatT"], po["Bhat"].transpose(0, 2, 1))
    if scale:
        assert np.array_equal(p["sA"], po["sA"]) and np.array_equal(p["sB"], po["sB"])
    # block products (fp32 accumulation on tensor cores vs fp64) and decode
    assert gu.rel_fro(p["M"], po["M"]) <= 1e-5
    assert gu.rel_fro(C, Co) <= TOL_FRO


@pytest.mark.parametrize("order", ["strassen_outside", "classical_outside"])
@pytest.mark.parametrize("Pd,scale", [("bf16", 0), ("e4m3", 1)])
def test_hybrid_of_one_strassen_and_one_classical_level(lib, order, Pd, scale):
    """One level of Strassen nested with one classical level, <4,4,4;56> (the nesting the paper's first repaired
    algorithm uses, Appendix C): every step against the oracle's Kronecker scheme, in both nesting orders; the
    classical level adds no block sums of its own, so the largest block sum has two terms, not four."""
    At, Bt, A64, B64 = _inputs(17, 512, 768, 544, "bf16", "llm")
    st, cl = lib.scheme_builtin("strassen222"), lib.scheme_builtin("classical222")
    ost, ocl = oracle.strassen(), oracle.classical_scheme(2, 2, 2)
    s = lib.scheme_kron(st, cl) if order == "strassen_outside" else lib.scheme_kron(cl, st)
    so = oracle.kron(ost, ocl) if order == "strassen_outside" else oracle.kron(ocl, ost)
    assert s.dims == (4, 4, 4, 56)
    assert oracle.criteria(so)["L_A"] == 2
    C, p, _ = gu.run_scheme_gemm(s, At, Bt, "bf16", Pd, "bf16", scale_mode=scale, parts=True)
    Co, po = oracle.scheme_gemm(so, A64, B64, pd=Pd, od="bf16", scale_mode=scale, parts=True)
    assert np.array_equal(p["Ahat"], po["Ahat"])
    assert np.array_equal(p["BhatT"], po["Bhat"].transpose(0, 2, 1))
    if scale:
        assert np.array_equal(p["sA"], po["sA"]) and np.array_equal(p["sB"], po["sB"])
    assert gu.rel_fro(p["M"], po["M"]) <= 1e-5
    assert gu.rel_fro(C, Co) <= TOL_FRO


@pytest.mark.parametrize("scheme,M,K,N,S,Pd,O,kind,scale", [
    ("strassen444", 1024, 1024, 2048, "bf16", "bf16", "bf16", "llm", 0),    # CTA-pair kernel, bf16 products
    ("strassen444", 384, 320, 288, "bf16", "bf16", "f32", "llm", 0),        # ragged tiles
    ("strassen444", 512, 1024, 544, "bf16", "e4m3", "bf16", "t3", 1),       # per-tensor scales folded into the decode
    ("strassen222", 200, 2240, 272, "bf16", "e4m3", "f32", "llm", 2),       # row / column scales applied before the rounding
    ("strassen444", 512, 2048, 1024, "bf16", "e4m3", "bf16", "t3", 3),      # the paper's whole model schedule: group scales, bf16 products
])
def test_products_returned_in_bf16(lib, scheme, M, K, N, S, Pd, O, kind, scale):
    """FMM_FLAG_PRODUCTS_BF16, the paper's model schedule: every product rounded once to bf16, combined in fp32.
    The device rounds an fp32 accumulation where the oracle rounds an fp64 one, so a few products may land one
    bf16 step apart: the products are compared in norm, and at most 1 in 1000 of them may differ at all."""
    At, Bt, A64, B64 = _inputs(3, M, K, N, S, kind)
    s, so = lib.scheme_builtin(scheme), gu.oracle_scheme(scheme)
    C, p, _ = gu.run_scheme_gemm(s, At, Bt, S, Pd, O, scale_mode=scale, flags=lib.FLAG_PRODUCTS_BF16, parts=True)
    Co, po = oracle.scheme_gemm(so, A64, B64, pd=Pd, od=O, scale_mode=scale, parts=True, md="bf16")
    assert np.array_equal(p["Ahat"], po["Ahat"])
    assert np.mean(p["M"] != po["M"]) <= 1e-3
    # never more than one bf16 step, plus the fp32 accumulation error where a product cancels to almost nothing
    assert np.all(np.abs(p["M"] - po["M"]) <= 2.0 ** -7 * np.abs(po["M"]) + 1e-5 * np.abs(po["M"]).max())
    assert gu.rel_fro(C, Co) <= TOL_FRO
    # and it is a different operator from the fp32-product default
    C32 = gu.run_scheme_gemm(s, At, Bt, S, Pd, O, scale_mode=scale)
    assert not np.array_equal(C, C32)


@pytest.mark.parametrize("scheme,M,K,N,S,Pd,O,bound", [
    ("strassen222", 256, 256, 256, "f32", "bf16", "f32", 8),       # config 1 shape, L*b <= 2^8
    ("strassen444", 512, 512, 384, "bf16", "bf16", "f32", 7),      # two-level, 16*bk*(4*7)^2 < 2^24
    ("strassen444", 256, 1024, 256, "bf16", "e4m3", "f32", 4),     # e4m3 dense codebook: |code| <= 4, L = 4
    ("strassen222", 384, 640, 272, "bf16", "bf16", "bf16", 2),     # bf16 output still exact (small values)
])
def test_integer_inputs_bit_exact(lib, scheme, M, K, N, S, Pd, O, bound):
    At, Bt, A64, B64 = _inputs(5, M, K, N, S, "int", bound)
    s, so = lib.scheme_builtin(scheme), gu.oracle_scheme(scheme)
    C = gu.run_scheme_gemm(s, At, Bt, S, Pd, O)
    ref = A64 @ B64
    if O == "bf16":
        assert np.abs(ref).max() < 256
    assert np.array_equal(C, ref)
    assert np.array_equal(oracle.scheme_gemm(so, A64, B64, pd=Pd, od=O), ref)
    assert np.array_equal(gu.run_classical(At, Bt, S, Pd, O), ref)
    assert np.array_equal(gu.run_exact(At, Bt, S).cpu().numpy(), ref)


def test_sign_variants_give_one_integer_product_and_flipped_w_breaks_it(lib):
    At, Bt, A64, B64 = _inputs(6, 128, 256, 128, "bf16", "int", 4)
    s2 = lib.scheme_builtin("strassen444")
    ref = A64 @ B64
    for d, e, f in oracle.sign_variants(4, 4, 4)[::41]:
        g = lib.gauge_apply(s2, np.diag(d), np.diag(e), np.diag(f))
        assert np.array_equal(gu.run_scheme_gemm(g, At, Bt, "bf16", "e4m3", "f32"), ref)
    # negative control: a single flipped decoding coefficient must break parity (loaded with the Brent
    # check disabled by a huge tolerance)
    U, V, W = s2.coefficients()
    W[5, 1, 2] = -W[5, 1, 2] if W[5, 1, 2] != 0 else 1.0
    bad = lib.scheme_load(U, V, W, brent_tol=1e9)
    assert not np.array_equal(gu.run_scheme_gemm(bad, At, Bt, "bf16", "e4m3", "f32"), ref)


def test_layouts_flags_and_identity_gauge(lib):
    At, Bt, A64, B64 = _inputs(7, 512, 768, 640, "bf16", "llm")
    s = lib.scheme_builtin("strassen444")
    C_kn, _, ws = gu.run_scheme_gemm(s, At, Bt, "bf16", "bf16", "bf16", parts=True)
    # weight layout [N,K] gives the same bits as [K,N]
    C_w = gu.run_scheme_gemm(s, At, Bt.t().contiguous(), "bf16", "bf16", "bf16", weight_layout=True)
    assert np.array_equal(C_kn, C_w)
    # reuse of the encoded weights left in the workspace
    C_re = gu.run_scheme_gemm(s, At, Bt, "bf16", "bf16", "bf16", flags=lib.FLAG_REUSE_BHAT, ws=ws)
    assert np.array_equal(C_kn, C_re)
    # identity gauge equals the base scheme bit for bit; run-to-run bit identity
    g = lib.gauge_apply(s, np.eye(4), np.eye(4), np.eye(4))
    assert np.array_equal(gu.run_scheme_gemm(g, At, Bt, "bf16", "bf16", "bf16"), C_kn)
    assert np.array_equal(gu.run_scheme_gemm(s, At, Bt, "bf16", "bf16", "bf16"), C_kn)
    # strided operands (leading dimensions larger than the rows)
    M, K, N = 512, 768, 640
    Abig = torch.zeros((M, K + 64), dtype=torch.bfloat16, device="cuda"); Abig[:, :K] = At
    Cbig = torch.zeros((M, N + 32), dtype=torch.bfloat16, device="cuda")
    d = lib.GemmDesc.make(M, K, N, "bf16", "bf16", "bf16", lda=K + 64, ldc=N + 32)
    lib.scheme_gemm(s, d, Abig, Bt, Cbig, ws)
    lib.device_status(ws)
    assert np.array_equal(Cbig[:, :N].double().cpu().numpy(), C_kn)
    assert float(Cbig[:, N:].abs().max()) == 0.0


def test_row_leak_pattern_on_gpu(lib):
    """Appendix B.2 structure: with rounded block sums, replacing row 40 (of 40, padded to 48) changes
    output rows 4, 16, 28 and 40 only; the classical product changes row 40 only."""
    A = np.zeros((48, 512))
    A[:40] = gen.normal(21, 1, (40, 512))
    B = gen.normal(21, 2, (512, 512))
    A2 = A.copy()
    A2[39] = gen.normal(21, 89, (512,))
    s = lib.scheme_builtin("strassen444")
    outs, outs_cl = [], []
    for a in (A, A2):
        At, _ = gu.storage_pair(a, "f32")
        Bt, _ = gu.storage_pair(B, "f32")
        # M/m = 12 rows per block is legal (no alignment rule on rows)
        outs.append(gu.run_scheme_gemm(s, At, Bt, "f32", "e4m3", "f32"))
        outs_cl.append(gu.run_classical(At, Bt, "f32", "e4m3", "f32"))
    changed = {i for i in range(48) if np.any(outs[0][i] != outs[1][i])}
    assert changed == {3, 15, 27, 39}
    assert {i for i in range(48) if np.any(outs_cl[0][i] != outs_cl[1][i])} == {39}


# ---------------------------------------------------------------------------- controls and references
@pytest.mark.parametrize("M,K,N,S,Pd,O,scale,wl", [
    (384, 320, 264, "bf16", "bf16", "f32", 0, False),      # direct path (operands read in place after transpose)
    (512, 1024, 768, "bf16", "bf16", "bf16", 0, True),     # direct path, weight layout
    (256, 256, 256, "f32", "bf16", "f32", 0, False),       # conversion pass fp32 -> bf16
    (384, 2240, 264, "bf16", "e4m3", "bf16", 1, False),    # fp8 with per-tensor scales
    (384, 2240, 264, "bf16", "e4m3", "f32", 2, False),     # fp8 with per-row / per-column scales
    (128, 128, 128, "f32", "e4m3", "f32", 2, True),
    (384, 2048, 528, "bf16", "e4m3", "bf16", 3, True),     # the deployed FP8 kernel's schedule: 1 x 128 and 128 x 128 scales
    (200, 1024, 264, "f32", "e4m3", "f32", 3, False),
])
def test_classical_and_exact_match_oracle(lib, M, K, N, S, Pd, O, scale, wl):
    At, Bt, A64, B64 = _inputs(9, M, K, N, S, "llm")
    Bdev = Bt.t().contiguous() if wl else Bt
    Cc = gu.run_classical(At, Bdev, S, Pd, O, weight_layout=wl, scale_mode=scale)
    assert gu.rel_fro(Cc, oracle.classical_gemm(A64, B64, Pd, O, scale)) <= TOL_FRO
    Cs = gu.run_exact(At, Bdev, S, weight_layout=wl).cpu().numpy()
    assert gu.rel_fro(Cs, oracle.exact_gemm(A64, B64)) <= 1e-14


def test_error_frobenius_matches_oracle(lib):
    At, Bt, A64, B64 = _inputs(10, 384, 320, 264, "bf16", "llm")
    Cs = gu.run_exact(At, Bt, "bf16")
    for O, td in (("bf16", torch.bfloat16), ("f32", torch.float32)):
        Cc64 = gu.run_classical(At, Bt, "bf16", "bf16", O)
        Cc = torch.from_numpy(Cc64).to(td).cuda()
        d = lib.GemmDesc.make(384, 320, 264, "bf16", "bf16", O)
        out = torch.zeros(2, dtype=torch.float64, device="cuda")
        ws = gu.workspace(64 * 1024)
        lib.error_frobenius(d, Cc, Cs, out, ws)
        e, nrm = out.cpu().tolist()
        eo, no = oracle.fro_err(Cc64, Cs.cpu().numpy())
        assert math.isclose(e, eo, rel_tol=1e-10) and math.isclose(nrm, no, rel_tol=1e-10)


# ---------------------------------------------------------------------------- sweeps
def _oracle_ratios(so, P, Q, S, A64, B64, Pd, O, scale=0, level=0):
    Cs = oracle.exact_gemm(A64, B64)
    Ecl = oracle.rel_error(oracle.classical_gemm(A64, B64, Pd, O, scale), Cs)
    out = []
    for g in range(P.shape[0]):
        if level == 1:
            s1 = oracle.strassen()
            sg = oracle.kron(oracle.gauge(s1, P[g], Q[g], S[g]), s1)
        else:
            sg = oracle.gauge(so, P[g], Q[g], S[g])
        out.append(oracle.error_ratio(oracle.rel_error(oracle.scheme_gemm(sg, A64, B64, Pd, O, scale), Cs), Ecl))
    return np.array(out), Ecl


def test_config1_identity_plus_8_gauges(lib):
    """Config 1: one-level Strassen on fp32 256^3, bf16 products; identity + 8 GL2 gauges with cond <= 10."""
    At, Bt, A64, B64 = _inputs(0, 256, 256, 256, "f32", "normal")
    P = np.stack([np.eye(2)] + [gen.gauge_cond_limited(0, 3 * g, 2) for g in range(8)])
    Q = np.stack([np.eye(2)] + [gen.gauge_cond_limited(0, 3 * g + 1, 2) for g in range(8)])
    S = np.stack([np.eye(2)] + [gen.gauge_cond_limited(0, 3 * g + 2, 2) for g in range(8)])
    s1, so = lib.scheme_builtin("strassen222"), oracle.strassen()
    d = lib.GemmDesc.make(256, 256, 256, "f32", "bf16", "f32")
    ws = gu.workspace(lib.error_sweep_workspace(s1, d, 9))
    ratios, summ = lib.error_sweep(s1, 0, P, Q, S, d, At, Bt, ws)
    want, Ecl = _oracle_ratios(so, P, Q, S, A64, B64, "bf16", "f32")
    assert np.all(np.abs(ratios - want) <= TOL_RATIO * want)
    assert math.isclose(summ["e_classical_rel"], Ecl, rel_tol=TOL_RATIO)
    ws_sum = oracle.summary(ratios)
    for key in ("min", "median", "max", "spread", "count_gt2"):
        assert summ[key] == ws_sum[key]
    # C itself for the identity gauge and every cond <= 10 gauge
    for g in range(9):
        sg = lib.gauge_apply(s1, P[g], Q[g], S[g], cond_limit=10.0)
        C = gu.run_scheme_gemm(sg, At, Bt, "f32", "bf16", "f32")
        Co = oracle.scheme_gemm(oracle.gauge(so, P[g], Q[g], S[g]), A64, B64, "bf16", "f32")
        assert gu.rel_fro(C, Co) <= TOL_FRO


def test_sweep_log_uniform_gauges_bf16_and_outer_level_fp8(lib):
    At, Bt, A64, B64 = _inputs(11, 256, 512, 384, "bf16", "llm")
    G = 6
    P = np.stack([gen.gauge_log_uniform_cond(1, 3 * g, 2) for g in range(G)])
    Q = np.stack([gen.gauge_log_uniform_cond(1, 3 * g + 1, 2) for g in range(G)])
    S = np.stack([gen.gauge_log_uniform_cond(1, 3 * g + 2, 2) for g in range(G)])
    # one level, bf16 (config 3 in small)
    s1 = lib.scheme_builtin("strassen222")
    d = lib.GemmDesc.make(256, 512, 384, "bf16", "bf16", "bf16")
    ws = gu.workspace(lib.error_sweep_workspace(s1, d, G))
    ratios, _ = lib.error_sweep(s1, 0, P, Q, S, d, At, Bt, ws)
    want, _ = _oracle_ratios(oracle.strassen(), P, Q, S, A64, B64, "bf16", "bf16")
    assert np.all(np.abs(ratios - want) <= TOL_RATIO * want)
    # two level, gauge on the outer factor, fp8 with scales (config 5 in small), reference supplied
    s2 = lib.scheme_builtin("strassen444")
    d2 = lib.GemmDesc.make(256, 512, 384, "bf16", "e4m3", "bf16", scale_mode=1)
    ws2 = gu.workspace(lib.error_sweep_workspace(s2, d2, G))
    Cs = gu.run_exact(At, Bt, "bf16")
    ratios2, _ = lib.error_sweep(s2, 1, P, Q, S, d2, At, Bt, ws2, Cstar=Cs)
    want2, _ = _oracle_ratios(None, P, Q, S, A64, B64, "e4m3", "bf16", scale=1, level=1)
    assert np.all(np.abs(ratios2 - want2) <= TOL_RATIO * want2)
    # 512 sign variants through the same entry point: a sample of them, diagonal +-1 in GL4
    var = oracle.sign_variants(4, 4, 4)[::103]
    Pd_ = np.stack([np.diag(v[0]) for v in var]); Qd = np.stack([np.diag(v[1]) for v in var]); Sd = np.stack([np.diag(v[2]) for v in var])
    ws3 = gu.workspace(lib.error_sweep_workspace(s2, d2, len(var)))
    ratios3, _ = lib.error_sweep(s2, 0, Pd_, Qd, Sd, d2, At, Bt, ws3, Cstar=Cs)
    o2 = gu.oracle_scheme("strassen444")
    Cs64 = Cs.cpu().numpy()
    Ecl = oracle.rel_error(oracle.classical_gemm(A64, B64, "e4m3", "bf16", 1), Cs64)
    for r, v in zip(ratios3, var):
        E = oracle.rel_error(oracle.scheme_gemm(oracle.sign_variant(o2, *v), A64, B64, "e4m3", "bf16", 1), Cs64)
        assert abs(r - E / Ecl) <= TOL_RATIO * E / Ecl


@pytest.mark.parametrize("Pd,scale", [("bf16", 0), ("e4m3", 1), ("e4m3", 2), ("e4m3", 3)])
def test_all_zero_operands(lib, Pd, scale):
    """Degenerate input: an all-zero operand gives scales of one (no division by a zero maximum), a zero product, and
    a ratio of 1 in the sweep (both errors vanish)."""
    M, K, N = 256, 512, 384
    At, Bt, A64, B64 = _inputs(13, M, K, N, "bf16", "llm")
    Z = torch.zeros_like(At)
    s, so = lib.scheme_builtin("strassen444"), gu.oracle_scheme("strassen444")
    C, p, _ = gu.run_scheme_gemm(s, Z, Bt, "bf16", Pd, "bf16", scale_mode=scale, parts=True)
    Co, po = oracle.scheme_gemm(so, np.zeros_like(A64), B64, pd=Pd, od="bf16", scale_mode=scale, parts=True)
    assert np.all(C == 0.0) and np.all(Co == 0.0)
    assert np.all(p["Ahat"] == 0.0) and np.array_equal(p["BhatT"], po["Bhat"].transpose(0, 2, 1))
    if scale:
        assert np.all(p["sA"] == 1.0) and np.array_equal(p["sA"], po["sA"]) and np.array_equal(p["sB"], po["sB"])
    d = lib.GemmDesc.make(M, K, N, "bf16", Pd, "bf16", scale_mode=scale)
    I4 = np.eye(4)[None]
    ws = gu.workspace(lib.error_sweep_workspace(s, d, 1))
    ratios, summ = lib.error_sweep(s, 0, I4, I4, I4, d, Z, Bt, ws)
    assert ratios[0] == 1.0 and summ["e_classical_rel"] == 0.0 and summ["norm_ref"] == 0.0


def test_one_product_scheme_and_nan_containment(lib):
    """<1,1,1;1> (one product, no block sums) and <2,2,2;8> are the classical algorithm written as schemes: every step
    against the oracle.  A NaN in one block of A reaches exactly the outputs the oracle says it reaches: products whose
    block sum does not read that block are untouched (zero coefficients are skipped, not multiplied)."""
    At, Bt, A64, B64 = _inputs(14, 256, 256, 256, "bf16", "normal")
    for name, so in (("classical111", oracle.classical_scheme(1, 1, 1)), ("classical222", oracle.classical_scheme(2, 2, 2))):
        s = lib.scheme_builtin(name)
        C, p, _ = gu.run_scheme_gemm(s, At, Bt, "bf16", "bf16", "f32", parts=True)
        Co, po = oracle.scheme_gemm(so, A64, B64, pd="bf16", od="f32", parts=True)
        assert np.array_equal(p["Ahat"], po["Ahat"]) and gu.rel_fro(p["M"], po["M"]) <= 1e-5 and gu.rel_fro(C, Co) <= TOL_FRO
    An = At.clone(); An[3, 200] = float("nan")                 # block (0, 1) of a 2 x 2 grid
    A64n = A64.copy(); A64n[3, 200] = np.nan
    s1, o1 = lib.scheme_builtin("strassen222"), oracle.strassen()
    C = gu.run_scheme_gemm(s1, An, Bt, "bf16", "bf16", "f32")
    Co = oracle.scheme_gemm(o1, A64n, B64, "bf16", "f32")
    assert np.array_equal(np.isnan(C), np.isnan(Co))
    assert 0 < np.isnan(Co).sum() < Co.size                    # row 3 of the blocks fed by products that read A_12, nothing else
    ok = ~np.isnan(Co)
    assert gu.rel_fro(C[ok], Co[ok]) <= TOL_FRO


@pytest.mark.parametrize("scheme,M,K,N", [("strassen444", 4, 64, 32), ("strassen222", 2, 32, 16), ("strassen444", 12, 192, 96)])
@pytest.mark.parametrize("Pd,scale", [("bf16", 0), ("e4m3", 1), ("e4m3", 3)])
def test_smallest_legal_shapes(lib, scheme, M, K, N, Pd, scale):
    """One row per block, sixteen inner indices, eight columns: far below one tile in every dimension."""
    At, Bt, A64, B64 = _inputs(15, M, K, N, "bf16", "normal")
    s, so = lib.scheme_builtin(scheme), gu.oracle_scheme(scheme)
    C, p, _ = gu.run_scheme_gemm(s, At, Bt, "bf16", Pd, "f32", scale_mode=scale, parts=True)
    Co, po = oracle.scheme_gemm(so, A64, B64, pd=Pd, od="f32", scale_mode=scale, parts=True)
    assert np.array_equal(p["Ahat"], po["Ahat"]) and np.array_equal(p["BhatT"], po["Bhat"].transpose(0, 2, 1))
    assert gu.rel_fro(p["M"], po["M"]) <= 1e-5 and gu.rel_fro(C, Co) <= TOL_FRO
    m = so.dims[0]
    # the sweep with bf16 outputs: with bf16 storage and products the classical error is the output rounding alone
    d = lib.GemmDesc.make(M, K, N, "bf16", Pd, "bf16", scale_mode=scale)
    G = 5
    var = oracle.sign_variants(m, m, m)[:G]
    P = np.stack([np.diag(v[0]) for v in var]); Q = np.stack([np.diag(v[1]) for v in var]); S = np.stack([np.diag(v[2]) for v in var])
    ws = gu.workspace(lib.error_sweep_workspace(s, d, G))
    ratios, _ = lib.error_sweep(s, 0, P, Q, S, d, At, Bt, ws)
    Cs = A64 @ B64
    Ecl = oracle.rel_error(oracle.classical_gemm(A64, B64, Pd, "bf16", scale), Cs)
    for r, v in zip(ratios, var):
        E = oracle.rel_error(oracle.scheme_gemm(oracle.sign_variant(so, *v), A64, B64, Pd, "bf16", scale), Cs)
        assert abs(r - E / Ecl) <= TOL_RATIO * E / Ecl


def test_host_buffer_entry_point_is_the_same_operator(lib):
    """scheme_gemm_host: operands in (pinned) host memory with padded leading dimensions, result copied back; the
    same bits as scheme_gemm on device tensors, also with the weight's block sums reused and no weight passed."""
    M, K, N = 384, 320, 288
    At, Bt, A64, B64 = _inputs(5, M, K, N, "bf16", "llm")
    s = lib.scheme_builtin("strassen444")
    want = gu.run_scheme_gemm(s, At, Bt, "bf16", "e4m3", "bf16", scale_mode=1)
    lda, ldb, ldc = K + 8, N + 16, N + 24
    Ah = torch.zeros((M, lda), dtype=torch.bfloat16).pin_memory(); Ah[:, :K] = At.cpu()
    Bh = torch.zeros((K, ldb), dtype=torch.bfloat16).pin_memory(); Bh[:, :N] = Bt.cpu()
    Ch = torch.full((M, ldc), 7.0, dtype=torch.bfloat16).pin_memory()
    d = lib.GemmDesc.make(M, K, N, "bf16", "e4m3", "bf16", scale_mode=1)
    d.lda, d.ldb, d.ldc = lda, ldb, ldc
    ws = gu.workspace(lib.scheme_gemm_host_workspace(s, d))
    lib.scheme_gemm_host(s, d, Ah, Bh, Ch, ws)
    lib.scheme_gemm_host_status(s, d, ws)
    assert np.array_equal(Ch[:, :N].double().numpy(), want) and torch.all(Ch[:, N:] == 7.0)
    d2 = lib.GemmDesc.make(M, K, N, "bf16", "e4m3", "bf16", scale_mode=1, flags=lib.FLAG_REUSE_BHAT)
    d2.lda, d2.ldb, d2.ldc = lda, ldb, ldc
    Ch.fill_(0.0)
    lib.scheme_gemm_host(s, d2, Ah, None, Ch, ws)
    lib.scheme_gemm_host_status(s, d2, ws)
    assert np.array_equal(Ch[:, :N].double().numpy(), want)
    with pytest.raises(lib.FmmError):
        lib.scheme_gemm_host(s, d, Ah, None, Ch, ws)             # no weight and nothing to reuse


def test_sweep_batches_walk_several_tiles_per_block(lib):
    """Blocks of 512 x 1024 outputs: every decode block of the batched sweep walks four tiles, so the double-buffered
    stages (products and staged reference values) are reused; ratios against the oracle for 4 + 2 + 1 gauges."""
    At, Bt, A64, B64 = _inputs(21, 1024, 256, 2048, "bf16", "llm")
    G = 7
    P = np.stack([gen.gauge_log_uniform_cond(2, 3 * g, 2) for g in range(G)])
    Q = np.stack([gen.gauge_log_uniform_cond(2, 3 * g + 1, 2) for g in range(G)])
    S = np.stack([gen.gauge_log_uniform_cond(2, 3 * g + 2, 2) for g in range(G)])
    s1 = lib.scheme_builtin("strassen222")
    d = lib.GemmDesc.make(1024, 256, 2048, "bf16", "bf16", "bf16")
    ws = gu.workspace(lib.error_sweep_workspace(s1, d, G))
    ratios, _ = lib.error_sweep(s1, 0, P, Q, S, d, At, Bt, ws)
    want, _ = _oracle_ratios(oracle.strassen(), P, Q, S, A64, B64, "bf16", "bf16")
    assert np.all(np.abs(ratios - want) <= TOL_RATIO * want)
    # repeated runs give the same bits (Appendix B, repeated runs); a gauge swept alone gives the same ratio up to the
    # partition of its error sum (every C is the same bits, the squares are added in another grouping)
    again, _ = lib.error_sweep(s1, 0, P, Q, S, d, At, Bt, ws)
    assert np.array_equal(again, ratios)
    alone = np.array([lib.error_sweep(s1, 0, P[g:g + 1], Q[g:g + 1], S[g:g + 1], d, At, Bt, ws)[0][0] for g in range(G)])
    assert np.all(np.abs(alone - ratios) <= 1e-6 * ratios)


# ---------------------------------------------------------------------------- full size, sampled
def test_config3_full_size_sweep_against_the_oracle(lib):
    """The sweep exactly as bench.py times it (A 2048 x 4096, B 4096 x 4096 stored [N, K], bf16, batches of four
    algorithms, fourteen tiles per decode block): the ratios of five of the configuration's gauges against the
    oracle's full-size products (a 4 + 1 split of the batch)."""
    import bench
    At_h, Bt_h = bench.c3_inputs(0)
    At, Bt = At_h.cuda(), Bt_h.cuda()
    A64, B64 = At_h.double().numpy(), Bt_h.double().numpy().T.copy()
    P, Q, S = bench.sweep_gauges(512)
    pick = [0, 100, 200, 300, 511]
    P, Q, S = P[pick], Q[pick], S[pick]
    s1 = lib.scheme_builtin("strassen222")
    d = lib.GemmDesc.make(2048, 4096, 4096, "bf16", "bf16", "bf16", weight_layout=True)
    ws = gu.workspace(lib.error_sweep_workspace(s1, d, len(pick)))
    ratios, summ = lib.error_sweep(s1, 0, P, Q, S, d, At, Bt, ws)
    want, Ecl = _oracle_ratios(oracle.strassen(), P, Q, S, A64, B64, "bf16", "bf16")
    assert math.isclose(summ["e_classical_rel"], Ecl, rel_tol=TOL_RATIO)
    assert np.all(np.abs(ratios - want) <= TOL_RATIO * want), (ratios, want)


def test_config2_full_size_sampled_outputs(lib):
    """Config 2 at full size in the launch configuration the benchmark times (bf16, weight layout):
    sampled rows/columns recomputed by the oracle one by one (a scheme acts position-wise on blocks)."""
    M = K = N = 4096
    A = gen.activations_outlier(0, 1, M, K, frac=0.005, factor=100.0)
    B = gen.weights(0, 2, K, N)
    At, A64 = gu.storage_pair(A, "bf16")
    Bt, B64 = gu.storage_pair(B, "bf16")
    s = lib.scheme_builtin("strassen444")
    C = gu.run_scheme_gemm(s, At, Bt.t().contiguous(), "bf16", "bf16", "bf16", weight_layout=True)
    rows = [0, 1, 127, 128, 511, 640, 1000, 1023]
    cols = [0, 5, 255, 256, 300, 767, 1022, 1023]
    As, Bs, ridx, cidx = gu.subsample_problem(A64, B64, 4, 4, 4, rows, cols)
    Co = oracle.scheme_gemm(gu.oracle_scheme("strassen444"), As, Bs, "bf16", "bf16")
    got = C[np.ix_(ridx, cidx)]
    assert gu.rel_fro(got, Co) <= TOL_FRO
    # and the whole result is close to the exact product at the level the rounding allows
    Cs = gu.run_exact(At, Bt, "bf16").cpu().numpy()
    assert gu.rel_fro(C, Cs) < 0.05
    # every one of the 16.8 M outputs against the oracle's full-size run (about two seconds of host time): the block
    # sums are the same bits on both sides, so outputs differ only where fp32 against fp64 accumulation moves a value
    # across a bf16 rounding boundary — by one unit in the last place, on a small fraction of the entries (0.11 %)
    Cfull = oracle.scheme_gemm(gu.oracle_scheme("strassen444"), A64, B64, "bf16", "bf16")
    assert gu.rel_fro(C, Cfull) <= TOL_FRO
    diff = C != Cfull
    assert diff.mean() < 0.02, diff.mean()
    ulp = np.exp2(np.floor(np.log2(np.maximum(np.maximum(np.abs(Cfull), np.abs(C)), 1e-30))) - 7)   # of the larger neighbour
    noise = 2.0 ** -17 * np.sqrt(np.mean(Cfull ** 2))     # fp32 accumulation noise, visible where the terms of an output cancel
    assert np.all(np.abs(C - Cfull)[diff] <= 1.0001 * ulp[diff] + noise)


@pytest.mark.parametrize("Pd,scale", [("bf16", 0), ("e4m3", 2)])
def test_largest_benchmark_shape_sampled_outputs(lib, Pd, scale):
    """The largest GEMM of the benchmark configurations (8192 tokens, K = 5120, N = 27648; 2.8 GB of products),
    weight layout: sampled rows / columns against the oracle.  With row / column scales the sub-problem keeps the
    whole inner dimension, so its scales are the full problem's."""
    M, K, N = 8192, 5120, 27648
    A = gen.activations_outlier(2, 1, M, K, dist="t3", frac=0.001, factor=300.0, at_least=1)
    B = gen.weights(2, 2, K, N)
    At, A64 = gu.storage_pair(A, "bf16")
    Bt, B64 = gu.storage_pair(B, "bf16")
    s = lib.scheme_builtin("strassen444")
    C = gu.run_scheme_gemm(s, At, Bt.t().contiguous(), "bf16", Pd, "bf16", weight_layout=True, scale_mode=scale)
    rows = [0, 129, 1023, 1024, 2047]
    cols = [0, 7, 255, 256, 4095, 4096, 6911]
    As, Bs, ridx, cidx = gu.subsample_problem(A64, B64, 4, 4, 4, rows, cols)
    Co = oracle.scheme_gemm(gu.oracle_scheme("strassen444"), As, Bs, Pd, "bf16", scale_mode=scale)
    assert gu.rel_fro(C[np.ix_(ridx, cidx)], Co) <= TOL_FRO


# ---------------------------------------------------------------------------- failure reporting
def test_bounded_wait_expires_reports_timeout_and_context_survives(lib):
    """A wait that nothing will ever satisfy (the copy-issuing warp of one block is switched off) must run out,
    leave FMM_ERR_TIMEOUT in the status word and return; the next ordinary call must work."""
    ws = gu.workspace(256 * 1024)
    lib.selftest_timeout(ws, wait_ms=50)
    with pytest.raises(lib.FmmError) as err:
        lib.device_status(ws)
    assert err.value.code == 8
    torch.cuda.synchronize()
    At, Bt, A64, B64 = _inputs(13, 256, 256, 256, "bf16", "int", 3)
    C = gu.run_scheme_gemm(lib.scheme_builtin("strassen222"), At, Bt, "bf16", "bf16", "f32")
    assert np.array_equal(C, A64 @ B64)


def test_sign_variant_ensemble_on_the_device(lib):
    """Appendix B.1: all 512 sign variants of two-level Strassen on synthetic 128 x 128 operands, e4m3 block sums
    with one scale per row / column, through error_sweep.  Per-variant errors agree with the oracle on a sample;
    the ensemble statistics land where the paper prints them (2.59 / 0.9997 on U[0,1], 1.005 / 0.121 on U[-1,1])."""
    var = oracle.sign_variants(4, 4, 4)
    P = np.stack([np.diag(v[0]) for v in var]); Q = np.stack([np.diag(v[1]) for v in var]); S = np.stack([np.diag(v[2]) for v in var])
    s2, o2 = lib.scheme_builtin("strassen444"), gu.oracle_scheme("strassen444")
    d = lib.GemmDesc.make(128, 128, 128, "f32", "e4m3", "f32", scale_mode=2)
    ws = gu.workspace(lib.error_sweep_workspace(s2, d, len(var)))
    pairs = 24
    stats = {}
    for kind, seed in (("u01", 71), ("upm1", 72)):
        errs = np.empty((len(var), pairs))
        for p in range(pairs):
            At, Bt, A64, B64 = _inputs(seed + 100 * p, 128, 128, 128, "f32", kind)
            ratios, summ = lib.error_sweep(s2, 0, P, Q, S, d, At, Bt, ws)
            errs[:, p] = ratios * summ["e_classical_rel"]
            if p == 0:       # parity of a sample of variants against the oracle
                Cs = A64 @ B64
                Ecl = oracle.rel_error(oracle.classical_gemm(A64, B64, "e4m3", "f32", 2), Cs)
                assert math.isclose(summ["e_classical_rel"], Ecl, rel_tol=TOL_RATIO)
                for vi in range(0, len(var), 57):
                    E = oracle.rel_error(oracle.scheme_gemm(oracle.sign_variant(o2, *var[vi]), A64, B64, "e4m3", "f32", 2), Cs)
                    assert abs(errs[vi, 0] - E) <= TOL_RATIO * E
        avg = errs.mean(axis=1)
        stats[kind] = (avg.max() / avg.min(), float(np.corrcoef(errs[:, 0::2].mean(axis=1), errs[:, 1::2].mean(axis=1))[0, 1]))
    assert abs(stats["u01"][0] - 2.59) < 0.12 * 2.59 and stats["u01"][1] > 0.99, stats
    assert 1.0 <= stats["upm1"][0] < 1.03 and abs(stats["upm1"][1]) < 0.6, stats


def test_decode_order_is_part_of_the_operator(lib):
    """Products renumbered (Appendix B.1's summation-order observation): exact on integers, equal to the oracle run on
    the same renumbered coefficients, and on real data a different fp32 result from the original order."""
    s2, o2 = lib.scheme_builtin("strassen444"), gu.oracle_scheme("strassen444")
    perm = np.random.default_rng(9).permutation(49)
    sp = lib.scheme_permute_products(s2, perm)
    op = oracle.Scheme(o2.U[perm], o2.V[perm], o2.W[perm])
    At, Bt, A64, B64 = _inputs(15, 256, 512, 256, "bf16", "int", 4)
    assert np.array_equal(gu.run_scheme_gemm(sp, At, Bt, "bf16", "bf16", "f32"), A64 @ B64)
    At, Bt, A64, B64 = _inputs(16, 512, 1024, 512, "bf16", "llm")
    C0 = gu.run_scheme_gemm(s2, At, Bt, "bf16", "bf16", "f32")
    C1 = gu.run_scheme_gemm(sp, At, Bt, "bf16", "bf16", "f32")
    assert gu.rel_fro(C1, oracle.scheme_gemm(op, A64, B64, "bf16", "f32")) <= TOL_FRO
    assert not np.array_equal(C0, C1) and gu.rel_fro(C0, C1) < 1e-5


def test_sweep_under_the_model_schedule(lib):
    """error_sweep with the model schedule (group scales, products returned in bf16): ratios against the oracle."""
    At, Bt, A64, B64 = _inputs(19, 256, 1024, 512, "bf16", "t3")
    var = oracle.sign_variants(4, 4, 4)[::85]
    P = np.stack([np.diag(v[0]) for v in var]); Q = np.stack([np.diag(v[1]) for v in var]); S = np.stack([np.diag(v[2]) for v in var])
    s2, o2 = lib.scheme_builtin("strassen444"), gu.oracle_scheme("strassen444")
    d = lib.GemmDesc.make(256, 1024, 512, "bf16", "e4m3", "bf16", scale_mode=3, flags=lib.FLAG_PRODUCTS_BF16)
    ws = gu.workspace(lib.error_sweep_workspace(s2, d, len(var)))
    ratios, summ = lib.error_sweep(s2, 0, P, Q, S, d, At, Bt, ws)
    Cs = A64 @ B64
    Ecl = oracle.rel_error(oracle.classical_gemm(A64, B64, "e4m3", "bf16", 3), Cs)
    assert math.isclose(summ["e_classical_rel"], Ecl, rel_tol=TOL_RATIO)
    for r, v in zip(ratios, var):
        E = oracle.rel_error(oracle.scheme_gemm(oracle.sign_variant(o2, *v), A64, B64, "e4m3", "bf16", 3, md="bf16"), Cs)
        assert abs(r - E / Ecl) <= TOL_RATIO * E / Ecl
