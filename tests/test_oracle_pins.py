"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test is chosen so that a plausible mistake in the oracle (dropped term, wrong sign or
index, transposed operand, rounding in the wrong place, ties rounded away) fails it.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from fmm_inputs import generators as gen

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *v = line.split()
            out[k] = [float(x) for x in v]
    return out


S1 = oracle.strassen()
S2 = oracle.kron(S1, S1)


# ---------------------------------------------------------------- printed examples / constants
def test_hand_example_exact():
    g = _golden("strassen_hand_examples.txt")
    A = np.array(g["exact_A"]).reshape(2, 2)
    B = np.array(g["exact_B"]).reshape(2, 2)
    Cm, parts = oracle.scheme_gemm(S1, A, B, pd="f64", od="f64", parts=True)
    assert parts["M"].reshape(7).tolist() == g["exact_M"]
    assert Cm.reshape(4).tolist() == g["exact_C"]


def test_hand_example_rounding_placement():
    """Block sums, not inputs, are rounded; ties go to even."""
    g = _golden("strassen_hand_examples.txt")
    A = np.array(g["round_A"]).reshape(2, 2)
    B = np.array(g["round_B"]).reshape(2, 2)
    Cm, parts = oracle.scheme_gemm(S1, A, B, pd="bf16", od="f32", parts=True)
    assert parts["M"].reshape(7).tolist() == g["round_M"]
    assert Cm.reshape(4).tolist() == g["round_C"]
    Ccl = oracle.classical_gemm(A, B, pd="bf16", od="f32")
    assert Ccl.reshape(4).tolist() == g["round_classical_C"]
    assert oracle.exact_gemm(A, B).reshape(4).tolist() == g["round_classical_C"]


def test_printed_constants_two_level():
    g = _golden("two_level_strassen_constants.txt")
    m, k, n, R = S2.dims
    assert (m, k, n) == (4, 4, 4) and R == g["R"][0]
    assert m * k * n == g["R_classical"][0]
    assert round(R / (m * k * n), 4) == g["mult_ratio"][0]
    c = oracle.criteria(S2)
    for key in ("L_A", "L_B", "L_W", "Phi", "nnz", "maxabs"):
        assert c[key] == g[key][0], key
    b = math.floor(127 / c["L_A"])
    assert b == g["code_bound"][0]
    # largest h with L_W h (L_A b)(L_B b) < 2^31  (certificate condition (ii))
    h = (2 ** 31 - 1) // int(c["L_W"] * (c["L_A"] * b) * (c["L_B"] * b))
    assert h == g["h_max_int32"][0]
    assert round(127 / b, 4) == g["step_ratio"][0]
    assert len(oracle.sign_variants(4, 4, 4)) == g["sign_variants"][0]
    # the two remaining metadata entries: hand-evaluated from the printed product table (the paper prints no value)
    h = _golden("ballard_criteria_hand.txt")
    assert c["Q"] == h["Q_two_level"][0] and c["E"] == h["E_two_level"][0]
    c1 = oracle.criteria(S1)
    assert c1["Q"] == h["Q_one_level"][0] and c1["E"] == h["E_one_level"][0]


def test_strassen_reads_feeds_table():
    """Appendix A.1 table: which block rows of A each product reads, which rows of C it feeds."""
    reads = [{1, 2}, {2}, {1}, {2}, {1}, {1, 2}, {1, 2}]
    feeds = [{1, 2}, {2}, {1, 2}, {1, 2}, {1}, {2}, {1}]
    for r in range(7):
        assert {i + 1 for i in range(2) if np.any(S1.U[r, i, :] != 0)} == reads[r]
        assert {i + 1 for i in range(2) if np.any(S1.W[r, i, :] != 0)} == feeds[r]


# ---------------------------------------------------------------- Brent equations / exactness
def test_brent_exact_and_negative_control():
    assert oracle.brent_residual(S1) == 0.0
    assert oracle.brent_residual(S2) == 0.0
    W = S1.W.copy()
    W[3, 0, 0] = -W[3, 0, 0]          # deliberate sign flip in one decoding coefficient
    bad = oracle.Scheme(S1.U, S1.V, W)
    assert oracle.brent_residual(bad) >= 1.0
    A = gen.integer_matrix(3, 1, (8, 8), 5)
    B = gen.integer_matrix(3, 2, (8, 8), 5)
    assert not np.array_equal(oracle.scheme_gemm(bad, A, B, pd="bf16", od="f32"), A @ B)


def _triple_loop(A, B):
    M, K = A.shape
    N = B.shape[1]
    Cm = np.zeros((M, N))
    for i in range(M):
        for j in range(N):
            s = 0.0
            for t in range(K):
                s += A[i, t] * B[t, j]
            Cm[i, j] = s
    return Cm


@pytest.mark.parametrize("scheme,size", [(S1, 4), (S1, 8), (S2, 8), (S2, 12)])
def test_integer_matrices_reproduce_triple_loop(scheme, size):
    A = gen.integer_matrix(11, 1, (size, size), 7)
    B = gen.integer_matrix(11, 2, (size, size), 7)
    ref = _triple_loop(A, B)
    assert np.array_equal(oracle.scheme_gemm(scheme, A, B, pd="f64", od="f64"), ref)
    assert np.array_equal(oracle.scheme_gemm(scheme, A, B, pd="bf16", od="f32"), ref)
    assert np.array_equal(oracle.classical_gemm(A, B, pd="bf16", od="f32"), ref)
    assert np.array_equal(oracle.exact_gemm(A, B), ref)


def test_rectangular_blocks_and_transposition_sensitivity():
    """Non-square M,K,N with a non-symmetric grid catch transposed operands / swapped strides."""
    rect = oracle.kron(oracle.classical_scheme(1, 2, 1), S1)     # <2,4,2;14>
    assert oracle.brent_residual(rect) == 0.0
    A = gen.integer_matrix(5, 1, (6, 16), 6)
    B = gen.integer_matrix(5, 2, (16, 10), 6)
    assert np.array_equal(oracle.scheme_gemm(rect, A, B, pd="bf16", od="f32"), _triple_loop(A, B))
    assert np.array_equal(oracle.classical_gemm(A, B, pd="bf16", od="f32"), _triple_loop(A, B))


def test_hand_expanded_strassen_with_library_rounding():
    """Strassen's seven formulas typed out, block sums cast to bf16 by torch, fp64 products."""
    A = gen.normal(2, 1, (8, 8))
    B = gen.normal(2, 2, (8, 8))
    _, A = gen.to_storage(A, "f32")
    _, B = gen.to_storage(B, "f32")
    h = 4
    A11, A12, A21, A22 = A[:h, :h], A[:h, h:], A[h:, :h], A[h:, h:]
    B11, B12, B21, B22 = B[:h, :h], B[:h, h:], B[h:, :h], B[h:, h:]

    def q(x):  # fp32 sum of two fp32 values, then one bf16 cast
        return torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()

    f = np.float32
    M1 = q(f(A11) + f(A22)) @ q(f(B11) + f(B22))
    M2 = q(f(A21) + f(A22)) @ q(f(B11))
    M3 = q(f(A11)) @ q(f(B12) - f(B22))
    M4 = q(f(A22)) @ q(f(B21) - f(B11))
    M5 = q(f(A11) + f(A12)) @ q(f(B22))
    M6 = q(f(A21) - f(A11)) @ q(f(B11) + f(B12))
    M7 = q(f(A12) - f(A22)) @ q(f(B21) + f(B22))
    ref = np.block([[M1 + M4 - M5 + M7, M3 + M5], [M2 + M4, M1 - M2 + M3 + M6]])
    got = oracle.scheme_gemm(S1, A, B, pd="bf16", od="f64")
    assert np.allclose(got, ref, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- gauges
def test_all_sign_variants_exact_and_criteria_constant():
    base = oracle.criteria(S2)
    A = gen.integer_matrix(7, 1, (8, 8), 4)
    B = gen.integer_matrix(7, 2, (8, 8), 4)
    ref = A @ B
    variants = oracle.sign_variants(4, 4, 4)
    assert len(variants) == 512
    outs = set()
    for idx, (d, e, f) in enumerate(variants):
        s = oracle.sign_variant(S2, d, e, f)
        if idx % 16 == 0:
            assert oracle.brent_residual(s) == 0.0
        assert oracle.criteria(s) == base
        # e4m3 holds every sum of L=4 codes with |code| <= 4 (dense codebook bound)
        Cm = oracle.scheme_gemm(s, A, B, pd="e4m3", od="f32")
        outs.add(Cm.tobytes())
        # general gauge routine agrees with the printed sign formula
        if idx % 37 == 0:
            g = oracle.gauge(S2, np.diag(d), np.diag(e), np.diag(f))
            assert np.array_equal(g.U, s.U) and np.array_equal(g.V, s.V) and np.array_equal(g.W, s.W)
    assert len(outs) == 1 and outs.pop() == ref.tobytes()


def test_identity_gauge_is_bitwise_identity():
    for s in (S1, S2):
        m, k, n, _ = s.dims
        g = oracle.gauge(s, np.eye(m), np.eye(k), np.eye(n))
        assert np.array_equal(g.U, s.U) and np.array_equal(g.V, s.V) and np.array_equal(g.W, s.W)


def test_general_gauge_keeps_brent_and_exact_product():
    A = gen.normal(1, 1, (8, 12))
    B = gen.normal(1, 2, (12, 4))
    ref = oracle.exact_gemm(A, B)
    for idx in range(6):
        P = gen.gauge_log_uniform_cond(5, 3 * idx, 2)
        Q = gen.gauge_log_uniform_cond(5, 3 * idx + 1, 2)
        S = gen.gauge_cond_limited(5, 3 * idx + 2, 2)
        g = oracle.gauge(S1, P, Q, S)
        scale = 7 * np.abs(g.U).max() * np.abs(g.V).max() * np.abs(g.W).max()
        assert oracle.brent_residual(g) <= 1e-13 * scale
        Cm = oracle.scheme_gemm(g, A, B, pd="f64", od="f64")
        assert np.linalg.norm(Cm - ref) <= 1e-10 * scale * np.linalg.norm(ref)
    # a gauge on the outer factor of the nested algorithm
    P, Q, S = (gen.gauge_cond_limited(9, i, 2) for i in range(3))
    g2 = oracle.kron(oracle.gauge(S1, P, Q, S), S1)
    assert oracle.brent_residual(g2) < 1e-11
    with pytest.raises(ValueError):
        oracle.gauge(S1, np.zeros((2, 2)), np.eye(2), np.eye(2))


def test_gauge_equals_running_on_transformed_operands():
    """Definition check: the gauged algorithm on (A,B) forms the block sums of the base
    algorithm on A' = P A Q^-1, B' = Q B S^-1 (block-index action)."""
    P, Q, S = (gen.gauge_cond_limited(4, i, 2) for i in range(3))
    g = oracle.gauge(S1, P, Q, S)
    A = gen.normal(8, 1, (4, 6))
    B = gen.normal(8, 2, (6, 2))
    bm, bk, bn = 2, 3, 1
    Ab = A.reshape(2, bm, 2, bk).transpose(0, 2, 1, 3)     # [i,l,p,t]
    Bb = B.reshape(2, bk, 2, bn).transpose(0, 2, 1, 3)
    Ap = np.einsum("ia,alpt,lb->ibpt", P, Ab, np.linalg.inv(Q))
    Bp = np.einsum("la,ajpt,jb->lbpt", Q, Bb, np.linalg.inv(S))
    Apm = Ap.transpose(0, 2, 1, 3).reshape(4, 6)
    Bpm = Bp.transpose(0, 2, 1, 3).reshape(6, 2)
    _, base_parts = oracle.scheme_gemm(S1, Apm, Bpm, pd="f64", od="f64", parts=True)
    _, g_parts = oracle.scheme_gemm(g, A, B, pd="f64", od="f64", parts=True)
    assert np.allclose(base_parts["Ahat"], g_parts["Ahat"], atol=1e-12)
    assert np.allclose(base_parts["Bhat"], g_parts["Bhat"], atol=1e-12)


# ---------------------------------------------------------------- structure of the leak
def _changed_rows(f, A, B, row, seed):
    C0 = f(A, B)
    A2 = A.copy()
    _, A2[row] = gen.to_storage(gen.normal(seed, 50 + row, (A.shape[1],)), "f32")
    C1 = f(A2, B)
    return {i for i in range(A.shape[0]) if np.any(C0[i] != C1[i])}


def test_row_map_40_rows_padded_to_48():
    g = _golden("two_level_strassen_constants.txt")
    rows = int(g["rowmap_rows"][0])
    A = np.zeros((rows, 512))
    _, A[:40] = gen.to_storage(gen.normal(21, 1, (40, 512)), "f32")
    _, B = gen.to_storage(gen.normal(21, 2, (512, 512)), "f32")
    want = {int(x) - 1 for x in g["rowmap_changed"]}          # printed 1-based
    got = _changed_rows(lambda a, b: oracle.scheme_gemm(S2, a, b, pd="e4m3", od="f32"), A, B, 39, 21)
    assert got == want
    got_cl = _changed_rows(lambda a, b: oracle.classical_gemm(a, b, pd="e4m3", od="f32"), A, B, 39, 21)
    assert got_cl == {39}


def test_row_pairs_32_rows_in_4_blocks():
    g = _golden("two_level_strassen_constants.txt")
    _, A = gen.to_storage(gen.normal(22, 1, (32, 64)), "f32")
    _, B = gen.to_storage(gen.normal(22, 2, (64, 32)), "f32")
    Ai = gen.integer_matrix(22, 3, (32, 64), 4)
    Bi = gen.integer_matrix(22, 4, (64, 32), 4)
    pairs = moved = moved_int = 0
    C0 = oracle.scheme_gemm(S2, A, B, pd="e4m3", od="f32")
    C0i = oracle.scheme_gemm(S2, Ai, Bi, pd="e4m3", od="f32")
    for later in range(32):
        A2 = A.copy()
        _, A2[later] = gen.to_storage(gen.normal(22, 100 + later, (64,)), "f32")
        C1 = oracle.scheme_gemm(S2, A2, B, pd="e4m3", od="f32")
        A2i = Ai.copy()
        A2i[later] = gen.integer_matrix(22, 200 + later, (64,), 4)
        C1i = oracle.scheme_gemm(S2, A2i, Bi, pd="e4m3", od="f32")
        for earlier in range(later):
            pairs += 1
            if np.any(C0[earlier] != C1[earlier]):
                moved += 1
                assert earlier % 8 == later % 8          # same offset inside the blocks
            moved_int += int(np.any(C0i[earlier] != C1i[earlier]))
    assert pairs == g["row_pairs"][0]
    assert moved == g["moved_rounded"][0]
    assert moved_int == g["moved_integer"][0]


# ---------------------------------------------------------------- rounding helpers
def test_bf16_rounding_exhaustive_and_against_torch():
    bits = np.arange(65536, dtype=np.uint32) << 16
    with np.errstate(invalid="ignore"):
        vals = bits.view(np.float32).astype(np.float64)
    fin = np.isfinite(vals)
    assert np.array_equal(oracle.round_to(vals[fin], "bf16"), vals[fin])      # every bf16 is a fixed point
    x = gen.normal(3, 9, (200000,)).astype(np.float32) * np.float32(37.0)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(oracle.round_to(x.astype(np.float64), "bf16"), want)
    # ties to even: 257 -> 256, 259 -> 260; subnormal quantum 2^-133
    assert oracle.round_to([257.0, 259.0, 1.00390625], "bf16").tolist() == [256.0, 260.0, 1.0]
    tiny = 2.0 ** -133
    assert oracle.round_to([1.5 * tiny, 2.5 * tiny, 0.5 * tiny], "bf16").tolist() == [2 * tiny, 2 * tiny, 0.0]
    assert np.isinf(oracle.round_to([3.4e38], "bf16")[0])


def test_e4m3_rounding_exhaustive_and_against_torch():
    codes = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    fin = np.isfinite(codes)
    assert fin.sum() == 254 and np.nanmax(np.abs(codes[fin])) == 448.0
    assert np.array_equal(oracle.round_to(codes[fin], "e4m3"), codes[fin])
    x = gen.uniform(3, 10, (200000,), -448.0, 448.0).astype(np.float32)
    x = np.concatenate([x, (gen.normal(3, 11, (100000,)) * 0.01).astype(np.float32)])
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(oracle.round_to(x.astype(np.float64), "e4m3"), want)
    # ties to even at 4 significant bits, least subnormal 2^-9, saturation at 448
    assert oracle.round_to([17.0, 19.0, 2.0 ** -10, 3 * 2.0 ** -10, 449.0, 1e9, -1e9, np.inf], "e4m3").tolist() == \
        [16.0, 20.0, 0.0, 2.0 ** -8, 448.0, 448.0, -448.0, 448.0]
    assert np.isnan(oracle.round_to([np.nan], "e4m3")[0])


def test_dense_codebook_bound_e4m3():
    """Appendix D: with p = 4 and L = 4 codes per block sum, |code| <= 4 is the largest dense
    uniform codebook: every multiple up to L*J = 16 is representable, 17 is not."""
    ints = np.arange(-16, 17, dtype=np.float64)
    assert np.array_equal(oracle.round_to(ints, "e4m3"), ints)
    assert oracle.round_to([17.0], "e4m3")[0] != 17.0


# ---------------------------------------------------------------- scales, errors, summary
def test_power_of_two_scales_e4m3():
    A = gen.normal(6, 1, (8, 8)) * 1000.0
    B = gen.normal(6, 2, (8, 8)) * 1e-4
    _, A = gen.to_storage(A, "bf16")
    _, B = gen.to_storage(B, "bf16")
    Cm, parts = oracle.scheme_gemm(S1, A, B, pd="e4m3", od="f32", scale_mode=1, parts=True)
    for r in range(7):
        for s, hat in ((parts["sA"][r], parts["Ahat"][r]), (parts["sB"][r], parts["Bhat"][r])):
            assert math.log2(s) == int(math.log2(s))
            amax = np.abs(hat).max()
            assert 224.0 <= amax <= 448.0 or amax == 0.0      # fills the top binade of e4m3
    assert oracle.rel_error(Cm, oracle.exact_gemm(A, B)) < 0.2
    # integers inside the exact domain are untouched by scale mode 0
    Ai = gen.integer_matrix(6, 3, (8, 8), 4)
    Bi = gen.integer_matrix(6, 4, (8, 8), 4)
    assert np.array_equal(oracle.scheme_gemm(S2, Ai, Bi, pd="e4m3", od="f32", scale_mode=0), Ai @ Bi)


def test_error_ratio_and_summary_rules():
    Cs = np.array([[3.0, 4.0]])
    assert oracle.fro_err(np.array([[3.0, 5.0]]), Cs) == (1.0, 25.0)
    assert oracle.rel_error(np.array([[3.0, 5.0]]), Cs) == 0.2
    assert oracle.error_ratio(0.0, 0.0) == 1.0 and oracle.error_ratio(1.0, 0.0) == math.inf
    assert oracle.error_ratio(0.3, 0.1) == pytest.approx(3.0)
    s = oracle.summary([5.0, 1.0, 3.0, 2.5])              # even count: upper of the two middle values
    assert (s["min"], s["median"], s["max"], s["spread"], s["count_gt2"]) == (1.0, 3.0, 5.0, 5.0, 3)
    assert oracle.summary([4.0, 1.0, 2.0])["median"] == 2.0
    n = oracle.summary([4.0, math.nan, 1.0])              # a set with NaN has no order; the count skips it
    assert all(math.isnan(n[k]) for k in ("min", "median", "max", "spread")) and n["count_gt2"] == 1 and n["G"] == 3


def test_symmetric_vs_offset_operands_soft():
    """Appendix B.1 (soft): on operands uniform on [-1,1] sign variants are statistically alike;
    on [0,1] they differ markedly.  Small version: 16 variants x 6 pairs at 32 x 32."""
    variants = oracle.sign_variants(4, 4, 4)[::32]

    def spread(lo):
        errs = np.zeros(len(variants))
        for pair in range(6):
            _, A = gen.to_storage(gen.uniform(40, 2 * pair, (32, 32), lo, 1.0), "f32")
            _, B = gen.to_storage(gen.uniform(40, 2 * pair + 1, (32, 32), lo, 1.0), "f32")
            Cs = oracle.exact_gemm(A, B)
            for v, (d, e, f) in enumerate(variants):
                Cm = oracle.scheme_gemm(oracle.sign_variant(S2, d, e, f), A, B, pd="e4m3", od="f32", scale_mode=1)
                errs[v] += oracle.rel_error(Cm, Cs)
        return errs.max() / errs.min()

    assert spread(-1.0) < 1.25 < spread(0.0)


def test_generators_are_counter_based():
    a = gen.normal(0, 1, (5, 7))
    b = gen.normal(0, 1, (35,)).reshape(5, 7)
    assert np.array_equal(a, b) and not np.array_equal(a, gen.normal(1, 1, (5, 7)))
    big = gen.normal(0, 3, (300000,))
    assert abs(big.mean()) < 0.01 and abs(big.std() - 1.0) < 0.01
    A = gen.activations_outlier(0, 1, 16, 4096, frac=0.005, factor=100.0)
    assert (A.std(axis=0) > 20).sum() == 20
    assert np.linalg.cond(gen.gauge_cond_limited(0, 0, 2)) <= 10.0
    conds = [np.linalg.cond(gen.gauge_log_uniform_cond(1, i, 2)) for i in range(64)]
    assert 1.0 <= min(conds) < 3.0 and 300.0 < max(conds) <= 1000.0 + 1e-6


def test_products_rounded_to_bf16_special_cases():
    """Model schedule (Appendix B.1: each product is returned in bf16).  For the classical algorithm <1,1,1;1> the
    only product is A B itself, so the result is the exact product rounded once to bf16 (a library matmul plus
    the separately pinned rounding); on small integers the rounding is the identity; in general the result moves
    by at most sum_r |w_r| half-ulps of the largest product."""
    A = gen.integer_matrix(31, 1, (16, 32), 40).astype(np.float64)
    B = gen.integer_matrix(31, 2, (32, 24), 40).astype(np.float64)
    one = oracle.classical_scheme(1, 1, 1)
    got = oracle.scheme_gemm(one, A, B, "f64", "f64", md="bf16")
    assert np.array_equal(got, oracle.round_to(A @ B, "bf16")) and not np.array_equal(got, A @ B)
    s2 = oracle.kron(oracle.strassen(), oracle.strassen())
    a = gen.integer_matrix(32, 1, (8, 16), 1).astype(np.float64)
    b = gen.integer_matrix(32, 2, (16, 8), 1).astype(np.float64)
    assert np.array_equal(oracle.scheme_gemm(s2, a, b, "bf16", "f32", md="bf16"), a @ b)       # |M_r| <= 4*4*4 = 64: exact
    X = gen.normal(33, 1, (64, 64)); Y = gen.normal(33, 2, (64, 64))
    C0, p0 = oracle.scheme_gemm(s2, X, Y, "bf16", "f64", parts=True)
    C1, p1 = oracle.scheme_gemm(s2, X, Y, "bf16", "f64", parts=True, md="bf16")
    assert np.array_equal(p1["M"], oracle.round_to(p0["M"], "bf16"))
    assert 0 < np.abs(C1 - C0).max() <= 16 * 2.0 ** -9 * np.abs(p0["M"]).max()


def test_model_schedule_group_scales_invariances():
    """scale_mode 3 (Appendix B.1: e4m3 block sums of the input with one scale per 128 consecutive entries of a row,
    weight block sums first stored in bf16 then one scale per 128 x 128 block, groups accumulated separately).
    What the definition fixes without any reference values: (a) a power of two applied to one row position of A moves
    only scales, so those output rows scale exactly and the others keep their bits; (b) a power of two moved from one
    128-group of inner indices of A to the same group of B is absorbed by the two scales: identical bits; (c) on
    {-1, 0, 1} inputs every code is +-448 or 0 and the result is the exact product up to the fp32 rounding of 1/448;
    (d) finer scales help: the error is below the per-tensor schedule's on outlier-heavy inputs."""
    s2 = oracle.kron(oracle.strassen(), oracle.strassen())
    M, K, N = 64, 1024, 512                       # bm = 16, bk = 256 (2 groups), bn = 128 (1 block)
    A = gen.to_storage(gen.activations_outlier(41, 1, M, K, frac=0.02, factor=50.0), "bf16")[1]
    B = gen.to_storage(gen.weights(41, 2, K, N), "bf16")[1]
    C = oracle.scheme_gemm(s2, A, B, "e4m3", "f32", scale_mode=3)
    # (a)
    A2 = A.copy(); rows = [3 + i * 16 for i in range(4)]
    A2[rows] *= 8.0
    C2 = oracle.scheme_gemm(s2, A2, B, "e4m3", "f32", scale_mode=3)
    keep = np.setdiff1d(np.arange(M), rows)
    assert np.array_equal(C2[rows], 8.0 * C[rows]) and np.array_equal(C2[keep], C[keep])
    # (b) group 1 of every block column of A (inner indices 128..255 of each 256-wide block) times 4, B rows divided
    idx = np.concatenate([l * 256 + np.arange(128, 256) for l in range(4)])
    A3 = A.copy(); B3 = B.copy()
    A3[:, idx] *= 4.0; B3[idx, :] /= 4.0
    assert np.array_equal(oracle.scheme_gemm(s2, A3, B3, "e4m3", "f32", scale_mode=3), C)
    assert np.array_equal(oracle.classical_gemm(A3, B3, "e4m3", "f32", 3), oracle.classical_gemm(A, B, "e4m3", "f32", 3))
    # (c)
    a = gen.integer_matrix(42, 1, (8, 512), 1).astype(np.float64); b = gen.integer_matrix(42, 2, (512, 128), 1).astype(np.float64)
    got = oracle.classical_gemm(a, b, "e4m3", "f32", 3)
    assert np.abs(got - a @ b).max() <= 1e-5 * np.abs(a @ b).max()
    # (d)
    Cs = A @ B
    e3 = oracle.rel_error(C, Cs); e1 = oracle.rel_error(oracle.scheme_gemm(s2, A, B, "e4m3", "f32", scale_mode=1), Cs)
    assert e3 < e1 and 1e-3 < e3 < 0.2
    _, parts = oracle.scheme_gemm(s2, A, B, "e4m3", "f32", scale_mode=3, parts=True)
    assert parts["sA"].shape == (49, 16, 2) and parts["sB"].shape == (49, 1, 2) and np.abs(parts["Ahat"]).max() == 448
