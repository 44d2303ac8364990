"""What the two forms of a block sum cost each other (no GPU).

The definition of a rounded block sum (Eq. 1 with the rounding of Section 2.3 / Appendix B.1) is the exact sum of
coefficient x entry, rounded ONCE to the product dtype: ``sum="f64"``.  The reading that lets quantised codes be
compared bit for bit with fp32 hardware forms the sum as an fp32 fused-multiply-add chain first: ``sum="f32chain"``.
The two can differ only where the fp32 chain rounds before the product dtype does.  These tests measure, on slices
of the benchmark recipes (outlier columns x100 / x300 make four-term sums that need more than 24 bits), how many
codes move, and assert that the result and the error-amplification ratio do not.
"""
import numpy as np
import pytest
import torch

import oracle
from fmm_inputs import generators as gen

S1 = oracle.strassen()
S2 = oracle.kron(S1, S1)


def _slice_problem(cfg, rows=64, cols=32):
    """Rows 0..rows-1 of every block row of A (full K) and columns 0..cols-1 of every block column of B, of the
    config-2 (normal activations, 20 of 4096 columns x100) or config-4 (Student-t, 4 columns x300) recipe."""
    K, M, N = 4096, 4096, 4096
    if cfg == "c2":
        A = gen.activations_outlier(0, 1, M, K, frac=0.005, factor=100.0)
    else:
        A = gen.activations_outlier(0, 1, M, K, dist="t3", frac=0.001, factor=300.0, at_least=1)
    B = gen.weights(0, 2, K, N)
    bm, bn = M // 4, N // 4
    ridx = np.concatenate([i * bm + np.arange(rows) for i in range(4)])
    cidx = np.concatenate([j * bn + np.arange(cols) for j in range(4)])
    _, A64 = gen.to_storage(A[ridx], "bf16")
    _, B64 = gen.to_storage(B[:, cidx], "bf16")
    return A64, B64


_CASES = [("c2", "bf16", 0), ("c4", "bf16", 0), ("c4", "e4m3", 1), ("c4", "e4m3", 2), ("c4", "e4m3", 3),
          ("c2", "e4m3", 1)]


@pytest.mark.parametrize("cfg,pd,scale", _CASES)
def test_f32_chain_against_the_definition(cfg, pd, scale, record_property):
    A, B = _slice_problem(cfg)
    Cs = oracle.exact_gemm(A, B)
    Ecl = oracle.rel_error(oracle.classical_gemm(A, B, pd, "bf16", scale), Cs)
    out = {}
    for mode in ("f32chain", "f64"):
        C, p = oracle.scheme_gemm(S2, A, B, pd, "bf16", scale, parts=True, sum=mode)
        out[mode] = (C, p)
    (Cc, pc), (Cd, pd_) = out["f32chain"], out["f64"]
    nA = pc["Ahat"].size
    diffA = int(np.sum(pc["Ahat"] != pd_["Ahat"]))
    diffB = int(np.sum(pc["Bhat"] != pd_["Bhat"]))
    record_property("codes_differing_A", f"{diffA}/{nA}")
    record_property("codes_differing_B", f"{diffB}/{pc['Bhat'].size}")
    print(f"{cfg} {pd} scale {scale}: A codes differing {diffA} of {nA} ({diffA / nA:.2e}), "
          f"B codes {diffB} of {pc['Bhat'].size}")
    # the double rounding can only move a code by one step of the product dtype, and only rarely
    assert diffA / nA < 2e-3 and diffB / pc["Bhat"].size < 2e-3
    # mode 1: the power-of-two scales are decided by the largest magnitude, which both forms agree on
    if scale == 1:
        assert np.array_equal(pc["sA"], pd_["sA"]) and np.array_equal(pc["sB"], pd_["sB"])
    rel = np.linalg.norm(Cc - Cd) / np.linalg.norm(Cd)
    assert rel <= 1e-3, rel
    rho_c = oracle.error_ratio(oracle.rel_error(Cc, Cs), Ecl)
    rho_d = oracle.error_ratio(oracle.rel_error(Cd, Cs), Ecl)
    assert abs(rho_c - rho_d) <= 0.02 * rho_d, (rho_c, rho_d)


def test_real_gauge_coefficients_move_a_few_codes_not_the_ratio():
    """With a general gauge the coefficients are fp32 reals, every product coefficient x entry needs about 32 bits and
    the fp32 chain rounds at every step: here the two forms do differ, by one step of the product dtype on a small
    share of the codes (config-3 recipe, one level of Strassen, log-uniform condition number)."""
    K, M, N = 4096, 2048, 4096
    A = gen.activations_outlier(0, 1, M, K, frac=0.005, factor=100.0)
    B = gen.weights(0, 2, K, N)
    ridx = np.concatenate([i * (M // 2) + np.arange(64) for i in range(2)])
    cidx = np.concatenate([j * (N // 2) + np.arange(32) for j in range(2)])
    _, A64 = gen.to_storage(A[ridx], "bf16")
    _, B64 = gen.to_storage(B[:, cidx], "bf16")
    Cs = oracle.exact_gemm(A64, B64)
    Ecl = oracle.rel_error(oracle.classical_gemm(A64, B64, "bf16", "bf16"), Cs)
    worst = 0.0
    for g in (0, 7, 19, -1):
        if g >= 0:
            P, Q, S = (gen.gauge_log_uniform_cond(1, 3 * g + i, 2) for i in range(3))
        else:       # condition number at most 10: here C itself is compared too
            P, Q, S = (gen.gauge_cond_limited(1, i, 2) for i in range(3))
        sg = oracle.gauge(S1, P, Q, S)
        Cc, pc = oracle.scheme_gemm(sg, A64, B64, "bf16", "bf16", parts=True, sum="f32chain")
        Cd, pd_ = oracle.scheme_gemm(sg, A64, B64, "bf16", "bf16", parts=True, sum="f64")
        frac = float(np.mean(pc["Ahat"] != pd_["Ahat"]))
        worst = max(worst, frac)
        step = np.abs(pc["Ahat"] - pd_["Ahat"])
        big = np.maximum(np.abs(pc["Ahat"]), np.abs(pd_["Ahat"]))
        # one bf16 step, or (sums that cancel) the fp32 chain's own error: four roundings of terms up to max|u| max|a|
        chain_err = 4 * 2.0 ** -23 * np.abs(sg.U).max() * np.abs(A64).max()
        assert np.all(step <= big * 2.0 ** -7 + chain_err)
        rho_c = oracle.error_ratio(oracle.rel_error(Cc, Cs), Ecl)
        rho_d = oracle.error_ratio(oracle.rel_error(Cd, Cs), Ecl)
        assert abs(rho_c - rho_d) <= 0.02 * rho_d, (g, rho_c, rho_d)
        if g < 0:   # ill-conditioned gauges amplify every rounding alike: for them parity is on the ratio only
            assert np.linalg.norm(Cc - Cd) <= 1e-3 * np.linalg.norm(Cd)
    print(f"gauged one-level Strassen: largest share of A codes differing {worst:.2e}")
    assert 0.0 < worst < 1e-3


def test_two_term_sums_single_rounding_differs_only_on_double_rounding():
    """One level of Strassen has at most two terms per sum: the fp32 chain is exact unless the exact sum needs
    more than 24 bits, so a code can move only when the fp32 result lands on a tie of the product dtype."""
    # a true double-rounding case: a sits on a bf16 tie, b is lost by fp32 and decides the direction in fp64
    a, b = 256.0 + 1.0, 2.0 ** -20          # 257 is the bf16 tie between 256 and 258
    A = np.array([[a, 0.0], [0.0, b]])      # M1 reads A11 + A22
    B = np.eye(2)
    _, pc = oracle.scheme_gemm(S1, A, B, "bf16", "f32", parts=True, sum="f32chain")
    _, pd_ = oracle.scheme_gemm(S1, A, B, "bf16", "f32", parts=True, sum="f64")
    assert pc["Ahat"][0, 0, 0] == 256.0     # fp32 drops 2^-20, then the tie goes to even
    assert pd_["Ahat"][0, 0, 0] == 258.0    # the exact sum is above the tie
    # and with b = 0 both forms see the same tie
    A[1, 1] = 0.0
    for mode in ("f32chain", "f64"):
        _, p = oracle.scheme_gemm(S1, A, B, "bf16", "f32", parts=True, sum=mode)
        assert p["Ahat"][0, 0, 0] == 256.0


def test_integer_domain_is_the_same_in_both_forms():
    A = gen.integer_matrix(5, 1, (32, 64), 7)
    B = gen.integer_matrix(5, 2, (64, 32), 7)
    ref = A @ B
    for mode in ("f32chain", "f64"):
        assert np.array_equal(oracle.scheme_gemm(S2, A, B, "bf16", "f32", sum=mode), ref)


def test_two_term_sums_of_bf16_values_are_the_same_in_both_forms_at_any_exponent_gap():
    """For TWO bf16 terms with coefficients +-1 the fp32 chain, the exact sum rounded once, and a single correctly
    rounded bf16 addition all agree — the fp32 sum is exact up to
    16 binades apart, and beyond that the small term cannot reach a rounding boundary of bf16.  One level of Strassen
    has only one- and two-term sums; operands span 60 binades and include exact ties."""
    rng = np.random.default_rng(3)
    n = 64
    mant = rng.integers(128, 256, size=(n, n)).astype(np.float64)            # 8 significant bits
    A = np.ldexp(mant, rng.integers(-30, 30, size=(n, n))) * rng.choice([-1.0, 1.0], size=(n, n))
    # force ties: A22 = half an ulp of A11 wherever the row index is even
    e11 = np.floor(np.log2(np.abs(A[:n // 2, :n // 2])))
    A[n // 2::2, n // 2:] = np.ldexp(1.0, (e11 - 8).astype(int))[::2]
    B = np.eye(n)
    _, pc = oracle.scheme_gemm(S1, A, B, "bf16", "f32", parts=True, sum="f32chain")
    _, pd_ = oracle.scheme_gemm(S1, A, B, "bf16", "f32", parts=True, sum="f64")
    assert np.array_equal(pc["Ahat"], pd_["Ahat"])
    # and torch's own bf16 addition (a library routine: one rounding of the exact sum) gives the same codes for M1 = A11 + A22
    a11 = torch.from_numpy(A[:n // 2, :n // 2]).to(torch.bfloat16)
    a22 = torch.from_numpy(A[n // 2:, n // 2:]).to(torch.bfloat16)
    assert np.array_equal((a11.double() + a22.double()).to(torch.bfloat16).double().numpy(), pc["Ahat"][0])
