"""Pins of the per-level rounding of a nested algorithm (no GPU).

"Strassen's algorithm applied to its own blocks" (Section 1) has two readings once block sums are rounded: the
flat one (the 49 block sums of the Kronecker coefficients, each rounded once — what the paper's two-level
algorithm does) and the literal recursion, in which the outer level's seven block sums are rounded, the inner
level forms its sums of those rounded values and rounds again.  The second is a different operator; these pins fix
it without reference to any implementation.
"""
import numpy as np
import pytest

import oracle
from fmm_inputs import generators as gen

S1 = oracle.strassen()
S2 = oracle.kron(S1, S1)
CL = oracle.classical_scheme(2, 2, 2)
ONE = oracle.classical_scheme(1, 1, 1)


def _ops(seed, M, K, N):
    _, A = gen.to_storage(gen.normal(seed, 1, (M, K)), "bf16")
    _, B = gen.to_storage(gen.normal(seed, 2, (K, N)), "bf16")
    return A, B


def test_nothing_rounded_equals_the_flat_algorithm_and_the_product():
    A, B = _ops(1, 32, 48, 40)
    C = oracle.scheme_gemm_per_level(S1, S1, A, B, "f64", "f64")
    assert np.allclose(C, A @ B, rtol=0, atol=1e-12 * np.abs(A @ B).max())
    assert np.allclose(C, oracle.scheme_gemm(S2, A, B, "f64", "f64"), rtol=0, atol=1e-12 * np.abs(C).max())


@pytest.mark.parametrize("pd,scale", [("bf16", 0), ("e4m3", 1)])
def test_trivial_levels_reduce_to_the_flat_operator(pd, scale):
    """A 1 x 1 x 1 level has a single coefficient 1: its 'block sum' is the operand itself.  As the INNER level it
    re-rounds values that are already in the product dtype (no change): the result is the flat one-level operator."""
    A, B = _ops(2, 32, 64, 32)
    for mode in ("f32chain", "f64"):
        want, pw = oracle.scheme_gemm(S1, A, B, pd, "bf16", scale, parts=True, sum=mode)
        got, pg = oracle.scheme_gemm_per_level(S1, ONE, A, B, pd, "bf16", scale, parts=True, sum=mode)
        assert np.array_equal(pg["Ahat"] * pg["sA"][:, None, None], pw["Ahat"] * pw["sA"][:, None, None])
        assert np.array_equal(got, want)
    # as the OUTER level of bf16 storage into bf16 products it rounds nothing either
    if pd == "bf16":
        want = oracle.scheme_gemm(S1, A, B, pd, "bf16", scale)
        assert np.array_equal(oracle.scheme_gemm_per_level(ONE, S1, A, B, pd, "bf16", scale), want)


def test_integer_domain_both_readings_are_exact():
    A = gen.integer_matrix(3, 1, (32, 64), 7)
    B = gen.integer_matrix(3, 2, (64, 48), 7)
    ref = A @ B
    assert np.array_equal(oracle.scheme_gemm_per_level(S1, S1, A, B, "bf16", "f32"), ref)
    assert np.array_equal(oracle.scheme_gemm(S2, A, B, "bf16", "f32"), ref)
    # e4m3: |a| <= 4 keeps the two-term outer sums (<= 8) and the inner sums of those (<= 16) on the code grid
    A4 = gen.integer_matrix(4, 1, (32, 64), 4)
    B4 = gen.integer_matrix(4, 2, (64, 48), 4)
    assert np.array_equal(oracle.scheme_gemm_per_level(S1, S1, A4, B4, "e4m3", "f32", 1), A4 @ B4)


def test_hand_example_where_the_two_readings_differ():
    """1 x 1 inner blocks, product (M1, M1): the flat sum A11 + A22 + A33 + A44 against rnd(rnd(A11 + A33) + rnd(A22 + A44))
    (outer M1 adds outer blocks 11 and 22, inner M1 adds inner blocks 11 and 22 of that sum).
    With A11 = 256, A33 = 1, A22 = 1, A44 = 0 ... the flat sum 258 is a bf16 value; per level rnd(257) = 256 (tie to
    even) and rnd(1) = 1 give rnd(257) = 256."""
    A = np.zeros((4, 4))
    A[0, 0], A[2, 2], A[1, 1], A[3, 3] = 256.0, 1.0, 1.0, 0.0
    B = np.eye(4)
    _, flat = oracle.scheme_gemm(S2, A, B, "bf16", "f32", parts=True, sum="f64")
    _, lvl = oracle.scheme_gemm_per_level(S1, S1, A, B, "bf16", "f32", parts=True, sum="f64")
    assert flat["Ahat"][0, 0, 0] == 258.0
    assert lvl["Ahat"][0, 0, 0] == 256.0
    # every product whose sums have at most two terms in total is untouched by the choice of reading
    two_term = [r for r in range(49) if np.count_nonzero(S2.U[r]) <= 2]
    assert two_term
    for r in two_term:
        if np.count_nonzero(S1.U[r // 7]) == 1 or np.count_nonzero(S1.U[r % 7]) == 1:
            assert flat["Ahat"][r, 0, 0] == lvl["Ahat"][r, 0, 0]


def test_differs_from_flat_on_real_data_and_is_no_better():
    A, B = _ops(5, 128, 256, 128)
    Cs = oracle.exact_gemm(A, B)
    Cf, pf = oracle.scheme_gemm(S2, A, B, "bf16", "bf16", parts=True)
    Cl, pl = oracle.scheme_gemm_per_level(S1, S1, A, B, "bf16", "bf16", parts=True)
    four = [r for r in range(49) if np.count_nonzero(S2.U[r]) == 4]
    frac = np.mean(pf["Ahat"][four] != pl["Ahat"][four])
    assert 0.05 < frac < 0.9, frac                     # a second rounding moves a fair share of the four-term codes
    one = [r for r in range(49) if np.count_nonzero(S2.U[r]) == 1]
    assert np.array_equal(pf["Ahat"][one], pl["Ahat"][one])
    Ef, El = oracle.rel_error(Cf, Cs), oracle.rel_error(Cl, Cs)
    assert El > 0.95 * Ef                              # rounding twice cannot systematically help
    assert abs(El - Ef) < 0.5 * Ef                     # and stays the same order of magnitude


def test_hybrid_levels_and_scale_bookkeeping():
    """Strassen outside, classical inside: the inner level has single-term sums, so per-level = flat, bit for bit,
    in both dtypes; with e4m3 the inner scale must then be exactly 1 relative to the outer codes or absorb a power
    of two without changing the decoded values."""
    A, B = _ops(6, 64, 64, 64)
    for pd, scale in (("bf16", 0), ("e4m3", 1)):
        want = oracle.scheme_gemm(oracle.kron(S1, CL), A, B, pd, "bf16", scale)
        got = oracle.scheme_gemm_per_level(S1, CL, A, B, pd, "bf16", scale)
        if pd == "bf16":
            assert np.array_equal(got, want)
        else:   # flat takes one scale per inner block sum, per level one per outer tensor first: close, not equal
            assert np.linalg.norm(got - want) <= 0.2 * np.linalg.norm(want - A @ B) + 1e-12


def test_rejects_row_scales():
    A, B = _ops(7, 16, 32, 16)
    with pytest.raises(ValueError):
        oracle.scheme_gemm_per_level(S1, S1, A, B, "e4m3", "bf16", 2)
