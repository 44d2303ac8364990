"""Per-level rounding of a nested algorithm on the device (FMM_FLAG_ROUND_PER_LEVEL) against the oracle, step by
step: twice-rounded block sums and their scales bit for bit, products to 1e-5, C to 1e-3; the flag must change the
operator on real data, leave it alone where the oracle says it must (integer domain, trivial levels), and be refused
where it has no meaning."""
import numpy as np
import pytest
import torch

import oracle
from fmm_inputs import generators as gen

import gpu_util as gu

pytestmark = pytest.mark.gpu

S1 = oracle.strassen()
CL = oracle.classical_scheme(2, 2, 2)


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__
    __graft_entry__.build()
    return gu.fmm()


def _pair(lib, outer, inner):
    names = {"s": "strassen222", "c": "classical222"}
    o = {"s": S1, "c": CL}
    return lib.scheme_kron(lib.scheme_builtin(names[outer]), lib.scheme_builtin(names[inner])), o[outer], o[inner]


@pytest.mark.parametrize("outer,inner,M,K,N,S,Pd,O,scale,kind", [
    ("s", "s", 384, 320, 288, "bf16", "bf16", "f32", 0, "llm"),        # ragged tiles
    ("s", "s", 1024, 1024, 2048, "bf16", "bf16", "bf16", 0, "llm"),    # several tiles per product, CTA pairs
    ("s", "s", 256, 512, 256, "f32", "bf16", "f32", 0, "normal"),      # fp32 storage: the outer level rounds fp32 sums
    ("s", "s", 512, 1024, 512, "bf16", "e4m3", "bf16", 1, "t3"),       # e4m3 codes as the inner level's source, two scales
    ("s", "s", 256, 2816, 288, "bf16", "e4m3", "f32", 1, "llm"),       # K / 4 = 704 = 5.5 stages
    ("s", "s", 128, 256, 128, "f32", "e4m3", "f32", 0, "u01"),         # e4m3 without scales
    ("s", "c", 256, 256, 256, "bf16", "bf16", "bf16", 0, "normal"),    # hybrid: single-term inner sums
    ("c", "s", 256, 256, 256, "bf16", "e4m3", "bf16", 1, "t3"),        # hybrid: single-term outer sums, scaled
])
def test_every_step_matches_oracle(lib, outer, inner, M, K, N, S, Pd, O, scale, kind):
    s, oo, oi = _pair(lib, outer, inner)
    if kind == "llm":
        A, B = gen.activations_outlier(3, 1, M, K, frac=0.01, factor=100.0), gen.weights(3, 2, K, N)
    elif kind == "t3":
        A, B = gen.activations_outlier(3, 1, M, K, dist="t3", frac=0.001, factor=300.0, at_least=1), gen.weights(3, 2, K, N)
    elif kind == "u01":
        A, B = gen.uniform(3, 1, (M, K)), gen.uniform(3, 2, (K, N))
    else:
        A, B = gen.normal(3, 1, (M, K)), gen.normal(3, 2, (K, N))
    At, A64 = gu.storage_pair(A, S)
    Bt, B64 = gu.storage_pair(B, S)
    C, p, _ = gu.run_scheme_gemm(s, At, Bt, S, Pd, O, scale_mode=scale, flags=lib.FLAG_ROUND_PER_LEVEL, parts=True)
    Co, po = oracle.scheme_gemm_per_level(oo, oi, A64, B64, Pd, O, scale, parts=True)
    assert np.array_equal(p["Ahat"], po["Ahat"])
    assert np.array_equal(p["BhatT"], po["Bhat"].transpose(0, 2, 1))
    if scale == 1:
        assert np.array_equal(p["sA"], po["sA"]) and np.array_equal(p["sB"], po["sB"])
    assert gu.rel_fro(p["M"], po["M"]) <= 1e-5
    assert gu.rel_fro(C, Co) <= 1e-3
    # against the definition (exact sums, rounded once per level): same tolerance on C
    Cd = oracle.scheme_gemm_per_level(oo, oi, A64, B64, Pd, O, scale, sum="f64")
    assert gu.rel_fro(C, Cd) <= 1e-3


def test_flag_changes_the_operator_only_where_it_should(lib):
    s, _, _ = _pair(lib, "s", "s")
    A, B = gen.normal(4, 1, (256, 512)), gen.normal(4, 2, (512, 256))
    At, _ = gu.storage_pair(A, "bf16")
    Bt, _ = gu.storage_pair(B, "bf16")
    flat, pf, _ = gu.run_scheme_gemm(s, At, Bt, "bf16", "bf16", "f32", parts=True)
    lvl, pl, _ = gu.run_scheme_gemm(s, At, Bt, "bf16", "bf16", "f32", flags=lib.FLAG_ROUND_PER_LEVEL, parts=True)
    U = oracle.kron(S1, S1).U
    four = [r for r in range(49) if np.count_nonzero(U[r]) == 4]
    one = [r for r in range(49) if np.count_nonzero(U[r]) == 1]
    assert np.mean(pf["Ahat"][four] != pl["Ahat"][four]) > 0.05      # a second rounding moves many four-term codes
    assert np.array_equal(pf["Ahat"][one], pl["Ahat"][one])          # and none of the single-term ones
    assert not np.array_equal(flat, lvl)
    # integer domain: both readings are the exact product
    Ai, Bi = gen.integer_matrix(5, 1, (128, 256), 7), gen.integer_matrix(5, 2, (256, 128), 7)
    Ait, _ = gu.storage_pair(Ai, "bf16")
    Bit, _ = gu.storage_pair(Bi, "bf16")
    got = gu.run_scheme_gemm(s, Ait, Bit, "bf16", "bf16", "f32", flags=lib.FLAG_ROUND_PER_LEVEL)
    assert np.array_equal(got, Ai @ Bi)
    # cached weights: a second call that reuses Bhat gives the same bits
    d = lib.GemmDesc.make(256, 512, 256, "bf16", "bf16", "f32", flags=lib.FLAG_ROUND_PER_LEVEL)
    ws = gu.workspace(lib.scheme_gemm_workspace(s, d))
    again = gu.run_scheme_gemm(s, At, Bt, "bf16", "bf16", "f32", flags=lib.FLAG_ROUND_PER_LEVEL, ws=ws)
    reuse = gu.run_scheme_gemm(s, At, Bt, "bf16", "bf16", "f32", flags=lib.FLAG_ROUND_PER_LEVEL | lib.FLAG_REUSE_BHAT, ws=ws)
    assert np.array_equal(again, lvl) and np.array_equal(reuse, lvl)


def test_flag_is_refused_without_factors_or_with_row_scales(lib):
    flat = lib.scheme_builtin("strassen222")
    d = lib.GemmDesc.make(256, 256, 256, "bf16", "bf16", "bf16", flags=lib.FLAG_ROUND_PER_LEVEL)
    assert lib.scheme_gemm_workspace(flat, d) == 0
    s, _, _ = _pair(lib, "s", "s")
    d2 = lib.GemmDesc.make(256, 256, 256, "bf16", "e4m3", "bf16", scale_mode=2, flags=lib.FLAG_ROUND_PER_LEVEL)
    assert lib.scheme_gemm_workspace(s, d2) == 0
    ok = lib.GemmDesc.make(256, 256, 256, "bf16", "e4m3", "bf16", scale_mode=1, flags=lib.FLAG_ROUND_PER_LEVEL)
    assert lib.scheme_gemm_workspace(s, ok) > lib.scheme_gemm_workspace(
        s, lib.GemmDesc.make(256, 256, 256, "bf16", "e4m3", "bf16", scale_mode=1))
    P = np.stack([np.eye(2)] * 2)
    A = torch.zeros((256, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.FmmError) as err:
        lib.error_sweep(s, 1, P, P, P, ok, A, A, gu.workspace(1 << 20))
    assert err.value.code == 1
