"""Parity at the stated benchmark configurations, at full size, in the launch configuration bench.py times
(weights stored [N, K], bf16 storage): configs 3, 4 and 5 against full-size runs of the CPU oracle.

Every comparison is against the oracle's own full-size result (per-tensor scales depend on the whole operand, so
no sub-problem can stand in for them).  Bars as everywhere: quantised codes and scales bit-exact, C within 1e-3 in
the Frobenius norm, ratios within 2 %.  Host time: the oracle multiplies at 40-50 GFLOP/s on 16 cores; the whole
file is a few minutes.
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


def _layer_inputs(T, K, N):
    """The recipe of configs 4 and 5 as bench.py draws it: Student-t(3) activations with max(1, floor(0.001 K))
    channels x300, weights N(0, 0.02^2) stored [N, K]."""
    A = gen.activations_outlier(0, 1, T, K, dist="t3", frac=0.001, factor=300.0, at_least=1)
    W = gen.normal(0, 2, (N, K), std=0.02)
    At, A64 = gen.to_storage(A, "bf16")
    Wt, W64 = gen.to_storage(W, "bf16")
    return At.cuda(), Wt.cuda(), A64, np.ascontiguousarray(W64.T)


def _check_full(lib, T, K, N, Pd, scale, codes_of=()):
    At, Wt, A64, B64 = _layer_inputs(T, K, N)
    s = lib.scheme_builtin("strassen444")
    o2 = gu.oracle_scheme("strassen444")
    C, p, ws = gu.run_scheme_gemm(s, At, Wt, "bf16", Pd, "bf16", weight_layout=True, scale_mode=scale, parts=True)
    want_parts = True if codes_of == "all" else "scales"
    Co, po = oracle.scheme_gemm(o2, A64, B64, Pd, "bf16", scale, parts=want_parts)
    if scale == 1:      # the 49 + 49 power-of-two scales, bit for bit
        assert np.array_equal(p["sA"], po["sA"]) and np.array_equal(p["sB"], po["sB"])
    if codes_of == "all":
        assert np.array_equal(p["Ahat"], po["Ahat"])
        assert np.array_equal(p["BhatT"], po["Bhat"].transpose(0, 2, 1))
    rel = gu.rel_fro(C, Co)
    assert rel <= TOL_FRO, rel
    del p, ws
    torch.cuda.empty_cache()
    return C, Co


@pytest.mark.parametrize("K,N", [(4096, 12288), (4096, 4096), (4096, 22016), (11008, 4096)])
def test_config4_every_gemm_full_size_e4m3_per_tensor_scales(lib, K, N):
    """Config 4: T = 2048, two-level Strassen, e4m3 block sums with one power-of-two scale per encoded tensor."""
    _check_full(lib, 2048, K, N, "e4m3", 1, codes_of="all")


@pytest.mark.parametrize("Pd,scale", [("bf16", 0), ("e4m3", 1)])
def test_config5_down_projection_full_size(lib, Pd, scale):
    """Config 5: T = 8192, K = 13824, N = 5120 (888 GFLOP of block products), bf16 and e4m3 with per-tensor scales."""
    _check_full(lib, 8192, 13824, 5120, Pd, scale)


def test_config5_outer_level_sweep_four_gauges_full_size(lib):
    """Four of the configuration's 512 outer-level gauges over the down projection at full size: the ratios against
    the oracle's (scheme, classical and exact products all at full size)."""
    T, K, N = 8192, 13824, 5120
    At, Wt, A64, B64 = _layer_inputs(T, K, N)
    import bench
    P, Q, S = bench.sweep_gauges(512)
    pick = [0, 170, 341, 511]
    P, Q, S = P[pick], Q[pick], S[pick]
    s1 = lib.scheme_builtin("strassen222")
    s2 = lib.scheme_kron(s1, s1)
    d = lib.GemmDesc.make(T, K, N, "bf16", "bf16", "bf16", weight_layout=True)
    ws = gu.workspace(lib.error_sweep_workspace(s2, d, len(pick)))
    ratios, summ = lib.error_sweep(s2, 1, P, Q, S, d, At, Wt, ws)
    del ws
    torch.cuda.empty_cache()
    Cs = oracle.exact_gemm(A64, B64)
    Ecl = oracle.rel_error(oracle.classical_gemm(A64, B64, "bf16", "bf16"), Cs)
    assert math.isclose(summ["e_classical_rel"], Ecl, rel_tol=TOL_RATIO)
    o1 = oracle.strassen()
    for g in range(len(pick)):
        sg = oracle.kron(oracle.gauge(o1, P[g], Q[g], S[g]), o1)
        want = oracle.error_ratio(oracle.rel_error(oracle.scheme_gemm(sg, A64, B64, "bf16", "bf16"), Cs), Ecl)
        assert abs(ratios[g] - want) <= TOL_RATIO * want, (g, ratios[g], want)


def _sweep_against_oracle(lib, At, Wt, A64, B64, P, Q, S):
    s1 = lib.scheme_builtin("strassen222")
    M, K = A64.shape
    N = B64.shape[1]
    d = lib.GemmDesc.make(M, K, N, "bf16", "bf16", "bf16", weight_layout=True)
    ws = gu.workspace(lib.error_sweep_workspace(s1, d, P.shape[0]))
    ratios, summ = lib.error_sweep(s1, 0, P, Q, S, d, At, Wt, ws)
    Cs = oracle.exact_gemm(A64, B64)
    Ecl = oracle.rel_error(oracle.classical_gemm(A64, B64, "bf16", "bf16"), Cs)
    assert math.isclose(summ["e_classical_rel"], Ecl, rel_tol=TOL_RATIO)
    o1 = oracle.strassen()
    want = np.array([oracle.error_ratio(oracle.rel_error(
        oracle.scheme_gemm(oracle.gauge(o1, P[g], Q[g], S[g]), A64, B64, "bf16", "bf16"), Cs), Ecl)
        for g in range(P.shape[0])])
    assert np.all(np.abs(ratios - want) <= TOL_RATIO * want), np.max(np.abs(ratios - want) / want)
    return ratios, want, summ


def test_config3_thirty_two_gauges_full_size(lib):
    """Config 3 as bench.py times it (A 2048 x 4096, B 4096 x 4096 stored [N, K]): every sixteenth of the
    configuration's 512 gauges at full size (four batches of eight in the sweep)."""
    import bench
    At_h, Bt_h = bench.c3_inputs(0)
    A64, B64 = At_h.double().numpy(), np.ascontiguousarray(Bt_h.double().numpy().T)
    P, Q, S = bench.sweep_gauges(512)
    pick = np.arange(0, 512, 16)
    _sweep_against_oracle(lib, At_h.cuda(), Bt_h.cuda(), A64, B64, P[pick], Q[pick], S[pick])


def test_config3_all_512_gauges_quarter_scale(lib):
    """All 512 gauges of config 3 on the quarter-scale problem 512 x 1024 x 1024 (same recipe), ratios and the
    summary statistics against the oracle's."""
    import bench
    M, K, N = 512, 1024, 1024
    A = gen.activations_outlier(0, 3, M, K, dist="normal", frac=0.005, factor=100.0)
    W = gen.weights(0, 4, K, N).T
    At, A64 = gen.to_storage(A, "bf16")
    Wt, W64 = gen.to_storage(np.ascontiguousarray(W), "bf16")
    P, Q, S = bench.sweep_gauges(512)
    ratios, want, summ = _sweep_against_oracle(lib, At.cuda(), Wt.cuda(), A64, np.ascontiguousarray(W64.T), P, Q, S)
    ws_sum = oracle.summary(ratios)
    for key in ("min", "median", "max", "spread", "count_gt2"):
        assert summ[key] == ws_sum[key]
    os_sum = oracle.summary(want)
    assert os_sum["count_gt2"] == summ["count_gt2"]
    for key in ("min", "median", "max"):
        assert abs(summ[key] - os_sum[key]) <= TOL_RATIO * os_sum[key]
