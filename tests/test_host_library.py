"""Host-side checks of the C-ABI library that need no GPU: the shared object loads and exports every
symbol the header declares; scheme handles, nesting, gauges and criteria agree with the oracle (the two
share no code); argument validation returns the documented status codes."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from fmm_inputs import generators as gen

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2609_39816_b200 as fmm
    return fmm


def test_header_symbols_are_exported(lib):
    header = open(os.path.join(ROOT, "include", "fmm_b200.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(\w+)\s*\([^;{]*\)\s*;", header))
    declared -= {"defined"}
    assert {"scheme_load", "gauge_apply", "scheme_gemm", "error_sweep"} <= declared
    so = ctypes.CDLL(lib.lib_path())
    for name in declared:
        assert hasattr(so, name), f"{name} declared in the header but not exported"
    assert declared == set(lib.EXPORTED_SYMBOLS)


def test_builtin_schemes_match_oracle_tables(lib):
    s1, s2 = oracle.strassen(), oracle.kron(oracle.strassen(), oracle.strassen())
    for name, o in (("strassen222", s1), ("strassen444", s2), ("classical222", oracle.classical_scheme(2, 2, 2))):
        s = lib.scheme_builtin(name)
        U, V, W = s.coefficients()
        assert s.dims == o.dims
        assert np.array_equal(U, o.U) and np.array_equal(V, o.V) and np.array_equal(W, o.W)
        info, crit = s.info, oracle.criteria(o)
        assert info == crit
    assert lib.scheme_builtin("strassen444").info["Phi"] == 1024.0


def _golden(name):
    out = {}
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                k, *v = line.split()
                out[k] = [float(x) for x in v]
    return out


def test_scheme_info_against_printed_and_hand_derived_constants(lib):
    """All eight metadata entries of scheme_info against the golden files (printed constants; Q and E evaluated by
    hand from the printed product table), not against the oracle."""
    g, h = _golden("two_level_strassen_constants.txt"), _golden("ballard_criteria_hand.txt")
    two = lib.scheme_builtin("strassen444").info
    for key in ("L_A", "L_B", "L_W", "Phi", "nnz", "maxabs"):
        assert two[key] == g[key][0], key
    assert two["Q"] == h["Q_two_level"][0] and two["E"] == h["E_two_level"][0]
    one = lib.scheme_builtin("strassen222").info
    assert one["Q"] == h["Q_one_level"][0] and one["E"] == h["E_one_level"][0]
    assert (one["L_A"], one["L_B"], one["L_W"], one["nnz"], one["maxabs"]) == (2.0, 2.0, 4.0, 36.0, 1.0)


def test_scheme_load_checks_brent(lib):
    o = oracle.strassen()
    s = lib.scheme_load(o.U, o.V, o.W)
    assert s.dims == (2, 2, 2, 7)
    W = o.W.copy()
    W[3, 0, 0] = -W[3, 0, 0]                         # one flipped decoding coefficient must be rejected
    with pytest.raises(lib.FmmError) as e:
        lib.scheme_load(o.U, o.V, W)
    assert e.value.code == 3
    big = oracle.classical_scheme(3, 3, 3)
    lib.scheme_load(big.U, big.V, big.W)
    with pytest.raises(lib.FmmError) as e:           # R = 125 > table limit
        c5 = oracle.classical_scheme(5, 5, 5)
        lib.scheme_load(c5.U, c5.V, c5.W)
    assert e.value.code == 9
    with pytest.raises(lib.FmmError):
        lib.scheme_builtin("no-such-scheme")


def test_kron_and_gauges_match_oracle(lib):
    o1 = oracle.strassen()
    s1 = lib.scheme_builtin("strassen222")
    s2 = lib.scheme_kron(s1, s1)
    o2 = oracle.kron(o1, o1)
    assert np.array_equal(s2.coefficients()[0], o2.U)
    # sign variants: exact, equal to the printed formula
    for d, e, f in oracle.sign_variants(4, 4, 4)[::73]:
        g = lib.gauge_apply(s2, np.diag(d), np.diag(e), np.diag(f))
        ov = oracle.sign_variant(o2, d, e, f)
        U, V, W = g.coefficients()
        assert np.array_equal(U, ov.U) and np.array_equal(V, ov.V) and np.array_equal(W, ov.W)
        assert g.info == s2.info
    # identity gauge is the base scheme bit for bit
    g = lib.gauge_apply(s1, np.eye(2), np.eye(2), np.eye(2))
    assert all(np.array_equal(a, b) for a, b in zip(g.coefficients(), s1.coefficients()))
    # general gauges, flat and on the outer factor
    for idx in range(4):
        P, Q, S = (gen.gauge_log_uniform_cond(3, 3 * idx + i, 2) for i in range(3))
        g = lib.gauge_apply(s1, P, Q, S)
        og = oracle.gauge(o1, P, Q, S)
        for a, b in zip(g.coefficients(), (og.U, og.V, og.W)):
            assert np.allclose(a, b, rtol=1e-12, atol=1e-12 * np.abs(b).max())
        g2 = lib.gauge_apply(s2, P, Q, S, level=1)
        og2 = oracle.kron(og, o1)
        for a, b in zip(g2.coefficients(), (og2.U, og2.V, og2.W)):
            assert np.allclose(a, b, rtol=1e-12, atol=1e-12 * np.abs(b).max())
        U2, V2, W2 = g2.coefficients()
        scale = 49 * np.abs(U2).max() * np.abs(V2).max() * np.abs(W2).max()
        assert oracle.brent_residual(oracle.Scheme(U2, V2, W2)) <= 1e-13 * scale
    with pytest.raises(lib.FmmError) as e:
        lib.gauge_apply(s1, np.zeros((2, 2)), np.eye(2), np.eye(2))
    assert e.value.code == 4
    with pytest.raises(lib.FmmError) as e:           # condition limit
        lib.gauge_apply(s1, np.diag([1.0, 1e-3]), np.eye(2), np.eye(2), cond_limit=10.0)
    assert e.value.code == 4
    with pytest.raises(lib.FmmError):                # level 1 needs a nested handle
        lib.gauge_apply(s1, np.eye(2), np.eye(2), np.eye(2), level=1)


def test_gauge_apply_against_the_numpy_definition(lib):
    """The library's gauge against the definition written with library routines of another kind (numpy's inverse and
    einsum), not against the oracle's loops, which have the same shape as the library's: U'_r = P^T U_r Q^-T,
    V'_r = Q^T V_r S^-T, W'_r = P^-1 W_r S; and running the gauged algorithm in exact arithmetic gives A B."""
    s1 = lib.scheme_builtin("strassen222")
    s2 = lib.scheme_builtin("strassen444")
    U1, V1, W1 = s1.coefficients()
    rng = np.random.default_rng(5)
    for idx in range(3):
        P, Q, S = (gen.gauge_log_uniform_cond(9, 3 * idx + i, 2) for i in range(3))
        Pi, Qi, Si = np.linalg.inv(P), np.linalg.inv(Q), np.linalg.inv(S)
        want = (np.einsum("ia,ril,bl->rab", P, U1, Qi), np.einsum("la,rlj,bj->rab", Q, V1, Si),
                np.einsum("ai,rij,jb->rab", Pi, W1, S))
        got = lib.gauge_apply(s1, P, Q, S).coefficients()
        for a, b in zip(got, want):
            assert np.allclose(a, b, rtol=1e-11, atol=1e-11 * np.abs(b).max())
        # level 1 on the nested handle = Kronecker product of the gauged outer factor with the inner one
        g2 = lib.gauge_apply(s2, P, Q, S, level=1).coefficients()
        kron = lambda X, Y: np.einsum("pab,qcd->pqacbd", X, Y).reshape(49, 4, 4)
        for a, X, Y in zip(g2, want, (U1, V1, W1)):
            assert np.allclose(a, kron(X, Y), rtol=1e-11, atol=1e-11 * np.abs(X).max())
        # Eq. 1 with the gauged coefficients, in fp64, on random 2 x 2 block matrices of scalars
        A, B = rng.standard_normal((2, 2)), rng.standard_normal((2, 2))
        Ug, Vg, Wg = got
        Mr = np.einsum("ril,il->r", Ug, A) * np.einsum("rlj,lj->r", Vg, B)
        C = np.einsum("rij,r->ij", Wg, Mr)
        assert np.allclose(C, A @ B, rtol=0, atol=1e-9 * np.abs(Ug).max() * np.abs(Vg).max() * np.abs(Wg).max())


def test_descriptor_validation_without_gpu(lib):
    s2 = lib.scheme_builtin("strassen444")
    ok = lib.GemmDesc.make(4096, 4096, 4096, "bf16", "bf16", "bf16")
    need = lib.scheme_gemm_workspace(s2, ok)
    bm = 1024
    assert need >= 49 * bm * bm * (2 + 2 + 4)
    assert lib.scheme_gemm_workspace(s2, lib.GemmDesc.make(4098, 4096, 4096, "bf16", "bf16", "bf16")) == 0
    assert lib.scheme_gemm_workspace(s2, lib.GemmDesc.make(4096, 4096 + 32, 4096, "bf16", "bf16", "bf16")) == 0
    assert lib.scheme_gemm_workspace(s2, lib.GemmDesc.make(4096, 4096, 4096, "bf16", "bf16", "bf16", scale_mode=1)) == 0
    assert lib.scheme_gemm_workspace(s2, lib.GemmDesc.make(4096, 4096, 4096, "bf16", "e4m3", "bf16", scale_mode=1)) > 0
    assert lib.error_sweep_workspace(s2, ok, 4) > need
    assert lib.classical_gemm_workspace(ok) > 0
    lay = lib.scheme_gemm_workspace_layout(s2, ok)
    assert lay["Ahat"] < lay["Bhat"] < lay["M"] < need
    assert all(lay[key] % 256 == 0 for key in ("Ahat", "Bhat", "M", "sA", "sB"))
    assert lay["stride_Ahat"] >= bm * bm and lay["stride_M"] >= bm * bm


def test_sweep_sharding_over_ranks_gloo():
    """Gauges are independent units: rank r of W takes gauges r, r+W, ...; results are gathered on rank 0.
    Run as two gloo ranks on CPU with a stand-in ratio function (the partitioning logic is what is tested)."""
    import torch.multiprocessing as mp
    from bench import shard_gauges  # noqa: F401  (import check)
    port = 29500 + os.getpid() % 1000
    mp.spawn(_shard_worker, args=(2, port), nprocs=2, join=True)


def _shard_worker(rank, world, port):
    import torch
    import torch.distributed as dist
    from bench import gather_ratios, shard_gauges
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    G = 13
    mine = shard_gauges(G, rank, world)
    local = torch.tensor([float(g) * 1.5 for g in mine], dtype=torch.float64)
    full = gather_ratios(local, mine, G, rank, world, device="cpu")
    if rank == 0:
        assert full.tolist() == [g * 1.5 for g in range(G)]
    dist.destroy_process_group()


def test_certificate_on_host_matches_oracle(lib):
    """Proposition 1 evaluated by the library agrees with the oracle's and with the printed constants."""
    s1 = lib.scheme_builtin("strassen222")
    s2 = lib.scheme_builtin("strassen444")
    o2 = oracle.kron(oracle.strassen(), oracle.strassen())
    for args in ((31, 31, 32, 128, 31), (31, 31, 32, 128, 24), (32, 31, 32, 128, 31), (31, 31, 8729, 4 * 8729, 31),
                 (31, 31, 8730, 4 * 8730, 31), (31, 31, 64, 128, 31)):
        got = lib.scheme_certificate(s2, *args)
        want = oracle.certificate(o2, *args)
        assert got[0] == want[0] and got[1] == want[1], args
    assert lib.scheme_certificate(s2, 31, 31, 32)[1]["LAbA"] == 124
    assert lib.scheme_certificate(s1, 63, 63, 64)[0] and not lib.scheme_certificate(s1, 64, 63, 64)[0]
    assert lib.scheme_certificate(None, 127, 127, 128)[0]
    # a gauged (non-integer) scheme never certifies
    P = gen.gauge_cond_limited(3, 0, 2)
    g = lib.gauge_apply(s1, P, P, P)
    assert not lib.scheme_certificate(g, 1, 1, 64)[0]
    # workspace query rejects what the path cannot tile
    assert lib.int8_gemm_workspace(s2, 64, 100, 64) == 0          # K not a multiple of 128
    assert lib.int8_gemm_workspace(s2, 66, 128, 64) == 0          # M not divisible by m
    assert lib.int8_gemm_workspace(s2, 64, 128, 64) > 0
    # the one-kernel realisation keeps int8 block sums (49 / 16 of an operand per side), the materialised form every
    # per-group fp32 product: R * K/128 blocks of bm x bn
    one = lib.int8_gemm_workspace(s2, 4096, 4096, 4096)
    mat = lib.int8_gemm_materialised_workspace(s2, 4096, 4096, 4096)
    sums = 2 * 13 * 32 * 1024 * 128                                # slabs of four products x groups x block rows x 128 bytes
    assert sums <= one <= sums + (4 << 20)
    assert mat >= 49 * 32 * 1024 * 1024 * 4
    assert lib.int8_gemm_materialised_workspace(s2, 64, 100, 64) == 0


def test_corrected_certificate_constants(lib):
    """Appendix D, certificate of the corrected computation: block sums up to 4 * 127 = 508, |R| <= 2, the terms
    of one rebuilt product within h (128 + 256 * 2)^2 = 13,107,200, sixteen of them below 2^31."""
    s1 = lib.scheme_builtin("strassen222")
    s2 = lib.scheme_kron(s1, s1)
    ok, c = lib.scheme_certificate_corrected(s2, 32)
    assert ok and c == dict(block_sum_max=508.0, r_max=2.0, product_terms=13107200.0, combination=16 * 13107200.0)
    ok1, c1 = lib.scheme_certificate_corrected(s1, 64)
    assert ok1 and c1["block_sum_max"] == 254 and c1["r_max"] == 1
    assert not lib.scheme_certificate_corrected(s2, 64)[0]          # a call of 256 indices over groups of 128
    P = gen.gauge_cond_limited(3, 0, 2)
    assert not lib.scheme_certificate_corrected(lib.gauge_apply(s1, P, P, P), 64)[0]
    assert lib.int8_gemm_corrected_workspace(s2, 64, 128, 64) > 0
    assert lib.int8_gemm_corrected_workspace(s2, 64, 100, 64) == 0


def test_empty_and_maximum_sizes_are_rejected_before_any_launch(lib):
    """Empty shapes and blocks beyond the kernels' 32-bit position index return no workspace (FMM_ERR_SHAPE)."""
    s2 = lib.scheme_builtin("strassen444")
    ok = lib.GemmDesc.make(4096, 4096, 4096, "bf16", "bf16", "bf16")
    assert lib.scheme_gemm_workspace(s2, ok) > 0
    for M, K, N in ((0, 64, 32), (64, 0, 32), (64, 64, 0)):
        assert lib.scheme_gemm_workspace(s2, lib.GemmDesc.make(M, K, N, "bf16", "bf16", "bf16")) == 0
        assert lib.classical_gemm_workspace(lib.GemmDesc.make(M, K, N, "bf16", "bf16", "bf16")) == 0
    # largest legal block: (M/4) * (K/4) * 2 / 16 vectors just under 2^31 - 4096; one step beyond is refused
    big_ok = lib.GemmDesc.make(4 * (1 << 20), 4 * 16368, 32, "bf16", "bf16", "bf16")       # 2^20 * 16368 / 8 = 2.1453e9
    assert (1 << 20) * 16368 // 8 < (1 << 31) - 4096 and lib.scheme_gemm_workspace(s2, big_ok) > 0
    too_big = lib.GemmDesc.make(4 * (1 << 20), 4 * 16400, 32, "bf16", "bf16", "bf16")
    assert (1 << 20) * 16400 // 8 >= (1 << 31) - 4096 and lib.scheme_gemm_workspace(s2, too_big) == 0
    assert lib.scheme_gemm_workspace(s2, lib.GemmDesc.make(4 * (1 << 17), 64, 4 * (1 << 17), "bf16", "bf16", "bf16")) == 0   # products
    assert lib.int8_gemm_workspace(s2, 0, 128, 64) == 0


def test_rotation_argument_checks_need_no_device(lib):
    """hadamard_rotate validates before it touches CUDA: bad arguments return their status and launch nothing."""
    f = lib.binding._lib.hadamard_rotate
    x = ctypes.c_void_p(1 << 20)                       # never dereferenced: every call below is refused
    assert f(0, None, 64, 4, 64, 32, None, x, 64, None) == 1               # FMM_ERR_ARG: null operand
    assert f(2, x, 64, 4, 64, 32, None, x, 64, None) == 5                  # FMM_ERR_DTYPE: e4m3 storage
    for h in (0, 1, 3, 48, 2048):
        assert f(0, x, 64, 4, 64, h, None, x, 64, None) == 2               # FMM_ERR_SHAPE: h
    assert f(0, x, 64, 0, 64, 32, None, x, 64, None) == 2                  # empty
    assert f(0, x, 48, 4, 48, 32, None, x, 48, None) == 2                  # K % h
    assert f(0, x, 32, 4, 64, 32, None, x, 64, None) == 2                  # ld < K
    assert f(1, x, 68, 4, 64, 32, None, x, 64, None) == 2                  # bf16 rows not 16-byte multiples
    assert f(0, ctypes.c_void_p((1 << 20) + 4), 64, 4, 64, 32, None, x, 64, None) == 2   # misaligned base


def test_repair_entry_points_validate_before_any_launch(lib):
    L = lib.binding._lib
    x = ctypes.c_void_p(1 << 20)
    assert L.row_pow2_scale(0, None, 64, 4, 64, x, x, 64, None) == 1            # FMM_ERR_ARG
    assert L.row_pow2_scale(2, x, 64, 4, 64, x, x, 64, None) == 5               # FMM_ERR_DTYPE: e4m3 storage
    assert L.row_pow2_scale(0, x, 32, 4, 64, x, x, 64, None) == 2               # FMM_ERR_SHAPE: ld < K
    assert L.row_unscale(0, x, 64, 0, 64, x, None) == 2                         # empty
    assert L.row_unscale(0, x, 64, 4, 64, None, None) == 1
    s1 = lib.scheme_builtin("strassen222")
    for pd, mode, want in (("bf16", 0, 5), ("e4m3", 1, 5), ("e4m3", 2, 5)):     # only the model schedule has the rule
        d = lib.GemmDesc.make(64, 256, 256, "bf16", pd, "bf16", weight_layout=True, scale_mode=mode)
        assert L.scheme_joint_round_weights(s1.handle, ctypes.byref(d), x, 12, x, 1 << 30, None) == want
    d3 = lib.GemmDesc.make(64, 256, 256, "bf16", "e4m3", "bf16", weight_layout=True, scale_mode=3)
    assert L.scheme_joint_round_weights(s1.handle, ctypes.byref(d3), x, -1, x, 1 << 30, None) == 1
    assert L.scheme_joint_round_weights(s1.handle, ctypes.byref(d3), x, 12, x, 16, None) == 6   # FMM_ERR_WORKSPACE


def test_host_buffer_entry_point_validates_before_any_copy(lib):
    L = lib.binding._lib
    s2 = lib.scheme_builtin("strassen444")
    d = lib.GemmDesc.make(256, 256, 256, "bf16", "bf16", "bf16")
    x = ctypes.c_void_p(1 << 20)
    need = lib.scheme_gemm_host_workspace(s2, d)
    assert need > lib.scheme_gemm_workspace(s2, d) + 3 * 256 * 256 * 2 - 1
    assert L.scheme_gemm_host(s2.handle, ctypes.byref(d), None, x, x, x, need, None) == 1       # FMM_ERR_ARG
    assert L.scheme_gemm_host(s2.handle, ctypes.byref(d), x, None, x, x, need, None) == 1       # no weight, no reuse flag
    assert L.scheme_gemm_host(s2.handle, ctypes.byref(d), x, x, x, x, need - 1, None) == 6      # FMM_ERR_WORKSPACE
    bad = lib.GemmDesc.make(250, 256, 256, "bf16", "bf16", "bf16")
    assert lib.scheme_gemm_host_workspace(s2, bad) == 0
    assert L.scheme_gemm_host(s2.handle, ctypes.byref(bad), x, x, x, x, need, None) == 2        # FMM_ERR_SHAPE


def test_permuted_products_are_the_same_algorithm(lib):
    """Renumbering the products keeps the Brent equations and every criterion; bad permutations are refused."""
    s2 = lib.scheme_builtin("strassen444")
    rng = np.random.default_rng(5)
    perm = rng.permutation(49)
    sp = lib.scheme_permute_products(s2, perm)
    U, V, W = s2.coefficients()
    Up, Vp, Wp = sp.coefficients()
    assert np.array_equal(Up, U[perm]) and np.array_equal(Vp, V[perm]) and np.array_equal(Wp, W[perm])
    assert sp.info == s2.info
    assert oracle.brent_residual(oracle.Scheme(Up, Vp, Wp)) == 0.0
    for bad in ([0] * 49, list(range(48)) + [49], list(range(48)) + [-1]):
        with pytest.raises(lib.FmmError):
            lib.scheme_permute_products(s2, bad)
