"""GPU parity of the certified int8 realisation (Section 4.2, Proposition 1, Appendix D) against the oracle:
integer work, so every comparison is bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from fmm_inputs import generators as gen
from gpu_util import fmm, workspace

pytestmark = pytest.mark.gpu

S1 = oracle.strassen()
S2 = oracle.kron(S1, S1)


def _lib_scheme(lib, o):
    return lib.scheme_load(o.U, o.V, o.W)


def _inputs(seed, M, K, N, dtype="f32"):
    At, A = gen.to_storage(gen.activations_outlier(seed, 1, M, K), dtype)
    Bt, B = gen.to_storage(gen.weights(seed, 2, N, K), dtype)
    return At.cuda(), A, Bt.cuda(), B


def _quantize(lib, X, b):
    rows, K = X.shape
    codes = torch.empty((rows, K), dtype=torch.int8, device="cuda")
    scales = torch.empty((rows, K // 128), dtype=torch.float32, device="cuda")
    lib.int8_quantize(X, b, codes, scales)
    torch.cuda.synchronize()
    return codes, scales


def _gemm(lib, s, b, cA, dA, cB, dB, out_dtype=torch.bfloat16, materialised=False):
    M, K = cA.shape
    N = cB.shape[0]
    C = torch.full((M, N), float("nan"), dtype=out_dtype, device="cuda")
    if materialised:
        ws = workspace(lib.int8_gemm_materialised_workspace(s, M, K, N))
        lib.int8_gemm_materialised(s, b, cA, dA, cB, dB, C, ws)
    else:
        ws = workspace(lib.int8_gemm_workspace(s, M, K, N))
        lib.int8_gemm(s, b, cA, dA, cB, dB, C, ws)
    lib.device_status(ws)
    return C.to(torch.float64).cpu().numpy()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("b", [31, 63, 127])
def test_quantiser_bit_exact(dtype, b):
    lib = fmm()
    At, A, _, _ = _inputs(11, 200, 512, 8, dtype)
    A[3, 128:256] = 0.0                      # an all-zero group: d = 1
    At[3, 128:256] = 0
    codes, scales = _quantize(lib, At, b)
    oc, od = oracle.quantize_rows(A, b)
    assert np.array_equal(scales.cpu().numpy().astype(np.float64), od)
    assert np.array_equal(codes.cpu().numpy().astype(np.float64), oc)
    assert np.abs(oc).max() == b and od[3, 1] == 1.0


@pytest.mark.parametrize("M,K,N", [(32, 128, 32), (512, 1024, 544), (200, 384, 96), (1040, 256, 2080), (4, 128, 32)])
def test_classical_and_certified_match_oracle_and_each_other(M, K, N):
    """Same bits from the classical int8 operator, the certified two-level realisation and the oracle."""
    lib = fmm()
    At, A, Bt, B = _inputs(21, M, K, N)
    cA, dA = _quantize(lib, At, 31)
    cB, dB = _quantize(lib, Bt, 31)
    oA, odA = oracle.quantize_rows(A, 31)
    oB, odB = oracle.quantize_rows(B, 31)
    want = oracle.int8_classical(oA, odA, oB, odB)
    got_cl = _gemm(lib, None, 31, cA, dA, cB, dB)          # one fused kernel: int8 MMAs, rescale in the epilogue
    assert np.array_equal(got_cl, want)
    one = lib.scheme_load(np.ones((1, 1, 1)), np.ones((1, 1, 1)), np.ones((1, 1, 1)))
    assert np.array_equal(_gemm(lib, one, 31, cA, dA, cB, dB), want)   # <1,1,1;1> through the one-kernel certified path
    assert np.array_equal(_gemm(lib, one, 31, cA, dA, cB, dB, materialised=True), want)   # and through the materialised pipeline
    s2 = _lib_scheme(lib, S2)
    got = _gemm(lib, s2, 31, cA, dA, cB, dB)              # one kernel: 49 int8 products per position in tensor memory
    assert np.array_equal(got, want)
    assert np.array_equal(_gemm(lib, s2, 31, cA, dA, cB, dB, materialised=True), want)    # every product written to memory
    if M % 2 == 0:
        s1 = _lib_scheme(lib, S1)                         # one level: blocks of 64 inner indices, two products per row
        cA6, dA6 = _quantize(lib, At, 63)
        cB6, dB6 = _quantize(lib, Bt, 63)
        ref6 = _gemm(lib, None, 63, cA6, dA6, cB6, dB6)
        assert np.array_equal(_gemm(lib, s1, 63, cA6, dA6, cB6, dB6), ref6)
    want_cert, mx = oracle.int8_certified(S2, oA, odA, oB, odB)
    assert np.array_equal(want_cert, want) and mx[0] <= 124 and mx[1] <= 124
    # fp32 output: the accumulated value itself, before the cast
    got32 = _gemm(lib, s2, 31, cA, dA, cB, dB, torch.float32)
    assert np.array_equal(got32, oracle.int8_classical(oA, odA, oB, odB, od="f32"))
    assert oracle.rel_error(got32, A @ B.T) < 0.2


def test_sign_variants_and_one_level_are_bit_identical():
    lib = fmm()
    M, K, N = 128, 256, 64
    At, A, Bt, B = _inputs(31, M, K, N)
    outs = set()
    variants = list(oracle.sign_variants(4, 4, 4))
    for b, base, picks in ((31, S2, variants[::37] + [variants[-1]]), (63, S1, list(oracle.sign_variants(2, 2, 2)))):
        cA, dA = _quantize(lib, At, b)
        cB, dB = _quantize(lib, Bt, b)
        ref = _gemm(lib, None, b, cA, dA, cB, dB, torch.float32)
        for d, e, f in picks:
            s = _lib_scheme(lib, oracle.sign_variant(base, d, e, f))
            got = _gemm(lib, s, b, cA, dA, cB, dB, torch.float32)
            assert np.array_equal(got, ref)
        oA, odA = oracle.quantize_rows(A, b)
        oB, odB = oracle.quantize_rows(B, b)
        assert np.array_equal(ref, oracle.int8_classical(oA, odA, oB, odB, od="f32"))
        outs.add(ref.tobytes())
    assert len(outs) == 2                     # b = 31 and b = 63 are different operators


def test_integer_weights_other_than_unit_and_undivided_groups():
    """Algorithms that the unit-weight fast path of the decode does not cover: <1,1,1;2> with C = 2 M1 - M2 (both
    products the plain one: k = 1, so a call spans the undivided group, h = 128, four MMAs per product) and Strassen
    with its first product doubled up as 2 M1 - M1' (R = 8, a weight of 2 and an extra product in two decode lists)."""
    lib = fmm()
    M, K, N = 200, 384, 96
    At, A, Bt, B = _inputs(61, M, K, N)
    one = oracle.Scheme(np.ones((2, 1, 1)), np.ones((2, 1, 1)), np.array([2.0, -1.0]).reshape(2, 1, 1))
    U = np.concatenate([S1.U, S1.U[:1]]); V = np.concatenate([S1.V, S1.V[:1]])
    W = np.concatenate([S1.W, -S1.W[:1]]); W[0] *= 2.0
    dup = oracle.Scheme(U, V, W)
    for o, b in ((one, 31), (dup, 31)):
        assert oracle.brent_residual(o) == 0.0
        cA, dA = _quantize(lib, At, b)
        cB, dB = _quantize(lib, Bt, b)
        ref = _gemm(lib, None, b, cA, dA, cB, dB, torch.float32)
        s = _lib_scheme(lib, o)
        assert np.array_equal(_gemm(lib, s, b, cA, dA, cB, dB, torch.float32), ref)
        assert np.array_equal(_gemm(lib, s, b, cA, dA, cB, dB, torch.float32, materialised=True), ref)
        oA, odA = oracle.quantize_rows(A, b)
        oB, odB = oracle.quantize_rows(B, b)
        assert np.array_equal(ref, oracle.int8_classical(oA, odA, oB, odB, od="f32"))


def test_certificate_is_enforced():
    lib = fmm()
    M, K, N = 32, 128, 32
    At, A, Bt, B = _inputs(41, M, K, N)
    cA, dA = _quantize(lib, At, 32)
    cB, dB = _quantize(lib, Bt, 32)
    s2 = _lib_scheme(lib, S2)
    ws = workspace(lib.int8_gemm_workspace(s2, M, K, N))
    C = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.FmmError) as ei:
        lib.int8_gemm(s2, 32, cA, dA, cB, dB, C, ws)        # L_A * 32 = 128 > 127
    assert ei.value.code == 10
    # a gauged scheme has non-integer coefficients: no certificate at any code bound
    P = gen.gauge_cond_limited(7, 0, 4)
    with pytest.raises(lib.FmmError) as ei:
        lib.int8_gemm(lib.gauge_apply(s2, P, P, P), 1, cA, dA, cB, dB, C, ws)
    assert ei.value.code == 10
    # one level of Strassen has L_A = 2 and admits the same codes
    s1 = _lib_scheme(lib, S1)
    ws1 = workspace(lib.int8_gemm_workspace(s1, M, K, N))
    lib.int8_gemm(s1, 32, cA, dA, cB, dB, C, ws1)
    lib.device_status(ws1)
    oA, odA = oracle.quantize_rows(A, 32)
    oB, odB = oracle.quantize_rows(B, 32)
    assert np.array_equal(C.to(torch.float64).cpu().numpy(), oracle.int8_classical(oA, odA, oB, odB))


def test_row_locality_on_device():
    """Section 4.2: changing a later token row leaves every earlier output row's bits alone (32 rows, 4 blocks)."""
    lib = fmm()
    M, K, N = 32, 256, 64
    At, A, Bt, B = _inputs(51, M, K, N)
    s2 = _lib_scheme(lib, S2)
    cB, dB = _quantize(lib, Bt, 31)
    cA, dA = _quantize(lib, At, 31)
    base = _gemm(lib, s2, 31, cA, dA, cB, dB)
    moved = 0
    for later in (1, 9, 17, 31):
        A2 = At.clone()
        A2[later] = gen.to_storage(gen.normal(51, 700 + later, (K,)), "f32")[0].cuda()
        c2, d2 = _quantize(lib, A2, 31)
        out = _gemm(lib, s2, 31, c2, d2, cB, dB)
        moved += sum(int(np.any(out[e] != base[e])) for e in range(later))
        assert np.any(out[later] != base[later])
    assert moved == 0


def test_fp8_schedule_moves_the_48_same_offset_pairs_on_device():
    """The FP8 counterpart (Section 4.2): block sums rounded before multiplying move exactly the 48 of 496 row pairs
    that share an offset in their blocks, with or without row-owned scales; the classical product moves none."""
    import gpu_util as gu
    lib = fmm()
    s2 = lib.scheme_builtin("strassen444")
    At, A = gen.to_storage(gen.normal(6, 1, (32, 128)), "f32")
    Bt, B = gen.to_storage(gen.normal(6, 2, (128, 32)), "f32")
    At, Bt = At.cuda(), Bt.cuda()
    want = {(e, l) for l in range(32) for e in range(l) if e % 8 == l % 8}

    def moved(run):
        base = run(At)
        out_set = set()
        for later in range(32):
            A2 = At.clone()
            A2[later] = gen.to_storage(gen.normal(77, 900 + later, (128,)), "f32")[0].cuda()
            out = run(A2)
            out_set |= {(e, later) for e in range(later) if np.any(out[e] != base[e])}
        return out_set

    for mode in (0, 2):
        assert moved(lambda X: gu.run_scheme_gemm(s2, X, Bt, "f32", "e4m3", "f32", scale_mode=mode)) == want
    assert moved(lambda X: gu.run_classical(X, Bt, "f32", "e4m3", "f32", scale_mode=2)) == set()


@pytest.mark.parametrize("M,K,N", [(32, 128, 32), (512, 1024, 544), (200, 384, 96)])
def test_overflow_corrected_full_range_codes(M, K, N):
    """Section 4.3: two-level Strassen at code bound 127 with the split X = X0 + 256 R gives classical int8's bits."""
    lib = fmm()
    At, A, Bt, B = _inputs(61, M, K, N)
    cA, dA = _quantize(lib, At, 127)
    cB, dB = _quantize(lib, Bt, 127)
    oA, odA = oracle.quantize_rows(A, 127)
    oB, odB = oracle.quantize_rows(B, 127)
    want = oracle.int8_classical(oA, odA, oB, odB)
    assert np.array_equal(_gemm(lib, None, 127, cA, dA, cB, dB), want)
    variants = list(oracle.sign_variants(4, 4, 4))
    for v in (variants[0], variants[203], variants[-1]):
        s = _lib_scheme(lib, oracle.sign_variant(S2, *v))
        ws = workspace(lib.int8_gemm_corrected_workspace(s, M, K, N))
        C = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        lib.int8_gemm_corrected(s, cA, dA, cB, dB, C, ws)
        lib.device_status(ws)
        assert np.array_equal(C.to(torch.float64).cpu().numpy(), want)
    want_corr, mx = oracle.int8_corrected(S2, oA, odA, oB, odB)
    assert np.array_equal(want_corr, want) and mx[0] == 0 and mx[1] <= 2
    # one level of Strassen (h = 64, |R| <= 1), fp32 output
    s1 = _lib_scheme(lib, S1)
    ws = workspace(lib.int8_gemm_corrected_workspace(s1, M, K, N))
    C32 = torch.empty((M, N), dtype=torch.float32, device="cuda")
    lib.int8_gemm_corrected(s1, cA, dA, cB, dB, C32, ws)
    lib.device_status(ws)
    assert np.array_equal(C32.to(torch.float64).cpu().numpy(), oracle.int8_classical(oA, odA, oB, odB, od="f32"))
    # the uncorrected call has no certificate at this code bound
    s2 = _lib_scheme(lib, S2)
    with pytest.raises(lib.FmmError) as ei:
        _gemm(lib, s2, 127, cA, dA, cB, dB)
    assert ei.value.code == 10


def test_fine_group_control_on_the_device():
    """Section 4.2, the control that breaks condition (iii) (scales on groups of 32 under a call of 128): the device's
    result is the oracle's bit for bit, and with one token row replaced at a time by a loud one every one of the 496
    (earlier, later) pairs moves — beside 0 for the certified call (test_row_locality...) and 48 for FP8 block sums."""
    lib = fmm()
    s1 = lib.scheme_builtin("strassen222")
    s2 = lib.scheme_kron(s1, s1)
    o2 = S2
    A = gen.to_storage(gen.normal(6, 1, (32, 128)), "f32")[1]
    Bt = gen.to_storage(gen.normal(6, 2, (32, 128)), "f32")[1]
    Bd = torch.from_numpy(Bt).float().cuda()
    ws = workspace(lib.int8_finegroup_control_workspace(s2, 32, 128, 32, 128))

    def run(X):
        C = torch.empty((32, 32), dtype=torch.float32, device="cuda")
        lib.int8_finegroup_control(s2, torch.from_numpy(X).float().cuda(), Bd, C, ws)
        return C.double().cpu().numpy()

    cB, dB = oracle.quantize_rows(Bt, 31, g=32)
    cA, dA = oracle.quantize_rows(A, 31, g=32)
    assert np.array_equal(run(A), oracle.int8_finegroup_control(o2, cA, dA, cB, dB, call=128, od="f32"))
    base = run(A)
    moved = 0
    for later in range(32):
        A2 = A.copy()
        A2[later] = gen.to_storage(gen.normal(77, 900 + later, (128,), std=4.0), "f32")[1]
        out = run(A2)
        moved += sum(int(np.any(out[e] != base[e])) for e in range(later))
    assert moved == 496
    # two calls along K, bf16 output, one level of Strassen (fine groups of 64): still the oracle's bits
    A3 = gen.to_storage(gen.normal(8, 1, (16, 256)), "f32")[1]
    B3 = gen.to_storage(gen.normal(8, 2, (24, 256)), "f32")[1]
    C3 = torch.empty((16, 24), dtype=torch.bfloat16, device="cuda")
    ws3 = workspace(lib.int8_finegroup_control_workspace(s1, 16, 256, 24, 128))
    lib.int8_finegroup_control(s1, torch.from_numpy(A3).float().cuda(), torch.from_numpy(B3).float().cuda(), C3, ws3, code_bound=63)
    c3a, d3a = oracle.quantize_rows(A3, 63, g=64)
    c3b, d3b = oracle.quantize_rows(B3, 63, g=64)
    want = oracle.int8_finegroup_control(oracle.strassen(), c3a, d3a, c3b, d3b, call=128, od="bf16")
    assert np.array_equal(C3.double().cpu().numpy(), want)
    assert lib.int8_finegroup_control_workspace(s2, 30, 128, 32, 128) == 0      # rows do not split into four blocks
