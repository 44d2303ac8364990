"""Pins of the oracle's certified int8 realisation (Section 4.2, Proposition 1, Appendix D) — no GPU."""
import numpy as np
import pytest

import oracle
from fmm_inputs import generators as gen

S1 = oracle.strassen()
S2 = oracle.kron(S1, S1)


def _quantised(seed, M, K, N, b):
    A = gen.to_storage(gen.normal(seed, 1, (M, K)), "f32")[1]
    Bt = gen.to_storage(gen.normal(seed, 2, (N, K)) * 0.02, "f32")[1]
    cA, dA = oracle.quantize_rows(A, b)
    cB, dB = oracle.quantize_rows(Bt, b)
    return A, Bt, cA, dA, cB, dB


def test_quantiser_rules():
    X = np.zeros((2, 256))
    X[0, :128] = np.linspace(-3.0, 3.0, 128)
    X[1, 128:] = 1e-3 * np.arange(128)
    c, d = oracle.quantize_rows(X, 31)
    assert d.shape == (2, 2) and d[0, 1] == 1.0 and d[1, 0] == 1.0          # all-zero group: d = 1
    assert np.float32(d[0, 0]) == np.float32(3.0) / np.float32(31)          # d = max|x| / b in fp32
    assert np.abs(c).max() == 31 and np.all(c == np.rint(c))                # no clipping needed: |code| <= b
    assert c[0, 0] == -31 and c[0, 127] == 31 and np.all(c[0, 128:] == 0)
    # ties to even: x/d = 0.5 -> 0, 1.5 -> 2, 2.5 -> 2   (d = 1 when max|x| = b)
    Y = np.zeros((1, 128)); Y[0, :4] = [31.0, 0.5, 1.5, 2.5]
    c2, d2 = oracle.quantize_rows(Y, 31)
    assert d2[0, 0] == 1.0 and c2[0, :4].tolist() == [31.0, 0.0, 2.0, 2.0]


def test_certificate_constants_of_two_level_strassen():
    """Section 4.2: L_A = L_B = 4 admit b = 31; with L_W = 16, g = 128 and h = 32 the certificate holds for
    int32 and for exact integers in fp32; inner length 8729 is the int32 limit; b = 32 breaks condition (i);
    a call spanning more than one group breaks condition (iii)."""
    ok, c = oracle.certificate(S2, 31, 31, 32, 128, 31)
    assert ok and c["LAbA"] == 124 and c["LBbB"] == 124 and c["largest"] == 16 * 32 * 124 * 124
    assert oracle.certificate(S2, 31, 31, 32, 128, 24)[0]                    # 7.87e6 < 2^24: fp32 emulation is exact
    assert not oracle.certificate(S2, 32, 31, 32, 128, 31)[0]                # 4 * 32 = 128 > 127
    assert oracle.certificate(S2, 31, 31, 8729, 4 * 8729, 31)[0]
    assert not oracle.certificate(S2, 31, 31, 8730, 4 * 8730, 31)[0]
    assert not oracle.certificate(S2, 31, 31, 64, 128, 31)[0]                # call of 256 over groups of 128
    ok1, c1 = oracle.certificate(S1, 63, 63, 64, 128, 31)                    # one level: L = 2 admits b = 63
    assert ok1 and c1["LAbA"] == 126


def test_certified_equals_classical_bit_for_bit_all_sign_variants():
    """All 512 sign variants compute one integer product and one output, the classical int8 operator's."""
    A, Bt, cA, dA, cB, dB = _quantised(3, 32, 256, 16, 31)
    ref, Pref = oracle.int8_classical(cA, dA, cB, dB, products=True)
    outs, prods = set(), set()
    for d, e, f in oracle.sign_variants(4, 4, 4):
        out, mx, P = oracle.int8_certified(oracle.sign_variant(S2, d, e, f), cA, dA, cB, dB, products=True)
        outs.add(out.tobytes()); prods.add(P.tobytes())
        assert mx[0] <= 124 and mx[1] <= 124 and mx[2] <= 16 * 32 * 124 * 124
    assert outs == {ref.tobytes()} and prods == {Pref.tobytes()}
    # the operator is close to the fp64 product at the accuracy 31 codes allow
    assert oracle.rel_error(ref, A @ Bt.T) < 0.05


def test_200_random_tiles_exact():
    for trial in range(200):
        cA = gen.integer_matrix(100 + trial, 1, (8, 128), 31)
        cB = gen.integer_matrix(100 + trial, 2, (8, 128), 31)
        one = np.ones((8, 1))
        _, mx, P = oracle.int8_certified(S2, cA, one, cB, one, products=True, od="f32")
        assert np.array_equal(P[0], cA @ cB.T)


def test_row_locality_zero_of_496_pairs_move():
    """Section 4.2: 32 token rows in four blocks, one row changed at a time: no earlier output row moves."""
    A, Bt, cA, dA, cB, dB = _quantised(5, 32, 128, 32, 31)
    base, _ = oracle.int8_certified(S2, cA, dA, cB, dB)
    moved = pairs = 0
    for later in range(32):
        A2 = A.copy()
        A2[later] = gen.to_storage(gen.normal(5, 300 + later, (128,)), "f32")[1]
        c2, d2 = oracle.quantize_rows(A2, 31)
        out, _ = oracle.int8_certified(S2, c2, d2, cB, dB)
        for earlier in range(later):
            pairs += 1
            moved += int(np.any(out[earlier] != base[earlier]))
        assert np.any(out[later] != base[later])
    assert pairs == 496 and moved == 0


def test_bound_is_sharp_and_violations_are_reported():
    """Codes whose signs follow the coefficients reach L_A * b (Appendix D: the bound is sharp); at b = 32 a
    block sum leaves the int8 range."""
    for b, limit in ((31, 124), (32, 128)):
        cA = np.zeros((4, 128)); cB = gen.integer_matrix(9, 2, (4, 128), b)
        r = int(np.argmax(np.abs(S2.U).sum(axis=(1, 2))))                  # a product with four nonzero u
        for i in range(4):
            for l in range(4):
                cA[i, 32 * l:32 * l + 32] = b * np.sign(S2.U[r, i, l])
        one = np.ones((4, 1))
        _, mx = oracle.int8_certified(S2, cA, one, cB, one, od="f32")
        assert mx[0] == limit
    with pytest.raises(ValueError):
        P = gen.gauge_cond_limited(1, 0, 2)
        oracle.int8_certified(oracle.gauge(S1, P, P, P), cA[:2], one[:2], cB[:2], one[:2])


def _pairs_moved(run, A, rows=32, std=1.0):
    base = run(A)
    moved = set()
    for later in range(rows):
        A2 = A.copy()
        A2[later] = gen.to_storage(gen.normal(77, 900 + later, (A.shape[1],), std=std), "f32")[1]
        out = run(A2)
        for earlier in range(later):
            if np.any(out[earlier] != base[earlier]):
                moved.add((earlier, later))
    return moved


def test_fp8_schedule_moves_exactly_the_48_same_offset_pairs():
    """Section 4.2: the same coefficients under an FP8 schedule that rounds the block sums before multiplying move
    48 of the 496 (earlier, later) row pairs — exactly those whose rows share an offset in their blocks (32 rows in
    four blocks of 8: 8 offsets x C(4,2) pairs).  Row-owned scales (one per row of each block sum) keep it at 48;
    the classical product at the same dtype moves none."""
    A = gen.to_storage(gen.normal(6, 1, (32, 128)), "f32")[1]
    B = gen.to_storage(gen.normal(6, 2, (128, 32)), "f32")[1]
    want = {(e, l) for l in range(32) for e in range(l) if e % 8 == l % 8}
    assert len(want) == 48
    for mode in (0, 2):
        moved = _pairs_moved(lambda X: oracle.scheme_gemm(S2, X, B, "e4m3", "f32", scale_mode=mode), A)
        assert moved == want, (mode, len(moved))
    assert _pairs_moved(lambda X: oracle.classical_gemm(X, B, "e4m3", "f32", 2), A) == set()


def test_fine_group_control_moves_all_496_pairs():
    """Section 4.2, the control that breaks condition (iii): scales on groups of 32 indices while a call spans 128.
    Every mixed block sum is rounded again with one scale set by its largest magnitude, which any of its rows can
    change: all 496 (earlier, later) pairs move — the third of the printed counts 0 / 48 / 496.  With the scales on
    groups of 128 (condition (iii) kept) the same inputs move none (test_row_locality_zero_of_496_pairs_move)."""
    A = gen.to_storage(gen.normal(6, 1, (32, 128)), "f32")[1]
    Bt = gen.to_storage(gen.normal(6, 2, (32, 128)), "f32")[1]
    cB, dB = oracle.quantize_rows(Bt, 31, g=32)

    def run(X):
        cA, dA = oracle.quantize_rows(X, 31, g=32)
        return oracle.int8_finegroup_control(S2, cA, dA, cB, dB, call=128, od="f32")
    # "which any of its rows can change": a replacement row loud enough (N(0, 4^2) among N(0, 1) rows) to take over the
    # largest magnitude of every block sum it enters changes every such scale, and every pair moves ...
    assert len(_pairs_moved(run, A, std=4.0)) == 496
    # ... while a replacement no louder than its neighbours changes a scale only when it held, or takes, the maximum:
    # most pairs move, not all
    quiet = len(_pairs_moved(run, A, std=1.0))
    assert 350 < quiet < 496
    # the same loud replacement leaves the two structural counts where they are: 0 for the certified call (scales on
    # the call's own group of 128), 48 for block sums rounded to FP8
    cB128, dB128 = oracle.quantize_rows(Bt, 31, g=128)

    def run_cert(X):
        cA, dA = oracle.quantize_rows(X, 31, g=128)
        return oracle.int8_certified(S2, cA, dA, cB128, dB128, od="f32")[0]
    assert _pairs_moved(run_cert, A, std=4.0) == set()
    assert len(_pairs_moved(lambda X: oracle.scheme_gemm(S2, X, Bt.T.copy(), "e4m3", "f32"), A, std=4.0)) == 48
    # the control is still a sound approximation of the product (it is the invariance that is lost, not the accuracy)
    ref = A @ Bt.T
    assert np.linalg.norm(run(A) - ref) <= 0.1 * np.linalg.norm(ref)     # code bound 31: a few per cent
    # one fine group per call (call = 32 with a <1,1,1;1> algorithm) is the classical operator on groups of 32: row local
    one = oracle.classical_scheme(1, 1, 1)

    def run_cl(X):
        cA, dA = oracle.quantize_rows(X, 31, g=32)
        return oracle.int8_classical(cA, dA, cB, dB, g=32, od="f32")
    assert _pairs_moved(run_cl, A, std=4.0) == set()


def test_fp8_block_sums_leave_no_sign_variant_exact_on_integer_codes():
    """Section 4.2: on a tile of integer codes every sign variant gives the one exact integer product, but with the
    block sums rounded to e4m3 (4 significant bits: sums up to 124 are not representable) none of the 512 does,
    and their largest errors differ severalfold (the paper's tile: 3.17x)."""
    cA = gen.integer_matrix(8, 1, (32, 128), 31)
    cB = gen.integer_matrix(8, 2, (128, 32), 31)
    exact = cA @ cB
    worst = []
    for d, e, f in oracle.sign_variants(4, 4, 4):
        sv = oracle.sign_variant(S2, d, e, f)
        worst.append(np.abs(oracle.scheme_gemm(sv, cA, cB, "e4m3", "f32") - exact).max())
    worst = np.array(worst)
    assert np.all(worst > 0)
    assert 1.5 < worst.max() / worst.min() < 8.0
    assert np.array_equal(oracle.scheme_gemm(S2, cA, cB, "f64", "f64"), exact)


def test_overflow_correction_full_range_codes():
    """Section 4.3 and its certificate: at code bound 127 the block sums reach L_A * 127 = 508, the split keeps
    every multiplicand in int8 with |R| <= 2, the terms of a rebuilt product stay within h (128 + 512)^2 =
    13,107,200, the combination within 16 times that (< 2^31), and the output is classical int8's bit for bit."""
    A, Bt, cA, dA, cB, dB = _quantised(13, 32, 256, 32, 127)
    ref, Pref = oracle.int8_classical(cA, dA, cB, dB, products=True)
    for v in oracle.sign_variants(4, 4, 4)[::57]:
        out, mx, P = oracle.int8_corrected(oracle.sign_variant(S2, *v), cA, dA, cB, dB, products=True)
        assert np.array_equal(P, Pref) and np.array_equal(out, ref)
        assert mx[0] == 0 and mx[1] <= 2 and mx[2] <= 32 * (128 + 512) ** 2 == 13107200
        assert mx[3] <= 16 * 13107200 < 2 ** 31 and 127 < mx[4] <= 508
    assert np.abs(Pref).max() <= 128 * 127 ** 2 == 2064512 < 2 ** 24
    # the uncorrected call at this code bound has no certificate: block sums leave the int8 range
    assert not oracle.certificate(S2, 127, 127, 32, 128, 31)[0]
    _, mx_plain = oracle.int8_certified(S2, cA, dA, cB, dB)
    assert mx_plain[0] > 127
    # sign-aligned codes reach the bound 508 and the largest correction |R| = 2
    cA2 = np.zeros((4, 128)); r = int(np.argmax(np.abs(S2.U).sum(axis=(1, 2))))
    for i in range(4):
        for l in range(4):
            cA2[i, 32 * l:32 * l + 32] = 127 * np.sign(S2.U[r, i, l])
    one = np.ones((4, 1))
    cB2 = gen.integer_matrix(9, 2, (4, 128), 127)
    outc, mx2, P2 = oracle.int8_corrected(S2, cA2, one, cB2, one, od="f32", products=True)
    assert mx2[4] == 508 and mx2[1] == 2 and np.array_equal(P2[0], cA2 @ cB2.T)
    # split identity on every residue: floor((x + 128) / 256), remainder in [-128, 127]
    for x in range(-508, 509):
        hi = (x + 128) // 256
        assert -128 <= x - 256 * hi <= 127 and abs(hi) <= 2
