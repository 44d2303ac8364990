"""Pins of the oracle's two repair rules (Appendix C, "The repair rules"): the power-of-two row scale and the joint
rounding of the weight's block sums.  The paper prints no number that a model-free test could reproduce for them, so
they are pinned to what their definitions fix: closed-form scale values and exact scale invariance; for the search —
the plain model-schedule codes when no sweep runs, candidates that bracket the bf16 value, an objective that never
rises, no change where H is diagonal (no coupling between products), coordinate-wise optimality at convergence checked
by brute force in fp64, and a lower measured error on operands with independent entries (the model behind e^T H e)."""
import itertools

import numpy as np
import pytest

import oracle
from fmm_inputs import generators as gen


def _bf16(x):
    return gen.to_storage(x, "bf16")[1]


def test_row_scale_closed_forms():
    K = 64
    rows = np.stack([np.full(K, 1.0), np.full(K, 1.0001), np.full(K, 0.75), np.full(K, 0.5), np.zeros(K),
                     np.full(K, 1e-3), np.full(K, 3.0), np.concatenate([[8.0], np.zeros(K - 1)])])
    want = [1.0, 2.0, 1.0, 0.5, 2.0 ** -9, 2.0 ** -9, 4.0, 1.0]           # RMS of the last row: 8 / sqrt(64) = 1
    assert np.array_equal(oracle.row_pow2_scales(rows), want)
    d = oracle.row_pow2_scales(gen.normal(1, 0, (50, 256)))
    assert np.all(np.log2(d) == np.round(np.log2(d)))                      # powers of two


def test_row_scale_makes_the_operator_scale_invariant_per_row():
    """Scaling a token row by a power of two scales d_t by the same factor: the scaled rows, and therefore every
    rounded block sum, keep their bits, and the output row scales exactly.  Without the rule the rows it is added to
    in the block sums change."""
    s2 = oracle.kron(oracle.strassen(), oracle.strassen())
    A, B = _bf16(gen.normal(2, 0, (64, 256))), _bf16(gen.weights(2, 1, 256, 128))
    A2 = A.copy(); A2[5] *= 64.0; A2[40] *= 2.0 ** -7
    outs = []
    for X in (A, A2):
        d = oracle.row_pow2_scales(X)
        outs.append(oracle.scheme_gemm(s2, X / d[:, None], B, "e4m3", "f32", 3, md="bf16") * d[:, None])
    f = np.ones(64); f[5] = 64.0; f[40] = 2.0 ** -7
    assert np.array_equal(outs[1], outs[0] * f[:, None])
    plain = [oracle.scheme_gemm(s2, X, B, "e4m3", "f32", 3, md="bf16") for X in (A, A2)]
    others = [t for t in range(64) if t not in (5, 40)]
    assert not np.array_equal(plain[1][others], plain[0][others])          # row 5 leaks into rows 21, 37, 53


def _block_sums_bf16(s, B):
    m, k, n, R = s.dims
    K, N = B.shape
    bk, bn = K // k, N // n
    V = np.asarray(s.V).reshape(R, k, n)
    out = np.zeros((R, bk, bn))
    for r in range(R):
        for l in range(k):
            for j in range(n):
                out[r] += V[r, l, j] * B[l * bk:(l + 1) * bk, j * bn:(j + 1) * bn]
    return oracle.round_to(out, "bf16")


def _H(s):
    m, k, n, R = s.dims
    U, W = np.asarray(s.U).reshape(R, -1), np.asarray(s.W).reshape(R, -1)
    return (W @ W.T) * (U @ U.T)


def test_no_sweep_gives_the_plain_model_schedule_codes():
    s2 = oracle.kron(oracle.strassen(), oracle.strassen())
    A, B = _bf16(gen.normal(3, 0, (64, 512))), _bf16(gen.weights(3, 1, 512, 640))      # 1 group, 2 column blocks (160)
    Bq, sB, st = oracle.joint_round_weights(s2, B, max_sweeps=0)
    C0, p = oracle.scheme_gemm(s2, A, B, "e4m3", "bf16", 3, parts=True, md="bf16")
    assert np.array_equal(Bq, p["Bhat"]) and np.array_equal(sB, p["sB"]) and st["moved"] == 0
    assert np.array_equal(oracle.scheme_gemm_weights(s2, A, B, Bq, sB), C0)


@pytest.mark.parametrize("name", ["classical111", "classical222"])
def test_uncoupled_products_keep_plain_rounding(name):
    """Classical algorithms: no two products share both an input and an output block, H is diagonal, and the nearer
    candidate is already optimal for every entry.  Only exact ties of the quotient b / s (common: bf16 values over a
    scale max|b| / 448) may switch, where fp32 rounding makes one decoded error a few ulps smaller than the other;
    the objective does not move."""
    s = oracle.classical_scheme(1, 1, 1) if name == "classical111" else oracle.classical_scheme(2, 2, 2)
    H = _H(s)
    assert np.array_equal(H, np.diag(np.diag(H)))
    B = _bf16(gen.weights(4, 1, 256, 256))
    Bq, sB, st = oracle.joint_round_weights(s, B)
    Bq0, _, _ = oracle.joint_round_weights(s, B, max_sweeps=0)
    assert st["sweeps"] <= 2 and st["moved"] < 0.01 * Bq.size
    assert abs(st["objective_after"] - st["objective_before"]) <= 1e-6 * st["objective_before"]
    sc = np.repeat(np.repeat(sB, 128, axis=1), 128, axis=2).transpose(0, 2, 1)[:, :Bq.shape[1], :Bq.shape[2]]
    mv = Bq != Bq0
    x = _block_sums_bf16(s, B)[mv] / sc[mv]
    assert np.all(np.abs(x - 0.5 * (Bq[mv] + Bq0[mv])) <= 1e-6 * np.abs(x))      # the moved ones sat on a midpoint


def test_search_properties_and_brute_force_on_strassen():
    s1 = oracle.strassen()
    B = _bf16(gen.weights(5, 1, 256, 256))
    Bq0, sB, _ = oracle.joint_round_weights(s1, B, max_sweeps=0)
    prev = None
    for sweeps in (1, 2, 12):
        Bq, sB2, st = oracle.joint_round_weights(s1, B, max_sweeps=sweeps)
        assert np.array_equal(sB2, sB)
        assert st["objective_after"] <= st["objective_before"]
        if prev is not None:
            assert st["objective_after"] <= prev * (1 + 1e-12)
        prev = st["objective_after"]
    assert 0 < st["moved"] and st["objective_after"] < 0.9 * st["objective_before"] and st["sweeps"] < 12
    # candidates bracket the bf16 block sum and are neighbours on the e4m3 grid
    b = _block_sums_bf16(s1, B)
    scale = np.repeat(np.repeat(sB, 128, axis=1)[:, :128], 128, axis=2)[:, :128, :128].transpose(0, 2, 1)
    import torch
    codes = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    grid = np.unique(codes[np.isfinite(codes)])                     # every finite e4m3 value, from the library's cast
    assert len(grid) == 253 and grid[0] == -448.0 and grid[-1] == 448.0
    assert np.all(np.isin(Bq, grid))
    moved = Bq != Bq0
    lo, hi = np.minimum(Bq, Bq0), np.maximum(Bq, Bq0)
    assert np.all((lo * scale <= b)[moved]) and np.all((b <= hi * scale)[moved])
    gi = np.searchsorted(grid, lo[moved])
    assert np.array_equal(grid[gi + 1], hi[moved])
    # brute force over the 2^7 candidate choices at sampled positions: the result is a coordinate-wise minimum of
    # e^T H e (fp64), and never worse than where it started
    H = _H(s1)
    for (t, c) in [(0, 0), (17, 93), (64, 5), (127, 127), (3, 70)]:
        bb, ss = b[:, t, c], scale[:, t, c]
        q_near, q_fin = Bq0[:, t, c], Bq[:, t, c]
        gi = np.searchsorted(grid, q_near)
        dq = ss * q_near
        other = np.where(dq < bb, grid[np.minimum(gi + 1, len(grid) - 1)], np.where(dq > bb, grid[np.maximum(gi - 1, 0)], q_near))
        def obj(qv):
            e = ss * qv - bb
            return float(e @ H @ e)
        assert set(np.where(q_fin != q_near)[0]) <= set(np.where(other != q_near)[0])
        assert np.all((q_fin == q_near) | (q_fin == other))
        best = min(obj(np.where(np.array(ch, dtype=bool), other, q_near)) for ch in itertools.product([0, 1], repeat=7))
        fin = obj(q_fin)
        assert best <= fin * (1 + 1e-9) <= obj(q_near) * (1 + 1e-6)
        for r in range(7):                                   # no single switch improves it (beyond fp32 noise)
            alt = q_fin.copy(); alt[r] = other[r] if q_fin[r] == q_near[r] else q_near[r]
            assert obj(alt) >= fin * (1 - 1e-5)


def test_joint_rounding_lowers_the_error_on_independent_entries():
    """e^T H e is the expected squared output error when the entries of A are independent with equal variance: on
    such operands the measured error falls, for the nesting the paper's first repaired algorithm uses."""
    hyb = oracle.kron(oracle.strassen(), oracle.classical_scheme(2, 2, 2))
    A, B = _bf16(gen.normal(6, 0, (256, 512))), _bf16(gen.weights(6, 1, 512, 512))
    Bq, sB, st = oracle.joint_round_weights(hyb, B)
    Bq0, _, _ = oracle.joint_round_weights(hyb, B, max_sweeps=0)
    Cs = A @ B
    # errors of the weight rounding alone: block sums of A kept exact by using the fp32 products of the codes
    E1 = oracle.rel_error(oracle.scheme_gemm_weights(hyb, A, B, Bq, sB, od="f32", md="f64"), Cs)
    E0 = oracle.rel_error(oracle.scheme_gemm_weights(hyb, A, B, Bq0, sB, od="f32", md="f64"), Cs)
    assert st["objective_after"] < 0.8 * st["objective_before"]
    assert E1 < E0
