"""GPU parity of the rotation pre-pass (Appendix B, "A rotation, other summation orders and repeated runs")
against the oracle's fp64 definition, through the C ABI.

Tolerance: the kernel runs the fast Walsh-Hadamard recursion in fp32 — log2(h) additions per output, each with
relative error 2^-24 of the running magnitude, which is bounded by sqrt(h) |x|_2 of the block — then one
multiplication by fl(1/sqrt(h)).  Per element that is at most (log2(h) + 2) 2^-24 |x|_2(block); for bf16 storage the
final rounding can land on the neighbouring code when the fp32 value sits within that distance of a tie, so a
small fraction of outputs may differ by one bf16 unit in the last place and no more."""
import math

import numpy as np
import pytest
import torch

import oracle
from fmm_inputs import generators as gen
import gpu_util as gu
from test_oracle_rotation import rotation_operands, _golden

pytestmark = pytest.mark.gpu

TOL_RATIO = 0.02


@pytest.fixture(scope="module")
def lib():
    return gu.fmm()


def _signs(seed, K):
    return np.where(gen.uniform(seed, 77, (K,)) < 0.5, -1.0, 1.0)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("h", [2, 4, 8, 64, 128, 256, 512, 1024])
def test_rotation_matches_the_definition(lib, dtype, h):
    rows, K, ld = 37, 2048, 2048 + 24            # ragged row count, padded leading dimension
    Xt, X64 = gu.storage_pair(gen.normal(9, h, (rows, K)), dtype)
    Xp = torch.zeros((rows, ld), dtype=Xt.dtype, device="cuda")
    Xp[:, :K] = Xt
    sg = _signs(h, K)
    sg_t = torch.from_numpy(sg.astype(np.int8)).cuda()
    out = torch.full((rows, ld), 7.0, dtype=Xt.dtype, device="cuda")
    lib.hadamard_rotate(Xp[:, :K], sg_t, h, out=out[:, :K])
    torch.cuda.synchronize()
    assert torch.all(out[:, K:] == 7.0)                      # padding untouched
    got = out[:, :K].to(torch.float64).cpu().numpy()
    want = oracle.hadamard_rotate(X64, sg, h)                # fp64, unrounded
    blk = np.linalg.norm(X64.reshape(rows, K // h, h), axis=2)
    bound = (math.log2(h) + 2) * 2.0 ** -24 * np.repeat(blk, h, axis=1)
    if dtype == "f32":
        assert np.all(np.abs(got - want) <= bound + 2.0 ** -22 * np.abs(want))
    else:
        ref = oracle.round_to(want, "bf16")
        diff = got != ref
        assert diff.mean() < 2e-3, diff.mean()
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(ref), 1e-30))) - 7)
        assert np.all(np.abs(got - ref)[diff] <= np.maximum(ulp[diff] * 1.0001, 2 * bound[diff]))   # cancelled entries: fp32 noise floor
        assert np.all(np.abs(got - want) <= bound + 2.0 ** -8 * np.abs(want))
    # in place, and without signs
    lib.hadamard_rotate(Xp[:, :K], sg_t, h, out=Xp[:, :K])
    assert torch.equal(Xp[:, :K], out[:, :K])
    Y0 = lib.hadamard_rotate(Xt, None, h)
    want0 = oracle.hadamard_rotate(X64, np.ones(K), h, dtype if dtype == "bf16" else "f64")
    assert gu.rel_fro(Y0.to(torch.float64).cpu().numpy(), want0) <= (1e-6 if dtype == "f32" else 1e-3)


def test_large_operand_spans_many_waves_and_keeps_the_product(lib):
    """4096 x 4096 bf16 (config 2's A): grid-stride path; sampled rows against the oracle; A H (B^T H)^T = A B^T."""
    At, A64 = gu.storage_pair(gen.normal(1, 0, (4096, 4096)), "f32")
    Bt, B64 = gu.storage_pair(gen.normal(1, 1, (512, 4096), std=0.02), "f32")
    sg = _signs(3, 4096)
    sg_t = torch.from_numpy(sg.astype(np.int8)).cuda()
    Ar, Br = lib.hadamard_rotate(At, sg_t, 128), lib.hadamard_rotate(Bt, sg_t, 128)
    rows = [0, 1, 777, 2048, 4095]
    want = oracle.hadamard_rotate(A64[rows], sg, 128)
    assert gu.rel_fro(Ar[rows].to(torch.float64).cpu().numpy(), want) <= 1e-6
    C0 = (At[:256].double() @ Bt.double().T).cpu().numpy()
    C1 = (Ar[:256].double() @ Br.double().T).cpu().numpy()
    assert gu.rel_fro(C1, C0) <= 1e-6
    # constant rows collapse onto one entry per block
    ones = torch.full((8, 1024), 0.75, dtype=torch.bfloat16, device="cuda")
    Y = lib.hadamard_rotate(ones, None, 256).float().cpu().numpy()
    want1 = np.zeros((8, 1024)); want1[:, ::256] = 0.75 * 16.0
    assert np.array_equal(Y, want1)


def test_single_row_and_single_block(lib):
    for dtype, K, h in (("f32", 4, 4), ("bf16", 8, 8), ("bf16", 1024, 1024), ("f32", 2, 2)):
        Xt, X64 = gu.storage_pair(gen.normal(4, K, (1, K)), dtype)
        if (K * Xt.element_size()) % 16:
            continue                                   # rows must be whole 16-byte vectors: checked elsewhere
        Y = lib.hadamard_rotate(Xt, None, h)
        want = oracle.hadamard_rotate(X64, np.ones(K), h, dtype if dtype == "bf16" else "f64")
        assert gu.rel_fro(Y.to(torch.float64).cpu().numpy(), want) <= (1e-6 if dtype == "f32" else 4e-3)


def test_argument_checks_launch_nothing(lib):
    X = torch.zeros((4, 64), dtype=torch.float32, device="cuda")
    for h in (0, 1, 3, 48, 2048):
        with pytest.raises(lib.FmmError):
            lib.hadamard_rotate(X, None, h)
    with pytest.raises(lib.FmmError):
        lib.hadamard_rotate(X[:, :48], None, 32)             # K % h
    with pytest.raises(lib.FmmError):
        lib.hadamard_rotate(X[:, 1:33], None, 32)            # misaligned base


def test_rotation_experiment_on_the_device(lib):
    """One-level Strassen, 128 x 128, e4m3 block sums with per-row / per-column scales, its 8 sign variants through
    error_sweep, before and after the rotation: per-variant errors agree with the oracle, and the spreads move the
    way the paper prints (2.137 -> 1.300 under a common offset; 1.240 -> 1.317 under outlier offsets)."""
    var = oracle.sign_variants(2, 2, 2)
    P = np.stack([np.diag(v[0]) for v in var]); Q = np.stack([np.diag(v[1]) for v in var]); S = np.stack([np.diag(v[2]) for v in var])
    s1, o1 = lib.scheme_builtin("strassen222"), oracle.strassen()
    d = lib.GemmDesc.make(128, 128, 128, "f32", "e4m3", "f32", scale_mode=2)
    ws = gu.workspace(lib.error_sweep_workspace(s1, d, len(var)))
    draws = 40
    gold = _golden()
    for case in ("uniform_offset", "outlier_offsets"):
        errs = np.empty((2, len(var), draws))
        for p in range(draws):
            A, B, signs = rotation_operands(case, 5, p)
            At, Bt = torch.from_numpy(A).float().cuda(), torch.from_numpy(B).float().cuda()
            sg_t = torch.from_numpy(signs.astype(np.int8)).cuda()
            Cs = gu.run_exact(At, Bt, "f32")
            Ar = lib.hadamard_rotate(At, sg_t, 128)
            Br = lib.hadamard_rotate(Bt.T.contiguous(), sg_t, 128).T.contiguous()
            for rot, (Ax, Bx) in enumerate(((At, Bt), (Ar, Br))):
                ratios, summ = lib.error_sweep(s1, 0, P, Q, S, d, Ax, Bx, ws, Cstar=Cs)
                errs[rot, :, p] = ratios * summ["e_classical_rel"]
            if p == 0:
                Cs64 = A @ B
                Ar64 = oracle.hadamard_rotate(A, signs, 128, "f32")
                Br64 = oracle.hadamard_rotate(B.T.copy(), signs, 128, "f32").T.copy()
                for vi in (0, 3, 7):
                    sv = oracle.sign_variant(o1, *var[vi])
                    E0 = oracle.rel_error(oracle.scheme_gemm(sv, A, B, "e4m3", "f32", 2), Cs64)
                    E1 = oracle.rel_error(oracle.scheme_gemm(sv, Ar64, Br64, "e4m3", "f32", 2), Cs64)
                    assert abs(errs[0, vi, 0] - E0) <= TOL_RATIO * E0
                    assert abs(errs[1, vi, 0] - E1) <= TOL_RATIO * E1
        avg = errs.mean(axis=2)
        plain, rot = avg[0].max() / avg[0].min(), avg[1].max() / avg[1].min()
        want_plain, want_rot = gold[case]
        assert abs(plain - want_plain) < 0.10 * want_plain and abs(rot - want_rot) < 0.06 * want_rot, (case, plain, rot)
        assert (rot < plain) == (case == "uniform_offset")
