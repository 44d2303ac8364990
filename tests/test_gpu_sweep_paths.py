"""The execution paths of error_sweep against one another and against its documented error behaviour.

The pipelined path (consecutive batches of gauges overlapped over the library's streams, two workspaces in flight)
must give the bits of the serial path (every stage back to back on the caller's stream); a sweep cut into two calls
must give the ratios of the one call (how a long sweep is resumed); a singular gauge anywhere in the list must be
refused before anything is enqueued; NaN in the operands must come out as NaN, not as an arbitrary order statistic.
"""
import math

import numpy as np
import pytest
import torch

from fmm_inputs import generators as gen

import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__
    __graft_entry__.build()
    return gu.fmm()


def _gauges(G, seed=4):
    P = np.stack([gen.gauge_log_uniform_cond(seed, 3 * g, 2) for g in range(G)])
    Q = np.stack([gen.gauge_log_uniform_cond(seed, 3 * g + 1, 2) for g in range(G)])
    S = np.stack([gen.gauge_log_uniform_cond(seed, 3 * g + 2, 2) for g in range(G)])
    return P, Q, S


def _ops(seed, M, K, N):
    A = gen.activations_outlier(seed, 1, M, K, dist="t3", frac=0.001, factor=300.0, at_least=1)
    W = gen.normal(seed, 2, (N, K), std=0.02)
    return gen.to_storage(A, "bf16")[0].cuda(), gen.to_storage(W, "bf16")[0].cuda()


@pytest.mark.parametrize("Pd,scale,level", [("e4m3", 1, 1), ("bf16", 0, 1), ("bf16", 0, 0), ("e4m3", 2, 0)])
def test_pipelined_sweep_gives_the_bits_of_the_serial_one(lib, Pd, scale, level):
    """Mid-size problems whose decode grid spans several waves behind the persistent product kernel: with one scale per
    encoded tensor the decode of batch c-2 reads scales that the encode of batch c rewrites, so the two must be
    ordered; every other buffer has the same hazard one stage earlier."""
    M, K, N, G = 2048, 2048, 2048, 12
    At, Wt = _ops(7, M, K, N)
    P, Q, S = _gauges(G)
    s1 = lib.scheme_builtin("strassen222")
    s = lib.scheme_kron(s1, s1) if level == 1 else s1
    d = lib.GemmDesc.make(M, K, N, "bf16", Pd, "bf16", weight_layout=True, scale_mode=scale, flags=lib.FLAG_SWEEP_UNFUSED)
    ds = lib.GemmDesc.make(M, K, N, "bf16", Pd, "bf16", weight_layout=True, scale_mode=scale, flags=lib.FLAG_SWEEP_SERIAL)
    ws = gu.workspace(lib.error_sweep_workspace(s, d, G))
    serial, _ = lib.error_sweep(s, level, P, Q, S, ds, At, Wt, ws)
    for _ in range(3):
        piped, _ = lib.error_sweep(s, level, P, Q, S, d, At, Wt, ws)
        assert np.array_equal(piped, serial)


@pytest.mark.parametrize("M,K,N,G,O", [(2048, 2048, 2048, 27, "bf16"), (1024, 512, 1536, 16, "f32"), (1024, 256, 2048, 17, "bf16")])
def test_fused_sweep_launches_against_the_serial_path(lib, M, K, N, G, O):
    """The fused launches (default where they apply): products of a batch, decode of the batch before and encode of the batch after in one launch.
    Every algorithm's C is the same bits as on the serial path; its error sum is added over another partition of the
    outputs (the fused launch has its own number of streaming blocks), so ratios agree to 1e-6, and run to run they are
    bit-identical.  G = 27 leaves a batch of two and one of one behind the fused batches (8 + 8 + 8 | 2 + 1)."""
    At, Wt = _ops(12, M, K, N)
    P, Q, S = _gauges(G, seed=9)
    s1 = lib.scheme_builtin("strassen222")
    mk = lambda fl: lib.GemmDesc.make(M, K, N, "bf16", "bf16", O, weight_layout=True, flags=fl)
    ws = gu.workspace(lib.error_sweep_workspace(s1, mk(0), G))
    serial, ss = lib.error_sweep(s1, 0, P, Q, S, mk(lib.FLAG_SWEEP_SERIAL), At, Wt, ws)
    n0 = lib.launch_count()
    fused, sf = lib.error_sweep(s1, 0, P, Q, S, mk(0), At, Wt, ws)
    n_fused = lib.launch_count() - n0
    n0 = lib.launch_count()
    piped, _ = lib.error_sweep(s1, 0, P, Q, S, mk(lib.FLAG_SWEEP_UNFUSED), At, Wt, ws)
    assert n_fused < lib.launch_count() - n0              # the fused path really ran: far fewer launches
    assert np.array_equal(piped, serial)                  # the three-stream pipeline uses the serial path's kernels
    assert np.all(np.abs(fused - serial) <= 1e-6 * serial)
    assert sf["count_gt2"] == ss["count_gt2"]
    again, _ = lib.error_sweep(s1, 0, P, Q, S, mk(0), At, Wt, ws)
    assert np.array_equal(again, fused)


def test_sweep_in_two_calls_is_the_sweep_in_one(lib):
    """Resuming: gauges [0, G1) in one call and [G1, G) in a second (pointer offset into the gauge arrays) give the
    ratios of the single call, up to the grouping of a batch's error partials (1e-6), and the same summary."""
    M, K, N, G, G1 = 512, 1024, 768, 21, 13
    At, Wt = _ops(8, M, K, N)
    P, Q, S = _gauges(G, seed=5)
    s1 = lib.scheme_builtin("strassen222")
    d = lib.GemmDesc.make(M, K, N, "bf16", "bf16", "bf16", weight_layout=True)
    ws = gu.workspace(lib.error_sweep_workspace(s1, d, G))
    whole, summ = lib.error_sweep(s1, 0, P, Q, S, d, At, Wt, ws)
    first, _ = lib.error_sweep(s1, 0, P[:G1], Q[:G1], S[:G1], d, At, Wt, ws)
    second, _ = lib.error_sweep(s1, 0, P[G1:], Q[G1:], S[G1:], d, At, Wt, ws)
    parts = np.concatenate([first, second])
    assert np.all(np.abs(parts - whole) <= 1e-6 * whole)
    import oracle
    so = oracle.summary(parts)
    assert so["count_gt2"] == summ["count_gt2"]
    for key in ("min", "median", "max"):
        assert math.isclose(so[key], summ[key], rel_tol=1e-6)


def test_singular_gauge_late_in_the_list_is_refused_before_any_launch(lib):
    M, K, N, G = 256, 512, 384, 40
    At, Wt = _ops(9, M, K, N)
    P, Q, S = _gauges(G, seed=6)
    Q[37] = np.array([[1.0, 2.0], [2.0, 4.0]])          # beyond the first group of tables the call builds
    s1 = lib.scheme_builtin("strassen222")
    d = lib.GemmDesc.make(M, K, N, "bf16", "bf16", "bf16", weight_layout=True)
    ws = gu.workspace(lib.error_sweep_workspace(s1, d, G))
    ws.fill_(0x5A)
    before = lib.launch_count()
    with pytest.raises(lib.FmmError) as err:
        lib.error_sweep(s1, 0, P, Q, S, d, At, Wt, ws)
    assert err.value.code == 4
    assert lib.launch_count() == before                    # nothing was enqueued
    torch.cuda.synchronize()
    assert bool((ws == 0x5A).all())                        # and nothing touched the workspace
    good, _ = lib.error_sweep(s1, 0, P[:37], Q[:37], S[:37], d, At, Wt, ws)
    assert np.all(np.isfinite(good))


def test_nan_operands_give_nan_summary(lib):
    M, K, N, G = 256, 512, 384, 5
    At, Wt = _ops(10, M, K, N)
    At[3, 5] = float("nan")
    P, Q, S = _gauges(G, seed=7)
    s1 = lib.scheme_builtin("strassen222")
    d = lib.GemmDesc.make(M, K, N, "bf16", "bf16", "bf16", weight_layout=True)
    ws = gu.workspace(lib.error_sweep_workspace(s1, d, G))
    ratios, summ = lib.error_sweep(s1, 0, P, Q, S, d, At, Wt, ws)
    assert np.all(np.isnan(ratios))
    assert all(math.isnan(summ[k]) for k in ("min", "median", "max", "spread")) and summ["count_gt2"] == 0
