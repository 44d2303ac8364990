"""GPU test of error_frobenius_noalloc, the entry point for callers that cannot allocate device memory
(graph capture, committed memory pools, hosts that forbid a library from allocating after start-up).

It is called twice in a row through the C ABI and compared with error_frobenius, the workspace-taking entry
point, on the same inputs; the second call checks that nothing left in the library's fixed scratch array by the
first call leaks into the result.  This file is named to be collected last, so a run that stops at the first
failure has already run everything else.
"""
import math

import pytest
import torch

from fmm_inputs import generators as gen

import gpu_util as gu

pytestmark = pytest.mark.gpu


def _reference(lib, d, Cmat, Cstar):
    out = torch.zeros(2, dtype=torch.float64, device="cuda")
    ws = gu.workspace(64 * 1024)
    lib.error_frobenius(d, Cmat, Cstar, out, ws)
    return out.cpu().tolist()


def test_noalloc_matches_workspace_variant_twice_in_a_row():
    import __graft_entry__
    __graft_entry__.build()
    lib = gu.fmm()
    # first call: a bf16 result with a padded leading dimension; second call: a smaller fp32 one
    cases = [(1024, 1536, torch.bfloat16, "bf16", 1536 + 64), (384, 264, torch.float32, "f32", 264)]
    for M, N, td, O, ldc in cases:
        Cstar = torch.from_numpy(gen.normal(31, M, (M, N))).cuda()
        Cbig = torch.zeros((M, ldc), dtype=td, device="cuda")
        Cbig[:, :N] = (Cstar + 1e-2 * torch.from_numpy(gen.normal(32, N, (M, N))).cuda()).to(td)
        d = lib.GemmDesc.make(M, 16, N, "bf16", "bf16", O, ldc=ldc)
        want = _reference(lib, d, Cbig, Cstar)
        got = torch.full((2,), -1.0, dtype=torch.float64, device="cuda")
        lib.error_frobenius_noalloc(d, Cbig, Cstar, got)
        e, nrm = got.cpu().tolist()
        assert math.isclose(e, want[0], rel_tol=1e-10) and math.isclose(nrm, want[1], rel_tol=1e-10)
    # sizes beyond the fixed array are refused, not truncated
    limit = lib.error_frobenius_noalloc_max_elements()
    too_big = lib.GemmDesc.make(limit // 1024 + 1, 16, 1024, "bf16", "bf16", "f32")
    with pytest.raises(lib.FmmError) as err:
        lib.error_frobenius_noalloc(too_big, Cbig, Cstar, got)
    assert err.value.code == 9
    # also when M * N does not fit 64 bits
    huge = lib.GemmDesc.make(2 ** 40, 16, 2 ** 40, "bf16", "bf16", "f32")
    with pytest.raises(lib.FmmError) as err:
        lib.error_frobenius_noalloc(huge, Cbig, Cstar, got)
    assert err.value.code == 9
