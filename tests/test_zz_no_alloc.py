"""ptq_sensitivity_order_static: the column-ordering call for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is not an option (a serving loop that must not allocate, a process
whose device memory is owned by another component's pool, a plug-in handed pointers but no allocator), so they
cannot provide the workspace that ptq_sensitivity_order needs.  The static variant keeps its scratch in an array
built into the library.  This test calls it through the C-ABI and checks it against the ordinary entry point:
same scores, same order, on two calls in a row (the second on a different shape, so anything the first call left
in the shared array would show), and checks that an oversized problem is refused on the host.

The file name keeps this module last in collection order, so that a run stopping at the first failure has already
run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2509_05576_b200 import ptq
from paper_2509_05576_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _inputs(rows, cols, seed, bits):
    W, _ = wl.make_layer(wl.LayerSpec("t", rows, cols, 8, bits, "kaiming", "halfnormal", seed))
    rng = np.random.Generator(np.random.PCG64(seed + 1))
    diag = rng.uniform(0.5, 2.0, cols)                     # stands in for diag(Hinv): any positive vector
    Wd = torch.from_numpy(W).cuda()
    scale = torch.empty(rows, dtype=torch.float32, device="cuda")
    zero = torch.empty(rows, dtype=torch.float32, device="cuda")
    st = ptq.new_status()
    ptq.minmax_grid(Wd, bits, scale, zero, st)
    return Wd, torch.from_numpy(diag).cuda(), scale, zero, st


def _both(rows, cols, seed, bits, mode):
    Wd, diag, scale, zero, st = _inputs(rows, cols, seed, bits)
    S_ref = torch.empty(cols, dtype=torch.float64, device="cuda")
    p_ref = torch.empty(cols, dtype=torch.int32, device="cuda")
    ptq.sensitivity_order(Wd, diag, scale, zero, bits, mode, S_ref, p_ref, ptq.Workspace(), st)
    S = torch.full((cols,), float("nan"), dtype=torch.float64, device="cuda")
    p = torch.full((cols,), -1, dtype=torch.int32, device="cuda")
    ptq.sensitivity_order_static(Wd, diag, scale, zero, bits, mode, S, p, st)
    torch.cuda.synchronize()
    ptq.check_status(st, "sensitivity_order_static")
    return S_ref.cpu().numpy(), p_ref.cpu().numpy(), S.cpu().numpy(), p.cpu().numpy()


def test_static_variant_matches_workspace_variant_on_two_calls_in_a_row():
    # first call: several row chunks and a ragged last one; second call: a smaller, differently shaped problem; then
    # the ascending order and the identity order (no sorting), which reads nothing from the array
    for rows, cols, seed, bits, mode in [(200, 333, 21, 4, ptq.SCORE_QERR), (70, 129, 22, 3, ptq.SCORE_PRUNE),
                                         (90, 77, 23, 4, ptq.SCORE_ERR | ptq.SCORE_ASCENDING),
                                         (33, 50, 24, 4, ptq.SCORE_NONE)]:
        S_ref, p_ref, S, p = _both(rows, cols, seed, bits, mode)
        # same kernels, same summation order: the scores agree to the tolerance of the score parity test (and in
        # fact bit for bit), the order exactly
        assert np.allclose(S, S_ref, rtol=1e-13, atol=0)
        assert np.array_equal(S, S_ref)
        assert np.array_equal(p, p_ref)
        assert sorted(p.tolist()) == list(range(cols))


def test_static_variant_allocates_nothing_and_takes_a_problem_exactly_at_the_limit():
    # 96 row chunks x 8192 columns x 8 bytes is exactly the size of the built-in array: accepted
    rows, cols, bits = 96 * 64, 8192, 4
    assert (rows // 64) * cols * 8 == ptq.STATIC_SCRATCH_BYTES
    Wd, diag, scale, zero, st = _inputs(rows, cols, 25, bits)
    S_ref = torch.empty(cols, dtype=torch.float64, device="cuda")
    p_ref = torch.empty(cols, dtype=torch.int32, device="cuda")
    ptq.sensitivity_order(Wd, diag, scale, zero, bits, ptq.SCORE_QERR, S_ref, p_ref, ptq.Workspace(), st)
    S = torch.empty(cols, dtype=torch.float64, device="cuda")
    p = torch.empty(cols, dtype=torch.int32, device="cuda")
    ptq.sensitivity_order_static(Wd, diag, scale, zero, bits, ptq.SCORE_QERR, S, p, st)     # first call: module set-up
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    ptq.sensitivity_order_static(Wd, diag, scale, zero, bits, ptq.SCORE_QERR, S, p, st)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before       # the device's free memory did not move
    ptq.check_status(st, "sensitivity_order_static")
    assert torch.equal(S, S_ref) and torch.equal(p, p_ref)


def test_static_variant_refuses_what_does_not_fit():
    L = ptq.lib()
    fake = ctypes.c_void_p(4096)            # never dereferenced: the size check comes before any launch
    rows, cols = 64 * 1024, 4096            # 1024 chunks x 4096 columns x 8 bytes = 32 MiB > the built-in array
    assert (rows // 64) * cols * 8 > ptq.STATIC_SCRATCH_BYTES
    rc = L.ptq_sensitivity_order_static(fake, rows, cols, cols, fake, fake, fake, 4, ptq.SCORE_QERR, fake, fake, fake,
                                        None)
    assert rc == ptq.ERR_STATIC_SCRATCH
    assert "built-in scratch" in ptq.status_string(rc)
    # the largest benchmark shape fits
    assert (4096 // 64) * 11008 * 8 <= ptq.STATIC_SCRATCH_BYTES
