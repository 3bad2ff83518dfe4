"""The float64 product on the int8 tensor path (C += alpha A B^T from error-free slices; the product behind the deferred
part of Eq. 11) against a float64 library matmul, entry by entry, with the error bound of a float64 dot product."""
import numpy as np
import pytest
import torch

from paper_2509_05576_b200 import ptq

pytestmark = pytest.mark.gpu


def _run(m, n, k, b_is_kn, alpha, seed, scale_rows=False, ld_pad=0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    A = torch.randn((m, k + ld_pad), dtype=torch.float64, device="cuda", generator=g)[:, :k]
    Bs = (k, n + ld_pad) if b_is_kn else (n, k + ld_pad)
    Bf = torch.randn(Bs, dtype=torch.float64, device="cuda", generator=g)
    B = Bf[:, :n] if b_is_kn else Bf[:, :k]
    if scale_rows:
        A = A * torch.logspace(-6, 5, m, dtype=torch.float64, device="cuda")[:, None]
        A[min(3, m - 1)] = 0.0                                        # a dead row
        if not b_is_kn:
            B = B * torch.logspace(3, -4, n, dtype=torch.float64, device="cuda")[:, None]
        A = A.clone() if ld_pad == 0 else A
    C0 = torch.randn((m, n), dtype=torch.float64, device="cuda", generator=g)
    C = C0.clone()
    st, ws = ptq.new_status(), ptq.Workspace()
    ptq.gemm_nt_sliced(C, A, B, alpha, ws, st, b_is_kn=b_is_kn)
    torch.cuda.synchronize()
    ptq.check_status(st, "gemm_nt_sliced")
    Bt = B if b_is_kn else B.T
    ref = C0 + alpha * (A @ Bt)
    bound = 8e-16 * (A.abs() @ Bt.abs()) * abs(alpha) + 4e-16 * ref.abs() + 1e-300
    # entries far below a row's largest magnitude are rounded at 2^-55 of that magnitude: add that term
    bound = bound + abs(alpha) * k * 2.0 ** -54 * (A.abs().amax(dim=1)[:, None] * Bt.abs().amax(dim=0)[None, :])
    err = (C - ref).abs()
    assert bool((err <= bound).all()), float((err / bound).max())
    return float((err / (A.abs() @ Bt.abs() + 1e-300)).max())


@pytest.mark.parametrize("m,n,k", [(128, 64, 64), (300, 200, 500), (1, 1, 1), (257, 129, 1000), (70, 333, 96)])
@pytest.mark.parametrize("b_is_kn", [False, True])
def test_sliced_product_matches_float64_matmul(m, n, k, b_is_kn):
    rel = _run(m, n, k, b_is_kn, -1.0, 100 + m + n + k)
    assert rel < 1e-15          # relative to sum |a||b|: a float64 dot product's accuracy


def test_rows_of_very_different_magnitude_and_strided_operands():
    _run(200, 150, 320, False, 0.5, 7, scale_rows=True, ld_pad=8)
    _run(200, 150, 320, True, -2.0, 8, scale_rows=True, ld_pad=6)


def test_the_shape_of_a_deferred_update_of_a_tall_wide_layer():
    # rows x later-columns x super-block: several waves of tiles, many K blocks
    rel = _run(2048, 3000, 1024, True, -1.0, 9)
    assert rel < 1e-15
