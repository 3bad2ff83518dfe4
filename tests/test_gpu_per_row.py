"""The non-parallel arm of the paper's ablation (Sec. 4.2: every row in its own sensitivity order, against its own copy
of the inverse Hessian) through the C-ABI against the CPU oracle, on identical inputs; and its cost beside the
row-parallel method on the same layer."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_05576_b200 import ptq
from paper_2509_05576_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _run(W, H, Hinv, sc, zp, bits, mode):
    rows, cols = W.shape
    codes = torch.empty((rows, cols), dtype=torch.uint8, device="cuda")
    What = torch.empty((rows, cols), dtype=torch.float32, device="cuda")
    perm_rows = torch.full((rows, cols), -1, dtype=torch.int32, device="cuda")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    st, ws = ptq.new_status(), ptq.Workspace()
    ptq.quantize_layer_per_row(_cuda(W), _cuda(Hinv), _cuda(sc), _cuda(zp), bits, mode, codes, What, perm_rows, _cuda(H),
                               loss, ws, st)
    torch.cuda.synchronize()
    ptq.check_status(st, "quantize_layer_per_row")
    return codes.cpu().numpy(), What.cpu().numpy(), perm_rows.cpu().numpy(), float(loss.item())


@pytest.mark.parametrize("rows,cols,n,bits", [(40, 128, 256, 4), (64, 64, 200, 3), (7, 33, 64, 8), (255, 128, 300, 4),
                                              (3, 1, 8, 4), (16, 108, 150, 4)])
@pytest.mark.parametrize("mode", [ptq.SCORE_QERR, ptq.SCORE_W | ptq.SCORE_ASCENDING])
def test_per_row_arm_matches_oracle(rows, cols, n, bits, mode):
    W, X = wl.make_layer(wl.LayerSpec("pr", rows, cols, n, bits, "kaiming", "halfnormal", 1400 + rows + cols))
    H = oracle.hessian_accumulate(X)
    Hinv, diag, _ = oracle.prepare_hinv(H)
    sc, zp = oracle.minmax_grid(W, bits)
    ref = oracle.quantize_layer_per_row(W, Hinv, diag, sc, zp, bits, mode, H_undamped=H)
    codes, What, perm_rows, loss = _run(W, H, Hinv, sc, zp, bits, mode)
    assert np.array_equal(perm_rows, ref["perm_rows"]), "a row's order differs"
    assert np.array_equal(codes, ref["codes"])
    assert np.array_equal(What, ref["What"])
    assert abs(loss - ref["loss"]) <= 1e-9 * ref["loss"]
    if rows > 1 and cols > 8:
        assert any(not np.array_equal(perm_rows[r], perm_rows[0]) for r in range(1, rows))   # the rows do differ


def test_wider_layers_are_refused():
    fake = torch.zeros(16, dtype=torch.float32, device="cuda")
    st, ws = ptq.new_status(), ptq.Workspace()
    W = torch.zeros((4, 129), dtype=torch.float32, device="cuda")
    Hinv = torch.eye(129, dtype=torch.float64, device="cuda")
    codes = torch.empty((4, 129), dtype=torch.uint8, device="cuda")
    pr = torch.empty((4, 129), dtype=torch.int32, device="cuda")
    with pytest.raises(ptq.PtqError) as ei:
        ptq.quantize_layer_per_row(W, Hinv, fake, fake, 4, 0, codes, None, pr, None, None, ws, st)
    assert ei.value.code == ptq.ERR_UNSUPPORTED
