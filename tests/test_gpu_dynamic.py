"""Dynamic re-ranking (Sec. 5: the sort inside the per-column loop) through the C-ABI against the CPU oracle's
literal statement of it, on identical inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_05576_b200 import ptq
from paper_2509_05576_b200 import workloads as wl
from parity import compare_codes, WHAT_RTOL, LOSS_RTOL

pytestmark = pytest.mark.gpu


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _inputs(rows, cols, n, bits, seed, xdist="halfnormal"):
    W, X = wl.make_layer(wl.LayerSpec("dyn", rows, cols, n, bits, "kaiming", xdist, seed))
    H = oracle.hessian_accumulate(X)
    Hinv, diag, _ = oracle.prepare_hinv(H)
    sc, zp = oracle.minmax_grid(W, bits)
    return W, H, Hinv, diag, sc, zp


def _gpu_dynamic(W, H, Hinv, sc, zp, bits, mode, block):
    rows, cols = W.shape
    codes = torch.empty((rows, cols), dtype=torch.uint8, device="cuda")
    What = torch.empty((rows, cols), dtype=torch.float32, device="cuda")
    order = torch.full((cols,), -1, dtype=torch.int32, device="cuda")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    st, ws = ptq.new_status(), ptq.Workspace()
    ptq.quantize_layer_dynamic(_cuda(W), _cuda(Hinv), _cuda(sc), _cuda(zp), bits, mode, block, codes, What, order,
                               _cuda(H), loss, ws, st)
    torch.cuda.synchronize()
    ptq.check_status(st, "quantize_layer_dynamic")
    return codes.cpu().numpy(), What.cpu().numpy(), order.cpu().numpy(), float(loss.item())


@pytest.mark.parametrize("rows,cols,n,bits,block", [(48, 200, 300, 4, 64), (130, 321, 512, 4, 128), (33, 256, 200, 3, 64),
                                                    (70, 640, 700, 4, 192), (300, 130, 256, 8, 64)])
@pytest.mark.parametrize("mode", [ptq.SCORE_QERR, ptq.SCORE_PRUNE | ptq.SCORE_ASCENDING])
def test_dynamic_reranking_matches_oracle(rows, cols, n, bits, block, mode):
    W, H, Hinv, diag, sc, zp = _inputs(rows, cols, n, bits, 1200 + cols)
    ref = oracle.quantize_layer_dynamic(W, Hinv, sc, zp, bits, block, mode, H_undamped=H, want_prer=True)
    codes, What, order, loss = _gpu_dynamic(W, H, Hinv, sc, zp, bits, mode, block)
    assert np.array_equal(order, ref["order"]), "column sequence differs"
    nm = compare_codes(codes, ref)
    assert nm == 0
    assert np.array_equal(What, ref["What"])
    assert abs(loss - ref["loss"]) <= 1e-9 * ref["loss"]
    # the re-ranking is not a no-op on these layers: the sequence differs from the static order
    _, perm_static = oracle.sensitivity_order(W, diag, sc, zp, bits, mode)
    assert not np.array_equal(order, perm_static)


def test_one_block_is_the_static_method():
    rows, cols, bits = 64, 200, 4
    W, H, Hinv, diag, sc, zp = _inputs(rows, cols, 300, bits, 1300)
    S, perm = oracle.sensitivity_order(W, diag, sc, zp, bits)
    ref = oracle.quantize_layer(W, Hinv, perm, sc, zp, bits, H_undamped=H, want_prer=True)
    for block in (cols, 100000):
        codes, What, order, loss = _gpu_dynamic(W, H, Hinv, sc, zp, bits, ptq.SCORE_QERR, block)
        assert np.array_equal(order, perm)
        assert compare_codes(codes, ref) == 0 and np.array_equal(What, ref["What"])
        assert abs(loss - ref["loss"]) <= 1e-9 * ref["loss"]
    # and the same bits as the ordinary two-call path on the GPU
    codes2 = torch.empty((rows, cols), dtype=torch.uint8, device="cuda")
    What2 = torch.empty((rows, cols), dtype=torch.float32, device="cuda")
    st, ws = ptq.new_status(), ptq.Workspace()
    ptq.quantize_layer(_cuda(W), _cuda(Hinv), _cuda(perm), _cuda(sc), _cuda(zp), bits, codes2, What2, None, None, ws, st)
    torch.cuda.synchronize()
    ptq.check_status(st)
    assert np.array_equal(codes2.cpu().numpy(), codes) and np.array_equal(What2.cpu().numpy(), What)


def test_no_sorting_mode_keeps_the_identity_sequence_whatever_the_block():
    W, H, Hinv, diag, sc, zp = _inputs(40, 192, 256, 4, 1301)
    ref = oracle.quantize_layer(W, Hinv, np.arange(192, dtype=np.int32), sc, zp, 4, H_undamped=H, want_prer=True)
    codes, What, order, loss = _gpu_dynamic(W, H, Hinv, sc, zp, 4, ptq.SCORE_NONE, 64)
    assert np.array_equal(order, np.arange(192))
    assert compare_codes(codes, ref) == 0 and np.array_equal(What, ref["What"])


def test_whole_path_with_dynamic_reranking_on_a_resnet_shaped_layer():
    """256 x 1152 (a layer2 3x3 convolution of the ResNet-50-shaped set), Hessian and inverse by the GPU path too."""
    spec = [s for s in wl.config3() if (s.rows, s.cols) == (128, 1152)][0]
    W, X = wl.make_layer(spec)
    Wd, Xd = _cuda(W), _cuda(X)
    bufs = ptq.quantize_layer_full(Wd, Xd, spec.bits, spec.damp)
    torch.cuda.synchronize()
    ptq.check_status(bufs.status)
    order = torch.empty(spec.cols, dtype=torch.int32, device="cuda")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    codes = torch.empty_like(bufs.codes)
    What = torch.empty_like(bufs.What)
    st, ws = ptq.new_status(), ptq.Workspace()
    ptq.quantize_layer_dynamic(Wd, bufs.Hinv, bufs.scale, bufs.zero, spec.bits, ptq.SCORE_QERR, 128, codes, What, order,
                               bufs.H, loss, ws, st)
    torch.cuda.synchronize()
    ptq.check_status(st)
    H = oracle.hessian_accumulate(X)
    Hinv, diag, _ = oracle.prepare_hinv(H, spec.damp)
    sc, zp = oracle.minmax_grid(W, spec.bits)
    ref = oracle.quantize_layer_dynamic(W, Hinv, sc, zp, spec.bits, 128, oracle.SCORE_QERR, H_undamped=H, want_prer=True)
    assert np.array_equal(order.cpu().numpy(), ref["order"])
    nm = compare_codes(codes.cpu().numpy(), ref)
    num = np.linalg.norm(What.cpu().numpy().astype(np.float64) - ref["What"].astype(np.float64))
    assert num <= WHAT_RTOL * np.linalg.norm(ref["What"].astype(np.float64))
    assert abs(float(loss.item()) - ref["loss"]) <= LOSS_RTOL * ref["loss"]
    assert nm == 0
