"""GPU parity of the convolution front end: the Hessian of a convolutional layer accumulated straight from the layer's
input (ptq_hessian_accumulate_conv, Sec. 3) against the CPU oracle, which writes the patch matrix out by definition,
and the whole path on convolutions shaped like those of the paper's networks."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_05576_b200 import ptq
from paper_2509_05576_b200 import workloads as wl
from parity import assert_layer_parity, oracle_layer

pytestmark = pytest.mark.gpu

H_RTOL = 2e-12          # same bound as for the matrix entry point: the products are exact, one rounding per chunk


def _gpu_conv_hessian(act_batches, spec):
    H = torch.zeros((spec.cols, spec.cols), dtype=torch.float64, device="cuda")
    st = ptq.new_status()
    ws = ptq.Workspace()
    for a in act_batches:
        ptq.hessian_accumulate_conv(H, torch.from_numpy(a).cuda(), spec.kh, spec.kw, spec.stride, spec.pad, ws, st)
    torch.cuda.synchronize()
    ptq.check_status(st, "hessian_accumulate_conv")
    return H


@pytest.mark.parametrize("spec", wl.conv_cases(), ids=lambda s: s.name)
def test_conv_hessian_matches_oracle(spec):
    _, act = wl.make_conv_layer(spec)
    Ho = oracle.hessian_accumulate_conv(act, spec.kh, spec.kw, spec.stride, spec.pad)
    Hg = _gpu_conv_hessian([act], spec).cpu().numpy()
    assert np.array_equal(Hg, Hg.T)
    assert np.max(np.abs(Hg - Ho)) <= H_RTOL * np.max(np.abs(Ho))
    # the matrix entry point on the written-out patches slices the very same numbers: bit-identical
    X = torch.from_numpy(oracle.unfold(act, spec.kh, spec.kw, spec.stride, spec.pad)).cuda()
    Hm = torch.zeros_like(torch.from_numpy(Hg)).cuda()
    st = ptq.new_status()
    ptq.hessian_accumulate(Hm, X, ptq.Workspace(), st)
    torch.cuda.synchronize()
    ptq.check_status(st, "hessian_accumulate")
    assert np.array_equal(Hm.cpu().numpy(), Hg)


def test_conv_hessian_accumulates_over_batches_and_chunks():
    """Three calibration batches, the first with more than 16384 output positions (several launches per call)."""
    spec = wl.ConvSpec("conv.big", 32, 16, 3, 3, 1, 1, 48, 48, 8, 4, "halfnormal", 7100)      # n = 18432, cols 144
    assert spec.n > 16384
    _, act = wl.make_conv_layer(spec)
    rng = np.random.Generator(np.random.PCG64(7101))
    more = [np.abs(rng.standard_normal((2, 16, 48, 48), dtype=np.float32)),
            np.abs(rng.standard_normal((1, 16, 17, 23), dtype=np.float32))]                  # another image size
    Ho = oracle.hessian_accumulate_conv(act, 3, 3, 1, 1)
    for a in more:
        oracle.hessian_accumulate_conv(a, 3, 3, 1, 1, H=Ho)
    Hg = _gpu_conv_hessian([act] + more, spec).cpu().numpy()
    assert np.max(np.abs(Hg - Ho)) <= H_RTOL * np.max(np.abs(Ho))


def test_conv_nonfinite_input_is_reported():
    spec = wl.conv_cases()[1]
    _, act = wl.make_conv_layer(spec)
    act[3, 5, 2, 7] = np.inf
    H = torch.zeros((spec.cols, spec.cols), dtype=torch.float64, device="cuda")
    st = ptq.new_status()
    ptq.hessian_accumulate_conv(H, torch.from_numpy(act).cuda(), 3, 3, 1, 1, ptq.Workspace(), st)
    torch.cuda.synchronize()
    code, index, _, _ = st.cpu().tolist()
    assert code == ptq.ERR_NONFINITE
    assert index // 9 == 5                      # a row of channel 5


def test_conv_bad_arguments_are_rejected_on_the_host():
    L = ptq.lib()
    import ctypes
    fake = ctypes.c_void_p(4096)
    args = dict(batch=1, channels=3, height=8, width=8, kh=3, kw=3, stride=1, pad=1)

    def call(**kw):
        a = dict(args, **kw)
        return L.ptq_hessian_accumulate_conv(fake, fake, a["batch"], a["channels"], a["height"], a["width"], a["kh"],
                                             a["kw"], a["stride"], a["pad"], fake, 1 << 30, fake, None)
    assert call(stride=0) == ptq.ERR_INVALID_ARG
    assert call(kh=12, pad=1) == ptq.ERR_INVALID_ARG          # kernel larger than the padded image
    assert call(pad=-1) == ptq.ERR_INVALID_ARG
    assert L.ptq_hessian_accumulate_conv(fake, fake, 1, 3, 8, 8, 3, 3, 1, 1, fake, 16, fake, None) == ptq.ERR_WORKSPACE


@pytest.mark.parametrize("spec", wl.conv_cases()[:6], ids=lambda s: s.name)
def test_conv_layer_whole_path_matches_oracle(spec):
    """Hessian from the activations in place, then inverse, order, sweep: codes equal to the oracle's on the patches."""
    W, act = wl.make_conv_layer(spec)
    X = oracle.unfold(act, spec.kh, spec.kw, spec.stride, spec.pad)
    ref = oracle_layer(W, X, spec.bits, spec.damp)
    half = spec.batch // 2
    batches = [torch.from_numpy(act[:half]).cuda(), torch.from_numpy(act[half:]).cuda()]    # two calibration batches
    bufs = ptq.quantize_layer_full(torch.from_numpy(W).cuda(), batches, spec.bits, spec.damp,
                                   conv=(spec.kh, spec.kw, spec.stride, spec.pad))
    torch.cuda.synchronize()
    ptq.check_status(bufs.status, "conv layer")
    g = {k: getattr(bufs, k).cpu().numpy() for k in ("perm", "scale", "zero", "codes", "What", "loss")}
    assert assert_layer_parity(g, ref) == 0
