"""Helpers shared by the GPU parity tests: run the CUDA path through the C-ABI binding, run the oracle on
the same seeded inputs, compare under the stated tolerances."""
import numpy as np
import torch

import oracle
from paper_2509_05576_b200 import ptq

# Tolerances: column order and integer codes bit-exact, except that codes whose
# pre-rounding value lies within 1e-4 (in units of the row's scale) of a rounding boundary may differ by one level on
# at most 0.1 % of the weights; dequantized weights within 1e-4 relative; reconstruction loss within 1e-3 relative.
BOUNDARY_TOL = 1e-4
MAX_MISMATCH_FRACTION = 1e-3
WHAT_RTOL = 1e-4
LOSS_RTOL = 1e-3


def gpu_layer(W, X, bits, damp=0.01, damp_mode=ptq.DAMP_REL_MEAN_DIAG, score_mode=ptq.SCORE_QERR, gram_f64=False):
    Wd = torch.from_numpy(W).cuda()
    Xd = torch.from_numpy(X).cuda()
    bufs = ptq.quantize_layer_full(Wd, Xd, bits, damp, damp_mode, score_mode, gram_f64=gram_f64)
    torch.cuda.synchronize()
    ptq.check_status(bufs.status, "quantize_layer_full")
    return {k: getattr(bufs, k).cpu().numpy() for k in
            ("H", "Hinv", "Hinv_diag", "lam", "scale", "zero", "S", "perm", "codes", "What", "loss")}


def compare_codes(codes_gpu, ref):
    """ref: oracle output dict with 'codes', 'prer', 'perm'.  Returns the number of mismatching codes."""
    mism = codes_gpu != ref["codes"]
    nm = int(mism.sum())
    if nm == 0:
        return 0
    assert nm <= MAX_MISMATCH_FRACTION * mism.size, f"{nm} of {mism.size} codes differ"
    diff = np.abs(codes_gpu.astype(np.int32) - ref["codes"].astype(np.int32))
    assert diff.max() <= 1, "codes differ by more than one level"
    # every mismatch must sit within BOUNDARY_TOL of a rounding boundary of the oracle's pre-rounding value
    v = ref["prer"][mism]
    dist = np.abs(np.abs(v - np.floor(v)) - 0.5)
    assert np.all(dist <= BOUNDARY_TOL), f"mismatch away from a boundary: max distance {dist.max()}"
    return nm


def assert_layer_parity(g, ref):
    assert np.array_equal(g["perm"], ref["perm"]), "column order differs"
    assert np.array_equal(g["scale"], ref["scale"]) and np.array_equal(g["zero"], ref["zero"])
    nm = compare_codes(g["codes"], ref)
    num = np.linalg.norm(g["What"].astype(np.float64) - ref["What"].astype(np.float64))
    den = np.linalg.norm(ref["What"].astype(np.float64))
    assert num <= WHAT_RTOL * den
    if nm == 0:
        assert np.array_equal(g["What"], ref["What"])
    assert abs(float(g["loss"][0]) - ref["loss"]) <= LOSS_RTOL * ref["loss"]
    return nm


def oracle_layer(W, X, bits, damp=0.01, damp_mode=oracle.DAMP_REL_MEAN_DIAG, score_mode=oracle.SCORE_QERR):
    return oracle.run_layer(W, X, bits, damp, damp_mode, score_mode, want_prer=True)
