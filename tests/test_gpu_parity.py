"""GPU parity tests: every stage and the whole path, through the C-ABI library, against the CPU oracle on the
same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_05576_b200 import ptq
from paper_2509_05576_b200 import workloads as wl
from parity import (assert_layer_parity, compare_codes, gpu_layer, oracle_layer, LOSS_RTOL, WHAT_RTOL)

pytestmark = pytest.mark.gpu


def _layer(rows, cols, n, seed, bits=4, xdist="halfnormal", wdist="kaiming"):
    return wl.make_layer(wl.LayerSpec("t", rows, cols, n, bits, wdist, xdist, seed))


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


# ------------------------------------------------------------------------------------------ Hessian
@pytest.mark.parametrize("cols,n", [(128, 1024), (147, 200), (64, 64), (200, 520), (333, 4096), (32, 36)])
@pytest.mark.parametrize("f64", [False, True])
def test_hessian_matches_oracle(cols, n, f64):
    _, X = _layer(4, cols, n, 100 + cols)
    ref = oracle.hessian_accumulate(X)
    H = torch.zeros((cols, cols), dtype=torch.float64, device="cuda")
    st, ws = ptq.new_status(), ptq.Workspace()
    ptq.hessian_accumulate(H, _cuda(X), ws, st, f64=f64)
    torch.cuda.synchronize()
    ptq.check_status(st)
    Hn = H.cpu().numpy()
    assert np.array_equal(Hn, Hn.T)
    assert np.max(np.abs(Hn - ref)) <= 2e-12 * np.max(np.abs(ref))


def test_hessian_sliced_last_wave_and_two_launches_per_call():
    """1600 columns are 169 output tiles: one full wave of the persistent grid and a last wave whose tiles are cut
    along the calibration length; 17000 calibration columns make the call two launches (16384 + 616).  The sliced
    tiles must come out exactly as whole ones would: compared with the oracle and, bit for bit, with the same call on
    a matrix whose tile count leaves no partial wave to slice (the first 1280 columns: 110 tiles, more than half a wave)."""
    cols, n = 1600, 17000
    _, X = _layer(4, cols, n, 4242)
    ref = oracle.hessian_accumulate(X)
    st, ws = ptq.new_status(), ptq.Workspace()
    H = torch.zeros((cols, cols), dtype=torch.float64, device="cuda")
    ptq.hessian_accumulate(H, _cuda(X), ws, st)
    sub = 1280
    Hs = torch.zeros((sub, sub), dtype=torch.float64, device="cuda")
    ptq.hessian_accumulate(Hs, _cuda(X[:sub]), ws, st)
    torch.cuda.synchronize()
    ptq.check_status(st)
    Hn = H.cpu().numpy()
    assert np.array_equal(Hn, Hn.T)
    assert np.max(np.abs(Hn - ref)) <= 2e-12 * np.max(np.abs(ref))
    assert np.array_equal(Hs.cpu().numpy(), Hn[:sub, :sub])


@pytest.mark.parametrize("xdist", ["normal", "silu", "halfnormal_sparse30"])
def test_hessian_signed_and_sparse_inputs_accumulate_in_chunks(xdist):
    cols, n = 190, 768
    _, X = _layer(4, cols, n, 7, xdist=xdist)
    X[5] = 0.0                      # a dead input channel
    X[9] *= 1e-6                    # rows of very different magnitude
    X[11] *= 3e4
    ref = oracle.hessian_accumulate(X)
    H = torch.zeros((cols, cols), dtype=torch.float64, device="cuda")
    st, ws = ptq.new_status(), ptq.Workspace()
    Xd = _cuda(X)
    ptq.hessian_accumulate(H, Xd[:, :256], ws, st)       # strided views: ldx = 768
    ptq.hessian_accumulate(H, Xd[:, 256:], ws, st)
    torch.cuda.synchronize()
    ptq.check_status(st)
    Hn = H.cpu().numpy()
    scale = np.sqrt(np.outer(np.diag(ref), np.diag(ref))) + 1e-300
    assert np.max(np.abs(Hn - ref) / scale) <= 1e-11
    assert np.all(Hn[5] == 0) and np.all(Hn[:, 5] == 0)


def test_hessian_reports_nonfinite_input():
    _, X = _layer(4, 64, 128, 8)
    X[3, 17] = np.inf
    H = torch.zeros((64, 64), dtype=torch.float64, device="cuda")
    st, ws = ptq.new_status(), ptq.Workspace()
    ptq.hessian_accumulate(H, _cuda(X), ws, st)
    torch.cuda.synchronize()
    with pytest.raises(ptq.PtqError) as ei:
        ptq.check_status(st)
    assert ei.value.code == ptq.ERR_NONFINITE and ei.value.index == 3


# ------------------------------------------------------------------------------------------ damped inverse
@pytest.mark.parametrize("cols,n", [(64, 256), (100, 300), (128, 1024), (257, 200), (600, 700)])
def test_inverse_matches_oracle(cols, n):
    _, X = _layer(4, cols, n, 200 + cols)
    H = oracle.hessian_accumulate(X)
    ref, ref_diag, ref_lam = oracle.prepare_hinv(H, 0.01, oracle.DAMP_REL_MEAN_DIAG)
    Hd = _cuda(H)
    Hinv = torch.empty_like(Hd)
    diag = torch.empty(cols, dtype=torch.float64, device="cuda")
    lam = torch.empty(1, dtype=torch.float64, device="cuda")
    st, ws = ptq.new_status(), ptq.Workspace()
    ptq.prepare_hinv(Hd, 0.01, ptq.DAMP_REL_MEAN_DIAG, Hinv, diag, lam, ws, st)
    torch.cuda.synchronize()
    ptq.check_status(st)
    G = Hinv.cpu().numpy()
    assert abs(lam.item() - ref_lam) <= 1e-14 * ref_lam
    cond = np.linalg.cond(H + ref_lam * np.eye(cols))
    assert np.max(np.abs(G - ref)) <= 1e-15 * cond * np.max(np.abs(ref)) * 20
    assert np.array_equal(G, G.T)
    assert np.array_equal(diag.cpu().numpy(), np.diag(G))
    assert np.max(np.abs(np.diag(G) - ref_diag) / ref_diag) <= 1e-15 * cond * 20
    assert torch.equal(Hd, _cuda(H)), "input H must not be modified"


def test_inverse_absolute_damping_and_not_spd_status():
    _, X = _layer(4, 70, 30, 9)       # rank 30 < 70
    H = oracle.hessian_accumulate(X)
    ref, _, _ = oracle.prepare_hinv(H, 0.1, oracle.DAMP_ABS)
    Hd = _cuda(H)
    Hinv = torch.empty_like(Hd)
    diag = torch.empty(70, dtype=torch.float64, device="cuda")
    lam = torch.empty(1, dtype=torch.float64, device="cuda")
    st, ws = ptq.new_status(), ptq.Workspace()
    ptq.prepare_hinv(Hd, 0.1, ptq.DAMP_ABS, Hinv, diag, lam, ws, st)
    torch.cuda.synchronize()
    ptq.check_status(st)
    assert lam.item() == 0.1
    assert np.max(np.abs(Hinv.cpu().numpy() - ref)) <= 1e-9 * np.max(np.abs(ref))
    # not positive definite: reported through the status word, nothing traps
    bad = _cuda(-np.eye(70))
    st2 = ptq.new_status()
    ptq.prepare_hinv(bad, 0.0, ptq.DAMP_ABS, Hinv, diag, lam, ws, st2)
    torch.cuda.synchronize()
    with pytest.raises(ptq.PtqError) as ei:
        ptq.check_status(st2)
    assert ei.value.code == ptq.ERR_NOT_SPD and ei.value.index == 0


# ------------------------------------------------------------------------------------------ grid, scores, order
@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_grid_is_bit_exact(bits):
    W, _ = _layer(70, 333, 8, 300 + bits)
    W[5] = np.abs(W[5]); W[6] = 0.0; W[7] = -np.abs(W[7])
    ref_s, ref_z = oracle.minmax_grid(W, bits)
    scale = torch.empty(70, dtype=torch.float32, device="cuda")
    zero = torch.empty(70, dtype=torch.float32, device="cuda")
    st = ptq.new_status()
    ptq.minmax_grid(_cuda(W), bits, scale, zero, st)
    torch.cuda.synchronize()
    ptq.check_status(st)
    assert np.array_equal(scale.cpu().numpy(), ref_s) and np.array_equal(zero.cpu().numpy(), ref_z)


@pytest.mark.parametrize("mode", [ptq.SCORE_QERR, ptq.SCORE_PRUNE, ptq.SCORE_ERR, ptq.SCORE_W, ptq.SCORE_NONE])
@pytest.mark.parametrize("rows,cols", [(70, 333), (200, 64), (1, 5)])
def test_scores_and_order_match_oracle(mode, rows, cols):
    W, X = _layer(rows, cols, 400, 400 + rows)
    if cols > 20:
        W[:, 17] = W[:, 3]              # exact ties must keep the lower index first
    _, diag, _ = oracle.prepare_hinv(oracle.hessian_accumulate(X))
    if cols > 20:
        diag[17] = diag[3]
    sc, zp = oracle.minmax_grid(W, 4)
    ref_S, ref_perm = oracle.sensitivity_order(W, diag, sc, zp, 4, mode)
    S = torch.empty(cols, dtype=torch.float64, device="cuda")
    perm = torch.empty(cols, dtype=torch.int32, device="cuda")
    st, ws = ptq.new_status(), ptq.Workspace()
    ptq.sensitivity_order(_cuda(W), _cuda(diag), _cuda(sc), _cuda(zp), 4, mode, S, perm, ws, st)
    torch.cuda.synchronize()
    ptq.check_status(st)
    assert np.allclose(S.cpu().numpy(), ref_S, rtol=1e-13, atol=0)
    assert np.array_equal(perm.cpu().numpy(), ref_perm)


@pytest.mark.parametrize("mode", [ptq.SCORE_QERR, ptq.SCORE_PRUNE, ptq.SCORE_ERR, ptq.SCORE_W])
def test_ascending_order_matches_oracle_and_whole_path(mode):
    """The "asc" keys of Sec. 4.1: same scores, ascending stable order; then the whole path in that order."""
    W, X = _layer(70, 333, 400, 471)
    W[:, 17] = W[:, 3]
    H = oracle.hessian_accumulate(X)
    Hinv, diag, _ = oracle.prepare_hinv(H)
    diag[17] = diag[3]
    sc, zp = oracle.minmax_grid(W, 4)
    ref_S, ref_perm = oracle.sensitivity_order(W, diag, sc, zp, 4, mode | oracle.SCORE_ASCENDING)
    S = torch.empty(333, dtype=torch.float64, device="cuda")
    perm = torch.empty(333, dtype=torch.int32, device="cuda")
    st, ws = ptq.new_status(), ptq.Workspace()
    ptq.sensitivity_order(_cuda(W), _cuda(diag), _cuda(sc), _cuda(zp), 4, mode | ptq.SCORE_ASCENDING, S, perm, ws, st)
    # the sort alone, from scores the caller already has
    perm2 = torch.empty(333, dtype=torch.int32, device="cuda")
    ptq.sort_scores(S, perm2, ascending=True)
    perm3 = torch.empty(333, dtype=torch.int32, device="cuda")
    ptq.sort_scores(S, perm3, ascending=False)
    torch.cuda.synchronize()
    ptq.check_status(st)
    assert np.allclose(S.cpu().numpy(), ref_S, rtol=1e-13, atol=0)
    assert np.array_equal(perm.cpu().numpy(), ref_perm)
    assert np.array_equal(perm2.cpu().numpy(), ref_perm)
    _, ref_desc = oracle.sensitivity_order(W, diag, sc, zp, 4, mode)
    assert np.array_equal(perm3.cpu().numpy(), ref_desc)
    ref = oracle_layer(W, X, 4, score_mode=mode | oracle.SCORE_ASCENDING)
    g = gpu_layer(W, X, 4, score_mode=mode | ptq.SCORE_ASCENDING)
    assert assert_layer_parity(g, ref) == 0


# ------------------------------------------------------------------------------------------ bounded waits
@pytest.mark.parametrize("which", [0, 1])
def test_bounded_wait_runs_out_and_the_context_stays_usable(which):
    """The factorisation's grid barrier (0) and the sweep's counter wait (1) are asked, with a limit of a few thousand
    cycles, for something that never comes: the kernel must return with PTQ_ERR_TIMEOUT in the status word, and an
    ordinary call made afterwards on the same stream must give exactly what it gave before."""
    W, X = _layer(48, 200, 300, 480)
    before = gpu_layer(W, X, 4)
    st, ws = ptq.new_status(), ptq.Workspace()
    ptq.selftest_wait_timeout(which, 5000, ws, st)
    torch.cuda.synchronize()
    with pytest.raises(ptq.PtqError) as ei:
        ptq.check_status(st)
    assert ei.value.code == ptq.ERR_TIMEOUT
    assert int(st.cpu()[2]) == 1 + which
    after = gpu_layer(W, X, 4)
    for k in ("H", "Hinv", "S", "perm", "codes", "What", "loss"):
        assert np.array_equal(before[k], after[k]), k


# ------------------------------------------------------------------------------------------ column sweep
def _sweep(W, Hinv, perm, sc, zp, bits, H=None):
    rows, cols = W.shape
    codes = torch.empty((rows, cols), dtype=torch.uint8, device="cuda")
    What = torch.empty((rows, cols), dtype=torch.float32, device="cuda")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    st, ws = ptq.new_status(), ptq.Workspace()
    ptq.quantize_layer(_cuda(W), _cuda(Hinv), _cuda(perm), _cuda(sc), _cuda(zp), bits, codes, What,
                       None if H is None else _cuda(H), None if H is None else loss, ws, st)
    torch.cuda.synchronize()
    ptq.check_status(st)
    return codes.cpu().numpy(), What.cpu().numpy(), loss.item()


@pytest.mark.parametrize("rows,cols,n,bits", [(64, 128, 1024, 4), (37, 147, 300, 4), (70, 200, 150, 3),
                                              (33, 64, 100, 8), (5, 9, 30, 2), (130, 321, 512, 4)])
def test_sweep_matches_oracle_on_identical_inputs(rows, cols, n, bits):
    W, X = _layer(rows, cols, n, 500 + cols)
    H = oracle.hessian_accumulate(X)
    Hinv, diag, _ = oracle.prepare_hinv(H)
    sc, zp = oracle.minmax_grid(W, bits)
    _, perm = oracle.sensitivity_order(W, diag, sc, zp, bits)
    ref = oracle.quantize_layer(W, Hinv, perm, sc, zp, bits, H_undamped=H, want_prer=True)
    codes, What, loss = _sweep(W, Hinv, perm, sc, zp, bits, H)
    nm = compare_codes(codes, ref)
    assert nm == 0
    assert np.array_equal(What, ref["What"])
    assert abs(loss - ref["loss"]) <= 1e-9 * ref["loss"]


def test_identity_inverse_hessian_gives_round_to_nearest():
    W, _ = _layer(40, 130, 8, 600)
    W[0, :8] = 0.0
    for bits in (2, 4, 8):
        sc, zp = oracle.minmax_grid(W, bits)
        perm = np.random.Generator(np.random.PCG64(1)).permutation(130).astype(np.int32)
        codes, What, _ = _sweep(W, np.eye(130), perm, sc, zp, bits)
        v = np.clip(np.rint(W.astype(np.float64) / sc[:, None].astype(np.float64)) + zp[:, None], 0, 2 ** bits - 1)
        assert np.array_equal(codes, v.astype(np.uint8))
        assert np.array_equal(What, (sc[:, None].astype(np.float64) * (v - zp[:, None])).astype(np.float32))


def test_invalid_permutation_is_reported_not_followed():
    W, X = _layer(8, 64, 100, 601)
    Hinv, diag, _ = oracle.prepare_hinv(oracle.hessian_accumulate(X))
    sc, zp = oracle.minmax_grid(W, 4)
    perm = np.arange(64, dtype=np.int32)
    perm[10] = 3                     # repeated entry
    perm[20] = 9999                  # out of range
    codes = torch.empty((8, 64), dtype=torch.uint8, device="cuda")
    st, ws = ptq.new_status(), ptq.Workspace()
    ptq.quantize_layer(_cuda(W), _cuda(Hinv), _cuda(perm), _cuda(sc), _cuda(zp), 4, codes, None, None, None, ws, st)
    torch.cuda.synchronize()
    with pytest.raises(ptq.PtqError) as ei:
        ptq.check_status(st)
    assert ei.value.code == ptq.ERR_INVALID_ARG


# ------------------------------------------------------------------------------------------ whole path
@pytest.mark.parametrize("rows,cols,n,bits,xdist", [
    (64, 128, 1024, 4, "halfnormal"),
    (37, 147, 260, 4, "halfnormal"),          # ragged: 7x7 stem width, n not a multiple of the K block
    (255, 128, 512, 8, "silu"),               # YOLO head: 255 rows
    (32, 108, 256, 4, "silu"),                # 6x6 stem
    (100, 300, 200, 3, "normal"),             # cols > n: rank-deficient before damping
    (1, 1, 4, 4, "normal"),                   # degenerate 1x1 layer
    (3, 2, 1, 2, "halfnormal"),
])
def test_whole_path_matches_oracle(rows, cols, n, bits, xdist):
    W, X = _layer(rows, cols, n, 700 + rows + cols, bits, xdist)
    ref = oracle_layer(W, X, bits)
    g = gpu_layer(W, X, bits)
    assert np.max(np.abs(g["H"] - ref["H"])) <= 2e-12 * np.max(np.abs(ref["H"]))
    assert assert_layer_parity(g, ref) == 0


def test_config1_bit_exact_and_deterministic():
    spec = wl.config1()[0]
    W, X = wl.make_layer(spec)
    ref = oracle_layer(W, X, spec.bits, spec.damp)
    runs = [gpu_layer(W, X, spec.bits, spec.damp) for _ in range(3)]
    assert assert_layer_parity(runs[0], ref) == 0
    for r in runs[1:]:
        for k in ("H", "Hinv", "S", "perm", "codes", "What", "loss"):
            assert np.array_equal(r[k], runs[0][k]), f"{k} is not bit-identical across runs"


@pytest.mark.parametrize("mode", [ptq.SCORE_PRUNE, ptq.SCORE_ERR, ptq.SCORE_W, ptq.SCORE_NONE])
def test_ordering_modes_whole_path(mode):
    W, X = _layer(48, 160, 400, 800 + mode)
    ref = oracle_layer(W, X, 4, score_mode=mode)
    g = gpu_layer(W, X, 4, score_mode=mode)
    assert assert_layer_parity(g, ref) == 0


def test_absolute_damping_whole_path():
    W, X = _layer(24, 96, 300, 810)
    ref = oracle_layer(W, X, 4, damp=0.1, damp_mode=oracle.DAMP_ABS)
    g = gpu_layer(W, X, 4, damp=0.1, damp_mode=ptq.DAMP_ABS)
    assert assert_layer_parity(g, ref) == 0


def test_config2_full_size():
    """The bench workload (256 x 2304, N = 4096, 30 % zeros) at full size, in the bench's launch configuration."""
    spec = wl.config2()[0]
    W, X = wl.make_layer(spec)
    ref = oracle_layer(W, X, spec.bits, spec.damp)
    g = gpu_layer(W, X, spec.bits, spec.damp)
    assert np.max(np.abs(g["H"] - ref["H"])) <= 2e-12 * np.max(np.abs(ref["H"]))
    assert np.max(np.abs(g["Hinv"] - ref["Hinv"])) <= 1e-10 * np.max(np.abs(ref["Hinv"]))
    assert_layer_parity(g, ref)
    assert abs(float(g["loss"][0]) - oracle.loss_direct(W, g["What"], X)) <= 1e-9 * ref["loss"]


def test_sharded_entry_on_one_rank_equals_the_single_gpu_path():
    """The multi-GPU entry (all-reduce of H over the calibration split, of the scores over the row split) on a group
    of one NCCL rank: the collectives are no-ops, so the result must be that of the ordinary path, bit for bit, and
    match the oracle.  (More ranks need more GPUs; the sharding logic itself runs as gloo ranks in the CPU suite.)"""
    import os
    import socket
    import torch.distributed as dist
    from paper_2509_05576_b200 import sharded
    W, X = _layer(70, 200, 300, 990)
    ref = oracle_layer(W, X, 4)
    g = gpu_layer(W, X, 4)
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        ops = sharded.GpuOps()
        res = sharded.quantize_layer_sharded(_cuda(W), _cuda(X), 200, 4, ops=ops)
        torch.cuda.synchronize()
        ops.check()
    finally:
        dist.destroy_process_group()
    for k in ("H", "Hinv", "S", "perm", "codes", "What"):
        assert np.array_equal(res[k].cpu().numpy(), g[k]), k
    assert float(res["loss"].item()) == float(g["loss"][0])
    out = {k: res[k].cpu().numpy() for k in ("perm", "scale", "zero", "codes", "What", "loss")}
    assert assert_layer_parity(out, ref) == 0


def test_layer_path_replayed_as_a_cuda_graph_matches_the_eager_path():
    """The whole path of a layer captured once and replayed: same bits as the call-by-call path, and new inputs written
    into the captured tensors give the new layer's result (checked against the oracle)."""
    W, X = _layer(96, 200, 512, 1500)
    g = gpu_layer(W, X, 4)
    Wd, Xd = _cuda(W), _cuda(X)
    lg = ptq.LayerGraph(Wd, Xd, 4)
    bufs = lg.replay()
    torch.cuda.synchronize()
    ptq.check_status(bufs.status, "graph replay")
    for k in ("H", "Hinv", "S", "perm", "codes", "What", "loss"):
        assert np.array_equal(getattr(bufs, k).cpu().numpy(), g[k]), k
    W2, X2 = _layer(96, 200, 512, 1501)
    Wd.copy_(_cuda(W2)); Xd.copy_(_cuda(X2))
    bufs = lg.replay()
    torch.cuda.synchronize()
    ptq.check_status(bufs.status, "graph replay 2")
    ref = oracle_layer(W2, X2, 4)
    out = {k: getattr(bufs, k).cpu().numpy() for k in ("perm", "scale", "zero", "codes", "What", "loss")}
    assert assert_layer_parity(out, ref) == 0


@pytest.mark.gpu
@pytest.mark.parametrize("rows,cols,limit", [(96, 700, 5), (300, 200, 3), (2500, 130, 20)])
def test_cta_limit_changes_the_grids_not_the_results(rows, cols, limit):
    """ptq_set_cta_limit holds the persistent cooperative kernels (factorisation, sweep) to a few CTAs; every array of the
    layer's result is the same, bit for bit, as with one CTA per SM.  The shapes give fewer CTAs than block rows of the
    factorisation, than row groups of the sweep, and fewer than either."""
    W, X = _layer(rows, cols, 384, 4242)
    g = gpu_layer(W, X, 4)
    ptq.set_cta_limit(limit)
    try:
        h = gpu_layer(W, X, 4)
    finally:
        ptq.set_cta_limit(0)
    for k in ("H", "Hinv", "S", "perm", "codes", "What", "loss"):
        assert np.array_equal(h[k], g[k]), k
    with pytest.raises(ptq.PtqError):
        ptq.set_cta_limit(-1)


@pytest.mark.gpu
def test_layer_set_on_several_streams_equals_the_layers_one_by_one():
    """ptq.LayerSet: independent layers side by side on three streams with limited cooperative grids; every layer's
    arrays are the same, bit for bit, as from its own call, whatever stream it landed on, and a second run of the same
    set object gives them again."""
    shapes = [(40, 300, 256, 4), (130, 64, 200, 3), (64, 520, 600, 8), (33, 147, 147, 4), (256, 128, 512, 4)]
    data = [_layer(r, c, n, 900 + i, bits=b) for i, (r, c, n, b) in enumerate(shapes)]
    single = [gpu_layer(W, X, b) for (W, X), (_, _, _, b) in zip(data, shapes)]
    ls = ptq.LayerSet([(_cuda(W), _cuda(X), b) for (W, X), (_, _, _, b) in zip(data, shapes)], n_streams=3, cta_limit=7)
    assert sorted(i for i, _ in ls.plan) == list(range(len(shapes)))
    for _ in range(2):
        outs = ls.run()
        torch.cuda.synchronize()
        for o, g in zip(outs, single):
            ptq.check_status(o.status, "layer set")
            for k in ("H", "Hinv", "S", "perm", "codes", "What", "loss"):
                assert np.array_equal(getattr(o, k).cpu().numpy(), g[k]), k
