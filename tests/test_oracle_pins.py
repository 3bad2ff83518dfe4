"""Pins for the float64 CPU oracle: it is checked against what the paper and the mathematics
fix (closed forms, invariants, library routines on special cases, brute force), never against
itself and never against the CUDA path."""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2509_05576_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def _small_layer(rows, cols, n, seed, xdist="halfnormal"):
    spec = wl.LayerSpec("t", rows, cols, n, 4, "kaiming", xdist, seed)
    return wl.make_layer(spec)


def _dequant(codes, scale, zero):
    return scale.astype(np.float64)[:, None] * (codes.astype(np.float64) - zero.astype(np.float64)[:, None])


def _rtn_codes(W, scale, zero, bits):
    v = W.astype(np.float64) / scale.astype(np.float64)[:, None]
    return np.clip(np.rint(v) + zero.astype(np.float64)[:, None], 0, 2 ** bits - 1).astype(np.uint8)


# ------------------------------------------------------------------ Hessian (Sec. 3, Eq. 2)
def test_hessian_matches_library_gram_and_trace():
    W, X = _small_layer(8, 37, 211, 1)
    H = oracle.hessian_accumulate(X)
    Xd = X.astype(np.float64)
    ref = 2.0 * (Xd @ Xd.T)  # BLAS: a different summation order
    assert np.array_equal(H, H.T)
    assert np.max(np.abs(H - ref)) <= 1e-12 * np.max(np.abs(ref))
    assert abs(np.trace(H) - 2.0 * np.sum(Xd * Xd)) <= 1e-12 * np.trace(H)
    for (i, j) in [(0, 0), (3, 17), (36, 2)]:
        assert oracle.hessian_entry(X, i, j) == H[i, j]


def test_hessian_is_second_derivative_of_layer_error():
    # E(w) = ||w X - w0 X||^2 for one row; finite differences of E must reproduce H = 2 X X^T
    _, X = _small_layer(1, 5, 40, 2)
    Xd = X.astype(np.float64)
    H = oracle.hessian_accumulate(X)
    w0 = _rng(3).standard_normal(5)

    def E(w):
        return float(np.sum(((w - w0) @ Xd) ** 2))

    h = 1e-3
    for a in range(5):
        for b in range(5):
            ea, eb = np.eye(5)[a] * h, np.eye(5)[b] * h
            fd = (E(w0 + ea + eb) - E(w0 + ea - eb) - E(w0 - ea + eb) + E(w0 - ea - eb)) / (4 * h * h)
            assert abs(fd - H[a, b]) <= 1e-6 * abs(H).max()


def test_hessian_accumulates_over_chunks():
    _, X = _small_layer(4, 19, 96, 4)
    H_full = oracle.hessian_accumulate(X)
    H = oracle.hessian_accumulate(X[:, :40])
    H = oracle.hessian_accumulate(X[:, 40:], H)
    assert np.max(np.abs(H - H_full)) <= 1e-13 * np.max(np.abs(H_full))


# ------------------------------------------------------------------ damped inverse (Sec. 5 item 1)
@pytest.mark.parametrize("spec", wl.conv_cases(), ids=lambda s: s.name)
def test_unfold_matches_library_unfold(spec):
    """The patch matrix of a convolution (Sec. 3) against torch's unfold, a library routine."""
    import torch
    _, act = wl.make_conv_layer(spec)
    X = oracle.unfold(act, spec.kh, spec.kw, spec.stride, spec.pad)
    assert X.shape == (spec.cols, spec.n)
    ref = torch.nn.functional.unfold(torch.from_numpy(act), (spec.kh, spec.kw), stride=spec.stride, padding=spec.pad)
    ref = ref.permute(1, 0, 2).reshape(spec.cols, -1).numpy()            # [cols, batch * positions]
    assert np.array_equal(X, ref)


@pytest.mark.parametrize("spec", wl.conv_cases()[:4] + wl.conv_cases()[5:], ids=lambda s: s.name)
def test_conv_hessian_is_energy_of_the_convolution_output(spec):
    """For any filter w, 1/2 w^T H w = ||w X||^2 is the squared norm of the convolution's output map, which torch's
    conv2d computes without ever forming patches: pins the row order (channel, ki, kj), stride and padding at once."""
    import torch
    W, act = wl.make_conv_layer(spec)
    H = oracle.hessian_accumulate_conv(act, spec.kh, spec.kw, spec.stride, spec.pad)
    assert np.array_equal(H, H.T)
    w = W[:3].astype(np.float64)
    out = torch.nn.functional.conv2d(torch.from_numpy(act).double(),
                                     torch.from_numpy(w).reshape(3, spec.channels, spec.kh, spec.kw),
                                     stride=spec.stride, padding=spec.pad).numpy()
    for r in range(3):
        energy = float(np.sum(out[:, r] ** 2))
        assert abs(0.5 * w[r] @ H @ w[r] - energy) <= 1e-11 * energy
    # two filters at once: the cross term, so that a transposed or permuted H would show
    cross = float(np.sum(out[:, 0] * out[:, 1]))
    assert abs(0.5 * w[0] @ H @ w[1] - cross) <= 1e-11 * np.sqrt(np.sum(out[:, 0] ** 2) * np.sum(out[:, 1] ** 2))


@pytest.mark.parametrize("cols,n,seed", [(16, 64, 5), (96, 64, 6), (200, 300, 7)])
def test_inverse_matches_lapack(cols, n, seed):
    _, X = _small_layer(4, cols, n, seed)
    H = oracle.hessian_accumulate(X)
    Hinv, diag, lam = oracle.prepare_hinv(H, 0.01, oracle.DAMP_REL_MEAN_DIAG)
    assert lam == pytest.approx(0.01 * np.mean(np.diag(H)), rel=1e-14)
    Hd = H + lam * np.eye(cols)
    ref = np.linalg.inv(Hd)
    cond = np.linalg.cond(Hd)
    assert np.max(np.abs(Hinv - ref)) <= 1e-15 * cond * np.max(np.abs(ref)) * 50
    assert np.max(np.abs(Hinv @ Hd - np.eye(cols))) <= 1e-15 * cond * 50
    assert np.array_equal(Hinv, Hinv.T)
    assert np.array_equal(diag, np.diag(Hinv))


def test_absolute_damping_and_not_spd():
    _, X = _small_layer(4, 12, 6, 8)  # rank 6 < 12: singular without damping
    H = oracle.hessian_accumulate(X)
    Hinv, _, lam = oracle.prepare_hinv(H, 0.1, oracle.DAMP_ABS)  # the paper's absolute 0.1
    assert lam == 0.1
    assert np.max(np.abs(Hinv @ (H + 0.1 * np.eye(12)) - np.eye(12))) < 1e-9
    Hneg = -np.eye(5)
    with pytest.raises(oracle.OracleError) as ei:
        oracle.prepare_hinv(Hneg, 0.0, oracle.DAMP_ABS)
    assert ei.value.code == oracle.ERR_NOT_SPD and ei.value.info == 0


# ------------------------------------------------------------------ grid and quant()
@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_grid_is_minmax_and_quant_is_nearest_level(bits):
    W, _ = _small_layer(6, 50, 8, 10 + bits)
    W[2] = np.abs(W[2])          # all-positive row: the range must still include 0
    W[3] = 0.0                   # degenerate row
    scale, zero = oracle.minmax_grid(W, bits)
    maxq = 2 ** bits - 1
    assert scale[3] == 1.0 and zero[3] == 0.0
    for i in range(6):
        if i == 3:
            continue
        lo, hi = min(W[i].min(), 0.0), max(W[i].max(), 0.0)
        assert scale[i] == np.float32((float(hi) - float(lo)) / maxq)
        assert zero[i] == np.rint(zero[i]) and 0 <= zero[i] <= maxq
        # the zero-point itself: level `zero` is the grid's 0, placed so that level 0 sits at the row minimum and the
        # top level at the row maximum, each to within half a step (an off-by-one zero-point shifts the whole grid by
        # one step and fails both)
        assert zero[i] == np.rint(-float(lo) / ((float(hi) - float(lo)) / maxq))
        levels = float(scale[i]) * (np.arange(maxq + 1) - float(zero[i]))
        half = 0.5 * float(scale[i]) * (1 + 1e-6)
        assert abs(levels[0] - float(lo)) <= half and abs(levels[maxq] - float(hi)) <= half
        assert levels[int(zero[i])] == 0.0
        for w in W[i].astype(np.float64):
            c = oracle.quant_code(w, scale[i], zero[i], bits)
            assert 0 <= c <= maxq
            d = np.abs(levels - w)
            assert d[c] <= d.min() * (1 + 1e-12) + 1e-300  # brute force over all 2^b levels


def test_quant_rounds_half_to_even_and_clamps():
    # scale 0.5, zero 2, 2 bits: levels -1, -0.5, 0, 0.5
    assert oracle.quant_code(0.25, 0.5, 2.0, 2) == 2     # 0.5 -> 0 (even), +2
    assert oracle.quant_code(0.75, 0.5, 2.0, 2) == 3     # 1.5 -> 2 then clamp(4) = 3
    assert oracle.quant_code(-0.25, 0.5, 2.0, 2) == 2    # -0.5 -> -0
    assert oracle.quant_code(-0.75, 0.5, 2.0, 2) == 0    # -1.5 -> -2
    assert oracle.quant_code(9.0, 0.5, 2.0, 2) == 3
    assert oracle.quant_code(-9.0, 0.5, 2.0, 2) == 0


# ------------------------------------------------------------------ ordering (Sec. 4.2 steps 1-3)
def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *v = line.split()
            out[k] = np.array([float(x) for x in v])
    return out


def test_ordering_hand_example():
    g = _read_golden("ordering_example.txt")
    W = np.stack([g["w_row0"], g["w_row1"]]).astype(np.float32)
    scale, zero = g["scale"].astype(np.float32), g["zero"].astype(np.float32)
    bits = int(g["bits"][0])
    S, perm = oracle.sensitivity_order(W, g["hinv_diag"], scale, zero, bits, oracle.SCORE_QERR)
    assert np.allclose(S, g["s_qerr"], rtol=1e-6) and list(perm) == list(g["order_qerr"].astype(int))
    S, perm = oracle.sensitivity_order(W, g["hinv_diag"], scale, zero, bits, oracle.SCORE_PRUNE)
    assert np.allclose(S, g["s_prune"], rtol=1e-6) and list(perm) == list(g["order_prune"].astype(int))
    # diagonal inverse Hessian: no compensation, codes are round-to-nearest under either order
    out = oracle.quantize_layer(W, np.diag(g["hinv_diag"]), perm, scale, zero, bits)
    assert np.array_equal(out["codes"], np.stack([g["codes_row0"], g["codes_row1"]]).astype(np.uint8))
    # ascending variants (Sec. 4.1): same scores, reversed order
    for mode, key_s, key_o in [(oracle.SCORE_QERR, "s_qerr", "order_qerr_asc"),
                               (oracle.SCORE_PRUNE, "s_prune", "order_prune_asc")]:
        S, perm = oracle.sensitivity_order(W, g["hinv_diag"], scale, zero, bits, mode | oracle.SCORE_ASCENDING)
        assert np.allclose(S, g[key_s], rtol=1e-6) and list(perm) == list(g[key_o].astype(int))
    # the non-parallel arm: each row in its own order; codes are still round-to-nearest (diagonal inverse Hessian)
    out = oracle.quantize_layer_per_row(W, np.diag(g["hinv_diag"]), g["hinv_diag"], scale, zero, bits)
    assert list(out["perm_rows"][0]) == list(g["order_row0"].astype(int))
    assert list(out["perm_rows"][1]) == list(g["order_row1"].astype(int))
    assert np.array_equal(out["codes"], np.stack([g["codes_row0"], g["codes_row1"]]).astype(np.uint8))


@pytest.mark.parametrize("mode", [oracle.SCORE_QERR, oracle.SCORE_PRUNE, oracle.SCORE_ERR, oracle.SCORE_W])
def test_scores_match_definition_and_sort_is_stable(mode):
    W, X = _small_layer(9, 24, 64, 20)
    W[:, 7] = W[:, 3]            # duplicated columns ...
    W[:, 15] = W[:, 3]
    Hinv, diag, _ = oracle.prepare_hinv(oracle.hessian_accumulate(X))
    diag[7] = diag[3]
    diag[15] = diag[3]           # ... with equal sensitivities -> exact ties
    scale, zero = oracle.minmax_grid(W, 3)
    S, perm = oracle.sensitivity_order(W, diag, scale, zero, 3, mode)
    Wd = W.astype(np.float64)
    err2 = (Wd - _dequant(_rtn_codes(W, scale, zero, 3), scale, zero)) ** 2
    num = err2 if mode in (oracle.SCORE_QERR, oracle.SCORE_ERR) else Wd ** 2
    den = 2.0 * diag[None, :] if mode in (oracle.SCORE_QERR, oracle.SCORE_PRUNE) else 1.0
    ref = (num / den).sum(axis=0)
    assert np.allclose(S, ref, rtol=1e-13)
    assert sorted(perm) == list(range(24))
    assert np.all(np.diff(S[perm]) <= 0)
    pos = {int(c): k for k, c in enumerate(perm)}
    assert S[3] == S[7] == S[15] and pos[3] < pos[7] < pos[15]
    assert pos[7] == pos[3] + 1 and pos[15] == pos[3] + 2


@pytest.mark.parametrize("mode", [oracle.SCORE_QERR, oracle.SCORE_W])
def test_ascending_order_is_stable_and_mirrors_descending(mode):
    W, X = _small_layer(9, 24, 64, 22)
    W[:, 7] = W[:, 3]
    W[:, 15] = W[:, 3]
    Hinv, diag, _ = oracle.prepare_hinv(oracle.hessian_accumulate(X))
    diag[7] = diag[3]
    diag[15] = diag[3]
    scale, zero = oracle.minmax_grid(W, 3)
    S_d, perm_d = oracle.sensitivity_order(W, diag, scale, zero, 3, mode)
    S_a, perm_a = oracle.sensitivity_order(W, diag, scale, zero, 3, mode | oracle.SCORE_ASCENDING)
    assert np.array_equal(S_a, S_d)                      # the direction changes the sort only
    assert sorted(perm_a) == list(range(24)) and np.all(np.diff(S_a[perm_a]) >= 0)
    pos = {int(c): k for k, c in enumerate(perm_a)}
    assert pos[7] == pos[3] + 1 and pos[15] == pos[3] + 2        # ties: lower column index first, as descending
    # away from the tie group the ascending order is the descending one read backwards
    rest_a = [c for c in perm_a if c not in (3, 7, 15)]
    rest_d = [c for c in perm_d if c not in (3, 7, 15)]
    assert rest_a == rest_d[::-1]
    assert list(perm_a) == list(np.argsort(S_a, kind="stable"))


def test_score_none_is_identity_order():
    W, _ = _small_layer(3, 11, 8, 21)
    S, perm = oracle.sensitivity_order(W, None, None, None, 4, oracle.SCORE_NONE)
    assert np.all(S == 0) and list(perm) == list(range(11))


# ------------------------------------------------------------------ column loop (Eq. 11, Eq. 12)
def test_identity_hessian_gives_round_to_nearest():
    W, _ = _small_layer(12, 40, 8, 30)
    W[0, :4] = np.float32(0.0)
    for bits in (2, 4, 8):
        scale, zero = oracle.minmax_grid(W, bits)
        perm = _rng(31).permutation(40).astype(np.int32)
        out = oracle.quantize_layer(W, np.eye(40), perm, scale, zero, bits, H_undamped=np.eye(40))
        rtn = _rtn_codes(W, scale, zero, bits)
        assert np.array_equal(out["codes"], rtn)
        assert np.array_equal(out["What"], _dequant(rtn, scale, zero).astype(np.float32))
        dW = W.astype(np.float64) - out["What"].astype(np.float64)
        assert out["loss"] == pytest.approx(0.5 * np.sum(dW * dW), rel=1e-12)


def _tiny(seed, rows=5, cols=9, n=30, bits=3):
    W, X = _small_layer(rows, cols, n, seed)
    H = oracle.hessian_accumulate(X)
    Hinv, diag, lam = oracle.prepare_hinv(H)
    scale, zero = oracle.minmax_grid(W, bits)
    S, perm = oracle.sensitivity_order(W, diag, scale, zero, bits)
    return W, X, H, Hinv, lam, scale, zero, perm, bits


@pytest.mark.parametrize("seed", [40, 41, 42])
def test_eq12_equals_direct_inverse_of_remaining_block(seed):
    W, X, H, Hinv, lam, scale, zero, perm, bits = _tiny(seed, cols=12)
    n = 12
    out = oracle.quantize_layer(W, Hinv, perm, scale, zero, bits, want_trace=True)
    Hd_p = (H + lam * np.eye(n))[np.ix_(perm, perm)]
    for p in range(n - 1):
        A = out["A_trace"][p]
        ref = np.linalg.inv(Hd_p[p + 1:, p + 1:])
        assert np.max(np.abs(A[p + 1:, p + 1:] - ref)) <= 1e-10 * np.max(np.abs(ref))
        assert np.all(A[:p + 1, :] == 0) and np.all(A[:, :p + 1] == 0)


@pytest.mark.parametrize("seed", [43, 44])
def test_eq11_equals_constrained_least_squares(seed):
    # After p columns are fixed to their grid values q_f, the OBS-optimal remaining weights are
    #   w_r = w0_r - Hd_rr^{-1} Hd_rf (q_f - w0_f)
    W, X, H, Hinv, lam, scale, zero, perm, bits = _tiny(seed, cols=10)
    n = 10
    out = oracle.quantize_layer(W, Hinv, perm, scale, zero, bits, want_trace=True)
    Hd_p = (H + lam * np.eye(n))[np.ix_(perm, perm)]
    W0 = W.astype(np.float64)[:, perm]
    for p in range(n - 1):
        Wp = out["W_trace"][p]
        f, r = slice(0, p + 1), slice(p + 1, n)
        qf = Wp[:, f]
        ref = W0[:, r] - (np.linalg.solve(Hd_p[r, r], Hd_p[r, f] @ (qf - W0[:, f]).T)).T
        assert np.max(np.abs(Wp[:, r] - ref)) <= 1e-10 * np.max(np.abs(W0))


@pytest.mark.parametrize("shape", [(5, 9, 30), (16, 64, 48), (32, 130, 256)])
def test_damped_loss_sum_identity(shape):
    # Eq. 10 summed over every quantization step equals 1/2 tr(dW Hd dW^T)
    rows, cols, n = shape
    W, X, H, Hinv, lam, scale, zero, perm, bits = _tiny(50 + rows, rows, cols, n, bits=4)
    out = oracle.quantize_layer(W, Hinv, perm, scale, zero, bits, H_undamped=H)
    dW = W.astype(np.float64) - _dequant(out["codes"], scale, zero)
    Hd = H + lam * np.eye(cols)
    quad = 0.5 * np.einsum("ij,jk,ik->", dW, Hd, dW)
    assert out["damped_sum"] == pytest.approx(quad, rel=1e-9)
    # and What is the float32 rounding of the grid value of each code
    assert np.array_equal(out["What"], _dequant(out["codes"], scale, zero).astype(np.float32))


def test_factor_form_identity():
    # Row p of A just before step p, divided by sqrt(A_pp), is row p of the upper Cholesky factor
    # of the permuted inverse Hessian -- the identity that licenses a blocked reformulation.
    W, X, H, Hinv, lam, scale, zero, perm, bits = _tiny(60, cols=14)
    out = oracle.quantize_layer(W, Hinv, perm, scale, zero, bits, want_trace=True)
    A0 = Hinv[np.ix_(perm, perm)]
    U = np.linalg.cholesky(A0).T
    for p in range(14):
        Ap = A0 if p == 0 else out["A_trace"][p - 1]
        assert np.allclose(Ap[p, p:] / np.sqrt(Ap[p, p]), U[p, p:], rtol=1e-9, atol=1e-14)


def test_oracle_factor_is_the_cholesky_factor_of_the_permuted_inverse():
    W, X, H, Hinv, lam, scale, zero, perm, bits = _tiny(62, 4, 33, 80)
    U = oracle.factor_upper(Hinv, perm)
    A0 = Hinv[np.ix_(perm, perm)]
    ref = np.linalg.cholesky(A0).T                       # LAPACK
    assert np.all(np.tril(U, -1) == 0)
    assert np.max(np.abs(U - ref)) <= 1e-12 * np.max(np.abs(ref))
    assert np.max(np.abs(U.T @ U - A0)) <= 1e-13 * np.max(np.abs(A0))
    with pytest.raises(oracle.OracleError) as ei:
        oracle.factor_upper(-np.eye(3), np.arange(3, dtype=np.int32))
    assert ei.value.code == oracle.ERR_NOT_SPD and ei.value.info == 0


@pytest.mark.parametrize("rows,cols,n,bits,xdist", [(5, 9, 30, 3, "halfnormal"), (16, 64, 48, 4, "halfnormal"),
                                                    (32, 130, 256, 4, "silu"), (24, 300, 200, 8, "normal"),
                                                    (12, 1024, 1500, 4, "halfnormal_sparse30"),
                                                    (8, 2304, 2048, 4, "halfnormal"), (6, 2304, 4096, 3, "halfnormal")])
def test_factor_form_sweep_equals_the_literal_loop(rows, cols, n, bits, xdist):
    """The factor-form mode against the literal Eq. 11 / Eq. 12 loop, up to the widest layers the literal loop
    reaches (2304 columns, with fewer calibration columns than weight columns in one case): same codes, same What,
    the same values before rounding."""
    W, X = _small_layer(rows, cols, n, 300 + cols + bits, xdist)
    H = oracle.hessian_accumulate(X)
    Hinv, diag, lam = oracle.prepare_hinv(H)
    scale, zero = oracle.minmax_grid(W, bits)
    S, perm = oracle.sensitivity_order(W, diag, scale, zero, bits)
    lit = oracle.quantize_layer(W, Hinv, perm, scale, zero, bits, want_prer=True)
    U = oracle.factor_upper(Hinv, perm)
    fac = oracle.quantize_rows_factor(W, U, perm, scale, zero, bits, want_prer=True)
    assert np.max(np.abs(fac["prer"] - lit["prer"])) <= 1e-7
    near = np.abs(np.abs(lit["prer"] - np.floor(lit["prer"])) - 0.5) <= 1e-6
    differ = fac["codes"] != lit["codes"]
    assert not np.any(differ & ~near)
    if not differ.any():
        assert np.array_equal(fac["What"], lit["What"])
    # rows are independent in this mode too
    sub = [rows - 1, 0]
    part = oracle.quantize_rows_factor(W[sub], U, perm, scale[sub], zero[sub], bits)
    assert np.array_equal(part["codes"], fac["codes"][sub])


# ------------------------------------------------------------------ dynamic re-ranking (Sec. 5)
@pytest.mark.parametrize("mode", [oracle.SCORE_QERR, oracle.SCORE_PRUNE | oracle.SCORE_ASCENDING])
def test_dynamic_with_one_block_is_the_static_method(mode):
    W, X, H, Hinv, lam, scale, zero, _, bits = _tiny(90, 7, 21, 64, bits=4)
    diag = np.diag(Hinv).copy()
    S, perm = oracle.sensitivity_order(W, diag, scale, zero, bits, mode)
    ref = oracle.quantize_layer(W, Hinv, perm, scale, zero, bits, H_undamped=H, want_prer=True)
    for block in (21, 1000):
        dyn = oracle.quantize_layer_dynamic(W, Hinv, scale, zero, bits, block, mode, H_undamped=H, want_prer=True)
        assert np.array_equal(dyn["order"], perm)
        assert np.array_equal(dyn["codes"], ref["codes"]) and np.array_equal(dyn["What"], ref["What"])
        assert np.array_equal(dyn["prer"], ref["prer"])
        assert dyn["loss"] == pytest.approx(ref["loss"], rel=1e-12)


@pytest.mark.parametrize("block", [1, 4])
def test_dynamic_order_follows_its_definition(block):
    """The state the dynamic loop ranks from is the state of the literal static loop run in the same column sequence:
    replay that sequence with the static loop (traces on), recompute the scores of the remaining columns from the
    traced weights and the traced inverse Hessian with numpy at every re-ranking point, and check that the dynamic
    loop picked the top `block` of them, in order."""
    bits = 3
    W, X, H, Hinv, lam, scale, zero, _, _ = _tiny(91, 6, 13, 40, bits=bits)
    n = 13
    dyn = oracle.quantize_layer_dynamic(W, Hinv, scale, zero, bits, block, oracle.SCORE_QERR)
    order = dyn["order"]
    assert sorted(order) == list(range(n))
    rep = oracle.quantize_layer(W, Hinv, order, scale, zero, bits, want_trace=True)
    assert np.array_equal(rep["codes"], dyn["codes"]) and np.array_equal(rep["What"], dyn["What"])
    sc, zp = scale.astype(np.float64)[:, None], zero.astype(np.float64)[:, None]
    for k in range(0, n, block):
        if k == 0:
            Wcur, Acur = W.astype(np.float64)[:, order], Hinv[np.ix_(order, order)]
        else:
            Wcur, Acur = rep["W_trace"][k - 1], rep["A_trace"][k - 1]          # permuted by `order`
        rem = np.arange(k, n)
        w = Wcur[:, rem]
        q = sc * (np.clip(np.rint(w / sc) + zp, 0, 2 ** bits - 1) - zp)
        Srem = ((w - q) ** 2 / (2.0 * np.diag(Acur)[rem][None, :])).sum(axis=0)
        # stable descending by score, ties by lower ORIGINAL column index
        want = sorted(range(len(rem)), key=lambda t: (-Srem[t], order[rem[t]]))[:block]
        assert [int(order[rem[t]]) for t in want] == [int(c) for c in order[k:k + block]]
    # re-ranking changes the sequence on this layer (otherwise the test would not bite)
    _, perm_static = oracle.sensitivity_order(W, np.diag(Hinv).copy(), scale, zero, bits)
    assert not np.array_equal(order, perm_static)


# ------------------------------------------------------------------ the non-parallel arm (Sec. 4.2)
def test_per_row_mode_ranks_and_quantizes_every_row_on_its_own():
    bits = 4
    W, X, H, Hinv, lam, scale, zero, perm, _ = _tiny(92, 6, 17, 50, bits=bits)
    diag = np.diag(Hinv).copy()
    out = oracle.quantize_layer_per_row(W, Hinv, diag, scale, zero, bits, H_undamped=H)
    Wd = W.astype(np.float64)
    err2 = (Wd - _dequant(_rtn_codes(W, scale, zero, bits), scale, zero)) ** 2
    L = err2 / (2.0 * diag[None, :])
    total = 0.0
    for i in range(6):
        perm_i = np.argsort(-L[i], kind="stable").astype(np.int32)
        assert np.array_equal(out["perm_rows"][i], perm_i)
        one = oracle.quantize_layer(W[i:i + 1], Hinv, perm_i, scale[i:i + 1], zero[i:i + 1], bits, H_undamped=H)
        assert np.array_equal(out["codes"][i], one["codes"][0]) and np.array_equal(out["What"][i], one["What"][0])
        total += one["loss"]
    assert out["loss"] == pytest.approx(total, rel=1e-12)
    dW = Wd - out["What"].astype(np.float64)
    assert out["loss"] == pytest.approx(0.5 * np.einsum("ij,jk,ik->", dW, H, dW), rel=1e-10)
    # the rows do not share one order on this layer
    assert any(not np.array_equal(out["perm_rows"][i], out["perm_rows"][0]) for i in range(1, 6))


def test_loss_from_hessian_equals_loss_from_inputs():
    W, X, H, Hinv, lam, scale, zero, perm, bits = _tiny(61, 7, 20, 100)
    out = oracle.quantize_layer(W, Hinv, perm, scale, zero, bits, H_undamped=H)
    direct = oracle.loss_direct(W, out["What"], X)
    Xd = X.astype(np.float64)
    lib = float(np.sum(((W.astype(np.float64) - out["What"].astype(np.float64)) @ Xd) ** 2))
    assert out["loss"] == pytest.approx(direct, rel=1e-11)
    assert direct == pytest.approx(lib, rel=1e-11)


def test_bruteforce_enumeration_on_tiny_rows():
    # 2-bit grid, 8 weights per row: enumerate all 4^8 code vectors.
    bits, cols, rows = 2, 8, 6
    W, X = _small_layer(rows, cols, 24, 70)
    H = oracle.hessian_accumulate(X)
    Hinv, diag, lam = oracle.prepare_hinv(H)
    scale, zero = oracle.minmax_grid(W, bits)
    S, perm = oracle.sensitivity_order(W, diag, scale, zero, bits)
    out = oracle.quantize_layer(W, Hinv, perm, scale, zero, bits, H_undamped=H)
    all_codes = np.array(list(itertools.product(range(4), repeat=cols)), dtype=np.float64)  # [65536, 8]
    Wd = W.astype(np.float64)
    rtn = _rtn_codes(W, scale, zero, bits)
    total_o = total_r = 0.0
    for i in range(rows):
        Q = float(scale[i]) * (all_codes - float(zero[i]))
        D = Wd[i][None, :] - Q
        losses = 0.5 * np.einsum("aj,jk,ak->a", D, H, D)
        idx_o = int(np.dot(out["codes"][i].astype(np.int64), 4 ** np.arange(cols - 1, -1, -1)))
        idx_r = int(np.dot(rtn[i].astype(np.int64), 4 ** np.arange(cols - 1, -1, -1)))
        assert losses[idx_o] >= losses.min() - 1e-12
        total_o += losses[idx_o]
        total_r += losses[idx_r]
    # the loss the oracle reports is the enumerated loss of its own code vectors
    # (What is the float32 rounding of the grid values, hence the 1e-6)
    assert out["loss"] == pytest.approx(total_o, rel=1e-5)
    assert total_o <= total_r


def test_compensation_beats_rtn_on_average_and_forced_codes_roundtrip():
    W, X, H, Hinv, lam, scale, zero, perm, bits = _tiny(80, 24, 48, 96, bits=4)
    out = oracle.quantize_layer(W, Hinv, perm, scale, zero, bits, H_undamped=H, want_prer=True)
    rtn = _dequant(_rtn_codes(W, scale, zero, bits), scale, zero).astype(np.float32)
    assert out["loss"] < oracle.loss_direct(W, rtn, X)
    again = oracle.quantize_layer(W, Hinv, perm, scale, zero, bits, H_undamped=H,
                                  forced_codes=out["codes"], want_prer=True)
    assert np.array_equal(again["codes"], out["codes"]) and np.array_equal(again["What"], out["What"])
    assert np.array_equal(again["prer"], out["prer"])
    # each code is the nearest level of the value seen before rounding
    v = np.clip(np.rint(out["prer"]) + zero[:, None].astype(np.float64), 0, 15)
    assert np.array_equal(v.astype(np.uint8), out["codes"])


def test_rows_are_independent_given_order_and_inverse():
    W, X, H, Hinv, lam, scale, zero, perm, bits = _tiny(81, 10, 20, 64)
    full = oracle.quantize_layer(W, Hinv, perm, scale, zero, bits)
    sub = [7, 2, 9]
    part = oracle.quantize_layer(W[sub], Hinv, perm, scale[sub], zero[sub], bits)
    assert np.array_equal(part["codes"], full["codes"][sub])
    assert np.array_equal(part["What"], full["What"][sub])


def test_config1_layer_runs_and_improves_on_rtn():
    spec = wl.config1()[0]
    W, X = wl.make_layer(spec)
    out = oracle.run_layer(W, X, spec.bits, spec.damp)
    rtn = _dequant(_rtn_codes(W, out["scale"], out["zero"], 4), out["scale"], out["zero"]).astype(np.float32)
    assert out["loss"] < 0.6 * oracle.loss_direct(W, rtn, X)
    assert out["loss"] == pytest.approx(oracle.loss_direct(W, out["What"], X), rel=1e-10)
