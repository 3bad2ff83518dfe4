"""ctypes loader for the float64 CPU oracle (``oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the bench's
CPU-baseline leg.  The CUDA library never imports or links anything from here, and this
package imports nothing from the CUDA package.

Every wrapper takes and returns numpy arrays on the host; argument marshalling is all
that happens in Python -- the arithmetic is in ``oracle.c``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from ctypes import POINTER, c_double, c_float, c_int, c_int32, c_int64, c_uint8, c_void_p

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

OK, ERR_INVALID_ARG, ERR_NOT_SPD, ERR_NOMEM = 0, 1, 4, 9
DAMP_REL_MEAN_DIAG, DAMP_ABS = 0, 1
SCORE_QERR, SCORE_PRUNE, SCORE_ERR, SCORE_W, SCORE_NONE = 0, 1, 2, 3, 4
SCORE_ASCENDING = 16          # added to a score mode: sort by S ascending (the "asc" keys of Sec. 4.1)


class OracleError(RuntimeError):
    def __init__(self, code, what, info=None):
        super().__init__(f"oracle {what} failed with status {code}" + (f" (index {info})" if info is not None else ""))
        self.code = code
        self.info = info


def build(force: bool = False) -> str:
    """Compile ``oracle.c`` with gcc into ``liboracle.so`` next to it (no-op when up to date)."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
           "-fno-fast-math", "-o", _LIB + ".tmp", _SRC, "-lm"]
    subprocess.run(cmd, check=True, cwd=_HERE)
    os.replace(_LIB + ".tmp", _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        pf, pd, pi, pu = POINTER(c_float), POINTER(c_double), POINTER(c_int32), POINTER(c_uint8)
        L.oracle_version.restype = c_int
        L.oracle_num_threads.restype = c_int
        L.oracle_hessian_accumulate.argtypes = [pd, pf, c_int, c_int, c_int64]
        L.oracle_hessian_entry.argtypes = [pf, c_int, c_int64, c_int, c_int]
        L.oracle_unfold.argtypes = [pf, pf] + [c_int] * 8
        L.oracle_hessian_entry.restype = c_double
        L.oracle_prepare_hinv.argtypes = [pd, c_int, c_int, c_double, pd, pd, pd, POINTER(c_int)]
        L.oracle_minmax_grid.argtypes = [pf, c_int, c_int, c_int64, c_int, pf, pf]
        L.oracle_quant_code.argtypes = [c_double, c_float, c_float, c_int]
        L.oracle_sensitivity_order.argtypes = [pf, c_int, c_int, c_int64, pd, pf, pf, c_int, c_int, pd, pi]
        L.oracle_quantize_layer_ex.argtypes = [pf, c_int, c_int, c_int64, pd, pi, pf, pf, c_int, pu, pf,
                                               pd, pd, pu, pd, pd, pd, pd]
        L.oracle_loss_direct.argtypes = [pf, pf, c_int, c_int, c_int64, c_int64, pf, c_int, c_int64]
        L.oracle_factor_upper.argtypes = [pd, pi, c_int, pd, POINTER(c_int)]
        L.oracle_quantize_rows_factor.argtypes = [pf, c_int, c_int, c_int64, pd, pi, pf, pf, c_int, pu, pf, pd]
        L.oracle_quantize_layer_dynamic.argtypes = [pf, c_int, c_int, c_int64, pd, pf, pf, c_int, c_int, c_int, pu,
                                                    pf, pi, pd, pd, pd]
        L.oracle_quantize_layer_per_row.argtypes = [pf, c_int, c_int, c_int64, pd, pd, pf, pf, c_int, c_int, pu, pf,
                                                    pi, pd, pd]
        L.oracle_loss_direct.restype = c_double
        _lib = L
    return _lib


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(POINTER(ct))


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    assert a.ndim == 2
    return a


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def hessian_accumulate(X, H=None):
    """H += 2 X X^T (Sec. 3, Eq. 2).  X: [cols, n] float32.  Returns H [cols, cols] float64."""
    X = _f32(X)
    cols, n = X.shape
    if H is None:
        H = np.zeros((cols, cols), dtype=np.float64)
    assert H.shape == (cols, cols) and H.dtype == np.float64 and H.flags.c_contiguous
    st = lib().oracle_hessian_accumulate(_p(H, c_double), _p(X, c_float), cols, n, X.strides[0] // 4)
    if st:
        raise OracleError(st, "hessian_accumulate")
    return H


def unfold(act, kh, kw, stride=1, pad=0):
    """Input patches of a convolution as the columns of X (Sec. 3): act [batch, channels, height, width] float32 ->
    X [channels kh kw, batch out_h out_w] float32, rows ordered like a flattened filter (channel, ki, kj)."""
    act = np.ascontiguousarray(act, dtype=np.float32)
    assert act.ndim == 4
    b, c, h, w = act.shape
    oh, ow = (h + 2 * pad - kh) // stride + 1, (w + 2 * pad - kw) // stride + 1
    X = np.empty((c * kh * kw, b * oh * ow), dtype=np.float32)
    st = lib().oracle_unfold(_p(X, c_float), _p(act, c_float), b, c, h, w, int(kh), int(kw), int(stride), int(pad))
    if st:
        raise OracleError(st, "unfold")
    return X


def hessian_accumulate_conv(act, kh, kw, stride=1, pad=0, H=None):
    """H += 2 X X^T with X = unfold(act): the Hessian of a convolutional layer (Sec. 3, Eq. 2)."""
    return hessian_accumulate(unfold(act, kh, kw, stride, pad), H)


def hessian_entry(X, i, j) -> float:
    X = _f32(X)
    return float(lib().oracle_hessian_entry(_p(X, c_float), X.shape[1], X.strides[0] // 4, int(i), int(j)))


def prepare_hinv(H, damp=0.01, mode=DAMP_REL_MEAN_DIAG):
    """Returns (Hinv, Hinv_diag, lambda) for Hd = H + lambda I (Sec. 5 item 1)."""
    H = np.ascontiguousarray(H, dtype=np.float64)
    cols = H.shape[0]
    Hinv = np.empty_like(H)
    diag = np.empty(cols, dtype=np.float64)
    lam = c_double(0.0)
    info = c_int(-1)
    st = lib().oracle_prepare_hinv(_p(H, c_double), cols, int(mode), float(damp), _p(Hinv, c_double),
                                   _p(diag, c_double), ctypes.byref(lam), ctypes.byref(info))
    if st:
        raise OracleError(st, "prepare_hinv", info.value)
    return Hinv, diag, lam.value


def minmax_grid(W, bits):
    W = _f32(W)
    rows, cols = W.shape
    scale = np.empty(rows, dtype=np.float32)
    zero = np.empty(rows, dtype=np.float32)
    st = lib().oracle_minmax_grid(_p(W, c_float), rows, cols, W.strides[0] // 4, int(bits), _p(scale, c_float),
                                  _p(zero, c_float))
    if st:
        raise OracleError(st, "minmax_grid")
    return scale, zero


def quant_code(w, scale, zero, bits) -> int:
    return int(lib().oracle_quant_code(float(w), float(scale), float(zero), int(bits)))


def sensitivity_order(W, Hinv_diag, scale, zero, bits, mode=SCORE_QERR):
    """Returns (S [cols] float64, perm [cols] int32): Sec. 4.2 steps 1-3."""
    W = _f32(W)
    rows, cols = W.shape
    S = np.empty(cols, dtype=np.float64)
    perm = np.empty(cols, dtype=np.int32)
    d = None if Hinv_diag is None else np.ascontiguousarray(Hinv_diag, dtype=np.float64)
    sc = None if scale is None else np.ascontiguousarray(scale, dtype=np.float32)
    zp = None if zero is None else np.ascontiguousarray(zero, dtype=np.float32)
    st = lib().oracle_sensitivity_order(_p(W, c_float), rows, cols, W.strides[0] // 4, _p(d, c_double),
                                        _p(sc, c_float), _p(zp, c_float), int(bits), int(mode),
                                        _p(S, c_double), _p(perm, c_int32))
    if st:
        raise OracleError(st, "sensitivity_order")
    return S, perm


def quantize_layer(W, Hinv, perm, scale, zero, bits, H_undamped=None, forced_codes=None,
                   want_prer=False, want_trace=False):
    """Sec. 4.2 steps 3-5 (Eq. 11, Eq. 12).  Returns a dict with codes, What and the extras asked for."""
    W = _f32(W)
    rows, cols = W.shape
    Hinv = np.ascontiguousarray(Hinv, dtype=np.float64)
    perm = np.ascontiguousarray(perm, dtype=np.int32)
    scale = np.ascontiguousarray(scale, dtype=np.float32)
    zero = np.ascontiguousarray(zero, dtype=np.float32)
    codes = np.empty((rows, cols), dtype=np.uint8)
    What = np.empty((rows, cols), dtype=np.float32)
    Hu = None if H_undamped is None else np.ascontiguousarray(H_undamped, dtype=np.float64)
    loss = c_double(float("nan"))
    dsum = c_double(float("nan"))
    fc = None if forced_codes is None else np.ascontiguousarray(forced_codes, dtype=np.uint8)
    prer = np.empty((rows, cols), dtype=np.float64) if want_prer else None
    A_tr = np.empty((cols, cols, cols), dtype=np.float64) if want_trace else None
    W_tr = np.empty((cols, rows, cols), dtype=np.float64) if want_trace else None
    st = lib().oracle_quantize_layer_ex(
        _p(W, c_float), rows, cols, W.strides[0] // 4, _p(Hinv, c_double), _p(perm, c_int32),
        _p(scale, c_float), _p(zero, c_float), int(bits), _p(codes, c_uint8), _p(What, c_float),
        _p(Hu, c_double), ctypes.byref(loss) if Hu is not None else None, _p(fc, c_uint8),
        _p(prer, c_double), _p(A_tr, c_double), _p(W_tr, c_double), ctypes.byref(dsum))
    if st:
        raise OracleError(st, "quantize_layer")
    out = {"codes": codes, "What": What, "damped_sum": dsum.value}
    if Hu is not None:
        out["loss"] = loss.value
    if want_prer:
        out["prer"] = prer
    if want_trace:
        out["A_trace"], out["W_trace"] = A_tr, W_tr
    return out


def factor_upper(Hinv, perm):
    """U with Hinv[perm][:, perm] = U^T U (upper triangular), by the oracle's own plain Cholesky."""
    Hinv = np.ascontiguousarray(Hinv, dtype=np.float64)
    perm = np.ascontiguousarray(perm, dtype=np.int32)
    cols = Hinv.shape[0]
    U = np.empty((cols, cols), dtype=np.float64)
    info = c_int(-1)
    st = lib().oracle_factor_upper(_p(Hinv, c_double), _p(perm, c_int32), cols, _p(U, c_double), ctypes.byref(info))
    if st:
        raise OracleError(st, "factor_upper", info.value)
    return U


def quantize_rows_factor(W, U, perm, scale, zero, bits, want_prer=False):
    """The column loop in factor form (e = (w - q) / U_pp, w_j -= e U_pj) on the given rows.  Licensed by its pin
    against the literal Eq. 11 / Eq. 12 loop; for layers too wide for that loop."""
    W = _f32(W)
    rows, cols = W.shape
    U = np.ascontiguousarray(U, dtype=np.float64)
    perm = np.ascontiguousarray(perm, dtype=np.int32)
    scale = np.ascontiguousarray(scale, dtype=np.float32)
    zero = np.ascontiguousarray(zero, dtype=np.float32)
    codes = np.empty((rows, cols), dtype=np.uint8)
    What = np.empty((rows, cols), dtype=np.float32)
    prer = np.empty((rows, cols), dtype=np.float64) if want_prer else None
    st = lib().oracle_quantize_rows_factor(_p(W, c_float), rows, cols, W.strides[0] // 4, _p(U, c_double),
                                           _p(perm, c_int32), _p(scale, c_float), _p(zero, c_float), int(bits),
                                           _p(codes, c_uint8), _p(What, c_float), _p(prer, c_double))
    if st:
        raise OracleError(st, "quantize_rows_factor")
    out = {"codes": codes, "What": What}
    if want_prer:
        out["prer"] = prer
    return out


def quantize_layer_dynamic(W, Hinv, scale, zero, bits, block, mode=SCORE_QERR, H_undamped=None, want_prer=False):
    """Dynamic re-ranking (Sec. 5): the remaining columns are re-scored from the current weights and the current
    inverse Hessian every `block` columns.  Returns codes, What, order (the sequence of columns) and the extras."""
    W = _f32(W)
    rows, cols = W.shape
    Hinv = np.ascontiguousarray(Hinv, dtype=np.float64)
    scale = np.ascontiguousarray(scale, dtype=np.float32)
    zero = np.ascontiguousarray(zero, dtype=np.float32)
    codes = np.empty((rows, cols), dtype=np.uint8)
    What = np.empty((rows, cols), dtype=np.float32)
    order = np.empty(cols, dtype=np.int32)
    Hu = None if H_undamped is None else np.ascontiguousarray(H_undamped, dtype=np.float64)
    loss = c_double(float("nan"))
    prer = np.empty((rows, cols), dtype=np.float64) if want_prer else None
    st = lib().oracle_quantize_layer_dynamic(_p(W, c_float), rows, cols, W.strides[0] // 4, _p(Hinv, c_double),
                                             _p(scale, c_float), _p(zero, c_float), int(bits), int(mode), int(block),
                                             _p(codes, c_uint8), _p(What, c_float), _p(order, c_int32),
                                             _p(Hu, c_double), ctypes.byref(loss) if Hu is not None else None,
                                             _p(prer, c_double))
    if st:
        raise OracleError(st, "quantize_layer_dynamic")
    out = {"codes": codes, "What": What, "order": order}
    if Hu is not None:
        out["loss"] = loss.value
    if want_prer:
        out["prer"] = prer
    return out


def quantize_layer_per_row(W, Hinv, Hinv_diag, scale, zero, bits, mode=SCORE_QERR, H_undamped=None):
    """The non-parallel arm (Sec. 4.2): every row ranked by its own sensitivities and quantized against its own copy
    of the inverse Hessian.  Returns codes, What, perm_rows [rows, cols] and the loss when H is given."""
    W = _f32(W)
    rows, cols = W.shape
    Hinv = np.ascontiguousarray(Hinv, dtype=np.float64)
    diag = None if Hinv_diag is None else np.ascontiguousarray(Hinv_diag, dtype=np.float64)
    scale = np.ascontiguousarray(scale, dtype=np.float32)
    zero = np.ascontiguousarray(zero, dtype=np.float32)
    codes = np.empty((rows, cols), dtype=np.uint8)
    What = np.empty((rows, cols), dtype=np.float32)
    perm_rows = np.empty((rows, cols), dtype=np.int32)
    Hu = None if H_undamped is None else np.ascontiguousarray(H_undamped, dtype=np.float64)
    loss = c_double(float("nan"))
    st = lib().oracle_quantize_layer_per_row(_p(W, c_float), rows, cols, W.strides[0] // 4, _p(Hinv, c_double),
                                             _p(diag, c_double), _p(scale, c_float), _p(zero, c_float), int(bits),
                                             int(mode), _p(codes, c_uint8), _p(What, c_float), _p(perm_rows, c_int32),
                                             _p(Hu, c_double), ctypes.byref(loss) if Hu is not None else None)
    if st:
        raise OracleError(st, "quantize_layer_per_row")
    out = {"codes": codes, "What": What, "perm_rows": perm_rows}
    if Hu is not None:
        out["loss"] = loss.value
    return out


def loss_direct(W, What, X) -> float:
    """Eq. 2 evaluated from the calibration inputs."""
    W, What, X = _f32(W), _f32(What), _f32(X)
    rows, cols = W.shape
    return float(lib().oracle_loss_direct(_p(W, c_float), _p(What, c_float), rows, cols, W.strides[0] // 4,
                                          What.strides[0] // 4, _p(X, c_float), X.shape[1], X.strides[0] // 4))


def run_layer(W, X, bits, damp=0.01, damp_mode=DAMP_REL_MEAN_DIAG, score_mode=SCORE_QERR, want_prer=False):
    """The whole path on one layer: Hessian, damped inverse, grid, order, column loop, loss."""
    H = hessian_accumulate(X)
    Hinv, diag, lam = prepare_hinv(H, damp, damp_mode)
    scale, zero = minmax_grid(W, bits)
    S, perm = sensitivity_order(W, diag, scale, zero, bits, score_mode)
    out = quantize_layer(W, Hinv, perm, scale, zero, bits, H_undamped=H, want_prer=want_prer)
    out.update(H=H, Hinv=Hinv, Hinv_diag=diag, lam=lam, scale=scale, zero=zero, S=S, perm=perm)
    return out
