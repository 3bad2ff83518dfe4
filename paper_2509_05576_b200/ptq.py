"""Thin binding over the C-ABI CUDA library ``libptq.so`` (declared in ``include/ptq.h``).

Only argument marshalling happens here: every step of the path runs in the library's kernels.
torch is used for device memory and streams.  There is no CPU fallback: if the library is missing
or no CUDA device is present, the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_double, c_int, c_int64, c_size_t, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libptq.so")

OK, ERR_INVALID_ARG, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_NOT_SPD, ERR_NONFINITE, ERR_TIMEOUT, ERR_CUDA, ERR_UNSUPPORTED = range(9)
ERR_STATIC_SCRATCH = 9
STATIC_SCRATCH_BYTES = 6 << 20
DAMP_REL_MEAN_DIAG, DAMP_ABS = 0, 1
SCORE_QERR, SCORE_PRUNE, SCORE_ERR, SCORE_W, SCORE_NONE = 0, 1, 2, 3, 4
SCORE_ASCENDING = 16          # added to a score mode: sort by S ascending
CALL_HESSIAN_ACCUMULATE, CALL_PREPARE_HINV, CALL_SENSITIVITY_ORDER, CALL_QUANTIZE_LAYER, CALL_HESSIAN_ACCUMULATE_F64 = range(5)
CALL_QUANTIZE_LAYER_DYNAMIC = 5
CALL_QUANTIZE_LAYER_PER_ROW = 6

EXPORTS = ["ptq_workspace_bytes", "ptq_hessian_accumulate", "ptq_hessian_accumulate_conv", "ptq_hessian_accumulate_f64", "ptq_prepare_hinv",
           "ptq_minmax_grid", "ptq_sensitivity_order", "ptq_sensitivity_order_static", "ptq_quantize_layer", "ptq_status_string", "ptq_version",
           "ptq_sort_scores", "ptq_gemm_nt_sliced", "ptq_gemm_nt_sliced_workspace_bytes", "ptq_quantize_layer_dynamic", "ptq_quantize_layer_per_row", "ptq_selftest_wait_timeout", "ptq_fp64_probe",
           "ptq_kernel_count", "ptq_kernel_name", "ptq_launch_count", "ptq_profile_enable", "ptq_profile_read",
           "ptq_set_cta_limit"]


class PtqError(RuntimeError):
    def __init__(self, code, where, index=None):
        msg = f"{where}: {status_string(code)} (status {code})"
        if index is not None:
            msg += f", index {index}"
        super().__init__(msg)
        self.code = code
        self.index = index


_lib = None


def lib():
    """Loads ``libptq.so`` (built in-tree by ``paper_2509_05576_b200.build``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2509_05576_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp = c_void_p
        L.ptq_workspace_bytes.argtypes = [c_int, c_int, c_int, c_int]
        L.ptq_workspace_bytes.restype = c_size_t
        for name in ("ptq_hessian_accumulate", "ptq_hessian_accumulate_f64"):
            getattr(L, name).argtypes = [vp, vp, c_int, c_int, c_int64, vp, c_size_t, vp, vp]
        L.ptq_hessian_accumulate_conv.argtypes = [vp, vp, c_int, c_int, c_int, c_int, c_int, c_int, c_int, c_int, vp,
                                                  c_size_t, vp, vp]
        L.ptq_prepare_hinv.argtypes = [vp, c_int, c_int, c_double, vp, vp, vp, vp, c_size_t, vp, vp]
        L.ptq_minmax_grid.argtypes = [vp, c_int, c_int, c_int64, c_int, vp, vp, vp, vp]
        L.ptq_sensitivity_order.argtypes = [vp, c_int, c_int, c_int64, vp, vp, vp, c_int, c_int, vp, vp, vp, c_size_t,
                                            vp, vp]
        L.ptq_sensitivity_order_static.argtypes = [vp, c_int, c_int, c_int64, vp, vp, vp, c_int, c_int, vp, vp, vp, vp]
        L.ptq_quantize_layer.argtypes = [vp, c_int, c_int, c_int64, vp, vp, vp, vp, c_int, vp, vp, vp, vp, vp,
                                         c_size_t, vp, vp]
        L.ptq_sort_scores.argtypes = [vp, c_int, c_int, vp, vp]
        L.ptq_gemm_nt_sliced_workspace_bytes.argtypes = [c_int, c_int, c_int]
        L.ptq_gemm_nt_sliced_workspace_bytes.restype = c_size_t
        L.ptq_gemm_nt_sliced.argtypes = [vp, c_int64, vp, c_int64, vp, c_int64, c_int, c_int, c_int, c_int, c_double, vp,
                                         c_size_t, vp, vp]
        L.ptq_quantize_layer_per_row.argtypes = [vp, c_int, c_int, c_int64, vp, vp, vp, c_int, c_int, vp, vp, vp, vp, vp,
                                                 vp, c_size_t, vp, vp]
        L.ptq_quantize_layer_dynamic.argtypes = [vp, c_int, c_int, c_int64, vp, vp, vp, c_int, c_int, c_int, vp, vp,
                                                 vp, vp, vp, vp, c_size_t, vp, vp]
        L.ptq_selftest_wait_timeout.argtypes = [c_int, ctypes.c_longlong, vp, c_size_t, vp, vp]
        L.ptq_fp64_probe.argtypes = [c_int, c_int, vp, ctypes.POINTER(c_double), vp]
        L.ptq_status_string.argtypes = [c_int]
        L.ptq_status_string.restype = ctypes.c_char_p
        L.ptq_version.restype = c_int
        L.ptq_kernel_count.restype = c_int
        L.ptq_kernel_name.argtypes = [c_int]
        L.ptq_kernel_name.restype = ctypes.c_char_p
        L.ptq_launch_count.argtypes = [c_int]
        L.ptq_launch_count.restype = ctypes.c_longlong
        L.ptq_profile_enable.argtypes = [c_int]
        L.ptq_set_cta_limit.argtypes = [c_int]
        L.ptq_profile_read.argtypes = [c_int, ctypes.POINTER(c_double), ctypes.POINTER(ctypes.c_longlong)]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().ptq_status_string(int(code)).decode()


def launch_count(kernel_id: int = -1) -> int:
    """Kernel launches made by the library in this process (all kernels when kernel_id < 0)."""
    return int(lib().ptq_launch_count(int(kernel_id)))


def set_cta_limit(limit: int):
    """At most `limit` CTAs per persistent cooperative kernel on the current device (0: one per SM)."""
    _check(lib().ptq_set_cta_limit(int(limit)), "ptq_set_cta_limit")


def profile_enable(on: bool):
    _check(lib().ptq_profile_enable(1 if on else 0), "ptq_profile_enable")


def profile_read():
    """Per-kernel device time of the launches recorded since ``profile_enable(True)``: {name: (ms, launches)}."""
    out = {}
    for k in range(lib().ptq_kernel_count()):
        ms, cnt = c_double(0.0), ctypes.c_longlong(0)
        _check(lib().ptq_profile_read(k, ctypes.byref(ms), ctypes.byref(cnt)), "ptq_profile_read")
        if cnt.value:
            out[lib().ptq_kernel_name(k).decode()] = (ms.value, cnt.value)
    return out


def workspace_bytes(call_id: int, rows: int, cols: int, n: int) -> int:
    return int(lib().ptq_workspace_bytes(int(call_id), int(rows), int(cols), int(n)))


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return c_void_p(s.cuda_stream)


def _dev(t, dtype, name):
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (the library has no CPU path)")
    if t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}")
    return t


def _rowmajor(t, name):
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError(f"{name} must be 2-D with unit column stride")
    return t.stride(0)


class Workspace:
    """A growable device scratch buffer handed to the library calls."""

    def __init__(self, device="cuda"):
        self.device = torch.device(device)
        self.buf = None

    def get(self, nbytes: int):
        if self.buf is None or self.buf.numel() < nbytes:
            self.buf = None
            self.buf = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=self.device)
        return self.buf


def new_status(device="cuda"):
    return torch.zeros(4, dtype=torch.int32, device=device)


def check_status(status, where="ptq"):
    """Synchronises and raises if a kernel recorded an error in the status word."""
    code, index, aux, _ = status.cpu().tolist()
    if code != OK:
        raise PtqError(code, where, index)


def _check(ret, where):
    if ret != OK:
        raise PtqError(ret, where)


def hessian_accumulate(H, X, ws, status, stream=None, f64=False):
    """H += 2 X X^T (Sec. 3).  H [cols, cols] float64, X [cols, n] float32, both on the device."""
    _dev(H, torch.float64, "H"); _dev(X, torch.float32, "X")
    cols, n = X.shape
    ldx = _rowmajor(X, "X")
    if H.shape != (cols, cols) or not H.is_contiguous():
        raise ValueError("H must be contiguous [cols, cols]")
    fn = lib().ptq_hessian_accumulate_f64 if f64 else lib().ptq_hessian_accumulate
    need = workspace_bytes(CALL_HESSIAN_ACCUMULATE_F64 if f64 else CALL_HESSIAN_ACCUMULATE, 0, cols, n)
    buf = ws.get(need)
    _check(fn(_ptr(H), _ptr(X), cols, n, ldx, _ptr(buf), buf.numel(), _ptr(status), _stream(stream)),
           "ptq_hessian_accumulate")


def conv_unfolded_shape(act_shape, kh, kw, stride=1, pad=0):
    """(cols, n) of the unfolded input of a convolution: channels kh kw rows, batch out_h out_w columns."""
    b, c, h, w = act_shape
    oh, ow = (h + 2 * pad - kh) // stride + 1, (w + 2 * pad - kw) // stride + 1
    return c * kh * kw, b * oh * ow


def hessian_accumulate_conv(H, act, kh, kw, stride, pad, ws, status, stream=None):
    """H += 2 X X^T with X the unfolded patches of act [batch, channels, height, width] (Sec. 3), read in place."""
    _dev(H, torch.float64, "H"); _dev(act, torch.float32, "act")
    if act.dim() != 4 or not act.is_contiguous():
        raise ValueError("act must be contiguous [batch, channels, height, width]")
    b, c, h, w = act.shape
    cols, n = conv_unfolded_shape(act.shape, kh, kw, stride, pad)
    if H.shape != (cols, cols) or not H.is_contiguous():
        raise ValueError("H must be contiguous [channels kh kw, channels kh kw]")
    buf = ws.get(workspace_bytes(CALL_HESSIAN_ACCUMULATE, 0, cols, n))
    _check(lib().ptq_hessian_accumulate_conv(_ptr(H), _ptr(act), b, c, h, w, int(kh), int(kw), int(stride), int(pad),
                                             _ptr(buf), buf.numel(), _ptr(status), _stream(stream)),
           "ptq_hessian_accumulate_conv")


def prepare_hinv(H, damp, damp_mode, Hinv, Hinv_diag, lambda_out, ws, status, stream=None):
    """Hinv = (H + lambda I)^-1 (Sec. 5 item 1); also its diagonal and lambda (device scalars)."""
    _dev(H, torch.float64, "H"); _dev(Hinv, torch.float64, "Hinv")
    cols = H.shape[0]
    buf = ws.get(workspace_bytes(CALL_PREPARE_HINV, 0, cols, 0))
    _check(lib().ptq_prepare_hinv(_ptr(H), cols, int(damp_mode), float(damp), _ptr(Hinv), _ptr(Hinv_diag),
                                  _ptr(lambda_out), _ptr(buf), buf.numel(), _ptr(status), _stream(stream)),
           "ptq_prepare_hinv")


def minmax_grid(W, bits, scale, zero, status, stream=None):
    _dev(W, torch.float32, "W")
    rows, cols = W.shape
    _check(lib().ptq_minmax_grid(_ptr(W), rows, cols, _rowmajor(W, "W"), int(bits), _ptr(scale), _ptr(zero),
                                 _ptr(status), _stream(stream)), "ptq_minmax_grid")


def sensitivity_order(W, Hinv_diag, scale, zero, bits, score_mode, S, perm, ws, status, stream=None):
    """Sec. 4.2 steps 1-3: column scores S and the descending, stable column order perm."""
    _dev(W, torch.float32, "W")
    rows, cols = W.shape
    buf = ws.get(workspace_bytes(CALL_SENSITIVITY_ORDER, rows, cols, 0))
    _check(lib().ptq_sensitivity_order(_ptr(W), rows, cols, _rowmajor(W, "W"), _ptr(Hinv_diag), _ptr(scale),
                                       _ptr(zero), int(bits), int(score_mode), _ptr(S), _ptr(perm), _ptr(buf),
                                       buf.numel(), _ptr(status), _stream(stream)), "ptq_sensitivity_order")


def sensitivity_order_static(W, Hinv_diag, scale, zero, bits, score_mode, S, perm, status, stream=None):
    """``sensitivity_order`` without a workspace argument, for callers that may not allocate device memory: the
    scratch is an array built into the library (``STATIC_SCRATCH_BYTES``).  Raises ``PtqError`` with
    ``ERR_STATIC_SCRATCH`` when ceil(rows / 64) * cols * 8 bytes exceeds it.  Calls share that array, so keep them
    ordered on one stream."""
    _dev(W, torch.float32, "W")
    rows, cols = W.shape
    _check(lib().ptq_sensitivity_order_static(_ptr(W), rows, cols, _rowmajor(W, "W"), _ptr(Hinv_diag), _ptr(scale),
                                              _ptr(zero), int(bits), int(score_mode), _ptr(S), _ptr(perm),
                                              _ptr(status), _stream(stream)), "ptq_sensitivity_order_static")


def sort_scores(S, perm, ascending=False, stream=None):
    """perm = indices sorted by S descending (or ascending), stable (Sec. 4.2 step 3)."""
    _dev(S, torch.float64, "S"); _dev(perm, torch.int32, "perm")
    _check(lib().ptq_sort_scores(_ptr(S), S.numel(), 1 if ascending else 0, _ptr(perm), _stream(stream)),
           "ptq_sort_scores")


def gemm_nt_sliced(C, A, B, alpha, ws, status, b_is_kn=False, stream=None):
    """C += alpha * A @ B.T (b_is_kn: C += alpha * A @ B) for float64 device tensors, on the int8 tensor path."""
    _dev(C, torch.float64, "C"); _dev(A, torch.float64, "A"); _dev(B, torch.float64, "B")
    m, k = A.shape
    n = B.shape[1] if b_is_kn else B.shape[0]
    buf = ws.get(int(lib().ptq_gemm_nt_sliced_workspace_bytes(m, n, k)))
    _check(lib().ptq_gemm_nt_sliced(_ptr(C), _rowmajor(C, "C"), _ptr(A), _rowmajor(A, "A"), _ptr(B), _rowmajor(B, "B"),
                                    1 if b_is_kn else 0, m, n, k, float(alpha), _ptr(buf), buf.numel(), _ptr(status),
                                    _stream(stream)), "ptq_gemm_nt_sliced")


def selftest_wait_timeout(which, limit_cycles, ws, status, stream=None):
    """Makes one of the library's bounded device-side waits run out (0: grid barrier, 1: sweep counter)."""
    buf = ws.get(256)
    _check(lib().ptq_selftest_wait_timeout(int(which), int(limit_cycles), _ptr(buf), buf.numel(), _ptr(status),
                                           _stream(stream)), "ptq_selftest_wait_timeout")


def fp64_probe(kind, iters, sink, stream=None) -> float:
    """Launches the float64 throughput probe (0: FMA, 1: tensor-core MMA); returns the flops of that launch."""
    flops = c_double(0.0)
    _check(lib().ptq_fp64_probe(int(kind), int(iters), _ptr(sink), ctypes.byref(flops), _stream(stream)),
           "ptq_fp64_probe")
    return flops.value


def quantize_layer(W, Hinv, perm, scale, zero, bits, codes, What, H_undamped, loss_out, ws, status, stream=None):
    """Sec. 4.2 steps 3-5 (Eq. 11, Eq. 12): the column-synchronous sweep.  Outputs in original column order."""
    _dev(W, torch.float32, "W"); _dev(Hinv, torch.float64, "Hinv"); _dev(perm, torch.int32, "perm")
    _dev(codes, torch.uint8, "codes")
    rows, cols = W.shape
    buf = ws.get(workspace_bytes(CALL_QUANTIZE_LAYER, rows, cols, 0))
    _check(lib().ptq_quantize_layer(_ptr(W), rows, cols, _rowmajor(W, "W"), _ptr(Hinv), _ptr(perm), _ptr(scale),
                                    _ptr(zero), int(bits), _ptr(codes), _ptr(What), _ptr(H_undamped), _ptr(loss_out),
                                    _ptr(buf), buf.numel(), _ptr(status), _stream(stream)), "ptq_quantize_layer")


def quantize_layer_dynamic(W, Hinv, scale, zero, bits, score_mode, block, codes, What, order_out, H_undamped, loss_out,
                           ws, status, stream=None):
    """The column loop with the remaining columns re-ranked every ``block`` columns (Sec. 5)."""
    _dev(W, torch.float32, "W"); _dev(Hinv, torch.float64, "Hinv"); _dev(codes, torch.uint8, "codes")
    _dev(order_out, torch.int32, "order_out")
    rows, cols = W.shape
    buf = ws.get(workspace_bytes(CALL_QUANTIZE_LAYER_DYNAMIC, rows, cols, 0))
    _check(lib().ptq_quantize_layer_dynamic(_ptr(W), rows, cols, _rowmajor(W, "W"), _ptr(Hinv), _ptr(scale), _ptr(zero),
                                            int(bits), int(score_mode), int(block), _ptr(codes), _ptr(What),
                                            _ptr(order_out), _ptr(H_undamped), _ptr(loss_out), _ptr(buf), buf.numel(),
                                            _ptr(status), _stream(stream)), "ptq_quantize_layer_dynamic")


def quantize_layer_per_row(W, Hinv, scale, zero, bits, score_mode, codes, What, perm_rows, H_undamped, loss_out, ws,
                           status, stream=None):
    """The non-parallel arm (Sec. 4.2): every row in its own order against its own inverse Hessian; cols <= 128."""
    _dev(W, torch.float32, "W"); _dev(Hinv, torch.float64, "Hinv"); _dev(codes, torch.uint8, "codes")
    _dev(perm_rows, torch.int32, "perm_rows")
    rows, cols = W.shape
    buf = ws.get(workspace_bytes(CALL_QUANTIZE_LAYER_PER_ROW, rows, cols, 0))
    _check(lib().ptq_quantize_layer_per_row(_ptr(W), rows, cols, _rowmajor(W, "W"), _ptr(Hinv), _ptr(scale), _ptr(zero),
                                            int(bits), int(score_mode), _ptr(codes), _ptr(What), _ptr(perm_rows),
                                            _ptr(H_undamped), _ptr(loss_out), _ptr(buf), buf.numel(), _ptr(status),
                                            _stream(stream)), "ptq_quantize_layer_per_row")


class LayerBuffers:
    """Device outputs and scratch of one layer shape, allocated once and reused across calls."""

    def __init__(self, rows, cols, device="cuda"):
        d = torch.device(device)
        self.rows, self.cols = rows, cols
        self.H = torch.empty((cols, cols), dtype=torch.float64, device=d)
        self.Hinv = torch.empty((cols, cols), dtype=torch.float64, device=d)
        self.Hinv_diag = torch.empty(cols, dtype=torch.float64, device=d)
        self.lam = torch.empty(1, dtype=torch.float64, device=d)
        self.scale = torch.empty(rows, dtype=torch.float32, device=d)
        self.zero = torch.empty(rows, dtype=torch.float32, device=d)
        self.S = torch.empty(cols, dtype=torch.float64, device=d)
        self.perm = torch.empty(cols, dtype=torch.int32, device=d)
        self.codes = torch.empty((rows, cols), dtype=torch.uint8, device=d)
        self.What = torch.empty((rows, cols), dtype=torch.float32, device=d)
        self.loss = torch.empty(1, dtype=torch.float64, device=d)
        self.status = new_status(d)


def quantize_layer_full(W, X, bits, damp=0.01, damp_mode=DAMP_REL_MEAN_DIAG, score_mode=SCORE_QERR, bufs=None, ws=None,
                        stream=None, want_loss=True, events=None, gram_f64=False, conv=None):
    """The whole hot path on one layer (all device-side, asynchronous on the stream):
    Hessian -> damped inverse -> grid -> scores + order -> column sweep -> codes, What, loss.

    ``conv``: None for a layer given by its input matrix X [cols, n]; for a convolution ``(kh, kw, stride, pad)``,
    and X is then the layer's input [batch, channels, height, width] or a list of such calibration batches, read in
    place by ``ptq_hessian_accumulate_conv`` (W is the weight flattened per filter, [out_channels, channels kh kw]).
    ``events``: optional list receiving (stage name, start event, end event) for per-stage timing.
    Returns the LayerBuffers holding the outputs; call ``check_status(bufs.status)`` after synchronising.
    """
    rows, cols = W.shape
    bufs = bufs or LayerBuffers(rows, cols, W.device)
    ws = ws or Workspace(W.device)
    st = bufs.status
    s = torch.cuda.current_stream() if stream is None else stream

    def timed(name, fn):
        if events is None:
            fn()
            return
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(s)
        fn()
        b.record(s)
        events.append((name, a, b))

    with torch.cuda.stream(s):
        st.zero_()
        bufs.H.zero_()
        if conv is None:
            timed("hessian", lambda: hessian_accumulate(bufs.H, X, ws, st, s, f64=gram_f64))
        else:
            kh, kw, stride, pad = conv
            batches = X if isinstance(X, (list, tuple)) else [X]
            timed("hessian", lambda: [hessian_accumulate_conv(bufs.H, a, kh, kw, stride, pad, ws, st, s)
                                      for a in batches])
        timed("inverse", lambda: prepare_hinv(bufs.H, damp, damp_mode, bufs.Hinv, bufs.Hinv_diag, bufs.lam, ws, st, s))
        timed("grid", lambda: minmax_grid(W, bits, bufs.scale, bufs.zero, st, s))
        timed("order", lambda: sensitivity_order(W, bufs.Hinv_diag, bufs.scale, bufs.zero, bits, score_mode, bufs.S,
                                                 bufs.perm, ws, st, s))
        timed("sweep", lambda: quantize_layer(W, bufs.Hinv, bufs.perm, bufs.scale, bufs.zero, bits, bufs.codes,
                                              bufs.What, bufs.H if want_loss else None,
                                              bufs.loss if want_loss else None, ws, st, s))
    return bufs


class LayerGraph:
    """The whole path of one layer captured once as a CUDA graph and replayed: for layers so small that launching
    their twenty-odd kernels one by one from the host takes longer than running them.

    The graph is tied to the tensors it was captured with (W, X, the LayerBuffers and the workspace): refill W and X
    in place and call ``replay()``.  Warm up the same call once before capturing (the first call on a device sets
    kernel attributes, which is not a stream operation)."""

    def __init__(self, W, X, bits, damp=0.01, damp_mode=DAMP_REL_MEAN_DIAG, score_mode=SCORE_QERR, bufs=None, ws=None):
        rows, cols = W.shape
        self.bufs = bufs or LayerBuffers(rows, cols, W.device)
        self.ws = ws or Workspace(W.device)
        self.stream = torch.cuda.Stream(device=W.device)
        args = (W, X, bits, damp, damp_mode, score_mode)
        self.stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(self.stream):
            quantize_layer_full(*args, bufs=self.bufs, ws=self.ws, stream=self.stream)       # warm-up, sizes the workspace
        self.stream.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph, stream=self.stream):
            quantize_layer_full(*args, bufs=self.bufs, ws=self.ws, stream=self.stream)

    def replay(self):
        self.graph.replay()
        return self.bufs


def estimate_layer_ms(rows, cols):
    """Rough device time of one layer in ms (fixed part, the two pivot chains per 64 columns, the cubic part), used only
    to deal the layers of a set onto streams."""
    return 0.1 + 0.04 * cols / 64 + 6.0 * (cols / 4608.0) ** 3 * (1 + rows / 4096.0)


def plan_layer_set(shapes, n_streams, longest_first=True):
    """[(layer index, stream index)] in issue order for layers of the given (rows, cols).  longest_first: the layers in
    descending order of their estimated time, each onto the stream with the least estimated work so far (ties: the lower
    stream index); otherwise round-robin in the given order."""
    n_streams = max(1, int(n_streams))
    if not longest_first:
        return [(i, i % n_streams) for i in range(len(shapes))]
    est = [estimate_layer_ms(r, c) for r, c in shapes]
    load = [0.0] * n_streams
    plan = []
    for i in sorted(range(len(shapes)), key=lambda q: (-est[q], q)):
        k = min(range(n_streams), key=lambda q: (load[q], q))
        load[k] += est[i]
        plan.append((i, k))
    return plan


class LayerSet:
    """Independent layers (a network's layers, each with its own calibration input) quantized side by side on several
    streams of one GPU.  Layers up to a few thousand columns are bound by dependency chains (the pivots of the
    factorisations, the columns of the sweep), not by the number of SMs, so several of them fit on the GPU at once --
    provided the two persistent cooperative kernels, which otherwise take one CTA per SM each, are held to a share of the
    SMs (``ptq_set_cta_limit``).  ``cta_limit`` None: a quarter of the SMs for layers below 3072 columns, half for wider
    ones; 0: no limit.  The layers are dealt longest first (a rough estimate from the shapes) onto the stream with the
    least work so far.  Every stream has its own workspace, every layer its own LayerBuffers, kept in ``self.bufs`` in
    the order the layers were given; results do not depend on the placement.

    ``layers``: list of (W, X, bits) or (W, X, bits, damp) with W [rows, cols] float32 and X [cols, n] float32 on the
    device.  ``run()`` issues the whole set asynchronously (the streams first wait for the current stream, which in turn
    waits for them at the end) and returns ``self.bufs``; synchronise and ``check_status`` before reading."""

    def __init__(self, layers, n_streams=8, cta_limit=None, score_mode=SCORE_QERR, damp_mode=DAMP_REL_MEAN_DIAG):
        self.layers = [tuple(l) if len(l) == 4 else (l[0], l[1], l[2], 0.01) for l in layers]
        dev = self.layers[0][0].device
        self.score_mode, self.damp_mode = score_mode, damp_mode
        self.streams = [torch.cuda.Stream(device=dev) for _ in range(max(1, n_streams))]
        self.wss = [Workspace(dev) for _ in self.streams]
        self.bufs = [LayerBuffers(W.shape[0], W.shape[1], dev) for W, _, _, _ in self.layers]
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        self.cta_limit = max(1, sms // 4) if cta_limit is None else int(cta_limit)
        self.plan = plan_layer_set([tuple(W.shape) for W, _, _, _ in self.layers], len(self.streams),
                                   longest_first=self.cta_limit > 0)

    def run(self):
        cur = torch.cuda.current_stream()
        for st_ in self.streams:
            st_.wait_stream(cur)
        try:
            for i, k in self.plan:
                W, X, bits, damp = self.layers[i]
                set_cta_limit(self.cta_limit if W.shape[1] < 3072 else 2 * self.cta_limit)
                quantize_layer_full(W, X, bits, damp, self.damp_mode, self.score_mode, bufs=self.bufs[i], ws=self.wss[k],
                                    stream=self.streams[k])
        finally:
            set_cta_limit(0)
        for st_ in self.streams:
            cur.wait_stream(st_)
        return self.bufs


class HostStaging:
    """Device landing buffers and the copy stream used by ``quantize_layer_from_host`` (allocated once per shape)."""

    def __init__(self, rows, cols, chunk_cols, device="cuda"):
        d = torch.device(device)
        self.W = torch.empty((rows, cols), dtype=torch.float32, device=d)
        self.X = [torch.empty((cols, nc), dtype=torch.float32, device=d) for nc in chunk_cols]
        self.copy_stream = torch.cuda.Stream(device=d)


def quantize_layer_from_host(W_host, X_batches_host, bits, damp=0.01, damp_mode=DAMP_REL_MEAN_DIAG,
                             score_mode=SCORE_QERR, bufs=None, ws=None, staging=None, stream=None, want_loss=True):
    """The whole path for a layer whose W and calibration activations sit in (pinned) host memory.

    ``X_batches_host`` is a list of contiguous [cols, n_i] float32 tensors, the calibration batches.  They are uploaded
    one after the other on a copy stream while the Hessian of the batches already on the device is being accumulated
    (``ptq_hessian_accumulate`` is additive over calibration columns), so most of the upload hides behind the Gram.
    Everything is asynchronous; returns the LayerBuffers (outputs on the device).
    """
    rows, cols = W_host.shape
    staging = staging or HostStaging(rows, cols, [x.shape[1] for x in X_batches_host])
    bufs = bufs or LayerBuffers(rows, cols)
    ws = ws or Workspace()
    s = torch.cuda.current_stream() if stream is None else stream
    cs = staging.copy_stream
    st = bufs.status
    cs.wait_stream(s)                       # the landing buffers are free once earlier work on the stream is done
    events = []
    with torch.cuda.stream(cs):
        for xd, xh in zip(staging.X, X_batches_host):
            xd.copy_(xh, non_blocking=True)
            ev = torch.cuda.Event()
            ev.record(cs)
            events.append(ev)
        staging.W.copy_(W_host, non_blocking=True)
        w_ready = torch.cuda.Event()
        w_ready.record(cs)
    with torch.cuda.stream(s):
        st.zero_()
        bufs.H.zero_()
        for xd, ev in zip(staging.X, events):
            s.wait_event(ev)
            hessian_accumulate(bufs.H, xd, ws, st, s)
        prepare_hinv(bufs.H, damp, damp_mode, bufs.Hinv, bufs.Hinv_diag, bufs.lam, ws, st, s)
        s.wait_event(w_ready)
        minmax_grid(staging.W, bits, bufs.scale, bufs.zero, st, s)
        sensitivity_order(staging.W, bufs.Hinv_diag, bufs.scale, bufs.zero, bits, score_mode, bufs.S, bufs.perm, ws, st, s)
        quantize_layer(staging.W, bufs.Hinv, bufs.perm, bufs.scale, bufs.zero, bits, bufs.codes, bufs.What,
                       bufs.H if want_loss else None, bufs.loss if want_loss else None, ws, st, s)
    return bufs
