"""One layer quantized by several GPUs: calibration columns and weight rows split over the ranks.

The path shards in two places (Sec. 3, Sec. 4.2):

* the Hessian is a sum over calibration columns, H = 2 sum_n x_n x_n^T, so each rank forms the Gram of ITS slice of
  the calibration set and one all-reduce (sum) of the cols x cols matrix gives every rank the whole H;
* rows never interact in the column loop (Sec. 4.2 step 4: all rows of a column are quantized at once, each against
  the same shared inverse Hessian), so each rank sweeps ITS rows.  The only quantity that couples the rows is the
  column score S_j, a sum over rows (Sec. 4.2 step 2): one all-reduce (sum) of a cols-vector, after which every rank
  sorts the same S and obtains the same column order.

Everything else (damped inverse, the factor of the permuted inverse Hessian) is computed redundantly by every rank
from the same H, so no further exchange is needed; the layer loss is summed at the end.  The collectives are plain
``torch.distributed`` all-reduces on ordinary device buffers (NCCL over NVLink on GPUs; any backend works).

``ops`` is the set of per-rank compute steps.  The default, ``GpuOps``, calls the CUDA library through the C-ABI
binding; there is no CPU implementation in this package (tests of the host logic supply their own ``ops``).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def split_range(total: int, world: int, rank: int):
    """Contiguous, balanced share of ``range(total)`` for ``rank`` of ``world``: the first ``total % world`` ranks get
    one element more.  Returns (start, stop); the shares tile the range in rank order and may be empty."""
    if world < 1 or not 0 <= rank < world or total < 0:
        raise ValueError("split_range: bad arguments")
    base, extra = divmod(total, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


class GpuOps:
    """The per-rank steps on this rank's GPU, through the C-ABI binding (device tensors in, device tensors out)."""

    def __init__(self, stream=None):
        from . import ptq
        self.ptq = ptq
        self.ws = ptq.Workspace()
        self.stream = stream
        self.status = ptq.new_status()

    def hessian(self, X, cols):
        H = torch.zeros((cols, cols), dtype=torch.float64, device="cuda")
        if X is not None and X.shape[1] > 0:
            self.ptq.hessian_accumulate(H, X, self.ws, self.status, self.stream)
        return H

    def prepare_hinv(self, H, damp, damp_mode):
        cols = H.shape[0]
        Hinv = torch.empty_like(H)
        diag = torch.empty(cols, dtype=torch.float64, device=H.device)
        lam = torch.empty(1, dtype=torch.float64, device=H.device)
        self.ptq.prepare_hinv(H, damp, damp_mode, Hinv, diag, lam, self.ws, self.status, self.stream)
        return Hinv, diag, lam

    def grid(self, W, bits):
        rows = W.shape[0]
        scale = torch.empty(rows, dtype=torch.float32, device=W.device)
        zero = torch.empty(rows, dtype=torch.float32, device=W.device)
        if rows:
            self.ptq.minmax_grid(W, bits, scale, zero, self.status, self.stream)
        return scale, zero

    def scores(self, W, diag, scale, zero, bits, score_mode):
        """This rank's share of S: the sum of the per-weight scores over ITS rows."""
        cols = W.shape[1]
        S = torch.zeros(cols, dtype=torch.float64, device=W.device)
        if W.shape[0]:
            perm = torch.empty(cols, dtype=torch.int32, device=W.device)
            self.ptq.sensitivity_order(W, diag, scale, zero, bits, score_mode, S, perm, self.ws, self.status, self.stream)
        return S

    def sort(self, S, ascending):
        perm = torch.empty(S.numel(), dtype=torch.int32, device=S.device)
        self.ptq.sort_scores(S, perm, ascending, self.stream)
        return perm

    def sweep(self, W, Hinv, perm, scale, zero, bits, H):
        rows, cols = W.shape
        codes = torch.empty((rows, cols), dtype=torch.uint8, device=W.device)
        What = torch.empty((rows, cols), dtype=torch.float32, device=W.device)
        loss = torch.zeros(1, dtype=torch.float64, device=W.device)
        if rows:
            self.ptq.quantize_layer(W, Hinv, perm, scale, zero, bits, codes, What, H, loss, self.ws, self.status,
                                    self.stream)
        return codes, What, loss

    def check(self, where="sharded layer"):
        self.ptq.check_status(self.status, where)


def quantize_layer_sharded(W_rows, X_cols, cols, bits, damp=0.01, damp_mode=0, score_mode=0, group=None, ops=None):
    """Quantizes one layer whose rows and calibration columns are spread over the ranks of ``group``.

    W_rows: this rank's rows of W, [rows_r, cols] float32 (``split_range(rows, world, rank)`` of the full matrix);
    X_cols: this rank's calibration columns, [cols, n_r] float32 (any split of the calibration set; None or zero
    columns allowed).  Returns a dict with this rank's ``codes`` and ``What`` (its rows), and the replicated
    ``H``, ``Hinv``, ``S``, ``perm``, ``lam`` and the whole layer's ``loss``.
    """
    ops = ops or GpuOps()
    ascending = bool(score_mode & 16)
    H = ops.hessian(X_cols, cols)
    dist.all_reduce(H, op=dist.ReduceOp.SUM, group=group)            # exchange 1: the Hessian over the calibration split
    Hinv, diag, lam = ops.prepare_hinv(H, damp, damp_mode)
    scale, zero = ops.grid(W_rows, bits)
    S = ops.scores(W_rows, diag, scale, zero, bits, score_mode & ~16)
    dist.all_reduce(S, op=dist.ReduceOp.SUM, group=group)            # exchange 2: the column scores over the row split
    perm = ops.sort(S, ascending)                                    # same S on every rank, so the same order
    codes, What, loss = ops.sweep(W_rows, Hinv, perm, scale, zero, bits, H)
    dist.all_reduce(loss, op=dist.ReduceOp.SUM, group=group)         # the layer loss is the sum over the rows
    return {"codes": codes, "What": What, "scale": scale, "zero": zero, "H": H, "Hinv": Hinv, "lam": lam, "S": S,
            "perm": perm, "loss": loss}
