"""Ordering / parallelism ablation on synthetic layers (the synthetic analogue of the paper's Table 3 and Figure 1):
for each layer, the row-parallel method with its static column order (Sec. 4.2), the same with the remaining columns
re-ranked every 64 columns (Sec. 5), the ascending and the unsorted orders (Sec. 4.1), and -- on layers of at most 128
columns -- the non-parallel arm in which every row has its own order and its own inverse Hessian (Sec. 4.2).
Reports device time of the ordering + column-loop stage and the reconstruction loss of each variant.

    python -m paper_2509_05576_b200.ablation_run [--config 3] [--max-cols 1152]
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import ptq
from . import workloads as wl


def _time(fn, stream, flush, reps=3):
    ts = []
    for r in range(reps + 1):
        flush.fill_(r)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fn()
        b.record(stream)
        torch.cuda.synchronize()
        if r:
            ts.append(a.elapsed_time(b))
    return float(np.median(ts))


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=3, choices=[3, 4, 6, 7])
    ap.add_argument("--max-cols", type=int, default=1152)
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise RuntimeError("ablation_run needs a CUDA device")
    specs, seen = [], set()
    for s in wl.CONFIGS[args.config]():
        if s.cols <= args.max_cols and (s.rows, s.cols) not in seen:
            seen.add((s.rows, s.cols))
            specs.append(s)
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 * 2 ** 20, dtype=torch.uint8, device="cuda")
    ws = ptq.Workspace()
    out = []
    print(f"{'layer':26s} {'rows':>5s} {'cols':>5s} | {'variant':22s} {'ms':>8s} {'loss':>12s} {'vs static':>9s}")
    for spec in specs:
        W, X = wl.make_layer(spec)
        Wd, Xd = torch.from_numpy(W).cuda(), torch.from_numpy(X).cuda()
        bufs = ptq.quantize_layer_full(Wd, Xd, spec.bits, spec.damp, ws=ws)
        torch.cuda.synchronize()
        ptq.check_status(bufs.status, spec.name)
        st = bufs.status
        order = torch.empty(spec.cols, dtype=torch.int32, device="cuda")
        perm_rows = torch.empty((spec.rows, spec.cols), dtype=torch.int32, device="cuda")

        def static(mode):
            def run():
                ptq.sensitivity_order(Wd, bufs.Hinv_diag, bufs.scale, bufs.zero, spec.bits, mode, bufs.S, bufs.perm, ws, st)
                ptq.quantize_layer(Wd, bufs.Hinv, bufs.perm, bufs.scale, bufs.zero, spec.bits, bufs.codes, bufs.What, bufs.H,
                                   bufs.loss, ws, st)
            return run

        def dynamic(block):
            return lambda: ptq.quantize_layer_dynamic(Wd, bufs.Hinv, bufs.scale, bufs.zero, spec.bits, ptq.SCORE_QERR, block,
                                                      bufs.codes, bufs.What, order, bufs.H, bufs.loss, ws, st)

        def per_row():
            ptq.quantize_layer_per_row(Wd, bufs.Hinv, bufs.scale, bufs.zero, spec.bits, ptq.SCORE_QERR, bufs.codes, bufs.What,
                                       perm_rows, bufs.H, bufs.loss, ws, st)

        variants = [("sensi_des, parallel", static(ptq.SCORE_QERR)),
                    ("sensi_asc, parallel", static(ptq.SCORE_QERR | ptq.SCORE_ASCENDING)),
                    ("err_des, parallel", static(ptq.SCORE_ERR)),
                    ("w_des, parallel", static(ptq.SCORE_W)),
                    ("no sorting, parallel", static(ptq.SCORE_NONE))]
        if spec.cols > 64:
            variants.append(("sensi_des, re-ranked/64", dynamic(64)))
        if spec.cols <= 128:
            variants.append(("sensi_des, per row", per_row))
        base = None
        for name, fn in variants:
            ms = _time(fn, stream, flush)
            ptq.check_status(st, spec.name + " " + name)
            loss = float(bufs.loss.item())
            base = base or (ms, loss)
            print(f"{spec.name:26s} {spec.rows:5d} {spec.cols:5d} | {name:22s} {ms:8.3f} {loss:12.5g} {ms / base[0]:8.1f}x")
            out.append({"layer": spec.name, "rows": spec.rows, "cols": spec.cols, "variant": name, "ms": ms, "loss": loss})
    print(json.dumps({"config": args.config, "results": out}))
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
