"""Runs one stage of the quantizer (or the whole path) a few times on one synthetic layer and prints the device
time of every repetition.  Meant for profiling and size sweeps:

    python -m paper_2509_05576_b200.stage_run --stage gram --rows 256 --cols 2304 --n 16384 --iters 3

Stages: gram (ptq_hessian_accumulate), inverse (ptq_prepare_hinv), order (ptq_minmax_grid +
ptq_sensitivity_order), sweep (ptq_quantize_layer), all (the whole path).  The inputs of a stage are produced by
running the earlier stages once, so every repetition sees valid data.  An L2-sized buffer is rewritten between
repetitions.  Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import ptq
from . import workloads as wl


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--stage", default="all", choices=["gram", "inverse", "order", "sweep", "all"])
    ap.add_argument("--rows", type=int, default=256)
    ap.add_argument("--cols", type=int, default=2304)
    ap.add_argument("--n", type=int, default=4096)
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--xdist", default="halfnormal")
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    ap.add_argument("--no-loss", action="store_true")
    ap.add_argument("--kernels", action="store_true", help="also one pass with the library's per-kernel event profiler")
    args = ap.parse_args(argv)

    if not torch.cuda.is_available():
        raise RuntimeError("stage_run needs a CUDA device")
    spec = wl.LayerSpec("stage", args.rows, args.cols, args.n, args.bits, "kaiming", args.xdist, args.seed)
    W, X = wl.make_layer(spec)
    Wd, Xd = torch.from_numpy(W).cuda(), torch.from_numpy(X).cuda()
    bufs = ptq.LayerBuffers(args.rows, args.cols)
    ws = ptq.Workspace()
    st = bufs.status
    s = torch.cuda.current_stream()
    flush = torch.empty(256 * 2 ** 20, dtype=torch.uint8, device="cuda")
    want_loss = not args.no_loss

    def gram():
        bufs.H.zero_()
        ptq.hessian_accumulate(bufs.H, Xd, ws, st, s)

    def inverse():
        ptq.prepare_hinv(bufs.H, spec.damp, ptq.DAMP_REL_MEAN_DIAG, bufs.Hinv, bufs.Hinv_diag, bufs.lam, ws, st, s)

    def order():
        ptq.minmax_grid(Wd, args.bits, bufs.scale, bufs.zero, st, s)
        ptq.sensitivity_order(Wd, bufs.Hinv_diag, bufs.scale, bufs.zero, args.bits, ptq.SCORE_QERR, bufs.S, bufs.perm,
                              ws, st, s)

    def sweep():
        ptq.quantize_layer(Wd, bufs.Hinv, bufs.perm, bufs.scale, bufs.zero, args.bits, bufs.codes, bufs.What,
                           bufs.H if want_loss else None, bufs.loss if want_loss else None, ws, st, s)

    stages = {"gram": gram, "inverse": inverse, "order": order, "sweep": sweep}

    def whole():
        for f in (gram, inverse, order, sweep):
            f()

    whole()                     # produces the inputs of every stage
    torch.cuda.synchronize()
    ptq.check_status(st, "set-up")
    fn = whole if args.stage == "all" else stages[args.stage]
    times = []
    for it in range(args.warmup + args.iters):
        flush.fill_(it & 0xFF)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(s)
        fn()
        b.record(s)
        torch.cuda.synchronize()
        if it >= args.warmup:
            times.append(a.elapsed_time(b))
    ptq.check_status(st, args.stage)
    kernels = None
    if args.kernels:
        ptq.profile_enable(True)
        flush.fill_(7)
        fn()
        torch.cuda.synchronize()
        kernels = {k: {"ms": round(ms, 4), "launches": cnt} for k, (ms, cnt) in ptq.profile_read().items()}
        ptq.profile_enable(False)
    print(json.dumps({"stage": args.stage, "rows": args.rows, "cols": args.cols, "n": args.n, "bits": args.bits,
                      "xdist": args.xdist, "ms": times, "ms_median": float(np.median(times)),
                      "loss": float(bufs.loss.item()) if want_loss else None, "kernels": kernels}))
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
