"""Times the Hessian of convolutional layers accumulated straight from the layer input (``ptq_hessian_accumulate_conv``)
against the same Hessian from written-out patches (``ptq_hessian_accumulate`` on X = unfold(act)), one GPU.

    python -m paper_2509_05576_b200.conv_run [--reps 5]

Both calls are bracketed by CUDA events on the launching stream; a 256 MiB buffer is rewritten before every timed
repetition.  The patch matrix of the second arm is produced beforehand by torch's unfold (not timed: it stands for
whatever produced X).  Prints one line per layer and checks that the two Hessians are bit-identical.
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
    ap.add_argument("--reps", type=int, default=5)
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise RuntimeError("conv_run needs a CUDA device")
    s = torch.cuda.current_stream()
    flush = torch.empty(256 * 2 ** 20, dtype=torch.uint8, device="cuda")
    ws = ptq.Workspace()
    st = ptq.new_status()
    out = []
    print(f"{'layer':20s} {'cols':>5s} {'n':>6s} {'act MB':>7s} {'X MB':>7s} {'in place ms':>11s} {'from X ms':>10s} {'same H':>6s}")
    for spec in wl.resnet_conv_specs():
        _, act = wl.make_conv_layer(spec)
        a = torch.from_numpy(act).cuda()
        X = torch.nn.functional.unfold(a, (spec.kh, spec.kw), stride=spec.stride, padding=spec.pad)
        X = X.permute(1, 0, 2).reshape(spec.cols, -1).contiguous()
        Hc = torch.zeros((spec.cols, spec.cols), dtype=torch.float64, device="cuda")
        Hm = torch.zeros_like(Hc)
        tc, tm = [], []
        for rep in range(args.reps + 1):
            for which in (0, 1):
                flush.fill_(rep)
                H = Hc if which == 0 else Hm
                H.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(s)
                if which == 0:
                    ptq.hessian_accumulate_conv(H, a, spec.kh, spec.kw, spec.stride, spec.pad, ws, st, s)
                else:
                    ptq.hessian_accumulate(H, X, ws, st, s)
                e1.record(s)
                torch.cuda.synchronize()
                if rep > 0:
                    (tc if which == 0 else tm).append(e0.elapsed_time(e1))
        ptq.check_status(st, spec.name)
        same = bool(torch.equal(Hc, Hm))
        row = {"layer": spec.name, "cols": spec.cols, "n": spec.n, "act_mb": a.numel() * 4 / 1e6,
               "x_mb": X.numel() * 4 / 1e6, "in_place_ms": float(np.median(tc)), "from_x_ms": float(np.median(tm)),
               "same": same}
        out.append(row)
        print(f"{spec.name:20s} {spec.cols:5d} {spec.n:6d} {row['act_mb']:7.1f} {row['x_mb']:7.1f} "
              f"{row['in_place_ms']:11.3f} {row['from_x_ms']:10.3f} {str(same):>6s}")
        del a, X, Hc, Hm
    print(json.dumps(out))
    return 0 if all(r["same"] for r in out) else 1


if __name__ == "__main__":
    raise SystemExit(main())
