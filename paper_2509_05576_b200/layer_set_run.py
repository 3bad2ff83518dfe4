"""Quantizes a whole synthetic layer set, layer by layer, on one GPU and reports per-layer and per-stage device time.

    python -m paper_2509_05576_b200.layer_set_run --config 3            # the 54 ResNet-50-shaped layers, 4-bit
    python -m paper_2509_05576_b200.layer_set_run --config 4 --bits 8   # the YOLOv5s-shaped stack
    python -m paper_2509_05576_b200.layer_set_run --config 5 --bits 4   # square / wide scaling shapes
    python -m paper_2509_05576_b200.layer_set_run --config 6            # ResNet-18-shaped (7: ResNet-34-shaped)
    python -m paper_2509_05576_b200.layer_set_run --config 3 --score-mode none   # the ordering ablation (Sec. 6)

Every layer goes through the five C-ABI calls (Hessian, damped inverse, grid, scores + order, sweep); each call is
bracketed by CUDA events on the launching stream, an L2-sized buffer is rewritten before every timed repetition.
Stage rooflines use the algorithmic work of the stage (MAC = 2 flops): Gram cols (cols + 1) n on the int8 tensor
pipe, inverse cols^3 (Cholesky + triangular inverse + V V^T) and sweep 4/3 cols^3 / 4 + ... on the float64 pipe --
see ``stage_work``.  Prints a table and one JSON line with the set totals.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch

from . import ptq
from . import workloads as wl

FP64_PEAK_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12      # stated upper bound: 148 SMs x 64 FP64 FMA / clk x 2 x 1.965 GHz
SCORE_MODES = {"qerr": ptq.SCORE_QERR, "prune": ptq.SCORE_PRUNE, "err": ptq.SCORE_ERR, "w": ptq.SCORE_W,
               "none": ptq.SCORE_NONE}
INT8_OVER_BF16 = 2.0


def _peaks():
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p["hbm_gbs"], p["bf16_tflops"], "measured"
    return 6650.0, 1590.0, "fallback"


def measure_fp64_peak(stream=None):
    """Float64 throughput of this GPU, measured with the library's probe kernels (eight independent chains of FMAs, or
    of tensor-core m8n8k4 MMAs, per thread and nothing else): best of five launches of each kind, timed with CUDA
    events on the launching stream after two warm-up launches."""
    stream = stream or torch.cuda.current_stream()
    sink = torch.zeros(1, dtype=torch.float64, device="cuda")
    out = {}
    for kind, name, iters in ((0, "dfma", 100000), (1, "dmma", 20000)):
        best = 0.0
        for rep in range(7):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            flops = ptq.fp64_probe(kind, iters, sink, stream)
            b.record(stream)
            torch.cuda.synchronize()
            if rep >= 2:
                best = max(best, flops / (a.elapsed_time(b) * 1e-3) / 1e12)
        out[name + "_tflops"] = best
    out["fp64_tflops"] = max(out["dfma_tflops"], out["dmma_tflops"])
    out["bound_tflops"] = FP64_PEAK_TFLOPS
    out["how"] = ("ptq_fp64_probe: 4 CTAs x 256 threads per SM, 8 independent chains per thread, 100000 (FMA) / 20000 (MMA) "
                  "rounds, best of 5 launches, CUDA events; bound = 148 SMs x 64 FMA/clk x 2 x 1.965 GHz")
    return out


def stage_work(spec):
    """Algorithmic flops per stage (MAC = 2 flops)."""
    r, c, n = spec.rows, spec.cols, spec.n
    return {
        "hessian": float(c) * (c + 1) * n,                 # symmetric half of 2 X X^T
        "inverse": float(c) ** 3,                          # Cholesky c^3/3 + triangular inverse c^3/3 + V V^T c^3/3
        "sweep": float(c) ** 3 / 3 + float(r) * c * c + 2.0 * r * c * c,   # Cholesky of the permuted inverse, Eq. 11, loss
    }


def run_specs(specs, reps=2, score_mode=ptq.SCORE_QERR, quiet=True, fp64_peak=FP64_PEAK_TFLOPS, ws=None, flush=None,
              graphs=False):
    """Quantizes the given layers one after the other on the current stream and times every C-ABI call with CUDA
    events (L2 flushed before every timed repetition, median over the repetitions).  Consecutive specs that describe
    the same seeded layer at another bit-width reuse its inputs.  Returns the per-layer records, the set totals, the
    per-stage totals and the per-stage roofline fractions of the whole set (sum of work / sum of time / peak).
    graphs=True also captures every layer's path as a CUDA graph and times its replay (``graph_ms`` per layer,
    ``graph_total_ms`` for the set): what a caller gets who does not issue the launches one by one."""
    hbm, bf16, src = _peaks()
    int8_peak = bf16 * INT8_OVER_BF16
    s = torch.cuda.current_stream()
    flush = flush if flush is not None else torch.empty(256 * 2 ** 20, dtype=torch.uint8, device="cuda")
    ws = ws or ptq.Workspace()
    rows_out = []
    totals = {"weights": 0, "ms": 0.0, "loss": 0.0}
    stage_tot, work_tot = {}, {}
    if not quiet:
        print(f"{'layer':28s} {'rows':>5s} {'cols':>6s} {'n':>5s} {'b':>2s} {'total ms':>9s} {'Mw/s':>8s} "
              f"{'hess':>7s} {'inv':>7s} {'order':>6s} {'sweep':>7s} {'%int8':>6s} {'%f64 inv':>8s} {'%f64 swp':>8s} {'loss':>12s}")
    key, Wd, Xd, bufs = None, None, None, None
    for spec in specs:
        k = (spec.rows, spec.cols, spec.n, spec.w_dist, spec.x_dist, spec.seed)
        if k != key:
            Wd = Xd = bufs = None
            W, X = wl.make_layer(spec)
            Wd, Xd = torch.from_numpy(W).cuda(), torch.from_numpy(X).cuda()
            bufs = ptq.LayerBuffers(spec.rows, spec.cols)
            key = k
        ptq.quantize_layer_full(Wd, Xd, spec.bits, spec.damp, score_mode=score_mode, bufs=bufs, ws=ws, stream=s)    # warm-up
        torch.cuda.synchronize()
        ptq.check_status(bufs.status, spec.name)
        per = {}
        for rep in range(reps):
            flush.fill_(rep)
            ev = []
            ptq.quantize_layer_full(Wd, Xd, spec.bits, spec.damp, score_mode=score_mode, bufs=bufs, ws=ws, stream=s, events=ev)
            torch.cuda.synchronize()
            for name, a, b in ev:
                per.setdefault(name, []).append(a.elapsed_time(b))
        ptq.check_status(bufs.status, spec.name)
        st = {k2: float(np.median(v)) for k2, v in per.items()}
        total = sum(st.values())
        work = stage_work(spec)
        frac = {"hessian": work["hessian"] / (st["hessian"] * 1e-3) / 1e12 / int8_peak,
                "inverse": work["inverse"] / (st["inverse"] * 1e-3) / 1e12 / fp64_peak,
                "sweep": work["sweep"] / (st["sweep"] * 1e-3) / 1e12 / fp64_peak}
        loss = float(bufs.loss.item())
        graph_ms = None
        if graphs:
            lg = ptq.LayerGraph(Wd, Xd, spec.bits, spec.damp, score_mode=score_mode, bufs=bufs, ws=ws)
            ts = []
            for rep in range(reps + 1):
                flush.fill_(rep)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(s)
                lg.replay()
                b.record(s)
                torch.cuda.synchronize()
                if rep:
                    ts.append(a.elapsed_time(b))
            ptq.check_status(bufs.status, spec.name + " (graph)")
            graph_ms = float(np.median(ts))
            del lg
        if not quiet:
            print(f"{spec.name:28s} {spec.rows:5d} {spec.cols:6d} {spec.n:5d} {spec.bits:2d} {total:9.3f} "
                  f"{spec.weights / total / 1e3:8.1f} {st['hessian']:7.3f} {st['inverse']:7.3f} "
                  f"{st['grid'] + st['order']:6.3f} {st['sweep']:7.3f} {100 * frac['hessian']:6.2f} "
                  f"{100 * frac['inverse']:8.2f} {100 * frac['sweep']:8.2f} {loss:12.5g}")
        rows_out.append({"layer": spec.name, "rows": spec.rows, "cols": spec.cols, "n": spec.n, "bits": spec.bits,
                         "ms": total, "stages_ms": st, "roofline_frac": frac, "loss": loss, "graph_ms": graph_ms})
        totals["weights"] += spec.weights
        totals["ms"] += total
        totals["loss"] += loss
        for k2, v in st.items():
            stage_tot[k2] = stage_tot.get(k2, 0.0) + v
        for k2, v in work.items():
            work_tot[k2] = work_tot.get(k2, 0.0) + v
    stage_frac = {"hessian": work_tot["hessian"] / (stage_tot["hessian"] * 1e-3) / 1e12 / int8_peak,
                  "inverse": work_tot["inverse"] / (stage_tot["inverse"] * 1e-3) / 1e12 / fp64_peak,
                  "sweep": work_tot["sweep"] / (stage_tot["sweep"] * 1e-3) / 1e12 / fp64_peak}
    graph_total = sum(r["graph_ms"] for r in rows_out) if graphs else None
    return {"layers": rows_out, "n_layers": len(rows_out), "weights": totals["weights"], "total_ms": totals["ms"],
            "graph_total_ms": graph_total,
            "weights_per_s": totals["weights"] / (totals["ms"] * 1e-3), "loss_sum": totals["loss"],
            "stage_total_ms": stage_tot, "stage_roofline_frac": stage_frac,
            "peaks": {"hbm_gbs": hbm, "int8_tflops": int8_peak, "fp64_tflops": fp64_peak, "source": src}}


def run_overlapped(specs, n_streams, reps=2, score_mode=ptq.SCORE_QERR, flush=None, cta_limit=0):
    """The whole set through ``ptq.LayerSet``: independent layers side by side on `n_streams` streams, the inputs of all
    layers put on the device first, one event pair around the whole set (median of `reps` timed passes after one warm-up
    pass).  cta_limit 0: layers dealt round-robin, cooperative kernels with one CTA per SM; > 0: see ``ptq.LayerSet``."""
    s = torch.cuda.current_stream()
    flush = flush if flush is not None else torch.empty(256 * 2 ** 20, dtype=torch.uint8, device="cuda")
    layers = []
    for spec in specs:
        W, X = wl.make_layer(spec)
        layers.append((torch.from_numpy(W).cuda(), torch.from_numpy(X).cuda(), spec.bits, spec.damp))
    ls = ptq.LayerSet(layers, n_streams, cta_limit, score_mode)
    times = []
    for rep in range(reps + 1):
        torch.cuda.synchronize()
        flush.fill_(rep)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s)
        outs = ls.run()
        e1.record(s)
        torch.cuda.synchronize()
        if rep > 0:
            times.append(e0.elapsed_time(e1))
    for o, spec in zip(outs, specs):
        ptq.check_status(o.status, spec.name)
    return {"streams": n_streams, "cta_limit": cta_limit, "set_ms": float(np.median(times)),
            "loss_sum": float(sum(o.loss.item() for o in outs))}


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=3, choices=[1, 2, 3, 4, 5, 6, 7])
    ap.add_argument("--bits", type=int, default=None, help="bit-width filter for configs 4 and 5")
    ap.add_argument("--reps", type=int, default=2)
    ap.add_argument("--limit", type=int, default=0, help="only the first LIMIT layers (0: all)")
    ap.add_argument("--max-cols", type=int, default=0, help="skip layers with more columns (0: none)")
    ap.add_argument("--streams", type=int, default=1,
                    help="> 1: also run the whole set with the layers dealt round-robin onto this many streams "
                         "(inputs resident, nothing synchronised in between) and report the wall time of that")
    ap.add_argument("--cta-limit", type=int, default=0,
                    help="with --streams: at most this many CTAs per persistent cooperative kernel (0: one per SM)")
    ap.add_argument("--score-mode", default="qerr", choices=sorted(SCORE_MODES),
                    help="column ordering: qerr (Eq. 10, the method's), prune (Eq. 8), err, w, none (no sorting)")
    ap.add_argument("--ascending", action="store_true", help="sort the scores ascending (the 'asc' keys of Sec. 4.1)")
    ap.add_argument("--graphs", action="store_true", help="also time every layer's path replayed as one CUDA graph")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise RuntimeError("layer_set_run needs a CUDA device")
    if args.config == 4:
        specs = wl.config4(bits=(args.bits,) if args.bits else (8, 4))
    elif args.config == 5:
        specs = wl.config5(bits=(args.bits,) if args.bits else (3, 4, 8))
    else:
        specs = wl.CONFIGS[args.config]()
    if args.max_cols:
        specs = [s for s in specs if s.cols <= args.max_cols]
    if args.limit:
        specs = specs[:args.limit]
    s = torch.cuda.current_stream()
    flush = torch.empty(256 * 2 ** 20, dtype=torch.uint8, device="cuda")
    mode = SCORE_MODES[args.score_mode] | (ptq.SCORE_ASCENDING if args.ascending else 0)
    fp64 = measure_fp64_peak(s)
    res = run_specs(specs, args.reps, mode, quiet=False, flush=flush, graphs=args.graphs, fp64_peak=fp64["fp64_tflops"])
    res["peaks"]["fp64_measured"] = fp64
    totals = {"ms": res["total_ms"]}
    overlapped = None
    if args.streams > 1:
        overlapped = run_overlapped(specs, args.streams, args.reps, mode, flush, args.cta_limit)
        print(f"whole set on {args.streams} streams: {overlapped['set_ms']:.2f} ms "
              f"(sum of the per-layer times on one stream: {totals['ms']:.2f} ms)")
    print(json.dumps({"config": args.config, "score_mode": args.score_mode, "ascending": bool(args.ascending),
                      "loss_sum": res["loss_sum"], "overlapped": overlapped,
                      "layers": res["n_layers"], "weights": res["weights"],
                      "total_ms": res["total_ms"], "weights_per_s": res["weights_per_s"],
                      "graph_total_ms": res["graph_total_ms"],
                      "stage_total_ms": res["stage_total_ms"], "stage_roofline_frac": res["stage_roofline_frac"],
                      "peaks": res["peaks"]}))
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
