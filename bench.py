#!/usr/bin/env python
"""Benchmark of the per-layer quantizer hot path on B200.

One "step" = one pass of the whole hot path over one synthetic layer: Hessian H = 2 X X^T, damped
inverse, grid, column scores + order, column-synchronous quantization sweep, codes / What / loss.
Workload at N = 1: the ResNet-50-shaped 3x3 convolution as a matrix (W 256 x 2304, X 2304 x 4096 with
30 % exact zeros, 4-bit per-row asymmetric grid, damping 0.01 * mean(diag H)).

`python bench.py [--gpus N] [--steps K] [--warmup W]` prints ONE JSON line (rank 0).  With N > 1 (torchrun)
every rank quantizes its own replica of the layer (the path is single-GPU: no collective on the data path);
`value` is the weights quantized per second by all ranks together, timed on the device, max over ranks.
`--impl reference` times the float64 CPU oracle on the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2509_05576_b200 import workloads as wl  # noqa: E402

METRIC = "weights quantized per second, whole per-layer path (ms_per_step = layer quantize time)"
UNIT = "weights/s"
FP64_PEAK_BOUND_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12  # stated upper bound: 148 SMs x 64 FP64 FMA / clk x 1965 MHz = 37.2
INT8_OVER_BF16 = 2.0                                   # nominal dense 4.5 / 2.25 PFLOP/s


# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised under
# profiles/, on the bench workload (Gram: scaled from the 16384-column capture by the calibration columns processed).
# Each entry names the kernel sources it was taken with; when they have changed since, the traffic is reported as null.
NCU_TRAFFIC = {
    "chol_coop": {"bytes_per_launch": (42.38e6 + 3.67e6 + 21.73e6 + 0.44e6) / 2, "sources": ["chol.cuh", "dgemm.cuh"],
                  "sha256_16": "26deddccb8d33464"},
    "sweep_coop": {"bytes_per_launch": 29.93e6 + 0.05e6, "sources": ["colloop.cuh"], "sha256_16": "dcc1e793b218823f"},
    "gram_i8_tcgen05": {"bytes_per_launch": (508.4e6 + 31.9e6) * 4096 / 16384, "sources": ["gram.cuh"],
                        "sha256_16": "67013082159ad65c"},
}


def ncu_traffic(kernel):
    import hashlib
    ent = NCU_TRAFFIC.get(kernel)
    if not ent:
        return None
    m = hashlib.sha256()
    for f in ent["sources"]:
        with open(os.path.join(ROOT, "paper_2509_05576_b200", "csrc", f), "rb") as fh:
            m.update(fh.read())
    return ent["bytes_per_launch"] if m.hexdigest()[:16] == ent["sha256_16"] else None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = str(gpu_index)
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.gpu, f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(value_ms, world, device):
    """Device time of a multi-rank run: the maximum over the ranks (every rank gets it)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value_ms)], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(weights_per_rank, world, ms_per_step):
    """Whole-job throughput of `world` independent replicas that each quantize `weights_per_rank` weights per step."""
    return world * weights_per_rank / (ms_per_step * 1e-3)


def bench_spec(rank=0):
    spec = wl.config2()[0]
    if rank:
        spec = wl.LayerSpec(spec.name, spec.rows, spec.cols, spec.n, spec.bits, spec.w_dist, spec.x_dist,
                            spec.seed + 100 * rank, spec.damp)
    return spec


def workload_config(spec, n_gpus):
    return {"workload": f"ResNet-50-shaped 3x3 conv as matrix: W {spec.rows}x{spec.cols} Kaiming-normal fp32, "
                        f"X {spec.cols}x{spec.n} half-normal with 30% exact zeros, {spec.bits}-bit per-row asymmetric "
                        f"min-max grid, damping {spec.damp}*mean(diag H), seed {spec.seed}",
            "rows": spec.rows, "cols": spec.cols, "n": spec.n, "bits": spec.bits,
            "l2": "L2 flushed (256 MiB write) before every timed step",
            "parallelism": "single GPU" if n_gpus == 1 else f"{n_gpus} independent replicas, one layer per GPU"}


# ------------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle as it stands
# ------------------------------------------------------------------------------------------------------
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    spec = bench_spec()
    W, X = wl.make_layer(spec)
    cores = oracle.num_threads()
    for _ in range(args.warmup):
        oracle.run_layer(W, X, spec.bits, spec.damp)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.run_layer(W, X, spec.bits, spec.damp)
    dt = (time.perf_counter() - t0) / args.steps
    value = spec.weights / dt
    sample = f"the whole {spec.rows}x{spec.cols} layer (N={spec.n}) per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": workload_config(spec, 1),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))
    return 0


# ------------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------------
def algorithmic_work(spec):
    """Algorithmic work of one step per kernel: (bound, flops or bytes).  MAC = 2 flops.

    tensor: int8 tensor pipe (Gram); alu: float64 pipe (factorisations, float64 MMA); hbm: bytes that must move."""
    r, c, n = spec.rows, spec.cols, spec.n
    return {
        "gram_i8_tcgen05": ("tensor", c * (c + 1) * n),            # symmetric half of 2 X X^T
        "gram_split": ("hbm", 4.0 * c * n + 6.0 * c * n),           # reads X once, writes six int8 planes
        # two launches: Cholesky of H + lambda I together with the inverse of its factor (c^3/3 + c^3/3, Sec. 5 item 1),
        # and the Cholesky of the permuted inverse Hessian (c^3/3, the blocked form of Eq. 12)
        "chol_coop": ("alu", 3 * (c ** 3 / 3.0)),
        "dgemm_lauum": ("alu", c ** 3 / 3.0),
        "dgemm_loss": ("alu", 1.0 * r * c * c),                     # H symmetric: half of the 2 r c^2 of the plain product
        # sweep: float64 W in and E out, codes out, the upper factor U once per 32-row group is NOT counted (L2)
        "sweep_coop": ("hbm", 8.0 * r * c + 8.0 * r * c + 1.0 * r * c + 8.0 * c * c / 2),
        "score_partial": ("hbm", 4.0 * r * c),
    }


def layer_set_totals(fp64_peak, flush, ws):
    """The configurations beyond the single bench layer, measured in this run: the ResNet-50-shaped set (4-bit), the
    YOLOv5s-shaped set (8- and 4-bit) and the scaling shapes at 3, 4 and 8 bits.  Per set: total ms, weights/s, per-stage
    ms and per-stage roofline fraction (sum of algorithmic work / sum of stage time / peak)."""
    import torch
    from paper_2509_05576_b200 import layer_set_run as lsr

    def brief(res, per_layer=False):
        out = {k: res[k] for k in ("n_layers", "weights", "total_ms", "weights_per_s", "graph_total_ms", "stage_total_ms",
                                   "stage_roofline_frac")}
        if per_layer:
            out["layers"] = [{"layer": r["layer"], "ms": r["ms"], "stages_ms": r["stages_ms"],
                              "roofline_frac": r["roofline_frac"]} for r in res["layers"]]
        return out

    sets = {}
    res3 = lsr.run_specs(wl.config3(), 2, fp64_peak=fp64_peak, ws=ws, flush=flush, graphs=True)
    sets["c3_resnet50_w4"] = brief(res3, per_layer=True)
    # the YOLOv5s-shaped layers at 8 and 4 bits share their inputs: run the two bit-widths of a layer back to back
    c4 = [s for pair in zip(wl.config4(bits=(8,)), wl.config4(bits=(4,))) for s in pair]
    res4 = lsr.run_specs(c4, 2, fp64_peak=fp64_peak, ws=ws, flush=flush, graphs=True)
    for b in (8, 4):
        rows = [r for r in res4["layers"] if r["bits"] == b]
        st = {}
        for r in rows:
            for k, v in r["stages_ms"].items():
                st[k] = st.get(k, 0.0) + v
        ms = sum(r["ms"] for r in rows)
        wts = sum(r["rows"] * r["cols"] for r in rows)
        sets[f"c4_yolov5s_w{b}"] = {"n_layers": len(rows), "weights": wts, "total_ms": ms,
                                    "weights_per_s": wts / (ms * 1e-3),
                                    "graph_total_ms": sum(r["graph_ms"] for r in rows), "stage_total_ms": st}
    sets["c4_yolov5s_w8"]["stage_roofline_frac_both_bit_widths"] = res4["stage_roofline_frac"]
    # Independent layers of a set overlapped on streams (the small layers leave most SMs idle on their own): four
    # streams as they come, and eight streams with the persistent cooperative kernels held to a quarter of the SMs each
    # (half for the wide layers), layers dealt longest first.  Same results either way (the sum of the losses is checked).
    def overlapped(specs, ref_loss):
        a4 = lsr.run_overlapped(specs, 4, 2, flush=flush)
        sms = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
        a8 = lsr.run_overlapped(specs, 8, 2, flush=flush, cta_limit=max(1, sms // 4))
        for a in (a4, a8):
            if abs(a["loss_sum"] - ref_loss) > 1e-9 * abs(ref_loss):
                raise RuntimeError("overlapped layer set: the losses differ from the one-stream run")
        return {"overlapped_4_streams_ms": a4["set_ms"], "overlapped_8_streams_cta_limited_ms": a8["set_ms"],
                "weights_per_s_overlapped": sum(sp.rows * sp.cols for sp in specs) / (a8["set_ms"] * 1e-3)}
    sets["c3_resnet50_w4"].update(overlapped(wl.config3(), sum(r["loss"] for r in res3["layers"])))
    for b in (8, 4):
        sets[f"c4_yolov5s_w{b}"].update(overlapped(wl.config4(bits=(b,)),
                                                   sum(r["loss"] for r in res4["layers"] if r["bits"] == b)))
    sets["c5_scaling_w3_w4_w8"] = brief(lsr.run_specs(wl.config5(), 2, fp64_peak=fp64_peak, ws=ws, flush=flush),
                                        per_layer=True)
    return sets


def kernel_rooflines(kernels, work, peaks):
    """Achieved rate of every kernel with a work model, against the peak of the unit that bounds it."""
    out = {}
    for name, (bound, amount) in work.items():
        k = kernels.get(name)
        if not k or k["ms_per_step"] <= 0:
            continue
        per_s = amount / (k["ms_per_step"] * 1e-3)
        if bound == "tensor":
            peak, unit, ach = peaks["bf16_tflops"] * INT8_OVER_BF16, "TFLOP/s", per_s / 1e12
            note = f"int8 dense = {peaks['source']} bf16 burst {peaks['bf16_tflops']} TF/s x nominal ratio 2"
        elif bound == "alu":
            peak, unit, ach = peaks["fp64_tflops"], "TFLOP/s", per_s / 1e12
            note = (f"float64 pipe, measured in this run by ptq_fp64_probe (FMA {peaks['fp64']['dfma_tflops']:.2f}, "
                    f"MMA {peaks['fp64']['dmma_tflops']:.2f} TFLOP/s); stated upper bound {FP64_PEAK_BOUND_TFLOPS:.2f}")
        else:
            peak, unit, ach = peaks["hbm_gbs"], "GB/s", per_s / 1e9
            note = f"{peaks['source']} copy bandwidth"
        out[name] = {"bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                     "ms_per_step": k["ms_per_step"], "launches_per_step": k["launches_per_step"], "peak_source": note}
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2509_05576_b200 import ptq
    import oracle

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the quantizer has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    ptq.lib()

    spec = bench_spec(rank)
    W, X = wl.make_layer(spec)
    Wd, Xd = torch.from_numpy(W).cuda(), torch.from_numpy(X).cuda()
    bufs = ptq.LayerBuffers(spec.rows, spec.cols)
    ws = ptq.Workspace()
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 * 2 ** 20, dtype=torch.uint8, device="cuda")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def step(events=None):
        ptq.quantize_layer_full(Wd, Xd, spec.bits, spec.damp, bufs=bufs, ws=ws, stream=stream, events=events)

    for _ in range(max(args.warmup, 3)):
        flush.fill_(1)
        step()
    torch.cuda.synchronize()
    ptq.check_status(bufs.status, "warm-up")

    # ---- timed region: K steps, device time by CUDA events on the launching stream, L2 flushed between steps
    sampler = ClockSampler(os.environ.get("CUDA_VISIBLE_DEVICES", str(local)).split(",")[0] if world == 1 else local)
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    launches0 = ptq.launch_count()
    barrier()
    sampler.start()
    for k in range(args.steps):
        flush.fill_(k & 0xFF)
        starts[k].record(stream)
        step()
        ends[k].record(stream)
    barrier()
    clocks = sampler.stop()
    launches = ptq.launch_count() - launches0
    ptq.check_status(bufs.status, "timed region")
    total_ms = max_over_ranks(sum(a.elapsed_time(b) for a, b in zip(starts, ends)), world, "cuda")
    ms_per_step = total_ms / args.steps
    value = aggregate_value(spec.weights, world, ms_per_step)

    # ---- per-stage times (events around each C-ABI call) and per-kernel times (library launch profiler)
    stage_ms = {}
    for _ in range(3):
        ev = []
        flush.fill_(3)
        step(ev)
        torch.cuda.synchronize()
        for name, a, b in ev:
            stage_ms.setdefault(name, []).append(a.elapsed_time(b))
    stage_ms = {k: float(np.median(v)) for k, v in stage_ms.items()}
    ptq.profile_enable(True)
    prof_steps = 3
    for _ in range(prof_steps):
        flush.fill_(5)
        step()
    torch.cuda.synchronize()
    prof = ptq.profile_read()
    ptq.profile_enable(False)
    kernels = {k: {"ms_per_step": ms / prof_steps, "launches_per_step": cnt // prof_steps} for k, (ms, cnt) in prof.items()}
    dominant = max(kernels, key=lambda k: kernels[k]["ms_per_step"])
    peaks = load_peaks()
    from paper_2509_05576_b200.layer_set_run import measure_fp64_peak
    peaks["fp64"] = measure_fp64_peak(stream)
    peaks["fp64_tflops"] = peaks["fp64"]["fp64_tflops"]
    work = algorithmic_work(spec)
    per_kernel = kernel_rooflines(kernels, work, peaks)
    traffic = ncu_traffic(dominant)
    dom = kernels[dominant]
    if dominant in per_kernel:
        pk = per_kernel[dominant]
        dom_launches = max(dom["launches_per_step"], 1)
        roofline = {"kernel": dominant, "bound": pk["bound"], "achieved": pk["achieved"], "peak": pk["peak"],
                    "unit": pk["unit"], "frac": pk["frac"], "traffic": traffic, "peak_source": pk["peak_source"],
                    "launch_ms": dom["ms_per_step"] / dom_launches, "launches_per_step": dom["launches_per_step"],
                    "algorithmic_work_per_launch": work[dominant][1] / dom_launches}
    else:
        roofline = {"kernel": dominant, "bound": "alu", "achieved": None, "peak": peaks["fp64_tflops"],
                    "unit": "TFLOP/s", "frac": None, "traffic": traffic}
    roofline["per_kernel"] = per_kernel
    gram = per_kernel.get("gram_i8_tcgen05")
    if gram:
        gram["issued"] = gram["achieved"] * 21          # 21 int8 slice-pair products per algorithmic product
        gram["frac_issued"] = gram["issued"] / gram["peak"]
    sw = kernels.get("sweep_coop")
    if sw:
        roofline["sweep_ns_per_column"] = sw["ms_per_step"] * 1e6 / spec.cols

    # ---- end to end through the C-ABI with HOST buffers: H2D of W and X, the path, D2H of codes and loss
    Wh = torch.from_numpy(W).pin_memory()
    n_batches = 4                                   # the calibration columns as four contiguous host batches
    cuts = [spec.n * i // n_batches for i in range(n_batches + 1)]
    Xh = [torch.from_numpy(np.ascontiguousarray(X[:, a:b])).pin_memory() for a, b in zip(cuts[:-1], cuts[1:])]
    codes_h = torch.empty((spec.rows, spec.cols), dtype=torch.uint8).pin_memory()
    loss_h = torch.empty(1, dtype=torch.float64).pin_memory()
    staging = ptq.HostStaging(spec.rows, spec.cols, [x.shape[1] for x in Xh])

    def e2e_step():
        # public entry point for host-resident layers: the calibration batches go up one by one on a copy stream while
        # the Hessian of the batches already there is accumulated; codes and loss come back at the end
        ptq.quantize_layer_from_host(Wh, Xh, spec.bits, spec.damp, bufs=bufs, ws=ws, staging=staging, stream=stream)
        codes_h.copy_(bufs.codes, non_blocking=True)
        loss_h.copy_(bufs.loss, non_blocking=True)

    for _ in range(2):
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2e_steps = max(3, min(args.steps, 10))
    e2e_ms = 0.0
    for k in range(e2e_steps):
        flush.fill_(k & 0xFF)
        e0.record(stream)
        e2e_step()
        e1.record(stream)
        torch.cuda.synchronize()
        e2e_ms += e0.elapsed_time(e1)
    barrier()
    e2e_ms = max_over_ranks(e2e_ms, world, "cuda")
    e2e_value = aggregate_value(spec.weights, world, e2e_ms / e2e_steps)
    e2e = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(W.nbytes + X.nbytes),
           "d2h_bytes_per_step": int(codes_h.numel() + 8), "ms_per_step": e2e_ms / e2e_steps}

    # ---- CPU baseline: the oracle as it stands, rank 0 at N = 1 only
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        t0 = time.perf_counter()
        ref = oracle.run_layer(W, X, spec.bits, spec.damp)
        dt = time.perf_counter() - t0
        cpu_baseline = {"value": spec.weights / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                        "sample": f"the whole {spec.rows}x{spec.cols} layer (N={spec.n}), one pass, {dt:.2f} s",
                        "codes_equal_to_gpu": bool(np.array_equal(ref["codes"], bufs.codes.cpu().numpy())),
                        "order_equal_to_gpu": bool(np.array_equal(ref["perm"], bufs.perm.cpu().numpy()))}

    # ---- the other configurations, measured in the same run (one GPU only)
    layer_sets = None
    if world == 1 and not args.no_sets:
        del Wd, Xd
        layer_sets = layer_set_totals(peaks["fp64_tflops"], flush, ws)
        if not args.no_cpu_baseline:
            # the oracle on a bounded sample of the ResNet-50-shaped set: every layer of at most 2304 columns (51 of the
            # 54; the three 512 x 4608 layers alone would take the oracle longer than all the others together)
            sample = [sp for sp in wl.config3() if sp.cols <= 2304]
            cpu_s = 0.0
            for sp in sample:
                Ws, Xs = wl.make_layer(sp)
                t0 = time.perf_counter()
                oracle.run_layer(Ws, Xs, sp.bits, sp.damp)
                cpu_s += time.perf_counter() - t0
            names = {sp.name for sp in sample}
            c3 = layer_sets["c3_resnet50_w4"]
            gpu_ms = sum(r["ms"] for r in c3["layers"] if r["layer"] in names)
            wts = sum(sp.weights for sp in sample)
            c3["cpu_baseline"] = {"value": wts / cpu_s, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                                  "sample": f"the {len(sample)} layers of the set with at most 2304 columns "
                                            f"({wts} weights), one pass each, {cpu_s:.1f} s",
                                  "gpu_ms_on_the_same_sample": gpu_ms}

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(spec, world), "clocks": clocks, "e2e": e2e,
            "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu_baseline,
            "stages_ms": stage_ms, "kernels": kernels, "fp64_peak": peaks["fp64"], "layer_sets": layer_sets,
            "context": "paper: ResNet-50 whole-model 80 s (FastOBQ) vs 9287 s (OBQ), hardware not stated"}))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sets", action="store_true", help="skip the layer-set totals (the single bench layer only)")
    args = ap.parse_args()
    if args.impl == "ours" and args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started plainly with --gpus N: become the launcher of N ranks, one per GPU
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(29500 + os.getpid() % 2000), os.path.abspath(__file__)]
        return subprocess.call(cmd + sys.argv[1:])
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
