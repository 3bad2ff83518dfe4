"""Host-side logic of the multi-GPU bench (N independent replicas, one layer per rank, no collective on the data
path): per-rank seeds, max-over-ranks timing and whole-job throughput, run as two gloo ranks on the CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        spec = bench.bench_spec(rank)
        my_ms = 10.0 + 5.0 * rank                       # rank 1 is the slower replica
        ms = bench.max_over_ranks(my_ms, world, "cpu")
        value = bench.aggregate_value(spec.weights, world, ms)
        out.put((rank, spec.seed, ms, value))
    finally:
        dist.destroy_process_group()


def test_two_replicas_take_the_slowest_rank_and_add_the_work():
    import bench
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    weights = bench.bench_spec(0).weights
    assert [g[1] for g in got] == [bench.bench_spec(0).seed, bench.bench_spec(0).seed + 100]   # different layers per rank
    for _, _, ms, value in got:
        assert ms == 15.0                                # the maximum over the ranks, on every rank
        assert value == world * weights / 15.0e-3


def test_reference_arm_runs_on_rank_zero_only(monkeypatch):
    import bench

    class Args:
        gpus, steps, warmup = 2, 1, 0
    monkeypatch.setenv("RANK", "1")
    assert bench.run_reference(Args()) == 0              # other ranks return at once, without work or output
