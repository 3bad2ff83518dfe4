"""Host logic of the multi-GPU sharding of one layer (calibration columns and weight rows split over the ranks; an
all-reduce of H, an all-reduce of the column scores, a sum of the loss), run as gloo ranks on the CPU.

The per-rank compute steps are injected: here they are the CPU oracle's functions on host tensors, so that what is
under test is the sharding itself -- the partition, which quantity is exchanged where, and that every rank ends up
with the same column order.  The result must equal the oracle's on the undivided layer."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2509_05576_b200 import sharded  # noqa: E402
from paper_2509_05576_b200 import workloads as wl  # noqa: E402


def test_split_range_tiles_the_range_in_rank_order():
    for total in (0, 1, 5, 64, 1000):
        for world in (1, 2, 3, 8):
            parts = [sharded.split_range(total, world, r) for r in range(world)]
            assert parts[0][0] == 0 and parts[-1][1] == total
            for (a0, a1), (b0, b1) in zip(parts[:-1], parts[1:]):
                assert a1 == b0 and a0 <= a1
            sizes = [b - a for a, b in parts]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        sharded.split_range(10, 2, 2)


class OracleOps:
    """The per-rank steps computed by the CPU oracle on host tensors (test stand-in for the CUDA library)."""

    def __init__(self):
        import oracle
        self.o = oracle

    def hessian(self, X, cols):
        H = np.zeros((cols, cols))
        if X is not None and X.shape[1] > 0:
            H = self.o.hessian_accumulate(X.numpy())
        return torch.from_numpy(H)

    def prepare_hinv(self, H, damp, damp_mode):
        Hinv, diag, lam = self.o.prepare_hinv(H.numpy(), damp, damp_mode)
        return torch.from_numpy(Hinv), torch.from_numpy(diag), torch.tensor([lam], dtype=torch.float64)

    def grid(self, W, bits):
        if W.shape[0] == 0:
            return torch.empty(0), torch.empty(0)
        s, z = self.o.minmax_grid(W.numpy(), bits)
        return torch.from_numpy(s), torch.from_numpy(z)

    def scores(self, W, diag, scale, zero, bits, mode):
        if W.shape[0] == 0:
            return torch.zeros(W.shape[1], dtype=torch.float64)
        S, _ = self.o.sensitivity_order(W.numpy(), diag.numpy(), scale.numpy(), zero.numpy(), bits, mode)
        return torch.from_numpy(S)

    def sort(self, S, ascending):
        Sn = S.numpy()
        order = sorted(range(len(Sn)), key=lambda j: ((Sn[j] if ascending else -Sn[j]), j))
        return torch.tensor(order, dtype=torch.int32)

    def sweep(self, W, Hinv, perm, scale, zero, bits, H):
        rows, cols = W.shape
        if rows == 0:
            return (torch.empty((0, cols), dtype=torch.uint8), torch.empty((0, cols)),
                    torch.zeros(1, dtype=torch.float64))
        out = self.o.quantize_layer(W.numpy(), Hinv.numpy(), perm.numpy(), scale.numpy(), zero.numpy(), bits,
                                    H_undamped=H.numpy())
        return (torch.from_numpy(out["codes"]), torch.from_numpy(out["What"]),
                torch.tensor([out["loss"]], dtype=torch.float64))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


SPEC = wl.LayerSpec("shard", 37, 45, 96, 4, "kaiming", "halfnormal", 8800)


def _rank_main(rank, world, port, out, score_mode):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        W, X = wl.make_layer(SPEC)
        r0, r1 = sharded.split_range(SPEC.rows, world, rank)
        c0, c1 = sharded.split_range(SPEC.n, world, rank)
        res = sharded.quantize_layer_sharded(torch.from_numpy(W[r0:r1].copy()), torch.from_numpy(X[:, c0:c1].copy()),
                                             SPEC.cols, SPEC.bits, SPEC.damp, 0, score_mode, ops=OracleOps())
        out.put((rank, r0, r1, res["codes"].numpy(), res["What"].numpy(), res["perm"].numpy(), res["S"].numpy(),
                 res["H"].numpy(), float(res["loss"].item())))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,score_mode", [(2, 0), (3, 1 | 16)])
def test_sharded_layer_equals_the_undivided_layer(world, score_mode):
    import oracle
    port = _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out, score_mode)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted((out.get(timeout=180) for _ in range(world)), key=lambda g: g[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    W, X = wl.make_layer(SPEC)
    ref = oracle.run_layer(W, X, SPEC.bits, SPEC.damp, score_mode=score_mode)
    for rank, r0, r1, codes, What, perm, S, H, loss in got:
        assert np.array_equal(perm, ref["perm"])                     # every rank holds the whole layer's order
        assert np.allclose(S, ref["S"], rtol=1e-12, atol=0)
        assert np.max(np.abs(H - ref["H"])) <= 1e-12 * np.max(np.abs(ref["H"]))
        assert np.array_equal(codes, ref["codes"][r0:r1])            # and its own rows of the result
        assert np.array_equal(What, ref["What"][r0:r1])
        assert abs(loss - ref["loss"]) <= 1e-10 * ref["loss"]        # the whole layer's loss, on every rank
    assert [(g[1], g[2]) for g in got] == [sharded.split_range(SPEC.rows, world, r) for r in range(world)]
