"""The N > 1 path of the benchmark is "independent replicas": no data-path collective, only a barrier
and a max-over-ranks of the timings.  Its host logic runs here as two gloo ranks on CPU."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench

    local_ms = 100.0 + 50.0 * rank  # rank 1 is the slow replica
    dist.barrier()
    slowest = bench.max_over_ranks(local_ms, dist, torch.device("cpu"))
    value = bench.whole_job_value(20, world, slowest)
    out.put((rank, slowest, value))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_slowest_rank_and_summed_units():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, value in got:
        assert slowest == 150.0  # every rank sees the slowest rank's time
        assert abs(value - 2 * 20 / 0.150) < 1e-9  # both replicas' steps over that time


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(12.5, None, torch.device("cpu")) == 12.5
    assert bench.whole_job_value(10, 1, 5.0) == 2000.0
    assert bench.step_bytes(8, 60965224, 952583) == 12 * 8 * 60965224 + 8 * 60965224 + 16 * 8 * 952583 + 8 * 952583


# ---------------------------------------------------------------- workers spread over ranks (ShardedPruner)


class _NumpyEngine:
    """Test double for the per-rank CUDA engine: the four calls ShardedPruner makes, on CPU tensors, in plain
    numpy.  It lets the orchestration (who owns the chosen worker, what is broadcast, in which order the
    gathered values are summed) run as real gloo ranks; the CUDA engine itself is checked on the GPU."""

    def __init__(self, layer_sizes, W, ratio, eps):
        import math

        import numpy as np

        self.np = np
        self.n = list(layer_sizes)
        self.W, self.N = W, sum(self.n)
        self.k = [min(n, max(1, math.ceil(n / ratio))) for n in self.n]
        self.K = sum(self.k)
        self.eps = np.float32(eps)
        self.acc = np.zeros((W, self.N), np.float32)
        self.lists = None

    def shard_select(self, grads, weights, update):
        np = self.np
        self.acc = (self.acc + grads.numpy().reshape(self.W, self.N)).astype(np.float32)
        update.zero_()
        den = (np.abs(weights.numpy()) + self.eps).astype(np.float32)
        self.lists = []
        for w in range(self.W):
            key = (np.abs(self.acc[w]) / den).astype(np.float32).view(np.uint32).astype(np.int64)
            out, o = [], 0
            for n, k in zip(self.n, self.k):
                order = np.lexsort((np.arange(n), -key[o:o + n]))  # importance descending, index ascending
                out.append(np.sort(order[:k]) + o)
                o += n
            self.lists.append(np.concatenate(out))

    def selection(self, w):
        idx = self.lists[w]
        return torch.from_numpy(idx.astype(self.np.int32)), torch.from_numpy(self.acc[w, idx].copy())

    def shard_gather(self, idx):
        return torch.from_numpy(self.np.ascontiguousarray(self.acc[:, idx.numpy()]))

    def wire_pack(self, idx):
        np = self.np
        m = np.zeros(32 * ((self.N + 31) // 32), np.uint8)
        m[idx.numpy()] = 1
        return torch.from_numpy(np.packbits(m, bitorder="little"))

    def wire_unpack(self, bits, n):
        np = self.np
        idx = np.flatnonzero(np.unpackbits(bits.numpy(), bitorder="little"))
        assert idx.size == n
        return torch.from_numpy(idx.astype(np.int32))

    def shard_apply(self, idx, vals_all, update):
        np = self.np
        v = vals_all.numpy()
        s = v[0].copy()
        for w in range(1, v.shape[0]):
            s = (s + v[w]).astype(np.float32)
        update[idx.long()] = torch.from_numpy((np.float32(0) + s).astype(np.float32))
        self.acc[:, idx.numpy()] = 0

    def close(self):
        pass


def _sharded_rank_main(rank: int, world: int, port: int, out, wire="auto", ratio=8.0):
    import numpy as np

    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_1901_01544_b200.binding import ShardedPruner

    layers, W_total, eps, seed = [300, 17, 1000], 4, 1e-8, 5
    N, Wl = sum(layers), W_total // world
    sp = ShardedPruner(layers, W_total, ratio, eps, seed, engine=_NumpyEngine(layers, Wl, ratio, eps), wire=wire)
    orc = oracle.Oracle(layers, W_total, ratio, eps, seed)  # the whole job on one "node"
    rng = np.random.default_rng(3)  # the same stream on every rank
    weights = rng.standard_normal(N).astype(np.float32)
    ok, owners = True, set()
    for t in range(6):
        grads = rng.standard_normal((W_total, N)).astype(np.float32)
        want = orc.step(grads, weights)
        upd = torch.full((N,), float("nan"))
        sp.step(torch.from_numpy(grads[rank * Wl:(rank + 1) * Wl].copy()), torch.from_numpy(weights), upd)
        ok = ok and sp.leader == orc.leader and np.array_equal(upd.numpy().view(np.uint32), want.view(np.uint32))
        for w in range(Wl):
            ok = ok and np.array_equal(sp.local.acc[w].view(np.uint32), orc.residual(rank * Wl + w).view(np.uint32))
        owners.add(sp.leader // Wl)
    out.put((rank, bool(ok), sorted(owners), sp.last_wire, sp.wire_bytes))
    dist.barrier()
    dist.destroy_process_group()


# wire, ratio -> what must have travelled: at ratio 8 the mask (N / 8 bytes) is shorter than the list (N / 2
# bytes), at ratio 64 the list is
@pytest.mark.parametrize("wire,ratio,expect", [("auto", 8.0, "mask"), ("auto", 64.0, "list"), ("list", 8.0, "list"),
                                               ("mask", 64.0, "mask")])
def test_workers_spread_over_two_ranks_equal_one_node(wire, ratio, expect):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_sharded_rank_main, args=(r, 2, port, out, wire, ratio)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [True, True]
    assert got[0][2] == [0, 1]  # the chosen worker lived on either rank at some step
    assert [g[3] for g in got] == [expect, expect]
    N, K = 1317, sum(min(n, max(1, -(-n // int(ratio)))) for n in (300, 17, 1000))
    assert got[0][4] == (4 * ((N + 31) // 32) if expect == "mask" else 4 * K)


def _sharded_bad_split_main(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_1901_01544_b200.binding import ShardedPruner

    try:
        ShardedPruner([100], 3, 4.0, engine=_NumpyEngine([100], 1, 4.0, 1e-8))  # three workers over two ranks
        out.put((rank, "accepted"))
    except ValueError:
        out.put((rank, "rejected"))
    dist.barrier()
    dist.destroy_process_group()


def test_sharding_needs_the_workers_to_divide_over_the_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_sharded_bad_split_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, "rejected"), (1, "rejected")]
