"""Workers spread over several contexts (iwp_shard_select / iwp_shard_gather / iwp_shard_apply): parity with
the CPU oracle of the WHOLE job, bit for bit.  One GPU stands in for the ranks: the contexts run their phases
one after the other in one process and the two collectives are plain copies (nothing here waits on another
kernel); the transport itself runs as real ranks over gloo in tests/test_multirank_cpu.py and as a
one-rank NCCL group below."""
import os
import socket

import numpy as np
import pytest
import torch

import oracle
from paper_1901_01544_b200.binding import Pruner, ShardedPruner
from parity import assert_bits_equal

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _randn(shape, seed, scale=1.0):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return torch.randn(shape, generator=g, device=DEV, dtype=torch.float32) * scale


def _run_groups(sizes, W_total, groups, ratio, seed, steps, grads_fn, weights, options=None, wire="list"):
    N, Wl = sum(sizes), W_total // groups
    ctxs = [Pruner(sizes, Wl, ratio, 1e-8, seed) for _ in range(groups)]
    for c in ctxs:
        for k, v in (options or {}).items():
            c.set_option(k, v)
    orc = oracle.Oracle(sizes, W_total, ratio, 1e-8, seed)
    w_host = weights.cpu().numpy()
    upds = [torch.full((N,), float("nan"), device=DEV) for _ in range(groups)]
    for t in range(steps):
        g = grads_fn(t)
        want = orc.step(np.ascontiguousarray(g.cpu().numpy()), w_host)
        for r, c in enumerate(ctxs):
            c.shard_select(g[r * Wl:(r + 1) * Wl].contiguous(), weights, upds[r])
        owner, lw = divmod(orc.leader, Wl)
        assert orc.leader == oracle.leader(seed, t, W_total)
        idx = ctxs[owner].selection(lw)[0]                                # "broadcast"
        idx_at = [idx] * groups
        if wire == "mask":  # the encoded mask travels: packed on the owner, expanded by every other group
            bits = ctxs[owner].wire_pack(idx)
            idx_at = [idx if r == owner else c.wire_unpack(bits.clone(), idx.numel()) for r, c in enumerate(ctxs)]
            for r in range(groups):
                assert torch.equal(idx_at[r], idx), f"step {t}: group {r} expanded a different index list"
        vals_all = torch.cat([c.shard_gather(idx_at[r]) for r, c in enumerate(ctxs)], dim=0)  # "all-gather", worker order
        for r, c in enumerate(ctxs):
            c.shard_apply(idx_at[r], vals_all, upds[r])
        for r, c in enumerate(ctxs):
            assert c.sync_status() == 0 and c.t == t + 1
            assert_bits_equal(upds[r].cpu().numpy(), want, f"step {t}: update of group {r}")
            for w in range(Wl):
                gi, gv = c.selection(w)
                oi, ov = orc.selection(r * Wl + w)
                assert np.array_equal(gi.cpu().numpy().view(np.uint32), oi), f"step {t}: worker {r * Wl + w} list"
                assert_bits_equal(gv.cpu().numpy(), ov, f"step {t}: worker {r * Wl + w} list values")
                assert_bits_equal(c.residual(w).cpu().numpy(), orc.residual(r * Wl + w), f"step {t}: worker {r * Wl + w} residual")
            upds[r].fill_(float("nan"))
    for c in ctxs:
        c.close()
    orc.close()


@pytest.mark.parametrize("speculate", [1, 0])
@pytest.mark.parametrize("groups", [1, 2, 4])
def test_groups_of_workers_equal_the_whole_job(groups, speculate):
    sizes, W, ratio = [70000, 64, 16385, 300000, 9, 40000], 4, 32.0
    N = sum(sizes)
    weights = _randn((N,), 1, 0.05)
    weights[::53] = 0.0
    _run_groups(sizes, W, groups, ratio, 3, 4, lambda t: _randn((W, N), 900 + t), weights, {"speculate": speculate})


def test_groups_with_the_mask_as_wire_format():
    sizes, W, ratio = [70000, 64, 16385, 300001, 9, 40000], 4, 8.0  # N not a multiple of 32
    N = sum(sizes)
    weights = _randn((N,), 1, 0.05)
    _run_groups(sizes, W, 2, ratio, 3, 3, lambda t: _randn((W, N), 900 + t), weights, wire="mask")


@pytest.mark.parametrize("N,count", [(1, 1), (31, 0), (32, 32), (33, 5), (100003, 1563), (100003, 100003),
                                     (3 * 256 * 4 * 32 + 77, 50000)])
def test_wire_pack_and_unpack_against_numpy(N, count):
    pr = Pruner([N], 1, 2.0, 1e-8, 0)
    rng = np.random.default_rng(N + count)
    want = np.sort(rng.choice(N, size=count, replace=False)).astype(np.uint32)
    shuffled = rng.permutation(want)  # the pack takes any order
    bits = pr.wire_pack(torch.from_numpy(shuffled.view(np.int32)).to(DEV))
    ref = np.zeros(32 * ((N + 31) // 32), np.uint8)
    ref[want] = 1
    assert np.array_equal(bits.cpu().numpy(), np.packbits(ref, bitorder="little"))  # bit i % 8 of byte i / 8
    got = pr.wire_unpack(bits, count)
    assert np.array_equal(got.cpu().numpy().view(np.uint32), want)
    assert pr.sync_status() == 0
    pr.close()


def test_wire_format_error_reports():
    from paper_1901_01544_b200 import binding

    N = 5000
    pr = Pruner([N], 1, 2.0, 1e-8, 0)
    idx = torch.arange(0, 100, dtype=torch.int32, device=DEV)
    bits = pr.wire_pack(idx)
    short = pr.wire_unpack(bits, 60)  # fewer places than set bits: the surplus is dropped and reported
    assert np.array_equal(short.cpu().numpy(), np.arange(60))
    assert pr.sync_status() == binding.IWP_ERR_CAPACITY
    pr.reset()
    pr.wire_pack(torch.tensor([3, N, 7], dtype=torch.int32, device=DEV))  # N is not an element
    assert pr.sync_status() == binding.IWP_ERR_INTERNAL
    assert binding.iwp_wire_mask_bytes(N) == 4 * ((N + 31) // 32) and binding.iwp_wire_mask_bytes(0) == 0
    pr.close()


def test_groups_with_ties_and_fallbacks():
    sizes, W, ratio = [70000, 300, 20000], 6, 16.0
    N = sum(sizes)
    g0 = torch.Generator(device=DEV)
    g0.manual_seed(7)
    weights = torch.randint(-3, 4, (N,), generator=g0, device=DEV).float() * 0.25

    def grads(t):
        gg = torch.Generator(device=DEV)
        gg.manual_seed(950 + t)
        if t % 2:
            return torch.randint(-4, 5, (W, N), generator=gg, device=DEV).float() / 8.0
        return torch.randn((W, N), generator=gg, device=DEV) * 1e-3

    _run_groups(sizes, W, 3, ratio, 4, 5, grads, weights)


def test_sharded_argument_checks():
    pr = Pruner([5000], 2, 4.0, 1e-8, 0)
    idx = torch.zeros(4, dtype=torch.int32, device=DEV)
    vals = torch.zeros((1, 4), device=DEV)
    upd = torch.zeros(5000, device=DEV)
    from paper_1901_01544_b200 import binding

    with pytest.raises(binding.IwpError):
        pr.shard_apply(idx, vals, upd)  # fewer rows than this context has workers
    thr = Pruner([5000], 2, None, 1e-8, 0, thresholds=[1.0])
    with pytest.raises(binding.IwpError):
        thr.shard_select(torch.zeros((2, 5000), device=DEV), torch.ones(5000, device=DEV), upd)  # ratio mode only
    thr.close()
    pr.close()


@pytest.mark.parametrize("wire", ["list", "mask"])
def test_sharded_pruner_over_a_one_rank_nccl_group(wire):
    import torch.distributed as dist

    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        sizes, W, ratio, seed = [70000, 64, 30000], 4, 16.0, 9
        N = sum(sizes)
        weights = _randn((N,), 2, 0.05)
        sp = ShardedPruner(sizes, W, ratio, 1e-8, seed, wire=wire)
        orc = oracle.Oracle(sizes, W, ratio, 1e-8, seed)
        upd = torch.full((N,), float("nan"), device=DEV)
        for t in range(3):
            g = _randn((W, N), 970 + t)
            sp.step(g, weights, upd)
            want = orc.step(np.ascontiguousarray(g.cpu().numpy()), weights.cpu().numpy())
            assert sp.leader == orc.leader and sp.last_wire == wire
            assert_bits_equal(upd.cpu().numpy(), want, f"step {t}: update")
            for w in range(W):
                assert_bits_equal(sp.local.residual(w).cpu().numpy(), orc.residual(w), f"step {t}: worker {w} residual")
        sp.close()
        orc.close()
    finally:
        dist.destroy_process_group()


# ------------------------------------------------------------------ real ranks on real GPUs (when the box has them)


def _nccl_rank_main(rank: int, world: int, port: int, wire: str, out):
    import torch.distributed as dist

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    torch.cuda.set_device(rank)
    dev = torch.device("cuda", rank)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    ok, why = True, ""
    try:
        from paper_1901_01544_b200 import workloads as wl

        c = wl.single_layer()  # configuration 1: one layer of 2^20, four workers
        Wl = c.W // world
        sp = ShardedPruner(c.layer_sizes, c.W, c.ratio, c.eps, c.seed, wire=wire)
        orc = oracle.Oracle(c.layer_sizes, c.W, c.ratio, c.eps, c.seed)  # the whole job, on every rank
        weights = c.weights(dev)
        w_host = weights.cpu().numpy()
        upd = torch.full((c.N,), float("nan"), device=dev)
        for t in range(c.steps):
            g = c.grads(t, dev)  # seeded: the same on every rank
            want = orc.step(np.ascontiguousarray(g.cpu().numpy()), w_host)
            sp.step(g[rank * Wl:(rank + 1) * Wl].contiguous(), weights, upd)
            same = sp.leader == orc.leader and np.array_equal(upd.cpu().numpy().view(np.uint32), want.view(np.uint32))
            for w in range(Wl):
                same = same and np.array_equal(sp.local.residual(w).cpu().numpy().view(np.uint32),
                                               orc.residual(rank * Wl + w).view(np.uint32))
            if not same:
                ok, why = False, f"step {t} differs from the oracle of the whole job"
                break
            upd.fill_(float("nan"))
        ok = ok and sp.local.sync_status() == 0 and sp.last_wire == wire
        sp.close()
        orc.close()
    except Exception as e:  # reported to the parent instead of a silent non-zero exit
        ok, why = False, f"{type(e).__name__}: {e}"
    out.put((rank, ok, why))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("wire", ["list", "mask"])
def test_sharded_pruner_on_two_gpus_over_nccl(wire):
    """Two ranks, one GPU each, NCCL broadcast + all-gather between them: the sharded step against the oracle of
    the whole job.  Needs two visible GPUs; on a one-GPU machine the test skips itself (the same orchestration runs
    as two gloo ranks on CPU and as a one-rank NCCL group above)."""
    import torch.multiprocessing as mp

    if torch.cuda.device_count() < 2:
        pytest.skip("needs two GPUs")
    world = 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_nccl_rank_main, args=(r, world, port, wire, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=600) for _ in procs)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert got == [(0, True, ""), (1, True, "")], got
