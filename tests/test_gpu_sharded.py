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


def _run_groups(sizes, W_total, groups, ratio, seed, steps, grads_fn, weights, options=None):
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
        vals_all = torch.cat([c.shard_gather(idx) for c in ctxs], dim=0)   # "all-gather", group order = worker order
        for r, c in enumerate(ctxs):
            c.shard_apply(idx, vals_all, upds[r])
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


def test_sharded_pruner_over_a_one_rank_nccl_group():
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
        sp = ShardedPruner(sizes, W, ratio, 1e-8, seed)
        orc = oracle.Oracle(sizes, W, ratio, 1e-8, seed)
        upd = torch.full((N,), float("nan"), device=DEV)
        for t in range(3):
            g = _randn((W, N), 970 + t)
            sp.step(g, weights, upd)
            want = orc.step(np.ascontiguousarray(g.cpu().numpy()), weights.cpu().numpy())
            assert sp.leader == orc.leader
            assert_bits_equal(upd.cpu().numpy(), want, f"step {t}: update")
            for w in range(W):
                assert_bits_equal(sp.local.residual(w).cpu().numpy(), orc.residual(w), f"step {t}: worker {w} residual")
        sp.close()
        orc.close()
    finally:
        dist.destroy_process_group()
