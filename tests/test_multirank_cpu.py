"""The N > 1 path of the benchmark is "independent replicas": no data-path collective, only a barrier
and a max-over-ranks of the timings.  Its host logic runs here as two gloo ranks on CPU."""
import os
import socket
import sys

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
