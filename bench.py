#!/usr/bin/env python
"""Benchmark of the importance-weighted pruning step (pruned all-reduce steps/s and achieved
HBM GB/s) on synthetic inputs of the AlexNet-shaped W=8 configuration by default.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

One JSON line is printed by rank 0.  A "step" is one pass of the whole hot path (accumulate,
importance, layer-wise top-k, compaction, leader gather, ordered worker sum, scatter, zeroing)
over one batch of W*N synthetic gradients.  The path has no inter-GPU exchange: with --gpus N
(under torchrun) every rank runs an independent replica of the same configuration.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "pruned_allreduce_steps_per_s"
UNIT = "steps/s"
NOMINAL_HBM_GBS = 8000.0
# DRAM traffic of the streaming kernel (both launches) relative to its algorithmic bytes, from the ncu captures in
# profiles/k_stream_alexnet_fc7_fc8_w8.md: 1.063 on the full-size default workload (1.026 for candidate slots, side
# values, the leader's record and the zero mask, plus the weights, which the second launch reads again once they
# no longer fit the L2); 1.026 when the weights of the tiled layers do fit (the small capture).
TRAFFIC_OVER_ALGORITHMIC = 1.063
TRAFFIC_OVER_ALGORITHMIC_WEIGHTS_IN_L2 = 1.026
L2_BYTES = 126e6
TRAFFIC_OVER_ALGORITHMIC_THRESHOLD = 1.022  # k_thr_fused, full-size capture (profiles/k_thr_fused_alexnet_fc7_fc8_w8.md)
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


def step_bytes(W, N, K):
    """Compulsory bytes of one step: every input read once, every output written once."""
    return 4 * W * N + 8 * W * N + 4 * N + 4 * N + 16 * W * K + 8 * K


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        try:
            self.proc.terminate()  # the exact process started above
            self.proc.wait(timeout=5)
        except Exception:
            pass
        try:
            rows = [r.strip().split(", ") for r in open(self.path) if r.strip()]
            os.unlink(self.path)
        except Exception:
            return out
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for nme, v in zip(names, r[3:7]):
                if v.strip().lower().startswith("active"):
                    reasons.add(nme)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def max_over_ranks(value: float, dist, device) -> float:
    """Slowest rank's value (each rank times its own replica on its own device)."""
    if dist is None:
        return float(value)
    import torch

    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(steps: int, world: int, ms_total_max: float) -> float:
    """Units all ranks processed divided by the slowest rank's time: every rank runs `steps` steps of
    its own replica (weak scaling, no data-path collective)."""
    return world * steps / (ms_total_max / 1e3)


def make_workload(name, layers=None):
    from paper_1901_01544_b200 import workloads as wl

    c = wl.CONFIGS[name]()
    if layers:
        lo, hi = (int(x) for x in layers.split(":"))
        c = wl.subset(c, lo, hi)
    return c


# ---------------------------------------------------------------------------------- CPU oracle legs


def oracle_timing(c, weights_host, grads_host_fn, steps, warmup):
    """Times the CPU oracle as it stands on the host cores; returns (steps/s, threads, seconds)."""
    import oracle

    orc = oracle.Oracle(c.layer_sizes, c.W, c.ratio, c.eps, c.seed)
    for t in range(warmup):
        orc.step(grads_host_fn(t), weights_host)
    t0 = time.perf_counter()
    for t in range(steps):
        orc.step(grads_host_fn(warmup + t), weights_host)
    dt = time.perf_counter() - t0
    threads = orc.threads
    orc.close()
    return steps / dt, threads, dt


def run_reference(args):
    """--impl reference: the CPU oracle on the same configuration, metric and unit."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch

    c = make_workload(args.config, args.layers)
    weights = c.weights("cpu").numpy()
    n_sets = 2
    sets = [c.grads(t, "cpu").numpy() for t in range(n_sets)]
    sps, threads, dt = oracle_timing(c, weights, lambda t: sets[t % n_sets], args.steps, args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": sps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 / sps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": c.name, "W": c.W, "N": c.N, "ratio": c.ratio, "layers": len(c.layer_sizes),
                   "note": "CPU oracle, every step a full step of the workload"},
        "cpu_baseline": {"value": sps, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": f"{args.steps} full steps of {c.name} after {args.warmup} warm-up steps"},
        "e2e": {"value": sps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------- workers spread over GPUs


def run_sharded(args):
    """--shard: the workload's W workers spread over the N ranks (W / N each), the chosen worker's index list
    broadcast and the gathered values all-gathered over NCCL (ShardedPruner).  Total work is fixed: strong
    scaling.  Not the default arm; on one GPU it measures the cost of the three-phase protocol itself."""
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the pruning path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world == 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29533")
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    from paper_1901_01544_b200 import build as lib_build

    if rank == 0:
        lib_build.build()
    dist.barrier()
    from paper_1901_01544_b200.binding import ShardedPruner

    c = make_workload(args.config, args.layers)
    if c.W % world != 0:
        raise SystemExit(f"--shard needs the workload's {c.W} workers to divide over {world} ranks")
    Wl, N = c.W // world, c.N
    weights = c.weights(dev)
    n_sets = args.grad_sets or 3
    sets = [c.grads(t, dev)[rank * Wl:(rank + 1) * Wl].contiguous() for t in range(n_sets)]
    update = torch.empty(N, dtype=torch.float32, device=dev)
    sp = ShardedPruner(c.layer_sizes, c.W, c.ratio, c.eps, c.seed)
    for t in range(args.warmup):
        sp.step(sets[t % n_sets], weights, update)
    torch.cuda.synchronize()
    dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(args.steps):
        sp.step(sets[(args.warmup + t) % n_sets], weights, update)
    e1.record()
    torch.cuda.synchronize()
    dist.barrier()
    ms_total = max_over_ranks(e0.elapsed_time(e1), dist, dev)
    assert sp.local.sync_status() == 0
    if rank == 0:
        line = {
            "metric": METRIC, "value": args.steps / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": c.name, "mode": "sharded", "W": c.W, "W_per_gpu": Wl, "N": N, "K": sp.K,
                       "collectives": "broadcast of K uint32 + all-gather of W x K fp32 per step (NCCL)"},
            "gpu_launches": sp.local.stat("launches"),
        }
        print(json.dumps(line), flush=True)
    dist.destroy_process_group()


# ---------------------------------------------------------------------------------- the CUDA arm


def run_ours(args):
    import torch

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the pruning path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    from paper_1901_01544_b200 import build as lib_build

    if rank == 0:
        lib_build.build()
    if dist is not None:
        dist.barrier()
    from paper_1901_01544_b200.binding import Pruner

    dev = torch.device("cuda", local)
    c = make_workload(args.config, args.layers)
    W, N = c.W, c.N
    weights = c.weights(dev)
    grad_bytes = 4 * W * N
    n_sets = max(2, min(5, int(24e9 // grad_bytes)))  # distinct gradient batches cycled through
    if args.grad_sets:
        n_sets = args.grad_sets
    sets = [c.grads(t, dev) for t in range(n_sets)]
    update = torch.empty(N, dtype=torch.float32, device=dev)
    if args.mode == "threshold":
        # Algorithm 1 as printed: absolute per-layer thresholds, set near the step-0 top-1/64 point of this
        # workload's value recipe (weight tensors 0.4; zero-initialised biases rank by |residual| / eps)
        thr = [0.4 if (c.tensors is None or tn.kind == "weight") else 2.0e4
               for tn in (c.tensors or [None] * len(c.layer_sizes))]
        pr = Pruner(c.layer_sizes, W, None, c.eps, c.seed, thresholds=thr)
        if args.layerwise:  # Section 3.4: thresholds from the chosen node's per-layer var/mean (Eq. 4)
            pr.set_layerwise(*(float(x) for x in args.layerwise.split(",")))
    else:
        pr = Pruner(c.layer_sizes, W, c.ratio, c.eps, c.seed)
    K = pr.K
    if args.speculate is not None:
        pr.set_option("speculate", args.speculate)
    for kv in args.option:
        k, v = kv.split("=")
        pr.set_option(k, int(v))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # warm-up (residuals carry over into the timed region, as in training)
    for t in range(args.warmup):
        pr.step(sets[t % n_sets], weights, update)
    pr.check()
    # two CUDA events per step, around the streaming stage (the dominant kernel, two launches of k_stream);
    # the full per-stage breakdown is taken in a separate, shorter pass after the timed region because
    # seven events per step cost about 1 % of the step
    pr.set_option("time_stages", 0 if args.no_stage_times else 2)
    launches0 = pr.stat("launches")
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(args.steps):
        pr.step(sets[(args.warmup + t) % n_sets], weights, update)
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    launches = pr.stat("launches") - launches0
    pr.check()
    if args.mode == "threshold":
        K = pr.list_length()  # size of the last step's index set
    k1_ms_live = pr.stat("time_gather_ns" if args.mode == "threshold" else "time_accumulate_ns") / 1e6 / args.steps
    spec = {"pairs": pr.stat("spec_pairs"), "failed": pr.stat("spec_failed")}
    stage_steps = 0 if args.no_stage_times else max(1, min(args.steps, args.stage_steps))
    stage_ms = None
    if stage_steps:
        pr.set_option("time_stages", 1)
        for t in range(stage_steps):
            pr.step(sets[(args.warmup + args.steps + t) % n_sets], weights, update)
        pr.check()
        stage_ms = {k: pr.stat(f"time_{k}_ns") / 1e6 / stage_steps for k in ("small", "sample", "accumulate", "select",
                                                                              "compact", "gather")}
        stage_ms["note"] = (f"separate pass of {stage_steps} steps in the serial schedule (no overlap of the selects with the "
                            "streaming pass) with an event at every stage boundary; 'small' runs on a side stream beside "
                            "the other stages, 'gather' includes waiting for the non-leader lists")
    pr.set_option("time_stages", 0)
    ms_total = max_over_ranks(ms_total, dist, dev)
    ms_per_step = ms_total / args.steps
    value = whole_job_value(args.steps, world, ms_total)

    # end to end through the host-buffer entry point: H2D of grads + weights and D2H of the update inside
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    e2e_value = None
    gh = wh = None
    if not args.no_e2e:
        gh = [sets[i].cpu().pin_memory() for i in range(min(2, n_sets))]
        wh = weights.cpu().pin_memory()
        uh = [torch.empty(N, dtype=torch.float32).pin_memory() for _ in range(2)]
        # host buffers in, host buffer out, every step; consecutive calls overlap their copies (the inputs of
        # step t + 1 travel while step t runs and its update travels back), the last update is waited for
        pr.step_host_async(gh[0], wh, uh[0])  # allocates the staging buffers
        pr.host_wait()
        barrier()
        t0 = time.perf_counter()
        for t in range(e2e_steps):
            pr.step_host_async(gh[t % len(gh)], wh, uh[t % 2])
        pr.host_wait()
        torch.cuda.synchronize()
        e2e_dt = time.perf_counter() - t0
        e2e_dt = max_over_ranks(e2e_dt, dist, dev)
        pr.check()
        e2e_value = whole_job_value(e2e_steps, world, e2e_dt * 1e3)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_src = measured_peak()
    B = step_bytes(W, N, K)
    plan = __import__("paper_1901_01544_b200.binding", fromlist=["x"]).iwp_plan_sizes(c.layer_sizes, W, c.ratio)
    Nt = sum(n for n in c.layer_sizes if n > 16384)  # elements on the tiled path
    # The dominant kernel is k_stream (fused accumulate + importance + candidate emission over all tiled
    # layers).  It is launched twice per step - once for the leader's worker, once for the W-1 others -
    # and the two launches together move, algorithmically: grads read, residual read and written
    # (12 bytes per worker and element), weights read and update zeroed once (8 bytes per element).
    k1_bytes = 12 * W * Nt + 8 * Nt
    k1_ms = k1_ms_live
    k1_name = "k_stream, both launches of a step (leader, then the other workers), timed together"
    k1_launches = 2 if W > 1 else 1
    k1_note = ("dram__bytes_read+write of both launches: ratio to algorithmic bytes from the ncu captures in "
               "profiles/k_stream_alexnet_fc7_fc8_w8.md (1.063 measured on the full-size default workload), "
               "scaled to this workload")
    k1_ratio = TRAFFIC_OVER_ALGORITHMIC if 4 * Nt > L2_BYTES else TRAFFIC_OVER_ALGORITHMIC_WEIGHTS_IN_L2
    k1_traffic = args.traffic_bytes if args.traffic_bytes else k1_ratio * k1_bytes
    if args.mode == "threshold":
        # The dominant kernel is k_thr_fused: residuals of all W workers read, gradients of the W - n
        # non-chosen workers read, their residuals written back, the update written, one set bit per element.
        nl = max(1, int(dict(o.split("=") for o in (args.option or [])).get("n_leaders", 1)))
        k1_bytes = 4 * N * (W + 2 * (W - nl) + 1) + N // 8
        k1_name, k1_launches = "k_thr_fused (accumulate the non-chosen workers, ordered sum, zeroing, update)", 1
        k1_note = ("dram__bytes_read+write of the launch: ratio to algorithmic bytes from the full-size ncu capture "
                   "(profiles/k_thr_fused_alexnet_fc7_fc8_w8.md), scaled to this workload")
        k1_traffic = args.traffic_bytes if args.traffic_bytes else TRAFFIC_OVER_ALGORITHMIC_THRESHOLD * k1_bytes
    achieved = k1_bytes / (k1_ms * 1e-3) / 1e9 if k1_ms > 0 else 0.0
    roofline = {
        "bound": "hbm", "kernel": k1_name,
        "achieved": achieved if k1_ms > 0 else None, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak if k1_ms > 0 else None, "peak_source": peak_src,
        "traffic": k1_traffic,
        "algorithmic_bytes_per_step_of_kernel": k1_bytes, "ms_per_step_of_kernel": k1_ms,
        "launches_per_step": k1_launches, "traffic_note": k1_note,
    }
    if stage_ms is not None:
        # the same kernel with nothing beside it (the serial stage pass): in the timed region the selects of
        # the overlapped schedule share the GPU with it
        alone_ms = stage_ms["gather" if args.mode == "threshold" else "accumulate"]
        if alone_ms > 0:
            alone = k1_bytes / (alone_ms * 1e-3) / 1e9
            roofline["alone"] = {"ms_per_step_of_kernel": alone_ms, "achieved": alone, "frac": alone / peak,
                                 "note": "separate serial pass, no other kernel running beside it"}
    eff = B / (ms_per_step * 1e-3) / 1e9
    step_eff = {"compulsory_bytes": B, "effective_gbs": eff, "frac_of_measured_peak": eff / peak,
                "frac_of_nominal_8tbs": eff / NOMINAL_HBM_GBS}

    # CPU baseline: the oracle as it stands, a bounded sample (a few full steps) on this machine's cores
    cpu = None
    if not args.no_cpu_baseline and args.mode == "ratio":
        w_host = weights.cpu().numpy()
        g_host = [sets[i].cpu().numpy() for i in range(min(2, n_sets))]
        sps, threads, dt = oracle_timing(c, w_host, lambda t: g_host[t % len(g_host)], args.cpu_steps, 1)
        cpu = {"value": sps, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"{args.cpu_steps} full steps of {c.name} after 1 warm-up step ({dt:.1f} s of CPU work)"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": c.name, "mode": args.mode + ("+layerwise" if args.layerwise else ""), "W": W, "N": N, "K": K,
                   "ratio": c.ratio if args.mode == "ratio" else None, "layers": len(c.layer_sizes),
                   "l2_policy": f"inputs larger than L2: {grad_bytes * 3 / 1e9:.2f} GB streamed per step, "
                                f"{n_sets} gradient batches cycled",
                   "multi_gpu": "independent replicas (the path has no inter-GPU exchange)",
                   "compression_N_over_K": N / K},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 4 * (W * N + N), "d2h_bytes_per_step": 4 * N,
                "steps": e2e_steps},
        "gpu_launches": launches,
        "roofline": roofline,
        "step_effective": step_eff,
        "stage_ms": stage_ms,
        "speculation": spec,
        "cpu_baseline": cpu,
        "clocks": clocks,
        "plan": plan,
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="alexnet_w8")
    ap.add_argument("--e2e-steps", type=int, default=8)
    ap.add_argument("--cpu-steps", type=int, default=15)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--speculate", type=int, default=None, choices=[0, 1])
    ap.add_argument("--mode", default="ratio", choices=["ratio", "threshold"],
                    help="ratio: exact layer-wise top-k at the configured compression (headline); threshold: "
                         "absolute per-layer thresholds on the chosen node (Algorithm 1 as printed)")
    ap.add_argument("--shard", action="store_true",
                    help="spread the workload's W workers over the ranks (ShardedPruner: NCCL broadcast + all-gather) "
                         "instead of running independent replicas")
    ap.add_argument("--layerwise", default=None,
                    help="alpha,beta,C - with --mode threshold: layer-wise thresholds alpha +/- beta var/mean (Eq. 4)")
    ap.add_argument("--layers", default=None, help="lo:hi - only these layers of the workload (small profiling case)")
    ap.add_argument("--grad-sets", type=int, default=None, help="distinct gradient batches kept on the device")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-stage-times", action="store_true", help="do not record per-stage CUDA events")
    ap.add_argument("--stage-steps", type=int, default=10, help="steps of the separate per-stage timing pass")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="DRAM bytes of the dominant kernel per step from an ncu capture (goes into roofline.traffic)")
    ap.add_argument("--option", action="append", default=[], help="key=value passed to iwp_set_option (experiments)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    elif args.shard:
        run_sharded(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
