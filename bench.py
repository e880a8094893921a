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
FALLBACK_HBM_GBS = 6650.0
# DRAM traffic of the dominant kernels relative to their algorithmic bytes, as captured with ncu: kept as data
# beside the ncu summaries, each entry with the git blob hash of the kernel source it was captured from
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "traffic_ratios.json")


def git_blob_hash(path: str) -> str:
    """The hash `git hash-object` gives the file: ties a captured figure to the kernel source it came from."""
    import hashlib

    data = open(path, "rb").read()
    return hashlib.sha1(b"blob %d\0" % len(data) + data).hexdigest()


def traffic_ratio(kernel: str, weights_fit_l2: bool):
    """(ratio of DRAM traffic to algorithmic bytes, note) of a dominant kernel from profiles/traffic_ratios.json;
    (None, why) if there is no capture.  A capture made from an older version of the kernel source is flagged."""
    try:
        ent = json.load(open(TRAFFIC_FILE))[kernel]
    except Exception as e:  # no capture on record: no traffic figure
        return None, f"no capture on record ({type(e).__name__})"
    ratio = ent["ratio_weights_in_l2"] if (weights_fit_l2 and "ratio_weights_in_l2" in ent) else ent["ratio"]
    src = os.path.join(ROOT, ent["source"])
    stale = (not os.path.exists(src)) or git_blob_hash(src) != ent["source_blob"]
    note = (f"dram__bytes_read+write per step of the kernel = {ratio} x algorithmic bytes, from the ncu capture in "
            f"{ent['profile']}, scaled to this workload" + ("; CAPTURED FROM AN OLDER VERSION OF THE KERNEL SOURCE" if stale else ""))
    return ratio, note


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


def oracle_timing(c, weights_host, grads_host_fn, steps, warmup, threads=0):
    """Times the CPU oracle as it stands on the host cores; returns (steps/s, threads, seconds)."""
    import oracle

    orc = oracle.Oracle(c.layer_sizes, c.W, c.ratio, c.eps, c.seed, threads=threads)
    for t in range(warmup):
        orc.step(grads_host_fn(t), weights_host)
    t0 = time.perf_counter()
    for t in range(steps):
        orc.step(grads_host_fn(warmup + t), weights_host)
    dt = time.perf_counter() - t0
    threads = orc.threads
    orc.close()
    return steps / dt, threads, dt


def config_dict(c, mode, K, n_sets):
    """The `config` object of the JSON line; both arms print exactly this for the same workload."""
    grad_bytes = 4 * c.W * c.N
    return {"workload": c.name, "mode": mode, "W": c.W, "N": c.N, "K": K,
            "ratio": c.ratio if mode.startswith("ratio") else None, "layers": len(c.layer_sizes),
            "l2_policy": f"inputs larger than L2: {grad_bytes * 3 / 1e9:.2f} GB streamed per step, "
                         f"{n_sets} gradient batches cycled",
            "multi_gpu": "independent replicas (the path has no inter-GPU exchange)",
            "compression_N_over_K": c.N / K}


def default_grad_sets(c, requested=None):
    if requested:
        return requested
    return max(2, min(5, int(24e9 // (4 * c.W * c.N))))  # distinct gradient batches cycled through


def run_reference(args):
    """--impl reference: the CPU oracle on the same configuration, metric and unit."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle

    c = make_workload(args.config, args.layers)
    weights = c.weights("cpu").numpy()
    n_sets = 2
    sets = [c.grads(t, "cpu").numpy() for t in range(n_sets)]
    sps, threads, dt = oracle_timing(c, weights, lambda t: sets[t % n_sets], args.steps, args.warmup)
    K = sum(oracle.keep_count(n, c.ratio) for n in c.layer_sizes)
    line = {
        "impl": "reference", "metric": METRIC, "value": sps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 / sps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_dict(c, "ratio", K, default_grad_sets(c, args.grad_sets)),
        "cpu_baseline": {"value": sps, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": f"{args.steps} full steps of {c.name} after {args.warmup} warm-up steps, the CPU "
                                   f"oracle as it stands ({dt:.1f} s of CPU work, 2 gradient batches cycled)"},
        "e2e": {"value": sps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------- workers spread over GPUs


def measure_sharded(c, dist, rank, world, dev, steps, warmup, grad_sets=None, wire="auto"):
    """The workload's W workers spread over the ranks (W / world each): ShardedPruner - NCCL broadcast of the chosen
    worker's index set (list or encoded mask, whichever is shorter) and all-gather of the gathered values.  Total
    work is fixed: strong scaling.  On one GPU it measures the cost of the three-phase protocol itself."""
    import torch

    from paper_1901_01544_b200.binding import ShardedPruner

    if c.W % world != 0:
        return {"error": f"the workload's {c.W} workers do not divide over {world} ranks"}
    Wl, N = c.W // world, c.N
    weights = c.weights(dev)
    n_sets = grad_sets or 3
    sets = [c.grads(t, dev)[rank * Wl:(rank + 1) * Wl].contiguous() for t in range(n_sets)]
    update = torch.empty(N, dtype=torch.float32, device=dev)
    sp = ShardedPruner(c.layer_sizes, c.W, c.ratio, c.eps, c.seed, wire=wire)
    for t in range(warmup):
        sp.step(sets[t % n_sets], weights, update)
    launches0 = sp.local.stat("launches")
    torch.cuda.synchronize()
    dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(steps):
        sp.step(sets[(warmup + t) % n_sets], weights, update)
    sp.local.join()
    e1.record()
    torch.cuda.synchronize()
    dist.barrier()
    ms_total = max_over_ranks(e0.elapsed_time(e1), dist, dev)
    assert sp.local.sync_status() == 0
    out = {"value": steps / (ms_total * 1e-3), "unit": UNIT, "ms_per_step": ms_total / steps, "scaling": "strong",
           "n_gpus": world, "steps": steps, "warmup": warmup, "W": c.W, "W_per_gpu": Wl, "N": N, "K": sp.K,
           "wire_format": sp.last_wire, "wire_bytes_per_step": sp.wire_bytes, "allgather_bytes_per_step": 4 * c.W * sp.K,
           "collectives": "broadcast of the index set (sorted uint32 list or one-bit-per-element mask, the shorter) + "
                          "all-gather of W x K fp32 per step (NCCL)",
           "gpu_launches": sp.local.stat("launches") - launches0}
    sp.close()
    del sets, weights, update, sp
    torch.cuda.empty_cache()
    return out


def run_sharded(args):
    """--shard: only the sharded arm (see measure_sharded), one JSON line from rank 0."""
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
    c = make_workload(args.config, args.layers)
    r = measure_sharded(c, dist, rank, world, dev, args.steps, args.warmup, args.grad_sets, args.wire)
    if "error" in r:
        raise SystemExit(r["error"])
    if rank == 0:
        line = {
            "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": c.name, "mode": "sharded", "W": c.W, "W_per_gpu": r["W_per_gpu"], "N": c.N, "K": r["K"],
                       "wire_format": r["wire_format"], "collectives": r["collectives"]},
            "gpu_launches": r["gpu_launches"],
        }
        print(json.dumps(line), flush=True)
    dist.destroy_process_group()


# ---------------------------------------------------------------------------------- the CUDA arm


def make_pruner(c, mode, layerwise, options, speculate=None):
    from paper_1901_01544_b200.binding import Pruner

    if mode == "threshold":
        # Algorithm 1 as printed: absolute per-layer thresholds, set near the step-0 top-1/64 point of this
        # workload's value recipe (weight tensors 0.4; zero-initialised biases rank by |residual| / eps)
        thr = [0.4 if (c.tensors is None or tn.kind == "weight") else 2.0e4
               for tn in (c.tensors or [None] * len(c.layer_sizes))]
        pr = Pruner(c.layer_sizes, c.W, None, c.eps, c.seed, thresholds=thr)
        if layerwise:  # Section 3.4: thresholds from the chosen node's per-layer var/mean (Eq. 4)
            pr.set_layerwise(*(float(x) for x in layerwise.split(",")))
    else:
        pr = Pruner(c.layer_sizes, c.W, c.ratio, c.eps, c.seed)
    if speculate is not None:
        pr.set_option("speculate", speculate)
    for kv in options:
        k, v = kv.split("=")
        pr.set_option(k, int(v))
    return pr


def timed_steps(pr, sets, weights, update, steps, warmup, barrier, threshold_mode, time_dominant=True):
    """`warmup` untimed steps, then `steps` steps between two CUDA events on the launching stream.
    Returns (ms of the timed region on this rank, launches in it, live ms per step of the dominant stage)."""
    import torch

    n_sets = len(sets)
    for t in range(warmup):  # residuals carry over into the timed region, as in training
        pr.step(sets[t % n_sets], weights, update)
    pr.check()
    # two CUDA events per step around the dominant streaming stage, created before the timed region
    pr.set_option("time_stages", 2 if time_dominant else 0)
    if time_dominant:
        pr.set_option("reserve_timed_steps", steps)
    launches0 = pr.stat("launches")
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(steps):
        pr.step(sets[(warmup + t) % n_sets], weights, update)
    pr.join()  # the last step's late selects (lists nobody consumes) are inside the timed region too
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    launches = pr.stat("launches") - launches0
    pr.check()
    live = None
    if time_dominant:
        live = pr.stat("time_gather_ns" if threshold_mode else "time_accumulate_ns") / 1e6 / steps
    pr.set_option("time_stages", 0)
    return ms, launches, live


def stage_pass(pr, sets, weights, update, steps, first):
    """Per-stage device times from a separate pass in the serial schedule (an event at every stage boundary)."""
    pr.set_option("time_stages", 1)
    pr.set_option("reserve_timed_steps", steps)
    for t in range(steps):
        pr.step(sets[(first + t) % len(sets)], weights, update)
    pr.check()
    out = {k: pr.stat(f"time_{k}_ns") / 1e6 / steps for k in ("small", "sample", "accumulate", "select", "compact", "gather")}
    out["note"] = (f"separate pass of {steps} steps in the serial schedule (no overlap of the selects with the "
                   "streaming pass) with an event at every stage boundary; 'small' runs on a side stream beside "
                   "the other stages, 'gather' includes waiting for the non-leader lists")
    pr.set_option("time_stages", 0)
    return out


def efficiency(B, ms_per_step, peak):
    eff = B / (ms_per_step * 1e-3) / 1e9
    return {"compulsory_bytes": B, "effective_gbs": eff, "frac_of_measured_peak": eff / peak,
            "frac_of_nominal_8tbs": eff / NOMINAL_HBM_GBS}


def measure_variant(name, dev, peak, steps, warmup, mode="ratio", layerwise=None, options=(), grad_sets=None):
    """One entry of the `configs` table: a workload (or a mode / option variant of one) timed like the headline,
    device-resident inputs, in this process."""
    import torch

    c = make_workload(name)
    n_sets = default_grad_sets(c, grad_sets)
    weights = c.weights(dev)
    sets = [c.grads(t, dev) for t in range(n_sets)]
    update = torch.empty(c.N, dtype=torch.float32, device=dev)
    pr = make_pruner(c, mode, layerwise, options)
    ms, launches, live = timed_steps(pr, sets, weights, update, steps, warmup, torch.cuda.synchronize, mode == "threshold")
    K = pr.list_length() if mode == "threshold" else pr.K
    B = step_bytes(c.W, c.N, K)
    spec_failed, spec_pairs = pr.stat("spec_failed"), pr.stat("spec_pairs")
    stages = stage_pass(pr, sets, weights, update, min(steps, 5), warmup + steps)
    stages.pop("note")
    out = {"workload": c.name, "mode": mode + ("+layerwise" if layerwise else ""), "options": list(options),
           "W": c.W, "N": c.N, "K": K, "layers": len(c.layer_sizes), "steps": steps, "warmup": warmup,
           "ms_per_step": ms / steps, "steps_per_s": steps / (ms * 1e-3), "gpu_launches_per_step": launches / steps,
           "dominant_stage_ms": live, "spec_failed": spec_failed, "spec_pairs": spec_pairs,
           "grad_batches": n_sets, "stage_ms_serial": {k: round(v, 5) for k, v in stages.items()}}
    out.update(efficiency(B, ms / steps, peak))
    pr.close()
    del sets, weights, update, pr
    torch.cuda.empty_cache()
    return out


# the other four configurations, then the mode and option variants on the headline workload
EXTRA_CONFIGS = ["single_layer", "resnet50_w8", "alexnet_w32", "flat_1g_w4"]
EXTRA_VARIANTS = [
    ("alexnet_w8:threshold", dict(name="alexnet_w8", mode="threshold")),
    ("alexnet_w8:threshold+layerwise", dict(name="alexnet_w8", mode="threshold", layerwise="0.4,0.0,1.0")),
    ("alexnet_w8:leader_only_select", dict(name="alexnet_w8", options=("leader_only_select=1",))),
    ("alexnet_w8:n_leaders=2", dict(name="alexnet_w8", options=("n_leaders=2",))),
    ("alexnet_w8:per_layer_leaders", dict(name="alexnet_w8", options=("per_layer_leaders=1",))),
]


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
    from paper_1901_01544_b200 import binding

    dev = torch.device("cuda", local)
    c = make_workload(args.config, args.layers)
    W, N = c.W, c.N
    weights = c.weights(dev)
    grad_bytes = 4 * W * N
    n_sets = default_grad_sets(c, args.grad_sets)
    sets = [c.grads(t, dev) for t in range(n_sets)]
    update = torch.empty(N, dtype=torch.float32, device=dev)
    pr = make_pruner(c, args.mode, args.layerwise, args.option, args.speculate)
    K = pr.K

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ms_total, launches, k1_ms_live = timed_steps(pr, sets, weights, update, args.steps, args.warmup, barrier,
                                                 args.mode == "threshold", time_dominant=not args.no_stage_times)
    clocks = sampler.stop() if rank == 0 else None
    if args.mode == "threshold":
        K = pr.list_length()  # size of the last step's index set
    spec = {"pairs": pr.stat("spec_pairs"), "failed": pr.stat("spec_failed")}
    stage_steps = 0 if args.no_stage_times else max(1, min(args.steps, args.stage_steps))
    stage_ms = stage_pass(pr, sets, weights, update, stage_steps, args.warmup + args.steps) if stage_steps else None
    ms_total = max_over_ranks(ms_total, dist, dev)
    ms_per_step = ms_total / args.steps
    value = whole_job_value(args.steps, world, ms_total)

    # end to end through the host-buffer entry point: H2D of grads + weights and D2H of the update inside
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    e2e_value = None
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
        del gh, wh, uh

    # N > 1: the same workload once more with its W workers spread over the ranks (the paper's deployment: the index
    # set and the gathered values cross NVLink), reported beside the replicas' number
    sharded = None
    if dist is not None:
        pr.close()
        del sets, weights, update, pr
        torch.cuda.empty_cache()
        sharded = measure_sharded(c, dist, rank, world, dev, args.steps, max(3, args.warmup), args.grad_sets, args.wire)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_src = measured_peak()
    B = step_bytes(W, N, K)
    plan = binding.iwp_plan_sizes(c.layer_sizes, W, c.ratio)
    l2_bytes = int(torch.cuda.get_device_properties(dev).L2_cache_size)
    Nt = sum(n for n in c.layer_sizes if n > 16384)  # elements on the tiled path
    # The dominant kernel is k_stream (fused accumulate + importance + candidate emission over all tiled
    # layers).  It is launched twice per step - once for the leader's worker, once for the W-1 others -
    # and the two launches together move, algorithmically: grads read, residual read and written
    # (12 bytes per worker and element), weights read and update zeroed once (8 bytes per element).
    k1_bytes = 12 * W * Nt + 8 * Nt
    k1_ms = k1_ms_live or 0.0
    k1_name = "k_stream, both launches of a step (leader, then the other workers), timed together"
    k1_launches = 2 if W > 1 else 1
    k1_ratio, k1_note = traffic_ratio("k_stream", weights_fit_l2=4 * Nt <= l2_bytes)
    if args.mode == "threshold":
        # The dominant kernel is k_thr_fused: residuals of all W workers read, gradients of the W - n
        # non-chosen workers read, their residuals written back, the update written, one set bit per element.
        nl = max(1, int(dict(o.split("=") for o in (args.option or [])).get("n_leaders", 1)))
        k1_bytes = 4 * N * (W + 2 * (W - nl) + 1) + N // 8
        k1_name, k1_launches = "k_thr_fused (accumulate the non-chosen workers, ordered sum, zeroing, update)", 1
        k1_ratio, k1_note = traffic_ratio("k_thr_fused", weights_fit_l2=False)
    k1_traffic = args.traffic_bytes if args.traffic_bytes else (k1_ratio * k1_bytes if k1_ratio else None)
    achieved = k1_bytes / (k1_ms * 1e-3) / 1e9 if k1_ms > 0 else 0.0
    roofline = {
        "bound": "hbm", "kernel": k1_name,
        "achieved": achieved if k1_ms > 0 else None, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak if k1_ms > 0 else None, "peak_source": peak_src,
        "traffic": k1_traffic,
        "algorithmic_bytes_per_step_of_kernel": k1_bytes, "ms_per_step_of_kernel": k1_ms,
        "launches_per_step": k1_launches, "traffic_note": k1_note, "l2_bytes": l2_bytes,
    }
    if stage_ms is not None:
        # the same kernel with nothing beside it (the serial stage pass): in the timed region the selects of
        # the overlapped schedule share the GPU with it
        alone_ms = stage_ms["gather" if args.mode == "threshold" else "accumulate"]
        if alone_ms > 0:
            alone = k1_bytes / (alone_ms * 1e-3) / 1e9
            roofline["alone"] = {"ms_per_step_of_kernel": alone_ms, "achieved": alone, "frac": alone / peak,
                                 "note": "separate serial pass, no other kernel running beside it"}
    step_eff = efficiency(B, ms_per_step, peak)

    # CPU baseline: the oracle as it stands, a bounded sample (a few full steps) on this machine's cores, and on one
    cpu = cpu1 = None
    if not args.no_cpu_baseline and args.mode == "ratio":
        w_host = c.weights("cpu").numpy() if dist is not None else weights.cpu().numpy()
        g_host = [(c.grads(i, "cpu") if dist is not None else sets[i].cpu()).numpy() for i in range(min(2, n_sets))]
        sps, threads, dt = oracle_timing(c, w_host, lambda t: g_host[t % len(g_host)], args.cpu_steps, 1)
        cpu = {"value": sps, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"{args.cpu_steps} full steps of {c.name} after 1 warm-up step ({dt:.1f} s of CPU work)"}
        if args.cpu1_steps > 0:
            sps1, threads1, dt1 = oracle_timing(c, w_host, lambda t: g_host[t % len(g_host)], args.cpu1_steps, 0, threads=1)
            cpu1 = {"value": sps1, "unit": UNIT, "cores": threads1, "kind": "oracle",
                    "sample": f"{args.cpu1_steps} full steps of {c.name}, no warm-up ({dt1:.1f} s of CPU work)"}
        del w_host, g_host

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": config_dict(c, args.mode + ("+layerwise" if args.layerwise else ""), K, n_sets),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 4 * (W * N + N), "d2h_bytes_per_step": 4 * N,
                "steps": e2e_steps},
        "gpu_launches": launches,
        "roofline": roofline,
        "step_effective": step_eff,
        "stage_ms": stage_ms,
        "speculation": spec,
        "cpu_baseline": cpu,
        "cpu_baseline_1core": cpu1,
        "clocks": clocks,
        "plan": plan,
    }
    if sharded is not None:
        line["sharded"] = sharded

    # The other configurations and the mode / option variants, each timed like the headline (device-resident
    # inputs, CUDA events around the timed steps), one after the other in this process at N = 1.
    if world == 1 and not args.no_extra_configs and args.mode == "ratio" and not args.layers and not args.option:
        pr.close()
        del sets, weights, update, pr
        torch.cuda.empty_cache()
        table = {}
        try:  # the three-phase protocol of the sharded deployment on this one GPU (a one-rank NCCL group)
            import torch.distributed as dist1

            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29533")
            dist1.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
            try:
                table[f"{args.config}:sharded_protocol_on_one_gpu"] = measure_sharded(
                    c, dist1, 0, 1, dev, args.extra_steps, max(3, args.warmup), args.grad_sets, args.wire)
            finally:
                dist1.destroy_process_group()
        except Exception as e:
            table[f"{args.config}:sharded_protocol_on_one_gpu"] = {"error": f"{type(e).__name__}: {e}"}
            torch.cuda.empty_cache()
        for name in EXTRA_CONFIGS:
            if name == args.config:
                continue
            try:
                table[name] = measure_variant(name, dev, peak, args.extra_steps, max(3, args.warmup))
            except Exception as e:  # reported, not hidden: an entry that failed carries the reason
                table[name] = {"error": f"{type(e).__name__}: {e}"}
                torch.cuda.empty_cache()
        for label, kw in EXTRA_VARIANTS:
            try:
                table[label] = measure_variant(dev=dev, peak=peak, steps=args.extra_steps, warmup=max(3, args.warmup), **kw)
            except Exception as e:
                table[label] = {"error": f"{type(e).__name__}: {e}"}
                torch.cuda.empty_cache()
        line["configs"] = table
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
    ap.add_argument("--cpu1-steps", type=int, default=2, help="full steps of the oracle timed on ONE core (0 = skip)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra-configs", action="store_true",
                    help="skip the table of the other configurations and variants (key `configs`)")
    ap.add_argument("--extra-steps", type=int, default=20, help="timed steps of every entry of that table")
    ap.add_argument("--speculate", type=int, default=None, choices=[0, 1])
    ap.add_argument("--mode", default="ratio", choices=["ratio", "threshold"],
                    help="ratio: exact layer-wise top-k at the configured compression (headline); threshold: "
                         "absolute per-layer thresholds on the chosen node (Algorithm 1 as printed)")
    ap.add_argument("--shard", action="store_true",
                    help="spread the workload's W workers over the ranks (ShardedPruner: NCCL broadcast + all-gather) "
                         "instead of running independent replicas")
    ap.add_argument("--wire", default="auto", choices=["auto", "list", "mask"],
                    help="what travels as the index set in the sharded arm (auto = the shorter encoding)")
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
