"""Seeded synthetic workloads: tensor-shape lists and value generators.

This module is the only code shared by the CPU oracle's tests and the CUDA
path's tests / bench.  It holds *no* arithmetic of the pruning method (no
importance, no keep-count, no selection, no leader draw): only the layer-size
lists of the five benchmark configurations and the random number recipes for
weights and per-step gradients.

The networks of the paper's experiments (AlexNet and ResNet-50 on ImageNet,
Section 4.1 / Table 1) are represented by their parameter-tensor shapes only;
values are drawn from the stated distributions, because neither the dataset
nor trained weights are available or needed for the data-parallel hot path.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Callable, List, Optional

import torch

# --------------------------------------------------------------------------
# tensor-shape lists
# --------------------------------------------------------------------------

# AlexNet (grouped-convolution variant): (out, in_per_group, kh, kw) / (out, in)
_ALEXNET_WEIGHT_SHAPES = [
    (96, 3, 11, 11),
    (256, 48, 5, 5),
    (384, 256, 3, 3),
    (384, 192, 3, 3),
    (256, 192, 3, 3),
    (4096, 9216),
    (4096, 4096),
    (1000, 4096),
]


def _prod(shape) -> int:
    p = 1
    for s in shape:
        p *= int(s)
    return p


@dataclass
class Tensor:
    """One selection unit ("layer" in Algorithm 1's loop over j)."""

    name: str
    numel: int
    kind: str  # "weight" | "zeros" | "ones"
    fan_in: int  # fan-in of the owning weight tensor (scales the gradients)


def alexnet_tensors() -> List[Tensor]:
    """w1, b1, w2, b2, ..., w8, b8 (16 tensors, 60 965 224 parameters)."""
    out: List[Tensor] = []
    for i, shp in enumerate(_ALEXNET_WEIGHT_SHAPES, start=1):
        fan_in = _prod(shp[1:])
        out.append(Tensor(f"w{i}", _prod(shp), "weight", fan_in))
        out.append(Tensor(f"b{i}", shp[0], "zeros", fan_in))
    return out


def resnet50_tensors() -> List[Tensor]:
    """ResNet-50 parameter tensors in module order: every convolution followed by
    its batch-norm gamma and beta; bottleneck stages [3, 4, 6, 3] with planes
    64/128/256/512 and expansion 4, a 1x1 downsample convolution + batch norm in
    the first block of each stage; a 1000x2048 classifier and its bias
    (161 tensors, 25 557 032 parameters)."""
    out: List[Tensor] = []

    def conv_bn(name: str, cout: int, cin: int, k: int) -> None:
        fan_in = cin * k * k
        out.append(Tensor(name + ".conv", cout * cin * k * k, "weight", fan_in))
        out.append(Tensor(name + ".gamma", cout, "ones", fan_in))
        out.append(Tensor(name + ".beta", cout, "zeros", fan_in))

    conv_bn("stem", 64, 3, 7)
    inplanes = 64
    for stage, (planes, blocks) in enumerate(zip((64, 128, 256, 512), (3, 4, 6, 3)), start=1):
        for b in range(blocks):
            p = f"s{stage}b{b}"
            conv_bn(p + ".c1", planes, inplanes, 1)
            conv_bn(p + ".c2", planes, planes, 3)
            conv_bn(p + ".c3", planes * 4, planes, 1)
            if b == 0:
                conv_bn(p + ".down", planes * 4, inplanes, 1)
            inplanes = planes * 4
    out.append(Tensor("fc.weight", 1000 * 2048, "weight", 2048))
    out.append(Tensor("fc.bias", 1000, "zeros", 2048))
    return out


# --------------------------------------------------------------------------
# configurations
# --------------------------------------------------------------------------


@dataclass
class Workload:
    name: str
    layer_sizes: List[int]
    W: int
    ratio: float
    eps: float
    steps: int
    seed: int
    describe: str
    _weights_fn: Callable[["Workload", torch.device], torch.Tensor] = field(repr=False, default=None)
    _grads_fn: Callable[["Workload", int, torch.Tensor], None] = field(repr=False, default=None)
    tensors: Optional[List[Tensor]] = field(repr=False, default=None)

    @property
    def N(self) -> int:
        return sum(self.layer_sizes)

    def offsets(self) -> List[int]:
        off, o = [], 0
        for n in self.layer_sizes:
            off.append(o)
            o += n
        return off

    def weights(self, device="cpu") -> torch.Tensor:
        """weights[N] fp32 on `device` (identical for every worker)."""
        return self._weights_fn(self, torch.device(device))

    def grads(self, t: int, device="cpu", out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """grads[W][N] fp32 for step t (worker-major, contiguous)."""
        device = torch.device(device)
        if out is None:
            out = torch.empty((self.W, self.N), dtype=torch.float32, device=device)
        self._grads_fn(self, t, out)
        return out


def _gen(device: torch.device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


_CHUNK = 1 << 26  # elements per temporary, bounds scratch memory for the 2^30 case


def _fill_normal(dst: torch.Tensor, std: float, g: torch.Generator) -> None:
    flat = dst.view(-1)
    for s in range(0, flat.numel(), _CHUNK):
        flat[s : s + _CHUNK].normal_(0.0, std, generator=g)


# ---- config 1: one layer of 2^20 ------------------------------------------


def _c1_weights(wl: Workload, device: torch.device) -> torch.Tensor:
    g = _gen(device, wl.seed * 7919 + 1)
    w = torch.empty(wl.N, dtype=torch.float32, device=device)
    w.normal_(0.0, 0.05, generator=g)
    nz = int(round(0.01 * wl.N))
    perm = torch.randperm(wl.N, generator=g, device=device)[:nz]
    w[perm] = 0.0
    return w


def _c1_grads(wl: Workload, t: int, out: torch.Tensor) -> None:
    g = _gen(out.device, wl.seed * 1000 + t + 17)
    _fill_normal(out, 1e-3, g)


# ---- He-normal weights for a tensor list ------------------------------------


def _tensorlist_weights(wl: Workload, device: torch.device) -> torch.Tensor:
    g = _gen(device, wl.seed * 7919 + 2)
    w = torch.empty(wl.N, dtype=torch.float32, device=device)
    o = 0
    for tn in wl.tensors:
        seg = w[o : o + tn.numel]
        if tn.kind == "weight":
            seg.normal_(0.0, math.sqrt(2.0 / tn.fan_in), generator=g)
        elif tn.kind == "ones":
            seg.fill_(1.0)
        else:
            seg.zero_()
        o += tn.numel
    return w


def _c2_grads(wl: Workload, t: int, out: torch.Tensor) -> None:
    g = _gen(out.device, wl.seed * 1000 + t + 29)
    for w in range(wl.W):
        o = 0
        for tn in wl.tensors:
            out[w, o : o + tn.numel].normal_(0.0, 0.01 * math.sqrt(2.0 / tn.fan_in), generator=g)
            o += tn.numel


def _c3_grads(wl: Workload, t: int, out: torch.Tensor) -> None:
    # Laplace(0, b): difference of two independent Exponential(1/b) draws.
    g = _gen(out.device, wl.seed * 1000 + t + 31)
    b = 1e-4
    flat = out.view(-1)
    for s in range(0, flat.numel(), _CHUNK):
        seg = flat[s : s + _CHUNK]
        tmp = torch.empty_like(seg)
        seg.exponential_(1.0 / b, generator=g)
        tmp.exponential_(1.0 / b, generator=g)
        seg.sub_(tmp)


def _c4_scales(wl: Workload, t: int) -> List[float]:
    # one scale per (weight layer, step), shared by the layer's bias and by all workers
    g = torch.Generator(device="cpu")
    g.manual_seed(wl.seed * 1000 + 4)
    n_groups = len(wl.tensors) // 2
    u = torch.rand((max(wl.steps, t + 1), n_groups), generator=g, dtype=torch.float64)
    lo, hi = math.log(1e-5), math.log(1e-2)
    return [math.exp(lo + (hi - lo) * float(u[t, j])) for j in range(n_groups)]


def _c4_grads(wl: Workload, t: int, out: torch.Tensor) -> None:
    g = _gen(out.device, wl.seed * 1000 + t + 37)
    scales = _c4_scales(wl, t)
    for w in range(wl.W):
        o = 0
        for j, tn in enumerate(wl.tensors):
            out[w, o : o + tn.numel].normal_(0.0, scales[j // 2], generator=g)
            o += tn.numel


# ---- config 5: flat 2^30 in 96 layers -----------------------------------------


def _c5_weights(wl: Workload, device: torch.device) -> torch.Tensor:
    g = _gen(device, wl.seed * 7919 + 5)
    w = torch.empty(wl.N, dtype=torch.float32, device=device)
    _fill_normal(w, 0.02, g)
    return w


def _c5_grads(wl: Workload, t: int, out: torch.Tensor) -> None:
    # Student-t(3) = z / sqrt(chi2_3 / 3), scaled by 1e-4
    g = _gen(out.device, wl.seed * 1000 + t + 41)
    flat = out.view(-1)
    for s in range(0, flat.numel(), _CHUNK):
        seg = flat[s : s + _CHUNK]
        chi = torch.zeros_like(seg)
        tmp = torch.empty_like(seg)
        for _ in range(3):
            tmp.normal_(0.0, 1.0, generator=g)
            chi.addcmul_(tmp, tmp)
        chi.div_(3.0).sqrt_()
        seg.normal_(0.0, 1.0, generator=g)
        seg.div_(chi).mul_(1e-4)


def split_equal(total: int, parts: int) -> List[int]:
    """`parts` sizes summing to `total`; the first (total % parts) get one extra."""
    base, extra = divmod(total, parts)
    return [base + (1 if i < extra else 0) for i in range(parts)]


# --------------------------------------------------------------------------
# registry
# --------------------------------------------------------------------------


def single_layer(seed: int = 0) -> Workload:
    return Workload(
        "single_layer_1m_w4", [1 << 20], 4, 64.0, 1e-8, 3, seed,
        "one fp32 layer of 2^20, W=4, keep 1/64; weights N(0,0.05) with 1% exact zeros, grads N(0,1e-3)",
        _c1_weights, _c1_grads,
    )


def alexnet_w8(seed: int = 0) -> Workload:
    ts = alexnet_tensors()
    return Workload(
        "alexnet_w8_r64", [t.numel for t in ts], 8, 64.0, 1e-8, 5, seed,
        "AlexNet-shaped 16 tensors, W=8, keep 1/64; He-normal weights, zero biases, grads N(0, 0.01*std)",
        _tensorlist_weights, _c2_grads, ts,
    )


def resnet50_w8(seed: int = 0) -> Workload:
    ts = resnet50_tensors()
    return Workload(
        "resnet50_w8_r58.8", [t.numel for t in ts], 8, 58.8, 1e-8, 5, seed,
        "ResNet-50-shaped 161 tensors, W=8, keep 1/58.8 rounded up; He-normal weights, gamma=1, beta=0, Laplace(0,1e-4) grads",
        _tensorlist_weights, _c3_grads, ts,
    )


def alexnet_w32(seed: int = 0) -> Workload:
    ts = alexnet_tensors()
    return Workload(
        "alexnet_w32_r256", [t.numel for t in ts], 32, 256.0, 1e-8, 20, seed,
        "AlexNet-shaped 16 tensors, W=32, keep 1/256; grads N(0, s) with s log-uniform in [1e-5,1e-2] per (layer, step)",
        _tensorlist_weights, _c4_grads, ts,
    )


def flat_1g_w4(seed: int = 0) -> Workload:
    return Workload(
        "flat_2p30_96l_w4_r1000", split_equal(1 << 30, 96), 4, 1000.0, 1e-8, 10, seed,
        "2^30 fp32 in 96 near-equal layers, W=4, keep 1/1000; weights N(0,0.02), grads 1e-4*Student-t(3)",
        _c5_weights, _c5_grads,
    )


def scaled(wl: Workload, layer_sizes: List[int], W: Optional[int] = None, steps: Optional[int] = None,
           name: Optional[str] = None) -> Workload:
    """Same value recipe on a different (usually smaller) size list; tensor kinds and
    fan-ins are kept position by position so that the value structure survives."""
    ts = None
    if wl.tensors is not None:
        assert len(layer_sizes) == len(wl.tensors)
        ts = [Tensor(t.name, int(n), t.kind, t.fan_in) for t, n in zip(wl.tensors, layer_sizes)]
    return Workload(
        name or (wl.name + "_scaled"), [int(n) for n in layer_sizes], W or wl.W, wl.ratio, wl.eps,
        steps or wl.steps, wl.seed, wl.describe + " (scaled sizes)", wl._weights_fn, wl._grads_fn, ts,
    )


def subset(wl: Workload, lo: int, hi: int, W: Optional[int] = None, name: Optional[str] = None) -> Workload:
    """Layers lo..hi-1 of a workload with the same value recipe (a smaller case of the same kind,
    e.g. for a profiler capture that must stay within a few GB)."""
    ts = wl.tensors[lo:hi] if wl.tensors is not None else None
    return Workload(
        name or f"{wl.name}[{lo}:{hi}]", wl.layer_sizes[lo:hi], W or wl.W, wl.ratio, wl.eps, wl.steps, wl.seed,
        wl.describe + f" (layers {lo}..{hi - 1} only)", wl._weights_fn, wl._grads_fn, ts,
    )


CONFIGS = {
    "single_layer": single_layer,
    "alexnet_w8": alexnet_w8,
    "resnet50_w8": resnet50_w8,
    "alexnet_w32": alexnet_w32,
    "flat_1g_w4": flat_1g_w4,
}
