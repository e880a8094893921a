"""Thin ctypes binding of the C-ABI library (include/iwp.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
torch supplies device memory and the stream.  There is no CPU fallback: if the shared
library is missing or a CUDA call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

HERE = os.path.dirname(os.path.abspath(__file__))
# IWP_LIB_VARIANT=debug loads the build with range and count checks in every kernel (same ABI, slower)
LIB_PATH = os.path.join(HERE, "libiwp_debug.so" if os.environ.get("IWP_LIB_VARIANT") == "debug" else "libiwp.so")

IWP_OK, IWP_ERR_INVALID, IWP_ERR_OOM, IWP_ERR_CUDA, IWP_ERR_INTERNAL, IWP_ERR_TIMEOUT = 0, -1, -2, -3, -4, -5
IWP_ERR_CAPACITY = -6

EXPORTS = [
    "iwp_strerror", "iwp_keep_count", "iwp_leader_at", "iwp_plan_sizes", "iwp_create", "iwp_destroy",
    "iwp_set_stream", "iwp_step", "iwp_step_host", "iwp_sync_status", "iwp_get_layout", "iwp_get_sizes",
    "iwp_get_step", "iwp_set_step", "iwp_get_leader", "iwp_get_residual", "iwp_set_residual",
    "iwp_get_selection", "iwp_get_mask", "iwp_reset", "iwp_set_option", "iwp_get_stat", "iwp_select_static",
    "iwp_set_momentum", "iwp_create_threshold", "iwp_set_thresholds", "iwp_get_list_length", "iwp_leaders_at",
    "iwp_set_layerwise", "iwp_get_layer_thresholds", "iwp_shard_select", "iwp_shard_gather", "iwp_shard_apply",
    "iwp_layer_leader_at", "iwp_encode_mask", "iwp_step_host_async", "iwp_host_wait", "iwp_select_static_status", "iwp_join", "iwp_wire_mask_bytes", "iwp_wire_pack", "iwp_wire_unpack",
]

_lib: Optional[C.CDLL] = None


class IwpError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {iwp_strerror(status)} ({status})")


def lib() -> C.CDLL:
    """Loads libiwp.so (built in-tree by paper_1901_01544_b200.build); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_1901_01544_b200.build` (needs nvcc); "
                "there is no CPU fallback")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, u64, f32, f64, cp = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_float, C.c_double, C.c_char_p
        L.iwp_strerror.restype, L.iwp_strerror.argtypes = cp, [C.c_int]
        L.iwp_keep_count.restype, L.iwp_keep_count.argtypes = i64, [i64, f64]
        L.iwp_leader_at.restype, L.iwp_leader_at.argtypes = i32, [u64, u64, i32]
        L.iwp_leaders_at.argtypes = [u64, u64, i32, i32, vp]
        L.iwp_layer_leader_at.restype, L.iwp_layer_leader_at.argtypes = i32, [u64, u64, i32, i32]
        L.iwp_plan_sizes.argtypes = [vp, i32, i32, f64, vp]
        L.iwp_create.argtypes = [C.POINTER(vp), vp, i32, i32, f64, f32, u64]
        L.iwp_create_threshold.argtypes = [C.POINTER(vp), vp, i32, i32, f32, u64, i64]
        L.iwp_set_thresholds.argtypes = [vp, vp]
        L.iwp_get_list_length.argtypes = [vp, vp]
        L.iwp_set_layerwise.argtypes = [vp, i32, f64, f64, f64]
        L.iwp_get_layer_thresholds.argtypes = [vp, vp, vp]
        L.iwp_destroy.argtypes = [vp]
        L.iwp_set_stream.argtypes = [vp, vp]
        L.iwp_set_momentum.argtypes = [vp, f32]
        L.iwp_step.argtypes = [vp, vp, vp, vp]
        L.iwp_step_host.argtypes = [vp, vp, vp, vp]
        L.iwp_step_host_async.argtypes = [vp, vp, vp, vp]
        L.iwp_host_wait.argtypes = [vp]
        L.iwp_shard_select.argtypes = [vp, vp, vp, vp]
        L.iwp_shard_gather.argtypes = [vp, vp, i64, vp]
        L.iwp_shard_apply.argtypes = [vp, vp, i64, vp, i32, vp]
        L.iwp_sync_status.argtypes = [vp]
        L.iwp_join.argtypes = [vp]
        L.iwp_wire_mask_bytes.restype, L.iwp_wire_mask_bytes.argtypes = i64, [i64]
        L.iwp_wire_pack.argtypes = [vp, vp, i64, vp]
        L.iwp_wire_unpack.argtypes = [vp, vp, vp, i64, vp]
        L.iwp_get_layout.argtypes = [vp, vp, vp]
        L.iwp_get_sizes.argtypes = [vp, vp]
        L.iwp_get_step.argtypes = [vp, vp]
        L.iwp_set_step.argtypes = [vp, i64]
        L.iwp_get_leader.argtypes = [vp, vp]
        L.iwp_get_residual.argtypes = [vp, i32, vp]
        L.iwp_set_residual.argtypes = [vp, i32, vp]
        L.iwp_get_selection.argtypes = [vp, i32, vp, vp]
        L.iwp_get_mask.argtypes = [vp, vp]
        L.iwp_encode_mask.argtypes = [vp, vp, vp]
        L.iwp_reset.argtypes = [vp]
        L.iwp_set_option.argtypes = [vp, cp, i64]
        L.iwp_get_stat.argtypes = [vp, cp, vp]
        L.iwp_select_static.argtypes = [vp, vp, i64, f64, f32, vp, vp, vp, vp]
        L.iwp_select_static_status.argtypes = [vp, vp]
        for name in EXPORTS:
            getattr(L, name)  # AttributeError if the library does not export a declared symbol
        _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != IWP_OK:
        raise IwpError(status, where)


# ---- functions with the C names (raw status codes are turned into exceptions) ---------------


def iwp_strerror(status: int) -> str:
    return lib().iwp_strerror(status).decode()


def iwp_keep_count(n: int, ratio: float) -> int:
    return int(lib().iwp_keep_count(n, ratio))


def iwp_leader_at(seed: int, t: int, W: int) -> int:
    return int(lib().iwp_leader_at(seed, t, W))


def iwp_leaders_at(seed: int, t: int, W: int, n: int) -> List[int]:
    out = (C.c_int32 * n)()
    _check(lib().iwp_leaders_at(seed, t, W, n, out), "iwp_leaders_at")
    return list(out)


def iwp_plan_sizes(layer_sizes: Sequence[int], W: int, ratio: float) -> dict:
    arr = (C.c_int64 * len(layer_sizes))(*layer_sizes)
    out = (C.c_int64 * 8)()
    _check(lib().iwp_plan_sizes(arr, len(layer_sizes), W, ratio, out), "iwp_plan_sizes")
    keys = ["N", "K", "small_layers", "tiled_layers", "tiles", "chunks", "device_bytes", "vector_ok"]
    return dict(zip(keys, [int(v) for v in out]))


def iwp_create(layer_sizes: Sequence[int], W: int, ratio: float, eps: float, seed: int) -> C.c_void_p:
    arr = (C.c_int64 * len(layer_sizes))(*layer_sizes)
    h = C.c_void_p()
    _check(lib().iwp_create(C.byref(h), arr, len(layer_sizes), W, ratio, eps, seed), "iwp_create")
    return h


def iwp_create_threshold(layer_sizes: Sequence[int], W: int, eps: float, seed: int, max_list: int = 0) -> C.c_void_p:
    arr = (C.c_int64 * len(layer_sizes))(*layer_sizes)
    h = C.c_void_p()
    _check(lib().iwp_create_threshold(C.byref(h), arr, len(layer_sizes), W, eps, seed, max_list),
           "iwp_create_threshold")
    return h


def iwp_destroy(h) -> None:
    _check(lib().iwp_destroy(h), "iwp_destroy")


def iwp_step(h, grads_ptr: int, weights_ptr: int, update_ptr: int) -> None:
    _check(lib().iwp_step(h, grads_ptr, weights_ptr, update_ptr), "iwp_step")


def iwp_step_host(h, grads_ptr: int, weights_ptr: int, update_ptr: int) -> None:
    _check(lib().iwp_step_host(h, grads_ptr, weights_ptr, update_ptr), "iwp_step_host")


def iwp_select_static(residual_ptr: int, weights_ptr: int, n: int, ratio: float, eps: float, idx_ptr: int,
                      val_ptr: int, stream: int = 0) -> int:
    """Top-k list of one layer without any allocation (see include/iwp.h); returns k."""
    k = C.c_int64()
    _check(lib().iwp_select_static(residual_ptr, weights_ptr, n, ratio, eps, idx_ptr, val_ptr, C.byref(k),
                                   C.c_void_p(stream)), "iwp_select_static")
    return int(k.value)


def iwp_wire_mask_bytes(N: int) -> int:
    return int(lib().iwp_wire_mask_bytes(N))


def iwp_select_static_status(stream: int = 0) -> int:
    """Device status word of the last iwp_select_static() call on the current device (waits for `stream`)."""
    v = C.c_int32()
    _check(lib().iwp_select_static_status(C.byref(v), C.c_void_p(stream)), "iwp_select_static_status")
    return int(v.value)


# ---- convenience wrapper over torch tensors ----------------------------------------------------


class Pruner:
    """Owns one iwp context; takes torch CUDA tensors (device memory and stream only)."""

    def __init__(self, layer_sizes: Sequence[int], W: int, ratio: Optional[float], eps: float = 1e-8, seed: int = 0,
                 thresholds: Optional[Sequence[float]] = None, max_list: int = 0):
        """ratio mode: `ratio` = compression factor.  Threshold mode (Algorithm 1 as printed): pass
        ratio=None and per-layer `thresholds`; `max_list` bounds the index list (0 = N entries)."""
        import torch

        if not torch.cuda.is_available():
            raise RuntimeError("iwp needs a CUDA device; there is no CPU fallback")
        self._torch = torch
        self.threshold_mode = ratio is None
        if self.threshold_mode:
            self._h = iwp_create_threshold(list(layer_sizes), W, float(eps), int(seed), int(max_list))
        else:
            self._h = iwp_create(list(layer_sizes), W, float(ratio), float(eps), int(seed))
        out = (C.c_int64 * 4)()
        _check(lib().iwp_get_sizes(self._h, out), "iwp_get_sizes")
        self.N, self.K, self.L, self.W = (int(v) for v in out)
        self.device = torch.device("cuda", torch.cuda.current_device())
        self.use_current_stream()
        if thresholds is not None:
            self.set_thresholds(thresholds)

    # life cycle
    def close(self) -> None:
        if getattr(self, "_h", None):
            iwp_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def use_current_stream(self) -> None:
        s = self._torch.cuda.current_stream().cuda_stream
        _check(lib().iwp_set_stream(self._h, C.c_void_p(s)), "iwp_set_stream")

    # the step
    def _check_inputs(self, grads, weights, update) -> None:
        t = self._torch
        assert grads.is_cuda and grads.dtype == t.float32 and grads.is_contiguous() and grads.numel() == self.W * self.N
        assert weights.is_cuda and weights.dtype == t.float32 and weights.is_contiguous() and weights.numel() == self.N
        assert update.is_cuda and update.dtype == t.float32 and update.is_contiguous() and update.numel() == self.N

    def step(self, grads, weights, update=None):
        t = self._torch
        if update is None:
            update = t.empty(self.N, dtype=t.float32, device=grads.device)
        self._check_inputs(grads, weights, update)
        iwp_step(self._h, grads.data_ptr(), weights.data_ptr(), update.data_ptr())
        return update

    def step_host(self, grads, weights, update):
        """Host (ideally pinned) tensors in, host tensor out; copies are inside the call."""
        t = self._torch
        for x, n in ((grads, self.W * self.N), (weights, self.N), (update, self.N)):
            assert (not x.is_cuda) and x.dtype == t.float32 and x.is_contiguous() and x.numel() == n
        iwp_step_host(self._h, grads.data_ptr(), weights.data_ptr(), update.data_ptr())
        return update

    def step_host_async(self, grads, weights, update) -> None:
        """Like step_host, but returns at once; consecutive calls overlap their copies.  Pinned host tensors,
        untouched until host_wait()."""
        t = self._torch
        for x, n in ((grads, self.W * self.N), (weights, self.N), (update, self.N)):
            assert (not x.is_cuda) and x.dtype == t.float32 and x.is_contiguous() and x.numel() == n and x.is_pinned()
        _check(lib().iwp_step_host_async(self._h, grads.data_ptr(), weights.data_ptr(), update.data_ptr()),
               "iwp_step_host_async")

    def host_wait(self) -> None:
        _check(lib().iwp_host_wait(self._h), "iwp_host_wait")

    # the three phases of a step whose workers are spread over several contexts (see ShardedPruner)
    def shard_select(self, grads, weights, update) -> None:
        self._check_inputs(grads, weights, update)
        _check(lib().iwp_shard_select(self._h, grads.data_ptr(), weights.data_ptr(), update.data_ptr()), "iwp_shard_select")

    def shard_gather(self, idx):
        t = self._torch
        assert idx.is_cuda and idx.dtype == t.int32 and idx.is_contiguous()
        vals = t.empty((self.W, idx.numel()), dtype=t.float32, device=self.device)
        _check(lib().iwp_shard_gather(self._h, idx.data_ptr(), idx.numel(), vals.data_ptr()), "iwp_shard_gather")
        return vals

    def shard_apply(self, idx, vals_all, update) -> None:
        t = self._torch
        assert vals_all.is_cuda and vals_all.dtype == t.float32 and vals_all.is_contiguous()
        assert vals_all.dim() == 2 and vals_all.shape[1] == idx.numel()
        _check(lib().iwp_shard_apply(self._h, idx.data_ptr(), idx.numel(), vals_all.data_ptr(), int(vals_all.shape[0]),
                                     update.data_ptr()), "iwp_shard_apply")

    # the two wire formats of an index set (see ShardedPruner)
    def wire_pack(self, idx):
        """Index list -> mask at one bit per element (uint8 tensor of iwp_wire_mask_bytes(N) bytes)."""
        t = self._torch
        assert idx.is_cuda and idx.dtype == t.int32 and idx.is_contiguous()
        bits = t.empty(iwp_wire_mask_bytes(self.N), dtype=t.uint8, device=self.device)
        _check(lib().iwp_wire_pack(self._h, idx.data_ptr(), idx.numel(), bits.data_ptr()), "iwp_wire_pack")
        return bits

    def wire_unpack(self, bits, n: int):
        """Mask at one bit per element -> ascending index list of n entries (n = the number of set bits)."""
        t = self._torch
        assert bits.is_cuda and bits.dtype == t.uint8 and bits.is_contiguous() and bits.numel() == iwp_wire_mask_bytes(self.N)
        idx = t.empty(n, dtype=t.int32, device=self.device)
        _check(lib().iwp_wire_unpack(self._h, bits.data_ptr(), idx.data_ptr(), n, None), "iwp_wire_unpack")
        return idx

    def set_thresholds(self, thr: Sequence[float]) -> None:
        arr = (C.c_float * self.L)(*[float(x) for x in thr])
        _check(lib().iwp_set_thresholds(self._h, arr), "iwp_set_thresholds")

    def set_layerwise(self, alpha: float, beta: float, c: float, on: bool = True) -> None:
        """Section 3.4: per-layer thresholds alpha +/- beta * var/mean from each chosen node's importances."""
        _check(lib().iwp_set_layerwise(self._h, int(on), float(alpha), float(beta), float(c)), "iwp_set_layerwise")

    def layer_thresholds(self):
        """[chosen node][layer] thresholds of the last layer-wise step (a CUDA float tensor)."""
        out = self._torch.empty((8, self.L), dtype=self._torch.float32, device=self.device)
        n = C.c_int32()
        _check(lib().iwp_get_layer_thresholds(self._h, out.data_ptr(), C.byref(n)), "iwp_get_layer_thresholds")
        return out[: int(n.value)]

    def list_length(self) -> int:
        v = C.c_int64()
        _check(lib().iwp_get_list_length(self._h, C.byref(v)), "iwp_get_list_length")
        return int(v.value)

    def set_momentum(self, m: float) -> None:
        _check(lib().iwp_set_momentum(self._h, float(m)), "iwp_set_momentum")

    def join(self) -> None:
        """Orders the context's stream behind everything the last step left running on side streams."""
        _check(lib().iwp_join(self._h), "iwp_join")

    def sync_status(self) -> int:
        return int(lib().iwp_sync_status(self._h))

    def check(self) -> None:
        _check(self.sync_status(), "iwp_sync_status")

    # state and accessors
    def layout(self) -> Tuple[List[int], List[int]]:
        off = (C.c_int64 * self.L)()
        k = (C.c_int64 * self.L)()
        _check(lib().iwp_get_layout(self._h, off, k), "iwp_get_layout")
        return list(off), list(k)

    @property
    def t(self) -> int:
        v = C.c_int64()
        _check(lib().iwp_get_step(self._h, C.byref(v)), "iwp_get_step")
        return int(v.value)

    def set_step(self, t: int) -> None:
        _check(lib().iwp_set_step(self._h, t), "iwp_set_step")

    @property
    def leader(self) -> int:
        v = C.c_int32()
        _check(lib().iwp_get_leader(self._h, C.byref(v)), "iwp_get_leader")
        return int(v.value)

    def residual(self, w: int):
        out = self._torch.empty(self.N, dtype=self._torch.float32, device=self.device)
        _check(lib().iwp_get_residual(self._h, w, out.data_ptr()), "iwp_get_residual")
        return out

    def set_residual(self, w: int, src) -> None:
        assert src.is_cuda and src.dtype == self._torch.float32 and src.is_contiguous() and src.numel() == self.N
        _check(lib().iwp_set_residual(self._h, w, src.data_ptr()), "iwp_set_residual")

    def selection(self, w: int):
        t = self._torch
        idx = t.empty(self.K, dtype=t.int32, device=self.device)  # uint32 bit patterns
        val = t.empty(self.K, dtype=t.float32, device=self.device)
        _check(lib().iwp_get_selection(self._h, w, idx.data_ptr(), val.data_ptr()), "iwp_get_selection")
        return idx, val

    def mask(self):
        m = self._torch.empty(self.N, dtype=self._torch.uint8, device=self.device)
        _check(lib().iwp_get_mask(self._h, m.data_ptr()), "iwp_get_mask")
        return m

    def mask_bits(self):
        """The index set of the last step at eight elements per byte (bit i % 8 of byte i / 8)."""
        m = self.mask()
        bits = self._torch.empty((self.N + 7) // 8, dtype=self._torch.uint8, device=self.device)
        _check(lib().iwp_encode_mask(self._h, m.data_ptr(), bits.data_ptr()), "iwp_encode_mask")
        return bits

    def reset(self) -> None:
        _check(lib().iwp_reset(self._h), "iwp_reset")

    def set_option(self, key: str, value: int) -> None:
        _check(lib().iwp_set_option(self._h, key.encode(), int(value)), f"iwp_set_option({key})")

    def stat(self, key: str) -> int:
        v = C.c_int64()
        _check(lib().iwp_get_stat(self._h, key.encode(), C.byref(v)), f"iwp_get_stat({key})")
        return int(v.value)


class ShardedPruner:
    """The W workers of a job spread over the ranks of a torch.distributed group, W / world consecutive
    workers per rank (rank r holds workers r * W_local .. (r + 1) * W_local - 1), one GPU per rank.

    A step is the ring deployment of the paper in three device phases and two collectives: every rank
    selects for its own workers; the chosen worker's index list is broadcast from the rank that holds it
    (Algorithm 1's AllGather of the encoded mask, here the sorted uint32 list); every rank gathers its
    workers' residuals at those indices; the gathered values are all-gathered (rank order = worker order)
    and every rank forms the sum over ALL workers in ascending order - bit for bit the update a single
    context of W workers computes - and zeroes what its own workers sent.  Only argument marshalling and
    the two collectives happen here; every step of the method runs in the library's kernels.

    What travels in the first collective (`wire`): "list" = the sorted uint32 index list (4 bytes per entry),
    "mask" = Algorithm 1's encoded mask at one bit per element (N / 8 bytes; packed on the owner and expanded
    on arrival by the library's kernels), "auto" (default) = whichever is shorter for the step's index set:
    the list when the set holds fewer than N / 32 entries.  `last_wire` names the last step's choice.

    `engine`: the per-rank object with shard_select / selection / shard_gather / shard_apply (default: a
    Pruner on the current CUDA device)."""

    def __init__(self, layer_sizes: Sequence[int], W_total: int, ratio: float, eps: float = 1e-8, seed: int = 0,
                 group=None, engine=None, wire: str = "auto"):
        import torch
        import torch.distributed as dist

        self._torch, self._dist, self.group = torch, dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        if W_total < 1 or W_total % self.world != 0:
            raise ValueError("the number of workers must be a positive multiple of the group size")
        self.W_total, self.W_local, self.seed, self.t = W_total, W_total // self.world, int(seed), 0
        self.leader_override = -1
        self.leader = -1
        if wire not in ("auto", "list", "mask"):
            raise ValueError("wire must be 'auto', 'list' or 'mask'")
        self.wire, self.last_wire, self.wire_bytes = wire, None, 0
        self.local = engine if engine is not None else Pruner(layer_sizes, self.W_local, ratio, eps, seed)
        self.N, self.K = self.local.N, self.local.K

    def _global_rank(self, group_rank: int) -> int:
        return group_rank if self.group is None else self._dist.get_global_rank(self.group, group_rank)

    def step(self, grads_local, weights, update):
        """grads_local: this rank's [W_local, N] gradients; weights [N]; update [N] (fully overwritten, the
        same on every rank)."""
        t, dist = self._torch, self._dist
        leader = self.leader_override if self.leader_override >= 0 else iwp_leader_at(self.seed, self.t, self.W_total)
        owner, local_worker = divmod(leader, self.W_local)
        self.local.shard_select(grads_local, weights, update)
        n = self.K  # ratio mode: every step's index set has K entries, known to every rank
        mask_bytes = 4 * ((self.N + 31) // 32)
        use_mask = self.wire == "mask" or (self.wire == "auto" and 4 * n >= mask_bytes)
        if use_mask:  # the encoded mask travels; every rank but the owner expands it back into the list
            if self.rank == owner:
                idx = self.local.selection(local_worker)[0]
                bits = self.local.wire_pack(idx)
            else:
                bits = t.empty(mask_bytes, dtype=t.uint8, device=update.device)
            dist.broadcast(bits, src=self._global_rank(owner), group=self.group)
            if self.rank != owner:
                idx = self.local.wire_unpack(bits, n)
        else:
            if self.rank == owner:
                idx = self.local.selection(local_worker)[0]
            else:
                idx = t.empty(n, dtype=t.int32, device=update.device)
            dist.broadcast(idx, src=self._global_rank(owner), group=self.group)
        self.last_wire, self.wire_bytes = ("mask" if use_mask else "list"), (mask_bytes if use_mask else 4 * n)
        vals_local = self.local.shard_gather(idx)
        vals_all = t.empty((self.W_total, self.K), dtype=t.float32, device=update.device)
        dist.all_gather_into_tensor(vals_all, vals_local, group=self.group)
        self.local.shard_apply(idx, vals_all, update)
        self.leader, self.t = leader, self.t + 1
        return update

    def close(self) -> None:
        self.local.close()
