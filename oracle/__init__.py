"""ctypes front end of the CPU oracle.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library and its Python binding never do.
"""
from __future__ import annotations

import ctypes as C
from typing import List, Sequence, Tuple

import numpy as np

from .build import build as _build

_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(_build())
        vp, i32, i64, u64, f32, f64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_float, C.c_double
        L.oracle_create.restype = vp
        L.oracle_create.argtypes = [vp, i32, i32, f64, f32, u64]
        L.oracle_destroy.argtypes = [vp]
        L.oracle_step.argtypes = [vp, vp, vp, vp]
        L.oracle_reset.argtypes = [vp]
        L.oracle_set_threads.argtypes = [vp, i32]
        L.oracle_threads_used.argtypes = [vp]
        L.oracle_threads_used.restype = i32
        L.oracle_set_leader_override.argtypes = [vp, i32]
        L.oracle_set_momentum.argtypes = [vp, f32]
        L.oracle_set_thresholds.argtypes = [vp, vp]
        L.oracle_set_n_leaders.argtypes = [vp, i32]
        L.oracle_set_random_select.argtypes = [vp, i32]
        L.oracle_set_per_layer_leaders.argtypes = [vp, i32]
        L.oracle_layer_leader.argtypes = [u64, u64, u64, i32]
        L.oracle_layer_leader.restype = i32
        L.oracle_union_length.argtypes = [vp]
        L.oracle_union_length.restype = i64
        L.oracle_get_union.argtypes = [vp, vp]
        L.oracle_set_layerwise.argtypes = [vp, i32, f64, f64, f64]
        L.oracle_get_layer_thresholds.argtypes = [vp, vp]
        L.oracle_get_layer_thresholds.restype = i32
        L.oracle_exact_sum.argtypes = [vp, i64]
        L.oracle_exact_sum.restype = f64
        L.oracle_layerwise_threshold.argtypes = [vp, vp, i64, f32, f64, f64, f64, vp]
        L.oracle_layerwise_threshold.restype = f32
        L.oracle_draw24.argtypes = [u64, u64, u64]
        L.oracle_draw24.restype = C.c_uint32
        L.oracle_leaders.argtypes = [u64, u64, i32, i32, vp]
        L.oracle_threshold_list_length.argtypes = [vp]
        L.oracle_threshold_list_length.restype = i64
        L.oracle_get_threshold_list.argtypes = [vp, vp, vp]
        L.oracle_total.argtypes = [vp]
        L.oracle_total.restype = i64
        L.oracle_total_keep.argtypes = [vp]
        L.oracle_total_keep.restype = i64
        L.oracle_get_step.argtypes = [vp]
        L.oracle_get_step.restype = i64
        L.oracle_get_leader.argtypes = [vp]
        L.oracle_get_leader.restype = i32
        L.oracle_get_layout.argtypes = [vp, vp, vp]
        L.oracle_get_residual.argtypes = [vp, i32, vp]
        L.oracle_set_residual.argtypes = [vp, i32, vp]
        L.oracle_get_selection.argtypes = [vp, i32, vp, vp]
        L.oracle_get_mask.argtypes = [vp, vp]
        L.oracle_leader.argtypes = [u64, u64, i32]
        L.oracle_leader.restype = i32
        L.oracle_mix64.argtypes = [u64]
        L.oracle_mix64.restype = u64
        L.oracle_keep_count.argtypes = [i64, f64]
        L.oracle_keep_count.restype = i64
        L.oracle_importance_bits.argtypes = [f32, f32, f32]
        L.oracle_importance_bits.restype = C.c_uint32
        L.oracle_select.argtypes = [vp, vp, i64, i64, f32, vp]
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def leader(seed: int, t: int, W: int) -> int:
    return int(lib().oracle_leader(seed, t, W))


def mix64(z: int) -> int:
    return int(lib().oracle_mix64(z))


def draw24(seed: int, t: int, i: int) -> int:
    return int(lib().oracle_draw24(seed, t, i))


def leaders(seed: int, t: int, W: int, n: int) -> List[int]:
    out = np.empty(n, dtype=np.int32)
    lib().oracle_leaders(seed, t, W, n, _p(out))
    return out.tolist()


def layer_leader(seed: int, t: int, l: int, W: int) -> int:
    return int(lib().oracle_layer_leader(seed, t, l, W))


def keep_count(n: int, ratio: float) -> int:
    return int(lib().oracle_keep_count(n, ratio))


def importance_bits(acc: float, w: float, eps: float) -> int:
    return int(lib().oracle_importance_bits(acc, w, eps))


def exact_sum(x: np.ndarray) -> float:
    """Sum of non-negative finite doubles, exact, rounded once to binary64."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    return float(lib().oracle_exact_sum(_p(x), x.size))


def layerwise_threshold(acc: np.ndarray, w: np.ndarray, eps: float, alpha: float, beta: float, c: float):
    """Eq. 4 for one node and layer -> (thr as np.float32, dict of S1, S2, mean, var, v)."""
    acc = np.ascontiguousarray(acc, dtype=np.float32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    st = np.empty(5, dtype=np.float64)
    thr = lib().oracle_layerwise_threshold(_p(acc), _p(w), acc.size, eps, alpha, beta, c, _p(st))
    return np.float32(thr), dict(zip(("S1", "S2", "mean", "var", "v"), st.tolist()))


def select(acc: np.ndarray, w: np.ndarray, k: int, eps: float) -> np.ndarray:
    acc = np.ascontiguousarray(acc, dtype=np.float32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    out = np.empty(k, dtype=np.uint32)
    lib().oracle_select(_p(acc), _p(w), acc.size, k, eps, _p(out))
    return out


class Oracle:
    """W simulated workers' residuals on the host and the step that updates them."""

    def __init__(self, layer_sizes: Sequence[int], W: int, ratio: float, eps: float, seed: int, threads: int = 0):
        ls = np.asarray(list(layer_sizes), dtype=np.int64)
        self._h = lib().oracle_create(_p(ls), len(ls), W, float(ratio), float(eps), int(seed))
        if not self._h:
            raise ValueError("oracle_create rejected the arguments")
        self.L, self.W = len(ls), W
        self.N = int(lib().oracle_total(self._h))
        self.K = int(lib().oracle_total_keep(self._h))
        if threads:
            lib().oracle_set_threads(self._h, threads)

    def close(self):
        if self._h:
            lib().oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    @property
    def threads(self) -> int:
        return int(lib().oracle_threads_used(self._h))

    def layout(self) -> Tuple[List[int], List[int]]:
        off = np.empty(self.L, dtype=np.int64)
        k = np.empty(self.L, dtype=np.int64)
        lib().oracle_get_layout(self._h, _p(off), _p(k))
        return off.tolist(), k.tolist()

    def set_thresholds(self, thr):
        """Per-layer absolute thresholds: Algorithm 1 as printed (None: back to the ratio mode)."""
        if thr is None:
            lib().oracle_set_thresholds(self._h, None)
            return
        a = np.ascontiguousarray(thr, dtype=np.float32)
        assert a.size == self.L
        lib().oracle_set_thresholds(self._h, _p(a))

    def set_random_select(self, on: bool):
        """Threshold mode: Section 3.3's P(update) = importance / threshold for elements below the threshold."""
        lib().oracle_set_random_select(self._h, 1 if on else 0)

    def set_n_leaders(self, n: int):
        """Threshold mode: OR the masks of n distinct chosen nodes (Algorithm 1's r_1..r_n)."""
        assert 1 <= n <= self.W
        lib().oracle_set_n_leaders(self._h, n)

    def threshold_list(self) -> Tuple[np.ndarray, np.ndarray]:
        n = int(lib().oracle_threshold_list_length(self._h))
        idx = np.empty(n, dtype=np.uint32)
        val = np.empty(n, dtype=np.float32)
        lib().oracle_get_threshold_list(self._h, _p(idx), _p(val))
        return idx, val

    def set_momentum(self, m: float):
        lib().oracle_set_momentum(self._h, float(m))

    def set_leader_override(self, leader: int):
        lib().oracle_set_leader_override(self._h, leader)

    def set_per_layer_leaders(self, on: bool = True):
        """Ratio mode: every layer draws its own chosen node each step."""
        lib().oracle_set_per_layer_leaders(self._h, 1 if on else 0)

    def index_set(self) -> np.ndarray:
        """Ratio mode: the index set of the last step (union of the chosen nodes' lists), ascending."""
        out = np.empty(int(lib().oracle_union_length(self._h)), dtype=np.uint32)
        lib().oracle_get_union(self._h, _p(out))
        return out

    def set_layerwise(self, alpha: float, beta: float, c: float, on: bool = True):
        """Section 3.4: per-layer thresholds from each chosen node's own importance statistics."""
        lib().oracle_set_layerwise(self._h, int(on), alpha, beta, c)

    def layer_thresholds(self) -> np.ndarray:
        """[chosen node][layer] thresholds the last step derived (layer-wise mode)."""
        out = np.empty(self.W * self.L, dtype=np.float32)
        n = lib().oracle_get_layer_thresholds(self._h, _p(out))
        return out[: n * self.L].reshape(n, self.L).copy()

    def reset(self):
        lib().oracle_reset(self._h)

    def step(self, grads: np.ndarray, weights: np.ndarray) -> np.ndarray:
        assert grads.dtype == np.float32 and grads.flags.c_contiguous and grads.size == self.W * self.N
        assert weights.dtype == np.float32 and weights.flags.c_contiguous and weights.size == self.N
        update = np.empty(self.N, dtype=np.float32)
        lib().oracle_step(self._h, _p(grads), _p(weights), _p(update))
        return update

    @property
    def t(self) -> int:
        return int(lib().oracle_get_step(self._h))

    @property
    def leader(self) -> int:
        return int(lib().oracle_get_leader(self._h))

    def residual(self, w: int) -> np.ndarray:
        out = np.empty(self.N, dtype=np.float32)
        lib().oracle_get_residual(self._h, w, _p(out))
        return out

    def set_residual(self, w: int, src: np.ndarray):
        src = np.ascontiguousarray(src, dtype=np.float32)
        assert src.size == self.N
        lib().oracle_set_residual(self._h, w, _p(src))

    def selection(self, w: int) -> Tuple[np.ndarray, np.ndarray]:
        idx = np.empty(self.K, dtype=np.uint32)
        val = np.empty(self.K, dtype=np.float32)
        lib().oracle_get_selection(self._h, w, _p(idx), _p(val))
        return idx, val

    def mask(self) -> np.ndarray:
        m = np.empty(self.N, dtype=np.uint8)
        lib().oracle_get_mask(self._h, _p(m))
        return m
