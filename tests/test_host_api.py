"""CPU-only checks of the C-ABI library: it builds, loads, exports every symbol the header
declares, and its pure host helpers agree with the printed tables.  No compute calls."""
import ctypes as C
import os
import re

import pytest

from paper_1901_01544_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLD = os.path.join(ROOT, "tests", "golden")


@pytest.fixture(scope="module")
def L():
    build.build()
    return binding.lib()


def _declared():
    src = open(os.path.join(ROOT, "include", "iwp.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(iwp_[a-z_0-9]+)\s*\(", src)))


def test_header_and_library_agree(L):
    names = _declared()
    assert len(names) >= 20 and {"iwp_create", "iwp_step", "iwp_destroy"} <= set(names)
    for n in names:
        assert hasattr(L, n), f"libiwp.so does not export {n}"
    assert sorted(binding.EXPORTS) == names  # the binding marshals every declared entry point


def test_keep_count_matches_table(L):
    for line in open(os.path.join(GOLD, "keep_counts.txt")):
        if line.startswith("#") or not line.strip():
            continue
        R, n, k = line.split()
        assert binding.iwp_keep_count(int(n), float(R)) == int(k), line
    assert binding.iwp_keep_count(0, 2.0) == 0 and binding.iwp_keep_count(5, 0.5) == 0
    assert binding.iwp_keep_count(5, float("nan")) == 0


def test_leader_matches_vectors(L):
    for line in open(os.path.join(GOLD, "leader_vectors.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, vals = line.split(":")
        seed, W = (int(x) for x in head.split())
        want = [int(x) for x in vals.split()]
        assert [binding.iwp_leader_at(seed, t, W) for t in range(len(want))] == want
    assert binding.iwp_leader_at(0, 0, 0) == -1


def test_leader_sets_match_vectors(L):
    for line in open(os.path.join(GOLD, "leader_sets.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, body = line.split(":")
        seed, W, n = (int(x) for x in head.split())
        for t, step in enumerate(body.split("|")):
            assert binding.iwp_leaders_at(seed, t, W, n) == [int(x) for x in step.split()]
    out = (C.c_int32 * 9)()
    E = binding.IWP_ERR_INVALID
    assert L.iwp_leaders_at(0, 0, 4, 5, out) == E and L.iwp_leaders_at(0, 0, 16, 9, out) == E
    assert L.iwp_leaders_at(0, 0, 4, 0, out) == E and L.iwp_leaders_at(0, 0, 4, 2, None) == E


def test_plan_sizes(L):
    from paper_1901_01544_b200 import workloads as wl

    a = binding.iwp_plan_sizes(wl.alexnet_w8().layer_sizes, 8, 64.0)
    assert (a["N"], a["K"]) == (60965224, 952583) and a["vector_ok"] == 1
    assert a["small_layers"] == 8 and a["tiled_layers"] == 8  # the eight bias vectors fit one CTA each
    r = binding.iwp_plan_sizes(wl.resnet50_w8().layer_sizes, 8, 58.8)
    assert (r["N"], r["K"]) == (25557032, 434735)
    assert r["small_layers"] + r["tiled_layers"] == 161 and r["small_layers"] >= 108
    f = binding.iwp_plan_sizes(wl.flat_1g_w4().layer_sizes, 4, 1000.0)
    assert (f["N"], f["K"]) == (1 << 30, 1073760) and f["tiled_layers"] == 96
    assert f["tiles"] >= (1 << 30) // 4096 and f["tiles"] <= (1 << 30) // 4096 + 96
    assert f["device_bytes"] >= 4 * 4 * (1 << 30)
    # chunk size by job size: 128-tile chunks for the large jobs, 8-tile chunks for one small layer
    assert a["tiles"] == 14889 and a["chunks"] == 121
    one = binding.iwp_plan_sizes(wl.single_layer().layer_sizes, 4, 64.0)
    assert (one["tiles"], one["chunks"]) == (256, 32)
    assert f["chunks"] == 96 * 22  # 2731 tiles per layer in chunks of 128
    odd = binding.iwp_plan_sizes([5, 17, 40001], 3, 2.0)
    assert odd["N"] == 40023 and odd["vector_ok"] == 0 and odd["small_layers"] == 2 and odd["tiled_layers"] == 1


def test_wire_mask_bytes_is_a_host_function(L):
    assert binding.iwp_wire_mask_bytes(0) == 0 and binding.iwp_wire_mask_bytes(1) == 4
    assert binding.iwp_wire_mask_bytes(32) == 4 and binding.iwp_wire_mask_bytes(33) == 8
    assert binding.iwp_wire_mask_bytes(60965224) == 4 * ((60965224 + 31) // 32) and binding.iwp_wire_mask_bytes(-1) == -1


def test_invalid_arguments_are_rejected_without_a_gpu(L):
    h = C.c_void_p()
    sizes = (C.c_int64 * 2)(8, 8)
    bad = (C.c_int64 * 2)(8, 0)
    E = binding.IWP_ERR_INVALID
    assert L.iwp_create(None, sizes, 2, 2, 2.0, 1e-8, 0) == E
    assert L.iwp_create(C.byref(h), None, 2, 2, 2.0, 1e-8, 0) == E and not h.value
    assert L.iwp_create(C.byref(h), sizes, 0, 2, 2.0, 1e-8, 0) == E
    assert L.iwp_create(C.byref(h), bad, 2, 2, 2.0, 1e-8, 0) == E
    assert L.iwp_create(C.byref(h), sizes, 2, 0, 2.0, 1e-8, 0) == E
    assert L.iwp_create(C.byref(h), sizes, 2, 65536, 2.0, 1e-8, 0) == E
    assert L.iwp_create_threshold(C.byref(h), sizes, 2, 0, 1e-8, 0, 0) == E
    assert L.iwp_create_threshold(C.byref(h), sizes, 2, 2, 1e-8, 0, -1) == E
    assert L.iwp_create_threshold(None, sizes, 2, 2, 1e-8, 0, 0) == E
    assert L.iwp_set_thresholds(None, None) == E and L.iwp_get_list_length(None, None) == E
    assert L.iwp_set_momentum(None, 0.5) == E
    assert L.iwp_create(C.byref(h), sizes, 2, 2, 0.5, 1e-8, 0) == E
    assert L.iwp_create(C.byref(h), sizes, 2, 2, float("inf"), 1e-8, 0) == E
    assert L.iwp_create(C.byref(h), sizes, 2, 2, 2.0, 0.0, 0) == E
    assert L.iwp_create(C.byref(h), sizes, 2, 2, 2.0, float("nan"), 0) == E
    huge = (C.c_int64 * 2)(1 << 31, 1 << 31)
    assert L.iwp_create(C.byref(h), huge, 2, 1, 2.0, 1e-8, 0) == E  # N >= 2^32
    assert L.iwp_destroy(None) == 0
    for fn in (L.iwp_step, L.iwp_step_host):
        assert fn(None, None, None, None) == E
    assert L.iwp_sync_status(None) == E and L.iwp_reset(None) == E
    assert L.iwp_set_option(None, b"speculate", 1) == E
    out = (C.c_int64 * 8)()
    assert L.iwp_plan_sizes(bad, 2, 2, 2.0, out) == E and L.iwp_plan_sizes(sizes, 2, 2, 2.0, None) == E
    assert binding.iwp_strerror(0) == "ok" and "invalid" in binding.iwp_strerror(E)
    assert binding.iwp_strerror(-99) == "unknown status"
