"""Pins of the CPU oracle against things other than itself: hand-worked values,
closed forms, brute force (full sort) on tiny inputs, invariants, library routines
and special cases that reduce to a textbook operation.  CPU only."""
import json
import math
import os

import numpy as np
import pytest
import torch

import oracle
from bruteforce import BruteForce, bits, importance

GOLD = os.path.join(os.path.dirname(__file__), "golden")
F = np.float32


def u32(a):
    return np.asarray(a, dtype=np.float32).view(np.uint32)


# ---------------------------------------------------------------- leader, keep count


def _leader_rows():
    rows = []
    for line in open(os.path.join(GOLD, "leader_vectors.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, vals = line.split(":")
        seed, W = (int(x) for x in head.split())
        rows.append((seed, W, [int(x) for x in vals.split()]))
    return rows


@pytest.mark.parametrize("seed,W,expect", _leader_rows())
def test_leader_vectors(seed, W, expect):
    assert [oracle.leader(seed, t, W) for t in range(len(expect))] == expect


def test_mix64_vector():
    assert oracle.mix64(0x9E3779B97F4A7C15) == 0xE220A8397B1DCDAF


def test_leader_range_and_spread():
    for W in (1, 2, 3, 7, 33):
        got = [oracle.leader(12345, t, W) for t in range(4000)]
        assert min(got) >= 0 and max(got) < W
        counts = np.bincount(got, minlength=W)
        assert counts.min() > 0.7 * 4000 / W  # every worker gets its turn


def test_keep_count_table():
    n_rows = 0
    for line in open(os.path.join(GOLD, "keep_counts.txt")):
        if line.startswith("#") or not line.strip():
            continue
        R, n, k = line.split()
        assert oracle.keep_count(int(n), float(R)) == int(k), line
        n_rows += 1
    assert n_rows > 50


def test_keep_count_totals_of_tensor_lists():
    from paper_1901_01544_b200 import workloads as wl

    a = wl.alexnet_tensors()
    r = wl.resnet50_tensors()
    assert len(a) == 16 and sum(t.numel for t in a) == 60965224
    assert len(r) == 161 and sum(t.numel for t in r) == 25557032
    assert sum(oracle.keep_count(t.numel, 64.0) for t in a) == 952583
    assert sum(oracle.keep_count(t.numel, 58.8) for t in r) == 434735
    assert sum(oracle.keep_count(t.numel, 256.0) for t in a) == 238148
    f = wl.split_equal(1 << 30, 96)
    assert f[:64] == [11184811] * 64 and f[64:] == [11184810] * 32
    assert sum(oracle.keep_count(n, 1000.0) for n in f) == 1073760
    # N/K reproduces the paper's Table 1 compression ratios by construction
    assert abs(60965224 / 952583 - 64.0) < 1e-3
    assert abs(25557032 / 434735 - 58.8) < 2e-2


# ---------------------------------------------------------------- importance


def test_importance_closed_forms():
    eps = F(1e-8)
    assert int(u32(eps)) == 0x322BCC77
    # |w| + eps rounds back to |w| for these, so importance = |acc| / |w| exactly
    for a, w, want in [(0.5, 1.0, 0.5), (-0.25, -0.5, 0.5), (0.125, 0.25, 0.5), (-1.0, -0.5, 2.0), (0.0, 1.0, 0.0),
                       (-0.0, 1.0, 0.0), (3.0, -1.0, 3.0)]:
        assert oracle.importance_bits(a, w, 1e-8) == int(u32(want)), (a, w)
    # w = 0: importance = |acc| / eps
    assert oracle.importance_bits(2.0 ** -20, 0.0, 1e-8) == 0x42BEBC20
    assert oracle.importance_bits(-(2.0 ** -21), -0.0, 1e-8) == 0x423EBC20
    # the guard is really added: 0.125 + 1e-8 is not 0.125 in binary32
    assert oracle.importance_bits(0.125, 0.125, 1e-8) != int(u32(1.0))
    assert oracle.importance_bits(0.125, 0.125, 1e-8) == int(u32(F(0.125) / (F(0.125) + eps)))
    # sign of either operand never matters; result is never negative
    rng = np.random.default_rng(0)
    for a, w in rng.normal(size=(200, 2)).astype(np.float32):
        b = oracle.importance_bits(a, w, 1e-8)
        assert b == oracle.importance_bits(-a, w, 1e-8) == oracle.importance_bits(a, -w, 1e-8)
        assert b < 0x80000000
        assert b == bits(importance(a, w, 1e-8))
    # denormals are kept, not flushed
    tiny = np.array([1], dtype=np.uint32).view(np.float32)[0]
    assert oracle.importance_bits(tiny, 1.0, 1e-8) == 1


def test_importance_monotone_in_magnitude():
    w = F(0.3)
    a = np.sort(np.abs(np.random.default_rng(1).normal(size=500)).astype(np.float32))
    keys = [oracle.importance_bits(x, w, 1e-8) for x in a]
    assert all(k0 <= k1 for k0, k1 in zip(keys, keys[1:]))


# ---------------------------------------------------------------- selection: brute force


def _brute_select(acc, w, k, eps):
    imp = [bits(importance(a, x, eps)) for a, x in zip(acc, w)]
    order = sorted(range(len(acc)), key=lambda i: (-imp[i], i))
    return sorted(order[:k])


def _adversarial(n, rng):
    yield np.zeros(n, np.float32), np.ones(n, np.float32)  # all keys equal (zero)
    yield np.full(n, 0.5, np.float32), np.full(n, -2.0, np.float32)  # all equal, non-zero
    yield rng.choice(np.array([0.25, 1.0], np.float32), n), np.ones(n, np.float32)  # two distinct values
    yield rng.normal(size=n).astype(np.float32), np.zeros(n, np.float32)  # every weight zero
    a = rng.normal(size=n).astype(np.float32)
    yield a, a.copy()  # importance ~ 1 everywhere, near-ties
    yield rng.integers(-3, 4, n).astype(np.float32), rng.integers(-2, 3, n).astype(np.float32)  # many ties, zeros


@pytest.mark.parametrize("n", [1, 2, 3, 7, 8, 31, 64])
def test_select_equals_full_sort(n):
    rng = np.random.default_rng(n)
    cases = list(_adversarial(n, rng))
    for _ in range(6):
        cases.append((rng.normal(size=n).astype(np.float32), (rng.normal(size=n) * (rng.random(n) > 0.2)).astype(np.float32)))
    for acc, w in cases:
        for k in sorted({1, max(1, n // 4), max(1, n // 2), n}):
            got = oracle.select(acc, w, k, 1e-8).tolist()
            assert got == _brute_select(acc, w, k, F(1e-8)), (n, k)


@pytest.mark.parametrize("layers,W,ratio", [([8], 2, 4.0), ([5, 1, 12, 3], 3, 3.0), ([64], 4, 64.0), ([17, 9], 1, 1.0),
                                            ([6, 6], 5, 2.5)])
def test_step_equals_bruteforce_model(layers, W, ratio):
    rng = np.random.default_rng(sum(layers) + W)
    N = sum(layers)
    weights = (rng.normal(size=N) * (rng.random(N) > 0.15)).astype(np.float32)
    orc = oracle.Oracle(layers, W, ratio, 1e-8, seed=3)
    bf = BruteForce(layers, W, ratio, 1e-8)
    for t in range(4):
        # coarse values make ties and exact cancellations frequent
        grads = (rng.integers(-4, 5, size=(W, N)) / 8.0).astype(np.float32)
        upd = orc.step(grads, weights)
        lists, upd_bf = bf.step(grads, weights, orc.leader)
        assert orc.leader == oracle.leader(3, t, W)
        assert np.array_equal(u32(upd), u32(upd_bf))
        for w in range(W):
            idx, val = orc.selection(w)
            assert idx.tolist() == [i for i, _ in lists[w]]
            assert np.array_equal(u32(val), u32(np.array([v for _, v in lists[w]], np.float32)))
            assert np.array_equal(u32(orc.residual(w)), u32(bf.residual(w)))


# ---------------------------------------------------------------- hand-worked example


def test_worked_example():
    g = json.load(open(os.path.join(GOLD, "worked_example.json")))
    orc = oracle.Oracle(g["layer_sizes"], g["W"], g["ratio"], g["eps"], seed=0)
    assert orc.layout() == ([0], [2])
    weights = np.array(g["weights"], np.float32)
    for st in g["steps"]:
        orc.set_leader_override(st["leader"])
        upd = orc.step(np.array(st["grads"], np.float32), weights)
        assert orc.leader == st["leader"]
        assert np.array_equal(u32(upd), u32(np.array(st["update"], np.float32)))  # includes +0 for the cancellation
        for w in range(g["W"]):
            idx, val = orc.selection(w)
            assert idx.tolist() == st["lists"][w]
            assert np.array_equal(u32(val), u32(np.array(st["list_vals"][w], np.float32)))
            assert np.array_equal(u32(orc.residual(w)), u32(np.array(st["residual"][w], np.float32)))
        mask = orc.mask()
        assert mask.tolist() == [1 if i in st["lists"][st["leader"]] else 0 for i in range(8)]
    assert oracle.importance_bits(2.0 ** -20, 0.0, 1e-8) == int(g["steps"][0]["importance_bits_w0_idx2"], 16)
    assert oracle.importance_bits(2.0 ** -21, 0.0, 1e-8) == int(g["steps"][1]["importance_bits_w1_idx2"], 16)
    m = g["mini"]
    o2 = oracle.Oracle(m["layer_sizes"], m["W"], m["ratio"], m["eps"], seed=0)
    o2.step(np.array(m["grads"], np.float32), np.array(m["weights"], np.float32))
    assert o2.selection(0)[0].tolist() == m["list"]


# ---------------------------------------------------------------- invariants and library routines


def _random_problem(layers, W, seed, zero_frac=0.05):
    rng = np.random.default_rng(seed)
    N = sum(layers)
    weights = (rng.normal(scale=0.05, size=N) * (rng.random(N) > zero_frac)).astype(np.float32)
    return rng, weights


def test_invariants_and_library_threshold():
    layers, W, R = [5000, 333, 20000, 64, 1], 4, 16.0
    rng, weights = _random_problem(layers, W, 11)
    N = sum(layers)
    orc = oracle.Oracle(layers, W, R, 1e-8, seed=5)
    off, ks = orc.layout()
    assert ks == [math.ceil(n / R) for n in layers]
    acc_model = np.zeros((W, N), np.float32)
    for t in range(3):
        grads = rng.normal(scale=1e-3, size=(W, N)).astype(np.float32)
        acc_model = acc_model + grads  # fp32 elementwise
        upd = orc.step(grads, weights)
        S, _ = orc.selection(orc.leader)
        assert len(S) == orc.K == sum(ks)
        imp = np.abs(acc_model) / (np.abs(weights) + F(1e-8))  # fp32 arithmetic in numpy
        assert imp.dtype == np.float32
        for w in range(W):
            idx, val = orc.selection(w)
            assert np.array_equal(u32(val), u32(acc_model[w, idx]))
            seg = 0
            for o, n, k in zip(off, layers, ks):
                loc = idx[seg:seg + k].astype(np.int64) - o
                seg += k
                assert np.all(np.diff(loc) > 0) and loc.min() >= 0 and loc.max() < n  # ascending, inside the layer
                li = imp[w, o:o + n]
                inside = np.zeros(n, bool)
                inside[loc] = True
                # threshold value = k-th largest, by two independent library routines
                T = li[inside].min()
                assert T == np.partition(li, n - k)[n - k]
                assert T == torch.kthvalue(torch.from_numpy(li.copy()), n - k + 1).values.item()
                if k < n:
                    assert T >= li[~inside].max()
                    ties_in = np.flatnonzero(inside & (li == T))
                    ties_out = np.flatnonzero(~inside & (li == T))
                    if len(ties_out):
                        assert ties_in.max() < ties_out.min()  # lower index wins the tie
                    else:
                        top = torch.topk(torch.from_numpy(li.copy()), k).indices.numpy()
                        assert set(top.tolist()) == set(loc.tolist())
        # shared index set keeps the reduced tensor sparse; everything off S is +0
        offS = np.ones(N, bool)
        offS[S] = False
        assert np.all(u32(upd[offS]) == 0) and np.count_nonzero(upd) <= orc.K
        # ordered worker sum at S
        s = acc_model[0, S].copy()
        for w in range(1, W):
            s = s + acc_model[w, S]
        assert np.array_equal(u32(upd[S]), u32(F(0) + s))
        # what was sent left every residual (+0), the rest is untouched: conservation
        sent = np.zeros_like(acc_model)
        sent[:, S] = acc_model[:, S]
        for w in range(W):
            r = orc.residual(w)
            assert np.all(u32(r[S]) == 0)
            assert np.array_equal(u32(r[offS]), u32(acc_model[w, offS]))
            assert np.array_equal(r + sent[w], acc_model[w])
        acc_model[:, S] = 0
        assert np.array_equal(orc.mask(), (~offS).astype(np.uint8))


def test_ratio_one_is_a_dense_allreduce():
    layers, W = [257, 1000, 3], 5
    rng, weights = _random_problem(layers, W, 2)
    N = sum(layers)
    orc = oracle.Oracle(layers, W, 1.0, 1e-8, seed=0)
    carry = np.zeros((W, N), np.float32)
    for t in range(2):
        grads = rng.normal(size=(W, N)).astype(np.float32)
        upd = orc.step(grads, weights)
        tot = grads[0].copy()
        for w in range(1, W):
            tot = tot + grads[w]
        assert np.array_equal(u32(upd), u32(F(0) + tot))
        for w in range(W):
            assert np.all(u32(orc.residual(w)) == 0)
            assert orc.selection(w)[0].tolist() == list(range(N))


def test_single_worker_conserves_gradient_mass():
    layers, W, R = [4096, 100], 1, 8.0
    rng, weights = _random_problem(layers, W, 4)
    N = sum(layers)
    orc = oracle.Oracle(layers, W, R, 1e-8, seed=0)
    seg_sum = np.zeros(N, np.float32)  # fp32 running sum since the element was last sent
    total_sent = np.zeros(N, np.float64)
    total_grad = np.zeros(N, np.float64)
    for t in range(12):
        g = rng.normal(scale=1e-2, size=(1, N)).astype(np.float32)
        seg_sum = seg_sum + g[0]
        upd = orc.step(g, weights)
        S = orc.selection(0)[0]
        assert np.array_equal(u32(upd[S]), u32(F(0) + seg_sum[S]))  # W = 1: update[S] is the residual itself
        total_sent += upd
        total_grad += g[0]
        seg_sum[S] = 0
        assert np.array_equal(u32(orc.residual(0)), u32(seg_sum))
    assert np.allclose(total_sent + orc.residual(0), total_grad, rtol=0, atol=1e-6)


def test_equal_denominators_reduce_to_magnitude_topk():
    # batch-norm gammas (all 1) or all-zero weights: ranking by importance = ranking by |residual|
    n, k = 3000, 100
    rng = np.random.default_rng(9)
    acc = rng.normal(size=n).astype(np.float32)
    for wval in (1.0, 0.0, -0.37):
        got = oracle.select(acc, np.full(n, wval, np.float32), k, 1e-8)
        want = torch.topk(torch.from_numpy(np.abs(acc)), k).indices.sort().values.numpy()
        assert np.array_equal(got, want.astype(np.uint32))


def test_zero_weights_dominate():
    # an element with w = 0 and any non-zero residual outranks every element with |w| >= 1e-3 and |residual| <= 1
    n = 512
    rng = np.random.default_rng(3)
    w = rng.uniform(1e-3, 1.0, n).astype(np.float32)
    acc = rng.uniform(-1, 1, n).astype(np.float32)
    zeros = [5, 77, 300]
    w[zeros] = 0.0
    acc[zeros] = [1e-4, -2e-4, 3e-4]
    assert oracle.select(acc, w, 3, 1e-8).tolist() == zeros


def test_create_rejects_bad_arguments():
    ok = dict(layer_sizes=[4, 4], W=2, ratio=2.0, eps=1e-8, seed=0)
    oracle.Oracle(**ok)
    for bad in (dict(layer_sizes=[4, 0]), dict(W=0), dict(ratio=0.5), dict(ratio=float("nan")), dict(eps=0.0),
                dict(eps=-1.0), dict(ratio=float("inf"))):
        with pytest.raises(ValueError):
            oracle.Oracle(**{**ok, **bad})


def test_reset_and_residual_roundtrip():
    layers, W = [100, 28], 2
    rng, weights = _random_problem(layers, W, 6)
    orc = oracle.Oracle(layers, W, 4.0, 1e-8, seed=1)
    g = rng.normal(size=(W, 128)).astype(np.float32)
    u0 = orc.step(g, weights)
    r = [orc.residual(w) for w in range(W)]
    orc.reset()
    assert orc.t == 0 and all(np.all(orc.residual(w) == 0) for w in range(W))
    u1 = orc.step(g, weights)
    assert np.array_equal(u32(u0), u32(u1))
    for w in range(W):
        orc.set_residual(w, r[w])
        assert np.array_equal(u32(orc.residual(w)), u32(r[w]))


# ---------------------------------------------------------------- momentum on the residual (Eq. 3)


def test_momentum_one_is_plain_accumulation_and_bruteforce_agrees():
    layers, W, ratio = [9, 20, 3], 3, 4.0
    rng = np.random.default_rng(77)
    N = sum(layers)
    weights = (rng.normal(size=N) * (rng.random(N) > 0.1)).astype(np.float32)
    for m in (1.0, 0.9, 0.5, 0.0):
        orc = oracle.Oracle(layers, W, ratio, 1e-8, seed=2)
        orc.set_momentum(m)
        bf = BruteForce(layers, W, ratio, 1e-8, momentum=m)
        plain = oracle.Oracle(layers, W, ratio, 1e-8, seed=2)
        for t in range(4):
            grads = (rng.integers(-8, 9, size=(W, N)) / 16.0).astype(np.float32)
            upd = orc.step(grads, weights)
            lists, upd_bf = bf.step(grads, weights, orc.leader)
            assert np.array_equal(u32(upd), u32(upd_bf)), (m, t)
            for w in range(W):
                assert orc.selection(w)[0].tolist() == [i for i, _ in lists[w]]
                assert np.array_equal(u32(orc.residual(w)), u32(bf.residual(w)))
            if m == 1.0:
                assert np.array_equal(u32(plain.step(grads, weights)), u32(upd))


def test_momentum_hand_worked():
    # one layer of 4, one worker, keep 1 of 4, weights 1: step 0 sends the largest, the rest is carried
    # scaled by m = 0.5 into step 1:  residual after step 0 = [0, 2, 1, 0.5]; step 1 adds [4, 0, 0, 0]
    # to 0.5 * residual = [0, 1, 0.5, 0.25]  ->  [4, 1, 0.5, 0.25]: index 0 is sent with value 4.
    orc = oracle.Oracle([4], 1, 4.0, 1e-8, seed=0)
    orc.set_momentum(0.5)
    w = np.ones(4, np.float32)
    u0 = orc.step(np.array([[8, 2, 1, 0.5]], np.float32), w)
    assert u0.tolist() == [8, 0, 0, 0] and orc.residual(0).tolist() == [0, 2, 1, 0.5]
    u1 = orc.step(np.array([[4, 0, 0, 0]], np.float32), w)
    assert u1.tolist() == [4, 0, 0, 0] and orc.residual(0).tolist() == [0, 1, 0.5, 0.25]
    # zero momentum forgets everything that was not sent
    o2 = oracle.Oracle([4], 1, 4.0, 1e-8, seed=0)
    o2.set_momentum(0.0)
    o2.step(np.array([[8, 2, 1, 0.5]], np.float32), w)
    u = o2.step(np.array([[0, 0, 0, 3]], np.float32), w)
    assert u.tolist() == [0, 0, 0, 3] and o2.residual(0).tolist() == [0, 0, 0, 0]


def test_momentum_geometric_carry_closed_form():
    # an element that is never sent and receives a constant gradient c carries c (1 + m + ... + m^t):
    # with c = 1 and m = 0.5 every partial sum is exactly representable
    n = 16
    orc = oracle.Oracle([n], 1, float(n), 1e-8, seed=0)  # keeps one element per step
    orc.set_momentum(0.5)
    w = np.ones(n, np.float32)
    g = np.ones((1, n), np.float32)
    g[0, 0] = 100.0  # index 0 always wins, the others are never sent
    for t in range(10):
        orc.step(g, w)
        want = 2.0 - 0.5 ** t
        assert np.all(orc.residual(0)[1:] == np.float32(want)), t


# ---------------------------------------------------------------- Algorithm 1 as printed: absolute thresholds


def _brute_threshold_step(acc, grads, weights, layers, thr, leader, eps, m=1.0):
    """Pure-Python statement of one threshold-mode step on lists of numpy float32 scalars."""
    W, N = len(acc), len(weights)
    for w in range(W):
        for i in range(N):
            acc[w][i] = F(F(F(m) * acc[w][i]) + F(grads[w][i]))
    S, o = [], 0
    for n, t in zip(layers, thr):
        S += [o + i for i in range(n) if importance(acc[leader][o + i], weights[o + i], eps) > F(t)]
        o += n
    upd = [F(0)] * N
    for i in S:
        s = acc[0][i]
        for w in range(1, W):
            s = F(s + acc[w][i])
        upd[i] = F(F(0) + s)
    vals = [acc[leader][i] for i in S]
    for i in S:
        for w in range(W):
            acc[w][i] = F(0)
    return S, vals, np.array(upd, np.float32)


def test_threshold_mode_equals_bruteforce():
    layers, W = [7, 1, 20, 4], 3
    N = sum(layers)
    rng = np.random.default_rng(31)
    weights = (rng.integers(-2, 3, N) * 0.5).astype(np.float32)  # includes zeros
    thr = [0.5, 0.0, 1.0, 1e9]
    orc = oracle.Oracle(layers, W, 2.0, 1e-8, seed=4)
    orc.set_thresholds(thr)
    acc = [[F(0)] * N for _ in range(W)]
    for t in range(5):
        grads = (rng.integers(-4, 5, size=(W, N)) / 4.0).astype(np.float32)  # importances hit the thresholds exactly
        upd = orc.step(grads, weights)
        S, vals, upd_bf = _brute_threshold_step(acc, grads, weights, layers, thr, orc.leader, F(1e-8))
        idx, val = orc.threshold_list()
        assert idx.tolist() == S and np.array_equal(u32(val), u32(np.array(vals, np.float32)))
        assert np.array_equal(u32(upd), u32(upd_bf))
        for w in range(W):
            assert np.array_equal(u32(orc.residual(w)), u32(np.array(acc[w], np.float32)))
        assert orc.mask().tolist() == [1 if i in S else 0 for i in range(N)]
        assert not any(i >= sum(layers[:3]) for i in S)  # the last layer's threshold of 1e9 is never passed


def test_threshold_mode_hand_worked_and_strictness():
    # weights 1, eps negligible: importance = |residual|.  thr = 0.5 is strict: 0.5 itself stays.
    orc = oracle.Oracle([4], 2, 2.0, 1e-8, seed=0)
    orc.set_thresholds([0.5])
    orc.set_leader_override(1)
    w = np.ones(4, np.float32)
    g = np.array([[1.0, 0.25, 0.5, -2.0], [0.5, 0.75, -0.5, 0.25]], np.float32)
    upd = orc.step(g, w)  # node 1's mask: |0.5|>0.5 no, 0.75 yes, |-0.5| no, 0.25 no  ->  S = {1}
    assert orc.threshold_list()[0].tolist() == [1] and upd.tolist() == [0, 1.0, 0, 0]
    assert orc.residual(0).tolist() == [1.0, 0, 0.5, -2.0] and orc.residual(1).tolist() == [0.5, 0, -0.5, 0.25]
    orc.set_leader_override(0)
    upd = orc.step(np.zeros((2, 4), np.float32), w)  # node 0: 1.0 and |-2| pass  ->  S = {0, 3}
    assert orc.threshold_list()[0].tolist() == [0, 3] and upd.tolist() == [1.5, 0, 0, -1.75]
    # thresholds 0 and +inf: everything non-zero / nothing
    o2 = oracle.Oracle([3, 3], 1, 2.0, 1e-8, seed=0)
    o2.set_thresholds([0.0, float("inf")])
    u = o2.step(np.array([[1, 0, -1, 5, 5, 5]], np.float32), np.ones(6, np.float32))
    assert o2.threshold_list()[0].tolist() == [0, 2] and u.tolist() == [1, 0, -1, 0, 0, 0]


def test_threshold_at_the_kplus1_th_importance_reproduces_the_ratio_mode():
    # with thr = the (k+1)-th largest importance of the chosen node's layer (continuous values, no ties)
    # the thresholded mask is that node's top-k set, so both modes must give the same update
    layers, W, R = [4000, 300], 3, 16.0
    rng, weights = _random_problem(layers, W, 55, zero_frac=0.0)
    N = sum(layers)
    grads = rng.normal(scale=1e-3, size=(W, N)).astype(np.float32)
    ratio = oracle.Oracle(layers, W, R, 1e-8, seed=9)
    upd_ratio = ratio.step(grads, weights)
    off, ks = ratio.layout()
    imp = np.abs(grads[ratio.leader]) / (np.abs(weights) + F(1e-8))
    thr = [np.sort(imp[o:o + n])[::-1][k] for o, n, k in zip(off, layers, ks)]
    th = oracle.Oracle(layers, W, R, 1e-8, seed=9)
    th.set_thresholds(thr)
    upd_thr = th.step(grads, weights)
    assert th.leader == ratio.leader
    assert np.array_equal(th.threshold_list()[0], ratio.selection(ratio.leader)[0])
    assert np.array_equal(u32(upd_thr), u32(upd_ratio))
    for w in range(W):
        assert np.array_equal(u32(th.residual(w)), u32(ratio.residual(w)))


# ---------------------------------------------------------------- several chosen nodes, masks OR-ed


def _leader_set_rows():
    rows = []
    for line in open(os.path.join(GOLD, "leader_sets.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, body = line.split(":")
        seed, W, n = (int(x) for x in head.split())
        rows.append((seed, W, n, [[int(x) for x in step.split()] for step in body.split("|")]))
    return rows


@pytest.mark.parametrize("seed,W,n,expect", _leader_set_rows())
def test_leader_sets(seed, W, n, expect):
    for t, want in enumerate(expect):
        got = oracle.leaders(seed, t, W, n)
        assert got == want
        assert len(set(got)) == n and got[0] == oracle.leader(seed, t, W)


def test_or_of_masks_equals_bruteforce_union():
    layers, W, n = [30, 6, 50], 5, 3
    N = sum(layers)
    rng = np.random.default_rng(5)
    weights = (rng.integers(-2, 3, N) * 0.5).astype(np.float32)
    thr = [0.75, 0.25, 1.5]
    orc = oracle.Oracle(layers, W, 2.0, 1e-8, seed=11)
    orc.set_thresholds(thr)
    orc.set_n_leaders(n)
    acc = np.zeros((W, N), np.float32)
    for t in range(4):
        grads = (rng.integers(-4, 5, size=(W, N)) / 4.0).astype(np.float32)
        acc = acc + grads
        upd = orc.step(grads, weights)
        rs = oracle.leaders(11, t, W, n)
        imp = np.abs(acc) / (np.abs(weights) + F(1e-8))
        layer_thr = np.repeat(np.array(thr, np.float32), layers)
        union = np.zeros(N, bool)
        for r in rs:
            union |= imp[r] > layer_thr
        S = np.flatnonzero(union)
        idx, val = orc.threshold_list()
        assert idx.tolist() == S.tolist() and orc.leader == rs[0]
        assert np.array_equal(u32(val), u32(acc[rs[0], S]))
        s = acc[0, S].copy()
        for w in range(1, W):
            s = s + acc[w, S]
        want = np.zeros(N, np.float32)
        want[S] = F(0) + s
        assert np.array_equal(u32(upd), u32(want))
        acc[:, S] = 0
        for w in range(W):
            assert np.array_equal(u32(orc.residual(w)), u32(acc[w]))
    # a union is never smaller than the first node's own mask
    one = oracle.Oracle(layers, W, 2.0, 1e-8, seed=11)
    one.set_thresholds(thr)
    g = (rng.integers(-4, 5, size=(W, N)) / 4.0).astype(np.float32)
    many = oracle.Oracle(layers, W, 2.0, 1e-8, seed=11)
    many.set_thresholds(thr)
    many.set_n_leaders(W)
    one.step(g, weights)
    many.step(g, weights)
    assert set(one.threshold_list()[0].tolist()) <= set(many.threshold_list()[0].tolist())


# ---------------------------------------------------------------- random sub-threshold selection (Section 3.3)


def test_random_select_draw_vectors_and_uniformity():
    for line in open(os.path.join(GOLD, "random_select_draws.txt")):
        if line.startswith("#") or not line.strip():
            continue
        seed, t, i, want = (int(x) for x in line.split())
        assert oracle.draw24(seed, t, i) == want
    u = np.array([oracle.draw24(3, 2, i) for i in range(20000)]) / 2.0 ** 24
    assert u.min() >= 0 and u.max() < 1 and abs(u.mean() - 0.5) < 0.01 and abs(u.var() - 1 / 12) < 0.005
    assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 0.03


def test_random_select_equals_bruteforce_and_has_the_right_rate():
    n, W = 6000, 2
    rng = np.random.default_rng(21)
    weights = np.ones(n, np.float32)
    thr = 1.0
    orc = oracle.Oracle([n], W, 2.0, 1e-8, seed=13)
    orc.set_thresholds([thr])
    orc.set_random_select(True)
    orc.set_leader_override(0)
    g = rng.uniform(0.0, 1.0, size=(W, n)).astype(np.float32)  # importance of node 0 = g[0] (weights 1): all below thr
    g[0, :10] = 0.0          # zero importance is never sent
    g[0, 10:20] = 2.0        # above the threshold: always sent
    upd = orc.step(g, weights)
    S = set(orc.threshold_list()[0].tolist())
    imp = np.abs(g[0]) / (np.abs(weights) + F(1e-8))
    want = set()
    for i in range(n):
        u = F(oracle.draw24(13, 0, i)) * F(2.0 ** -24)
        if imp[i] > F(thr) or u < F(imp[i] / F(thr)):
            want.add(i)
    assert S == want
    assert not (S & set(range(10))) and set(range(10, 20)) <= S
    # P(update) = importance / threshold: bucket the elements by importance and compare frequencies
    sel = np.zeros(n, bool)
    sel[list(S)] = True
    for lo in (0.1, 0.4, 0.7):
        band = (imp >= lo) & (imp < lo + 0.2) & (np.arange(n) >= 20)
        assert abs(sel[band].mean() - (lo + 0.1)) < 0.06
    # switched off: only the ten elements above the threshold go
    off = oracle.Oracle([n], W, 2.0, 1e-8, seed=13)
    off.set_thresholds([thr])
    off.set_leader_override(0)
    off.step(g, weights)
    assert off.threshold_list()[0].tolist() == list(range(10, 20))
    assert np.count_nonzero(upd) >= len(S) - 10


# ---------------------------------------------------------------- layer-wise threshold (Section 3.4, Eq. 4)


def _frac_round(values):
    """Exact sum by rational arithmetic, rounded once (Fraction -> float is correctly rounded)."""
    from fractions import Fraction

    return float(sum((Fraction(float(v)) for v in values), Fraction(0)))


def _eq4_by_fractions(acc, w, eps, alpha, beta, c):
    """Eq. 4 written out independently: exact moments by rational arithmetic, the rest in Python floats."""
    imp = [float(importance(a, b, eps)) for a, b in zip(acc, w)]
    S1, S2 = _frac_round(imp), _frac_round([x * x for x in imp])  # x * x is exact in binary64 for fp32 x
    n = float(len(imp))
    mean = S1 / n
    var = S2 / n - mean * mean
    v = var / mean if mean > 0.0 else 0.0
    t = alpha + beta * v if v > c else alpha - beta * v
    thr = F(t)
    return (F(0.0) if thr == 0 else thr), dict(S1=S1, S2=S2, mean=mean, var=var, v=v)


def test_exact_sum_equals_fsum_and_fractions():
    rng = np.random.default_rng(5)
    for n in (1, 2, 17, 1000, 100000):
        x = np.abs(rng.standard_normal(n)) * 10.0 ** rng.integers(-40, 40, n)  # 80 decades of magnitude
        assert oracle.exact_sum(x) == math.fsum(x.tolist())
    small = np.abs(rng.standard_normal(200)) * 10.0 ** rng.integers(-300, 10, 200)
    small[:5] = [5e-324, 1e-310, 2.2250738585072014e-308, 0.0, 4.9e-324]  # subnormals, the smallest normal, zero
    assert oracle.exact_sum(small) == math.fsum(small.tolist()) == _frac_round(small)
    assert oracle.exact_sum(np.zeros(3)) == 0.0 and oracle.exact_sum(np.zeros(0)) == 0.0
    # ties go to even, and anything beyond a tie rounds up
    assert oracle.exact_sum(np.array([2.0**53, 1.0])) == 2.0**53
    assert oracle.exact_sum(np.array([2.0**53, 1.0, 5e-324])) == 2.0**53 + 2
    assert oracle.exact_sum(np.array([2.0**53 + 2, 1.0])) == 2.0**53 + 4
    assert oracle.exact_sum(np.array([1.0, 2.0**-53])) == 1.0 and oracle.exact_sum(np.array([1.0, 2.0**-53, 2.0**-53])) == 1.0 + 2.0**-52
    # a plain left-to-right sum gets this one wrong: 1e16 + 1 + 1 + ... (1000 ones)
    x = np.array([1e16] + [1.0] * 1000)
    assert oracle.exact_sum(x) == 1e16 + 1000 and float(np.cumsum(x)[-1]) != 1e16 + 1000


def test_layerwise_threshold_closed_forms():
    eps = F(2.0**-30)
    w = np.full(1024, 1.0, np.float32)  # |w| + eps rounds back to 1, so importance = |acc|
    # a constant layer has no variance: thr = alpha
    thr, st = oracle.layerwise_threshold(np.full(1024, -0.25, np.float32), w, eps, 0.05, 3.0, 0.5)
    assert (st["S1"], st["S2"], st["mean"], st["var"], st["v"]) == (256.0, 64.0, 0.25, 0.0, 0.0) and thr == F(0.05)
    # half 1, half 3: mean 2, var 1, v = 0.5
    acc = np.where(np.arange(1024) % 2 == 0, 1.0, -3.0).astype(np.float32)
    thr, st = oracle.layerwise_threshold(acc, w, eps, 0.25, 0.5, 0.25)
    assert (st["mean"], st["var"], st["v"]) == (2.0, 1.0, 0.5) and thr == F(0.5)  # v > C: alpha + beta v
    thr, _ = oracle.layerwise_threshold(acc, w, eps, 0.25, 0.5, 0.5)
    assert thr == F(0.0)  # v == C is not "greater": alpha - beta v = 0
    thr, _ = oracle.layerwise_threshold(acc, w, eps, 0.25, 1.0, 1.0)
    assert thr == F(-0.25)  # a negative threshold is kept as it is
    # nothing accumulated: mean 0, v taken as 0
    thr, st = oracle.layerwise_threshold(np.zeros(64, np.float32), w[:64], eps, 0.125, 9.0, 0.0)
    assert st["mean"] == 0.0 and st["v"] == 0.0 and thr == F(0.125)
    # -0 becomes +0
    thr, _ = oracle.layerwise_threshold(np.zeros(64, np.float32), w[:64], eps, -0.0, 1.0, 0.0)
    assert u32([thr])[0] == 0


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_layerwise_threshold_equals_rational_arithmetic(seed):
    rng = np.random.default_rng(100 + seed)
    n = [257, 1000, 4096][seed]
    acc = (rng.standard_normal(n) * 10.0 ** rng.integers(-6, 3, n)).astype(np.float32)
    w = (rng.standard_normal(n) * 0.05).astype(np.float32)
    w[rng.random(n) < 0.05] = 0.0  # importances of 1e8 and more beside ones of 1e-6
    for alpha, beta, c in ((0.01, 1e-9, 1e6), (0.05, 0.001, 1e30), (0.0, 1.0, 0.0)):
        thr, st = oracle.layerwise_threshold(acc, w, F(1e-8), alpha, beta, c)
        thr_f, st_f = _eq4_by_fractions(acc, w, F(1e-8), alpha, beta, c)
        assert st == st_f and u32([thr])[0] == u32([thr_f])[0]


def test_layerwise_step_equals_bruteforce_with_two_chosen_nodes():
    layers, W = [40, 9, 64], 4
    N, eps = sum(layers), F(1e-8)
    rng = np.random.default_rng(77)
    weights = (rng.standard_normal(N) * 0.1).astype(np.float32)
    alpha, beta, c = 0.5, 0.02, 10.0
    orc = oracle.Oracle(layers, W, 2.0, eps, seed=9)
    orc.set_layerwise(alpha, beta, c)
    orc.set_n_leaders(2)
    acc = np.zeros((W, N), np.float32)
    saw_both_branches = set()
    for t in range(6):
        grads = (rng.standard_normal((W, N)) * (0.2 if t % 2 else 0.02)).astype(np.float32)
        upd = orc.step(grads, weights)
        acc = (acc + grads).astype(np.float32)
        chosen = oracle.leaders(9, t, W, 2)
        thr = orc.layer_thresholds()
        assert thr.shape == (2, len(layers))
        S, o = set(), 0
        for l, n in enumerate(layers):
            for j, r in enumerate(chosen):
                want, st = _eq4_by_fractions(acc[r, o:o + n], weights[o:o + n], eps, alpha, beta, c)
                saw_both_branches.add(st["v"] > c)
                assert u32([thr[j, l]])[0] == u32([want])[0]
                S |= {o + i for i in range(n) if importance(acc[r, o + i], weights[o + i], eps) > want}
            o += n
        idx, val = orc.threshold_list()
        assert idx.tolist() == sorted(S)
        want_upd = np.zeros(N, np.float32)
        for i in S:
            s = acc[0, i]
            for w_ in range(1, W):
                s = F(s + acc[w_, i])
            want_upd[i] = F(F(0) + s)
            acc[:, i] = 0
        assert np.array_equal(u32(upd), u32(want_upd))
        for w_ in range(W):
            assert np.array_equal(u32(orc.residual(w_)), u32(acc[w_]))
    assert saw_both_branches == {True, False}


# ---------------------------------------------------------------- several chosen nodes in the ratio mode


def test_ratio_mode_union_of_chosen_nodes_equals_bruteforce():
    # every worker's own top-k list comes from the full-sort model; the index set is the union of the
    # chosen nodes' lists, and sum / zeroing run over that union
    layers, W, n, ratio, eps = [30, 6, 50], 5, 3, 8.0, F(1e-8)
    N = sum(layers)
    rng = np.random.default_rng(21)
    weights = (rng.integers(-2, 3, N) * 0.5).astype(np.float32)
    orc = oracle.Oracle(layers, W, ratio, eps, seed=13)
    orc.set_n_leaders(n)
    k = [min(m, max(1, math.ceil(m / ratio))) for m in layers]
    acc = np.zeros((W, N), np.float32)
    sizes = set()
    for t in range(5):
        grads = (rng.integers(-4, 5, size=(W, N)) / 4.0).astype(np.float32)  # coarse: ties everywhere
        acc = (acc + grads).astype(np.float32)
        upd = orc.step(grads, weights)
        lists = []
        for w in range(W):
            lst, o = [], 0
            for m, kk in zip(layers, k):
                imp = [bits(importance(acc[w, o + i], weights[o + i], eps)) for i in range(m)]
                ranked = sorted(range(m), key=lambda i: (-imp[i], i))
                lst += sorted(o + i for i in ranked[:kk])
                o += m
            lists.append(lst)
            assert orc.selection(w)[0].tolist() == lst
        rs = oracle.leaders(13, t, W, n)
        assert orc.leader == rs[0]
        S = sorted(set().union(*(lists[r] for r in rs)))
        sizes.add(len(S))
        assert orc.index_set().tolist() == S and sum(k) <= len(S) <= n * sum(k)
        assert orc.mask().tolist() == [1 if i in set(S) else 0 for i in range(N)]
        want = np.zeros(N, np.float32)
        for i in S:
            s = acc[0, i]
            for w in range(1, W):
                s = F(s + acc[w, i])
            want[i] = F(F(0) + s)
            acc[:, i] = 0
        assert np.array_equal(u32(upd), u32(want))
        for w in range(W):
            assert np.array_equal(u32(orc.residual(w)), u32(acc[w]))
    assert any(s > sum(k) for s in sizes)  # the union really grew beyond one node's list


def test_ratio_mode_one_chosen_node_is_the_plain_path_and_all_nodes_cover_every_list():
    layers, W, ratio = [200, 64], 4, 16.0
    N = sum(layers)
    rng = np.random.default_rng(3)
    weights = rng.standard_normal(N).astype(np.float32)
    a, b, c = (oracle.Oracle(layers, W, ratio, 1e-8, seed=2) for _ in range(3))
    b.set_n_leaders(1)
    c.set_n_leaders(W)
    for t in range(3):
        g = rng.standard_normal((W, N)).astype(np.float32)
        ua, ub = a.step(g, weights), b.step(g, weights)
        assert np.array_equal(u32(ua), u32(ub)) and a.index_set().tolist() == a.selection(a.leader)[0].tolist()
        c.step(g, weights)
        every = set()
        for w in range(W):
            every |= set(c.selection(w)[0].tolist())
        assert set(c.index_set().tolist()) == every
        for w in range(W):  # everything any worker selected has left every residual
            assert not c.residual(w)[sorted(every)].any()


# ---------------------------------------------------------------- one chosen node per layer


def _layer_leader_rows():
    rows = []
    for line in open(os.path.join(GOLD, "layer_leaders.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, body = line.split(":")
        seed, W, L = (int(x) for x in head.split())
        rows.append((seed, W, L, [[int(x) for x in step.split()] for step in body.split("|")]))
    return rows


@pytest.mark.parametrize("seed,W,L,expect", _layer_leader_rows())
def test_layer_leader_vectors(seed, W, L, expect):
    assert [[oracle.layer_leader(seed, t, l, W) for l in range(L)] for t in range(len(expect))] == expect


def test_layer_leaders_are_uniform_and_differ_between_layers():
    W = 8
    draws = np.array([[oracle.layer_leader(3, t, l, W) for l in range(16)] for t in range(2000)])
    assert draws.min() == 0 and draws.max() == W - 1
    counts = np.bincount(draws.ravel(), minlength=W)
    assert np.all(np.abs(counts - draws.size / W) < 5 * math.sqrt(draws.size / W))  # within five sigma of uniform
    same = np.mean(draws[:, 0] == draws[:, 1])
    assert abs(same - 1 / W) < 0.03  # neighbouring layers agree about as often as independent draws would


def test_per_layer_leaders_equal_bruteforce():
    layers, W, ratio, eps = [30, 6, 50, 12], 4, 8.0, F(1e-8)
    N = sum(layers)
    rng = np.random.default_rng(41)
    weights = (rng.integers(-2, 3, N) * 0.5).astype(np.float32)
    orc = oracle.Oracle(layers, W, ratio, eps, seed=17)
    orc.set_per_layer_leaders()
    k = [min(m, max(1, math.ceil(m / ratio))) for m in layers]
    acc = np.zeros((W, N), np.float32)
    used = set()
    for t in range(5):
        grads = (rng.integers(-4, 5, size=(W, N)) / 4.0).astype(np.float32)
        acc = (acc + grads).astype(np.float32)
        upd = orc.step(grads, weights)
        S, o = [], 0
        for l, (m, kk) in enumerate(zip(layers, k)):
            r = oracle.layer_leader(17, t, l, W)
            used.add(r)
            imp = [bits(importance(acc[r, o + i], weights[o + i], eps)) for i in range(m)]
            ranked = sorted(range(m), key=lambda i: (-imp[i], i))
            S += sorted(o + i for i in ranked[:kk])
            o += m
        assert orc.index_set().tolist() == S and len(S) == sum(k)
        want = np.zeros(N, np.float32)
        for i in S:
            s = acc[0, i]
            for w in range(1, W):
                s = F(s + acc[w, i])
            want[i] = F(F(0) + s)
            acc[:, i] = 0
        assert np.array_equal(u32(upd), u32(want))
        for w in range(W):
            assert np.array_equal(u32(orc.residual(w)), u32(acc[w]))
    assert len(used) > 1


# ---------------------------------------------------------------- property tests (hypothesis)


def test_selection_properties_on_arbitrary_small_layers():
    from hypothesis import given, settings
    from hypothesis import strategies as st

    values = st.sampled_from([0.0, -0.0, 0.25, -0.25, 0.5, 1.0, -2.0, 3.0e-39, 1.0e30])  # ties, zeros, a denormal
    weights = st.sampled_from([0.0, 0.5, -0.5, 1.0, 2.0])

    @settings(max_examples=200, deadline=None)
    @given(st.lists(st.tuples(values, weights), min_size=1, max_size=40), st.integers(1, 40))
    def check(pairs, k):
        acc = np.array([p[0] for p in pairs], np.float32)
        w = np.array([p[1] for p in pairs], np.float32)
        k = min(k, acc.size)
        got = oracle.select(acc, w, k, 1e-8).tolist()
        imp = [bits(importance(a, b, F(1e-8))) for a, b in zip(acc, w)]
        assert got == sorted(got) and len(set(got)) == k  # ascending, distinct, exactly k
        inside, outside = [imp[i] for i in got], [imp[i] for i in range(acc.size) if i not in got]
        if outside:
            t = min(inside)
            assert t >= max(outside)  # nothing left out beats anything kept
            # at the threshold value the kept indices are the lowest ones
            at_t_in = [i for i in got if imp[i] == t]
            at_t_out = [i for i in range(acc.size) if i not in got and imp[i] == t]
            assert not at_t_out or max(at_t_in) < min(at_t_out)

    check()


def test_step_conserves_every_element_exactly():
    from hypothesis import given, settings
    from hypothesis import strategies as st

    @settings(max_examples=40, deadline=None)
    @given(st.integers(0, 2**31 - 1), st.integers(1, 4), st.sampled_from([1.0, 2.0, 7.0, 64.0]), st.integers(1, 3))
    def check(seed, W, ratio, n_leaders):
        rng = np.random.default_rng(seed)
        layers = [int(x) for x in rng.integers(1, 30, size=3)]
        N = sum(layers)
        orc = oracle.Oracle(layers, W, ratio, 1e-8, seed=seed)
        orc.set_n_leaders(min(n_leaders, W))
        weights = (rng.integers(-2, 3, N) * 0.5).astype(np.float32)
        before = np.zeros((W, N), np.float32)
        for t in range(3):
            g = (rng.integers(-4, 5, size=(W, N)) / 4.0).astype(np.float32)
            upd = orc.step(g, weights)
            mask = orc.mask().astype(bool)
            after = np.stack([orc.residual(w) for w in range(W)])
            acc = (before + g).astype(np.float32)
            assert not after[:, mask].any()  # what was sent has left every residual
            assert np.array_equal(u32(after[:, ~mask]), u32(acc[:, ~mask]))  # the rest is untouched
            assert not upd[~mask].any()  # nothing outside the index set
            s = acc[0].copy()
            for w in range(1, W):
                s = (s + acc[w]).astype(np.float32)
            assert np.array_equal(u32(upd[mask]), u32((F(0) + s)[mask]))  # the ordered sum inside it
            before = after

    check()
