"""GPU parity of the absolute-threshold mode (Algorithm 1 as printed: Mask = importance > thr on the
chosen node, variable-size index set) against the CPU oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_01544_b200 import binding
from paper_1901_01544_b200 import workloads as wl
from paper_1901_01544_b200.binding import Pruner
from parity import assert_bits_equal

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _randn(shape, seed, scale=1.0):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return torch.randn(shape, generator=g, device=DEV, dtype=torch.float32) * scale


def _run(sizes, W, thr, weights, grads_fn, steps, seed=3, momentum=None, max_list=0, force_scalar=False,
         residual_every=1, n_leaders=1, random_select=False, layerwise=None):
    """thr: fixed per-layer thresholds, or None with layerwise = (alpha, beta, C) of Eq. 4."""
    N = sum(sizes)
    pr = Pruner(sizes, W, None, 1e-8, seed, thresholds=thr, max_list=max_list)
    orc = oracle.Oracle(sizes, W, 2.0, 1e-8, seed)
    if layerwise is not None:
        pr.set_layerwise(*layerwise)
        orc.set_layerwise(*layerwise)
    else:
        orc.set_thresholds(thr)
    if momentum is not None:
        pr.set_momentum(momentum)
        orc.set_momentum(momentum)
    if force_scalar:
        pr.set_option("force_scalar", 1)
    if random_select:
        pr.set_option("random_select", 1)
        orc.set_random_select(True)
    if n_leaders > 1:
        pr.set_option("n_leaders", n_leaders)
        orc.set_n_leaders(n_leaders)
    w_host = weights.cpu().numpy()
    upd = torch.full((N,), float("nan"), device=DEV)
    seen_thr = []
    for t in range(steps):
        g = grads_fn(t)
        pr.step(g, weights, upd)
        want = orc.step(np.ascontiguousarray(g.cpu().numpy()), w_host)
        assert pr.sync_status() == 0 and pr.leader == orc.leader
        if layerwise is not None:  # the derived thresholds themselves, bit for bit, one row per chosen node
            assert_bits_equal(pr.layer_thresholds().cpu().numpy(), orc.layer_thresholds(), f"step {t}: thresholds")
            seen_thr.append(orc.layer_thresholds())
        oi, ov = orc.threshold_list()
        assert pr.list_length() == len(oi), f"step {t}: list length"
        gi, gv = pr.selection(pr.leader)
        assert np.array_equal(gi.cpu().numpy().view(np.uint32)[: len(oi)], oi), f"step {t}: indices"
        assert_bits_equal(gv.cpu().numpy()[: len(oi)], ov, f"step {t}: values")
        assert_bits_equal(upd.cpu().numpy(), want, f"step {t}: update")
        assert np.array_equal(pr.mask().cpu().numpy(), orc.mask()), f"step {t}: mask"
        assert np.array_equal(pr.mask_bits().cpu().numpy(), np.packbits(orc.mask(), bitorder="little")), f"step {t}: packed mask"
        if (t + 1) % residual_every == 0 or t == steps - 1:
            for w in range(W):
                assert_bits_equal(pr.residual(w).cpu().numpy(), orc.residual(w), f"step {t}: worker {w} residual")
        upd.fill_(float("nan"))
    pr.close()
    orc.close()
    return seen_thr


CASES = {
    "mixed_sizes": ([64, 16385, 256, 100000, 9408, 1, 36864, 1000], 4),
    "odd_total_scalar_path": ([20001, 17, 70003], 3),
    "unaligned_offsets": ([16389, 16387, 40000], 2),
    "many_chunks": ([128 * 4096 * 2 + 4097, 65536], 2),
    "one_worker": ([30000, 70], 1),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_threshold_mode_random_values(name):
    sizes, W = CASES[name]
    N = sum(sizes)
    weights = _randn((N,), 100, 0.05)
    weights[::53] = 0.0
    # importance of N(0,1e-3)/N(0,0.05) is heavy tailed; these thresholds keep from ~30 % down to ~0.5 %
    thr = [[0.02, 0.1, 0.5, 2.0][l % 4] for l in range(len(sizes))]
    _run(sizes, W, thr, weights, lambda t: _randn((W, N), 7 * t + 1, 1e-3), steps=4)


@pytest.mark.parametrize("n_leaders", [1, 2])
def test_threshold_mode_clustered_importances(n_leaders):
    # runs of consecutive elements far above the threshold (blocks of zero weights, one worker's hot gradients)
    # at segment, tile and chunk edges of the passes: whole mask words and whole chunks are set
    sizes, W = [300, 20000, 128 * 4096 + 70000], 4
    N = sum(sizes)
    weights = _randn((N,), 100, 0.05)
    weights = torch.where(weights.abs() < 1e-3, torch.full_like(weights, 1e-3), weights)
    off = sizes[0] + sizes[1]
    edge = ((off // 4096) + 128) * 4096
    for start, length in ((edge - 150, 300), (off + 8192, 513), (N - 280, 280), (100, 150), (4096 - 7, 257)):
        weights[start:start + length] = 0.0

    def grads(t):
        g = _randn((W, N), 300 + t, 1e-3)
        g[(t + 1) % W, off + 3 * 4096 + 500:off + 3 * 4096 + 900] *= 1000.0
        return g

    _run(sizes, W, [2.0, 1.0, 0.5], weights, grads, steps=4, n_leaders=n_leaders, residual_every=2)


def test_threshold_mode_ties_zero_and_infinite_thresholds():
    sizes, W = [50000, 300, 20000, 5], 3
    N = sum(sizes)
    g = torch.Generator(device=DEV)
    g.manual_seed(8)
    weights = torch.randint(-2, 3, (N,), generator=g, device=DEV).float() * 0.5

    def grads(t):
        gg = torch.Generator(device=DEV)
        gg.manual_seed(60 + t)
        return torch.randint(-4, 5, (W, N), generator=gg, device=DEV).float() / 8.0

    # many importances equal a threshold exactly (strict comparison); 0 sends every non-zero residual, inf nothing
    _run(sizes, W, [0.5, 0.0, 1.0, float("inf")], weights, grads, steps=4)


def test_threshold_mode_momentum_and_forced_scalar():
    sizes, W = [40000, 128, 16385], 4
    N = sum(sizes)
    weights = _randn((N,), 5, 0.05)
    _run(sizes, W, [0.3, 0.05, 1.0], weights, lambda t: _randn((W, N), 31 * t + 2, 1e-3), steps=4, momentum=0.9,
         force_scalar=True, residual_every=2)


def test_threshold_mode_capacity_error_and_argument_checks():
    sizes, W = [20000], 2
    weights = torch.ones(20000, device=DEV)
    pr = Pruner(sizes, W, None, 1e-8, 0, max_list=100)
    L = binding.lib()
    E = binding.IWP_ERR_INVALID
    g = _randn((W, 20000), 1, 1.0)
    assert L.iwp_step(pr._h, g.data_ptr(), weights.data_ptr(), weights.data_ptr()) == E  # no thresholds yet
    import ctypes as C

    bad = ((C.c_float * 1)(-1.0), (C.c_float * 1)(float("nan")))
    for arr in bad:
        assert L.iwp_set_thresholds(pr._h, arr) == E
    assert L.iwp_set_thresholds(pr._h, None) == E
    pr.set_thresholds([0.5])  # about 60 % of 20000 pass: far more than 100 entries
    pr.step(g, weights)
    assert pr.sync_status() == binding.IWP_ERR_CAPACITY
    assert pr.list_length() > 100
    assert "capacity" in binding.iwp_strerror(binding.IWP_ERR_CAPACITY)
    pr.close()
    ratio = Pruner(sizes, W, 4.0)
    assert L.iwp_set_thresholds(ratio._h, bad[0]) == E  # not a threshold-mode context
    assert ratio.list_length() == ratio.K
    ratio.close()


def test_threshold_mode_full_size_alexnet_shape():
    c = wl.alexnet_w8()
    weights = c.weights(DEV)
    # thresholds near the step-0 top-1/64 point of the He-normal / N(0, 0.01 std) recipe for weight tensors;
    # biases are zero-initialised (importance = |residual| / eps), so their thresholds sit at that scale
    thr = []
    for tns in c.tensors:
        thr.append(0.4 if tns.kind == "weight" else 2.0e4)
    buf = torch.empty((c.W, c.N), dtype=torch.float32, device=DEV)
    _run(c.layer_sizes, c.W, thr, weights, lambda t: c.grads(t, DEV, out=buf), steps=3, seed=c.seed, residual_every=3)


@pytest.mark.parametrize("n_leaders", [2, 4])
def test_threshold_mode_several_chosen_nodes(n_leaders):
    sizes, W = [70000, 300, 16385, 64], 5
    N = sum(sizes)
    weights = _randn((N,), 9, 0.05)
    weights[::31] = 0.0
    _run(sizes, W, [0.2, 0.05, 1.0, 0.5], weights, lambda t: _randn((W, N), 13 * t + 4, 1e-3), steps=5,
         n_leaders=n_leaders, residual_every=2)
    pr = Pruner(sizes, W, None, 1e-8, 0, thresholds=[1.0] * 4)
    L = binding.lib()
    assert L.iwp_set_option(pr._h, b"n_leaders", 6) == binding.IWP_ERR_INVALID  # more than W
    assert L.iwp_set_option(pr._h, b"n_leaders", 0) == binding.IWP_ERR_INVALID
    pr.close()
    ratio = Pruner(sizes, W, 4.0)
    assert L.iwp_set_option(ratio._h, b"n_leaders", 2) == 0  # the ratio mode takes several chosen nodes too
    assert L.iwp_set_option(ratio._h, b"n_leaders", 9) == binding.IWP_ERR_INVALID  # more than eight
    ratio.close()


@pytest.mark.parametrize("n_leaders", [1, 3])
def test_threshold_mode_random_sub_threshold_selection(n_leaders):
    sizes, W = [90000, 300, 16385], 4
    N = sum(sizes)
    weights = _randn((N,), 19, 0.05)
    weights[::41] = 0.0
    # high thresholds: most of what is sent is sent by the draw, not by the comparison
    _run(sizes, W, [5.0, 0.5, 20.0], weights, lambda t: _randn((W, N), 17 * t + 5, 1e-3), steps=5,
         n_leaders=n_leaders, random_select=True, momentum=0.9, residual_every=2)


def test_random_select_with_zero_and_infinite_thresholds():
    sizes, W = [20000, 20000], 2
    N = sum(sizes)
    weights = torch.ones(N, device=DEV)
    g = torch.Generator(device=DEV)
    g.manual_seed(3)
    grads = lambda t: torch.randint(-2, 3, (W, N), generator=g, device=DEV).float()  # many exact zeros
    _run(sizes, W, [0.0, float("inf")], weights, grads, steps=3, random_select=True)


# ------------------------------------------------------------------ layer-wise threshold (Section 3.4, Eq. 4)


@pytest.mark.parametrize("name", sorted(CASES))
def test_layerwise_threshold_random_values(name):
    sizes, W = CASES[name]
    N = sum(sizes)
    weights = _randn((N,), 100, 0.05)
    weights[::97] = 0.0  # importances of 1e6 and more beside ordinary ones: many exponents in one sum
    # C in the middle of the values var/mean takes here, so that both branches of Eq. 4 occur
    _run(sizes, W, None, weights, lambda t: _randn((W, N), 300 + t, 0.01 * (1 + 3 * (t % 2))), steps=4,
         layerwise=(0.3, 1e-9, 3e7), residual_every=2)


@pytest.mark.parametrize("n_leaders", [2, 3])
def test_layerwise_threshold_several_chosen_nodes_and_random_selection(n_leaders):
    sizes, W = [64, 16385, 256, 100000, 9408, 1, 36864], 4
    N = sum(sizes)
    weights = _randn((N,), 101, 0.05)
    _run(sizes, W, None, weights, lambda t: _randn((W, N), 400 + t, 0.02), steps=4, n_leaders=n_leaders,
         layerwise=(0.5, 0.01, 5.0), random_select=(n_leaders == 3), momentum=0.9)
    # each branch of Eq. 4 on its own: C below every var/mean, then above every one
    up = _run(sizes, W, None, weights, lambda t: _randn((W, N), 400 + t, 0.02), steps=2, n_leaders=n_leaders,
              layerwise=(0.5, 1e-6, -1.0))
    down = _run(sizes, W, None, weights, lambda t: _randn((W, N), 400 + t, 0.02), steps=2, n_leaders=n_leaders,
                layerwise=(0.5, 1e-6, 1e300))
    multi = [l for l, n in enumerate(sizes) if n > 1]  # a one-element layer has no variance
    assert all((thr[:, multi] > 0.5).all() for thr in up) and all((thr[:, multi] < 0.5).all() for thr in down)


def test_layerwise_threshold_degenerate_layers():
    # all-zero gradients (mean 0), a constant layer (variance 0), denormal importances, a negative
    # threshold (everything goes) and a threshold no importance reaches
    sizes, W = [4096, 20000, 5000, 70000], 3
    N = sum(sizes)
    weights = torch.ones(N, device=DEV)
    weights[4096 + 20000:4096 + 25000] = 1e30  # importances far below 1e-38 in the third layer

    def grads(t):
        g = _randn((W, N), 500 + t, 0.25)
        g[:, :4096] = 0.0
        g[:, 4096:24096] = 0.5 if t % 2 == 0 else -0.5
        return g

    _run(sizes, W, None, weights, grads, steps=3, layerwise=(0.2, 1.0, 0.1))
    _run(sizes, W, None, weights, grads, steps=2, layerwise=(-1.0, 0.0, 0.0))
    _run(sizes, W, None, weights, grads, steps=2, layerwise=(1e30, 0.0, 0.0))


def test_layerwise_argument_checks():
    pr = Pruner([5000, 300], 2, None, 1e-8, 0)
    for bad in ((float("nan"), 1.0, 1.0), (0.1, float("inf"), 1.0), (0.1, 1.0, float("nan"))):
        with pytest.raises(binding.IwpError):
            pr.set_layerwise(*bad)
    with pytest.raises(binding.IwpError):
        pr.layer_thresholds()  # not switched on
    pr.set_layerwise(0.1, 1.0, 1.0)
    assert pr.layer_thresholds().shape[0] == 0  # no step yet
    pr.set_layerwise(0.0, 0.0, 0.0, on=False)
    g = torch.zeros((2, 5300), device=DEV)
    with pytest.raises(binding.IwpError):
        pr.step(g, torch.ones(5300, device=DEV))  # back on fixed thresholds, and none were given
    pr.close()
    ratio_ctx = Pruner([5000], 2, 4.0, 1e-8, 0)
    with pytest.raises(binding.IwpError):
        ratio_ctx.set_layerwise(0.1, 1.0, 1.0)
    ratio_ctx.close()


def test_layerwise_threshold_full_size_alexnet_shape():
    c = wl.alexnet_w8()
    weights = c.weights(DEV)
    buf = torch.empty((c.W, c.N), dtype=torch.float32, device=DEV)
    _run(c.layer_sizes, c.W, None, weights, lambda t: c.grads(t, DEV, out=buf), steps=2, seed=c.seed,
         layerwise=(0.05, 1e-4, 100.0), residual_every=2)


# ------------------------------------------------------------------ seeded random shapes and options


@pytest.mark.parametrize("seed", range(int(__import__("os").environ.get("IWP_SHAPE_SEEDS", "8"))))
def test_threshold_mode_random_shapes(seed):
    rng = np.random.default_rng(6000 + seed)
    edges = [1, 3, 4, 5, 4095, 4096, 4097, 16383, 16384, 16385, 32767, 32768, 32769, 65537, 8 * 4096, 8 * 4096 + 1]
    sizes = [int(rng.choice(edges)) if rng.random() < 0.7 else int(rng.integers(1, 150000)) for _ in range(int(rng.integers(1, 6)))]
    if rng.random() < 0.5 and sum(sizes) % 4:
        sizes[-1] += 4 - sum(sizes) % 4
    W = int(rng.integers(1, 8))
    N = sum(sizes)
    weights = _randn((N,), 8000 + seed, 0.05)
    weights[:: int(rng.integers(7, 100))] = 0.0
    n_leaders = int(rng.integers(1, min(W, 4) + 1))
    kw = dict(steps=3, seed=seed, n_leaders=n_leaders, random_select=bool(rng.random() < 0.4),
              momentum=float(rng.choice([1.0, 0.5])), residual_every=int(rng.choice([1, 1000])))
    grads = lambda t: _randn((W, N), 9000 + 10 * seed + t, 1e-2)
    if rng.random() < 0.5:
        _run(sizes, W, None, weights, grads, layerwise=(float(rng.choice([0.0, 0.3, 2.0])), float(rng.choice([0.0, 1e-6, 0.05])),
                                                        float(rng.choice([0.0, 5.0, 1e9]))), **kw)
    else:
        _run(sizes, W, [float(rng.choice([0.0, 0.05, 0.5, 50.0])) for _ in sizes], weights, grads, **kw)
