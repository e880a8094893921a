"""GPU parity: the CUDA library against the CPU oracle, element by element and bit for bit
(update, residuals, ordered (index, value) lists, leader, byte mask), through the C ABI.

Tolerance: none.  Indices, masks and residuals are integer/bit work; the update is a sum in
a fixed worker order of IEEE binary32 additions on both sides, so it is compared bit-exactly
as well (the 1e-6 relative allowance would only apply to an unordered reduction, which
this library does not use)."""
import json
import os

import numpy as np
import pytest
import torch

from paper_1901_01544_b200 import workloads as wl
from parity import assert_bits_equal, run_parity

pytestmark = pytest.mark.gpu
GOLD = os.path.join(os.path.dirname(__file__), "golden")
DEV = "cuda"


def _randn(shape, seed, scale=1.0):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return torch.randn(shape, generator=g, device=DEV, dtype=torch.float32) * scale


def _weights(N, seed, zero_frac=0.05, scale=0.05):
    w = _randn((N,), seed, scale)
    g = torch.Generator(device=DEV)
    g.manual_seed(seed + 1)
    w[torch.rand(N, generator=g, device=DEV) < zero_frac] = 0.0
    return w


# ------------------------------------------------------------------ hand-worked example


def test_worked_example_on_gpu():
    g = json.load(open(os.path.join(GOLD, "worked_example.json")))
    from paper_1901_01544_b200.binding import Pruner

    pr = Pruner(g["layer_sizes"], g["W"], g["ratio"], g["eps"], 0)
    weights = torch.tensor(g["weights"], dtype=torch.float32, device=DEV)
    for st in g["steps"]:
        pr.set_option("leader_override", st["leader"])
        upd = pr.step(torch.tensor(st["grads"], dtype=torch.float32, device=DEV), weights)
        assert pr.sync_status() == 0 and pr.leader == st["leader"]
        assert_bits_equal(upd.cpu().numpy(), np.array(st["update"], np.float32), "update")
        for w in range(g["W"]):
            idx, val = pr.selection(w)
            assert idx.cpu().tolist() == st["lists"][w]
            assert_bits_equal(val.cpu().numpy(), np.array(st["list_vals"][w], np.float32), "list values")
            assert_bits_equal(pr.residual(w).cpu().numpy(), np.array(st["residual"][w], np.float32), "residual")
        assert pr.mask().cpu().tolist() == [1 if i in st["lists"][st["leader"]] else 0 for i in range(8)]
    pr.close()


# ------------------------------------------------------------------ tiny and adversarial inputs

CASES = {
    # name: (layer_sizes, W, ratio)
    "small_only": ([5, 1, 12, 3, 64, 300], 3, 3.0),
    "n_less_than_ratio": ([3, 2, 1, 40], 2, 64.0),
    "single_element": ([1], 4, 64.0),
    "one_tiled_layer": ([40000], 2, 16.0),
    "tiled_odd_total_scalar_path": ([20001, 17, 70003], 3, 10.0),
    "tiled_unaligned_offsets_vector_path": ([16389, 16387, 40000], 2, 7.0),
    "mixed_many": ([64, 16385, 256, 100000, 9408, 4096, 36864, 1000, 17000], 4, 58.8),
    "keep_everything": ([50000, 100], 3, 1.0),
    "one_worker": ([30000, 70], 1, 20.0),
    "thirty_three_workers": ([17000, 33], 33, 50.0),
    "chunk_boundaries": ([65536 * 2 + 4096 + 1, 65536], 2, 64.0),
}


# overlap: the schedule the library would only pick by itself for larger workloads is forced on as well
@pytest.mark.parametrize("overlap", [0, 1])
@pytest.mark.parametrize("name", sorted(CASES))
def test_random_values(name, overlap):
    sizes, W, ratio = CASES[name]
    N = sum(sizes)
    weights = _weights(N, 100 + N % 97)
    run_parity(sizes, W, ratio, 1e-8, seed=7, steps=3, weights=weights,
               grads_fn=lambda t: _randn((W, N), 1000 * t + 3, 1e-3), options={"overlap": overlap})


@pytest.mark.parametrize("overlap", [0, 1])
@pytest.mark.parametrize("name", ["mixed_many", "tiled_unaligned_offsets_vector_path", "one_tiled_layer"])
def test_many_ties(name, overlap):
    # coarse values: importances collide all the time, exact cancellations to +0 occur
    sizes, W, ratio = CASES[name]
    N = sum(sizes)
    g = torch.Generator(device=DEV)
    g.manual_seed(5)
    weights = torch.randint(-2, 3, (N,), generator=g, device=DEV).float() * 0.5

    def grads(t):
        gg = torch.Generator(device=DEV)
        gg.manual_seed(50 + t)
        return torch.randint(-4, 5, (W, N), generator=gg, device=DEV).float() / 8.0

    run_parity(sizes, W, ratio, 1e-8, seed=1, steps=4, weights=weights, grads_fn=grads, options={"overlap": overlap},
               state_every=1 + overlap)


@pytest.mark.parametrize("overlap", [0, 1])
@pytest.mark.parametrize("kind", ["all_equal", "all_zero", "two_values", "zero_weights", "tiny_values", "tiny_eps",
                                  "huge_values"])
def test_degenerate_layers(kind, overlap):
    sizes, W, ratio = [100000, 5000, 37], 3, 32.0
    N = sum(sizes)
    eps = 1e-8
    if kind == "tiny_values":  # importances far below 2^-60, some denormal
        weights = _weights(N, 3, zero_frac=0.0, scale=1.0) + 0.5
        grads = lambda t: _randn((W, N), 5 + t, 1e-38)
    elif kind == "tiny_eps":  # denominators down to 1e-30
        eps = 1e-30
        weights = _weights(N, 3, zero_frac=0.3)
        grads = lambda t: _randn((W, N), 6 + t, 1e-6)
    elif kind == "huge_values":  # importances up to ~1e37: products in the candidate pre-test overflow
        weights = _weights(N, 3, zero_frac=0.3)
        grads = lambda t: _randn((W, N), 7 + t, 1e29)
    elif kind == "all_equal":
        weights = torch.full((N,), -0.5, device=DEV)
        grads = lambda t: torch.full((W, N), 0.25, device=DEV)
    elif kind == "all_zero":
        weights = _weights(N, 3)
        grads = lambda t: torch.zeros((W, N), device=DEV)
    elif kind == "two_values":
        weights = torch.ones(N, device=DEV)
        g = torch.Generator(device=DEV)
        g.manual_seed(9)
        pick = torch.rand((W, N), generator=g, device=DEV) < 0.01  # fewer large values than k: ties at the small one
        grads = lambda t: torch.where(pick, torch.tensor(1.0, device=DEV), torch.tensor(0.25, device=DEV))
    else:
        weights = torch.zeros(N, device=DEV)
        grads = lambda t: _randn((W, N), 77 + t, 1e-3)
    run_parity(sizes, W, ratio, eps, seed=2, steps=3, weights=weights, grads_fn=grads, options={"overlap": overlap},
               state_every=1 + overlap)


def test_forced_scalar_path_and_leader_override():
    sizes, W, ratio = [40000, 128, 16385], 4, 16.0
    N = sum(sizes)
    weights = _weights(N, 11)
    run_parity(sizes, W, ratio, 1e-8, seed=0, steps=4, weights=weights,
               grads_fn=lambda t: _randn((W, N), 31 * t + 1, 1e-2), options={"force_scalar": 1},
               leader_overrides=[3, 0, 2, 2])


@pytest.mark.parametrize("overlap", [0, 1])
def test_select_chain_for_every_layer(overlap):
    # the one-launch select per (layer, worker) pair switched off: every tiled layer goes through the chain
    sizes, W, ratio = [300000, 128, 70000, 16385], 4, 64.0
    N = sum(sizes)
    weights = _weights(N, 13)
    run_parity(sizes, W, ratio, 1e-8, seed=0, steps=3, weights=weights,
               grads_fn=lambda t: _randn((W, N), 17 * t + 2, 1e-2), options={"pair_select": 0, "overlap": overlap})


def test_pair_select_next_to_the_chain_and_beyond_its_key_cache():
    # one layer above the limit of the one-launch select (641 tiles: chain), one of 600 tiles whose candidates
    # exceed what the kernel keeps in shared memory (the rest is re-read), and small ones
    sizes, W, ratio = [641 * 4096 - 100, 600 * 4096, 20000, 64], 3, 32.0
    N = sum(sizes)
    weights = _weights(N, 15, zero_frac=0.0)
    for overlap in (0, 1):
        run_parity(sizes, W, ratio, 1e-8, seed=2, steps=3, weights=weights,
                   grads_fn=lambda t: _randn((W, N), 19 * t + 5, 1e-2), options={"overlap": overlap, "pair_select": 1},
                   residual_every=3)


def test_exact_select_without_speculation():
    sizes, W, ratio = [300000, 128, 70000], 4, 64.0
    N = sum(sizes)
    weights = _weights(N, 13)
    run_parity(sizes, W, ratio, 1e-8, seed=0, steps=3, weights=weights,
               grads_fn=lambda t: _randn((W, N), 17 * t + 2, 1e-2), options={"speculate": 0})


def test_misaligned_caller_pointers():
    # caller buffers offset by one float: the library must fall back to scalar accesses
    sizes, W, ratio = [40000, 24], 2, 16.0
    N = sum(sizes)
    import oracle
    from paper_1901_01544_b200.binding import Pruner

    pr = Pruner(sizes, W, ratio, 1e-8, 4)
    orc = oracle.Oracle(sizes, W, ratio, 1e-8, 4)
    wbuf = torch.zeros(N + 1, device=DEV)
    wbuf[1:] = _weights(N, 5)
    gbuf = torch.zeros(W * N + 1, device=DEV)
    ubuf = torch.zeros(N + 1, device=DEV)
    for t in range(2):
        gbuf[1:] = _randn((W * N,), 90 + t, 1e-3)
        pr.step(gbuf[1:], wbuf[1:], ubuf[1:])
        want = orc.step(gbuf[1:].view(W, N).cpu().numpy().copy(), wbuf[1:].cpu().numpy().copy())
        assert pr.sync_status() == 0
        assert_bits_equal(ubuf[1:].cpu().numpy(), want, "update")
        for w in range(W):
            assert_bits_equal(pr.residual(w).cpu().numpy(), orc.residual(w), "residual")
            assert np.array_equal(pr.selection(w)[0].cpu().numpy().view(np.uint32), orc.selection(w)[0])
    pr.close()


# ------------------------------------------------------------------ the five configurations, scaled


def _scaled_case(name):
    if name == "single_layer":
        return wl.scaled(wl.single_layer(), [1 << 17], name="c1s")
    if name == "alexnet_w8":
        b = wl.alexnet_w8()
        return wl.scaled(b, [max(3, n // 48 + (n % 7)) for n in b.layer_sizes])
    if name == "resnet50_w8":
        b = wl.resnet50_w8()
        return wl.scaled(b, [max(2, n // 16 + (n % 5)) for n in b.layer_sizes], W=4)
    if name == "alexnet_w32":
        b = wl.alexnet_w32()
        return wl.scaled(b, [max(3, n // 192 + (n % 3)) for n in b.layer_sizes], steps=20)
    b = wl.flat_1g_w4()
    return wl.scaled(b, wl.split_equal((1 << 22) + 64, 96), steps=4)


@pytest.mark.parametrize("residual_every", [1, 1000])
@pytest.mark.parametrize("name", sorted(wl.CONFIGS))
def test_scaled_configs(name, residual_every):
    c = _scaled_case(name)
    weights = c.weights(DEV)
    run_parity(c.layer_sizes, c.W, c.ratio, c.eps, c.seed, c.steps, weights, lambda t: c.grads(t, DEV),
               residual_every=residual_every)


@pytest.mark.parametrize("overlap", [1, 0])
def test_long_run_into_the_steady_state(overlap):
    # 150 steps over five cycled gradient batches, as the bench runs them: residuals pile up, the chosen node's set
    # is zeroed on every worker step after step, thresholds settle.  The update is compared after every step, lists
    # and residuals now and then and at the end.
    c = _scaled_case("alexnet_w8")
    weights = c.weights(DEV)
    sets = [c.grads(t, DEV) for t in range(5)]
    run_parity(c.layer_sizes, c.W, c.ratio, c.eps, c.seed, 150, weights, lambda t: sets[t % 5],
               options={"overlap": overlap}, state_every=37, residual_every=74)


def test_residuals_left_alone_between_steps_with_ties_and_fallbacks():
    # coarse values: some pairs fall back to the multi-pass select, others stay on the single-read
    # path; residuals are read only at the end, and the option switch in the middle forces a flush
    sizes, W, ratio = [70000, 64, 16385, 300000], 4, 64.0
    N = sum(sizes)
    g = torch.Generator(device=DEV)
    g.manual_seed(17)
    weights = torch.randint(-3, 4, (N,), generator=g, device=DEV).float() * 0.25

    def grads(t):
        gg = torch.Generator(device=DEV)
        gg.manual_seed(500 + t)
        coarse = torch.randint(-4, 5, (W, N), generator=gg, device=DEV).float() / 8.0
        fine = torch.randn((W, N), generator=gg, device=DEV) * 1e-3
        return coarse if t % 3 == 2 else fine

    run_parity(sizes, W, ratio, 1e-8, seed=3, steps=7, weights=weights, grads_fn=grads, residual_every=1000)


# ------------------------------------------------------------------ selects left running past the end of a step


@pytest.mark.parametrize("state_every", [2, 3, 1000])
@pytest.mark.parametrize("overlap", [1, 0])
def test_steps_back_to_back_with_changing_weights(state_every, overlap):
    # Nobody asks for lists or residuals between most steps, so the other workers' selects of one step
    # run beside the head of the next; the weights change right after every step (the library must have
    # kept what a late fallback still needs), and coarse values make some pairs fall back while others
    # stay on the single-read path.
    sizes, W, ratio = [70000, 64, 16385, 300000, 40000], 5, 64.0
    N = sum(sizes)

    def weights_at(t):
        g = torch.Generator(device=DEV)
        g.manual_seed(900 + t)
        return torch.randint(-3, 4, (N,), generator=g, device=DEV).float() * 0.25

    def grads(t):
        gg = torch.Generator(device=DEV)
        gg.manual_seed(700 + t)
        coarse = torch.randint(-4, 5, (W, N), generator=gg, device=DEV).float() / 8.0
        fine = torch.randn((W, N), generator=gg, device=DEV) * 1e-3
        if t % 4 == 1:
            return coarse
        if t % 4 == 3:  # only two workers coarse: their pairs fall back, the others' do not
            fine[1] = coarse[1]
            fine[3] = coarse[3]
        return fine

    run_parity(sizes, W, ratio, 1e-8, seed=11, steps=9, weights=weights_at(0).clone(), grads_fn=grads,
               residual_every=1000, state_every=state_every, weights_fn=weights_at, options={"overlap": overlap})


@pytest.mark.parametrize("W", [2, 3])
def test_back_to_back_steps_with_few_workers(W):
    # W = 2: the leader and the next step's leader may be all there is
    sizes, ratio = [50000, 20000], 32.0
    N = sum(sizes)
    weights = _weights(N, 3)
    run_parity(sizes, W, ratio, 1e-8, seed=4, steps=8, weights=weights,
               grads_fn=lambda t: _randn((W, N), 40 + t), residual_every=1000, state_every=1000)


def test_back_to_back_steps_with_leader_overrides():
    # the leader the library foresaw for the next step is not the one it gets
    sizes, W, ratio = [50000, 20000, 100], 4, 32.0
    N = sum(sizes)
    weights = _weights(N, 5)
    run_parity(sizes, W, ratio, 1e-8, seed=4, steps=8, weights=weights, grads_fn=lambda t: _randn((W, N), 60 + t),
               leader_overrides=[0, 3, 3, 1, -1, 2, -1, 0], residual_every=1000, state_every=1000)


# ------------------------------------------------------------------ only the chosen node selects (option)


@pytest.mark.parametrize("speculate", [1, 0])
@pytest.mark.parametrize("overlap", [1, 0])
def test_leader_only_select(overlap, speculate):
    # Algorithm 1 consumes the chosen node's index set only; with the option on, no other worker makes a list.
    # Update, chosen node's list, mask and every residual are those of the default path.
    sizes, W, ratio = [70000, 64, 16385, 300000, 9, 40000], 5, 32.0
    N = sum(sizes)
    weights = _weights(N, 27)
    run_parity(sizes, W, ratio, 1e-8, seed=9, steps=6, weights=weights, grads_fn=lambda t: _randn((W, N), 600 + t),
               options={"leader_only_select": 1, "overlap": overlap, "speculate": speculate}, residual_every=2,
               leader_list_only=True)


def test_leader_only_select_switched_on_and_off_between_steps():
    import oracle
    from paper_1901_01544_b200.binding import Pruner
    from parity import compare_state

    c = _scaled_case("alexnet_w8")
    pr = Pruner(c.layer_sizes, c.W, c.ratio, c.eps, c.seed)
    orc = oracle.Oracle(c.layer_sizes, c.W, c.ratio, c.eps, c.seed)
    pr.set_option("overlap", 1)
    weights = c.weights(DEV)
    w_host = weights.cpu().numpy()
    update = torch.full((pr.N,), float("nan"), device=DEV)
    for t in range(8):
        only = t % 3 != 0
        pr.set_option("leader_only_select", int(only))
        g = c.grads(t, DEV)
        pr.step(g, weights, update)
        want = orc.step(np.ascontiguousarray(g.cpu().numpy()), w_host)
        compare_state(pr, orc, update, want, f"step {t}", check_residual=t % 2 == 1, leader_list_only=only)
        assert pr.stat("spec_failed") == 0
        update.fill_(float("nan"))
    pr.close()
    orc.close()


# ------------------------------------------------------------------ several chosen nodes (Mask = OR Mask_ri)


@pytest.mark.parametrize("speculate", [1, 0])
@pytest.mark.parametrize("n_leaders", [2, 4])
def test_union_of_several_chosen_nodes(n_leaders, speculate):
    sizes, W, ratio = [70000, 64, 16385, 300000, 9, 40000], 5, 32.0
    N = sum(sizes)
    weights = _weights(N, 21)
    run_parity(sizes, W, ratio, 1e-8, seed=6, steps=5, weights=weights, grads_fn=lambda t: _randn((W, N), 800 + t),
               n_leaders=n_leaders, options={"speculate": speculate}, residual_every=2)


def test_union_with_ties_fallbacks_and_identical_workers():
    # coarse values (ties, fallbacks) and two workers with the same gradients: their lists coincide, so every
    # element of the union has two entries competing for it
    sizes, W, ratio = [70000, 300, 20000], 4, 16.0
    N = sum(sizes)
    g0 = torch.Generator(device=DEV)
    g0.manual_seed(5)
    weights = torch.randint(-3, 4, (N,), generator=g0, device=DEV).float() * 0.25

    def grads(t):
        gg = torch.Generator(device=DEV)
        gg.manual_seed(870 + t)
        g = torch.randint(-4, 5, (W, N), generator=gg, device=DEV).float() / 8.0 if t % 2 else \
            torch.randn((W, N), generator=gg, device=DEV) * 1e-3
        g[2] = g[0]
        return g

    run_parity(sizes, W, ratio, 1e-8, seed=1, steps=5, weights=weights, grads_fn=grads, n_leaders=4)


def test_union_on_a_scaled_network_shape():
    c = _scaled_case("resnet50_w8")
    run_parity(c.layer_sizes, c.W, c.ratio, c.eps, c.seed, c.steps, c.weights(DEV), lambda t: c.grads(t, DEV), n_leaders=3,
               residual_every=1000)


# ------------------------------------------------------------------ one chosen node per layer


@pytest.mark.parametrize("speculate", [1, 0])
def test_one_chosen_node_per_layer(speculate):
    sizes, W, ratio = [70000, 64, 16385, 300000, 9, 40000, 1], 5, 32.0
    N = sum(sizes)
    weights = _weights(N, 23)
    run_parity(sizes, W, ratio, 1e-8, seed=8, steps=5, weights=weights, grads_fn=lambda t: _randn((W, N), 880 + t),
               per_layer_leaders=True, options={"speculate": speculate}, residual_every=2)


def test_one_chosen_node_per_layer_on_a_scaled_network_shape():
    from paper_1901_01544_b200 import binding

    c = _scaled_case("resnet50_w8")
    run_parity(c.layer_sizes, c.W, c.ratio, c.eps, c.seed, c.steps, c.weights(DEV), lambda t: c.grads(t, DEV),
               per_layer_leaders=True, residual_every=1000)
    got = [binding.lib().iwp_layer_leader_at(0, t, l, 8) for t in range(2) for l in range(6)]
    assert got == [2, 6, 1, 3, 7, 2, 7, 7, 5, 2, 7, 5]  # tests/golden/layer_leaders.txt, first row


# ------------------------------------------------------------------ momentum on the residual (Eq. 3)


@pytest.mark.parametrize("m", [0.9, 0.5, 0.0])
@pytest.mark.parametrize("speculate", [1, 0])
def test_momentum(m, speculate):
    sizes, W, ratio = [70000, 300, 16385, 64], 4, 64.0
    N = sum(sizes)
    weights = _weights(N, 21)
    run_parity(sizes, W, ratio, 1e-8, seed=5, steps=5, weights=weights,
               grads_fn=lambda t: _randn((W, N), 400 + t, 1e-3), options={"speculate": speculate}, momentum=m,
               residual_every=2)


def test_momentum_on_a_scaled_network_shape():
    c = _scaled_case("resnet50_w8")
    weights = c.weights(DEV)
    run_parity(c.layer_sizes, c.W, c.ratio, c.eps, c.seed, c.steps, weights, lambda t: c.grads(t, DEV), momentum=0.9,
               residual_every=1000)


# ------------------------------------------------------------------ option changes between steps


@pytest.mark.parametrize("seed", range(int(os.environ.get("IWP_WALK_SEEDS", "4"))))
def test_random_option_changes_between_steps(seed):
    """A seeded walk over the library's switches between steps - schedule, select path, number of chosen
    nodes, forced leaders, momentum, step counter, residual reads - against the oracle taking the same walk.
    Lists and residuals are compared only now and then, so late selects of one step meet all kinds of
    next steps."""
    import oracle
    from paper_1901_01544_b200.binding import Pruner
    from parity import compare_state

    rng = np.random.default_rng(1000 + seed)
    sizes, W, ratio = [70000, 64, 16385, 150000, 9, 40000], 4, 32.0
    N = sum(sizes)
    weights = _weights(N, 31 + seed)
    w_host = weights.cpu().numpy()
    pr = Pruner(sizes, W, ratio, 1e-8, seed)
    orc = oracle.Oracle(sizes, W, ratio, 1e-8, seed)
    pr.set_option("overlap", 1)  # the workload is below the size at which the library would choose it by itself
    update = torch.full((N,), float("nan"), device=DEV)
    for t in range(24):
        what = int(rng.integers(0, 9))
        if what == 0:
            pr.set_option("overlap", int(rng.integers(0, 2)))
        elif what == 1:
            pr.set_option("speculate", int(rng.integers(0, 2)))
        elif what == 2:
            n = int(rng.integers(1, W + 1))
            pr.set_option("n_leaders", n)
            orc.set_n_leaders(n)
        elif what == 3:
            lead = int(rng.integers(-1, W))
            pr.set_option("leader_override", lead)
            orc.set_leader_override(lead)
        elif what == 4:
            m = float(rng.choice([1.0, 0.9, 0.5]))
            pr.set_momentum(m)
            orc.set_momentum(m)
        elif what == 5:
            for w in range(W):  # forces the pending zeroing out
                assert_bits_equal(pr.residual(w).cpu().numpy(), orc.residual(w), f"before step {t}: worker {w} residual")
        elif what == 6:
            pr.set_option("time_stages", int(rng.integers(0, 3)))
        elif what == 7:
            pr.set_option("pair_select", int(rng.integers(-1, 2)))
        coarse = rng.random() < 0.3  # ties and fallbacks now and then
        if coarse:
            g = torch.randint(-4, 5, (W, N), device=DEV, generator=torch.Generator(device=DEV).manual_seed(t)).float() / 8.0
        else:
            g = _randn((W, N), 2000 + 100 * seed + t)
        pr.step(g, weights, update)
        upd_cpu = orc.step(np.ascontiguousarray(g.cpu().numpy()), w_host)
        assert pr.leader == orc.leader
        if rng.random() < 0.4 or t == 23:
            compare_state(pr, orc, update, upd_cpu, f"step {t}", check_residual=bool(rng.random() < 0.5) or t == 23)
        else:
            assert_bits_equal(update.cpu().numpy(), upd_cpu, f"step {t}: update")
        update.fill_(float("nan"))
    pr.set_option("time_stages", 0)
    pr.close()
    orc.close()


# ------------------------------------------------------------------ seeded random shapes


@pytest.mark.parametrize("seed", range(int(os.environ.get("IWP_SHAPE_SEEDS", "10"))))
def test_random_shapes(seed):
    """Layer lists drawn around the sizes where the code changes behaviour (one-CTA limit, tile and chunk edges,
    vector alignment), with random worker counts, ratios and schedules."""
    rng = np.random.default_rng(4000 + seed)
    edges = [1, 3, 4, 5, 4095, 4096, 4097, 8191, 16383, 16384, 16385, 16388, 65535, 65536, 65537, 128 * 4096, 128 * 4096 + 1]
    n_layers = int(rng.integers(1, 7))
    sizes = [int(rng.choice(edges)) if rng.random() < 0.7 else int(rng.integers(1, 200000)) for _ in range(n_layers)]
    if rng.random() < 0.5 and sum(sizes) % 4:  # half of the cases on the vector path
        sizes[-1] += 4 - sum(sizes) % 4
    W = int(rng.integers(1, 10))
    ratio = float(rng.choice([1.0, 2.0, 7.0, 58.8, 64.0, 1000.0]))
    N = sum(sizes)
    weights = _weights(N, 50 + seed)
    coarse = rng.random() < 0.3
    def grads(t):
        if coarse:
            return torch.randint(-4, 5, (W, N), device=DEV, generator=torch.Generator(device=DEV).manual_seed(seed * 100 + t)).float() / 8.0
        return _randn((W, N), 7000 + seed * 100 + t, 1e-2)
    run_parity(sizes, W, ratio, 1e-8, seed=seed, steps=4, weights=weights, grads_fn=grads,
               options={"overlap": int(rng.integers(0, 2)), "speculate": int(rng.random() < 0.8),
                        "pair_select": int(rng.random() < 0.7)},
               n_leaders=int(rng.integers(1, min(W, 3) + 1)), momentum=float(rng.choice([1.0, 0.9])),
               state_every=int(rng.choice([1, 2])), residual_every=int(rng.choice([1, 1000])))
