"""GPU parity on inputs whose importances are spatially clustered: runs of consecutive top-ranked
elements (a block of zero weights makes Algorithm 1's |grad / w| huge on the whole block; a hot filter
does the same through its gradients), placed at segment, tile and chunk edges of the streaming pass, on
the chosen node and on other workers.  Everything is compared with the CPU oracle bit for bit, as in
the other parity tests; tolerance: none.

Why these cases exist: the single-read path appends candidates to a per-(tile, worker) slot at ranks
computed from per-round counts inside a 512-element segment.  Independent random values never put more
than a handful of candidates into one segment, so only clustered inputs reach ranks above 255 inside a
segment, slots with more than 128 entries, and the tail loops of the select and the compaction."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_01544_b200.binding import Pruner
from parity import assert_bits_equal, compare_state, run_parity

pytestmark = pytest.mark.gpu
DEV = "cuda"
SEG, TILE, CHUNK = 512, 4096, 128 * 4096


def _randn(shape, seed, scale=1.0):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return torch.randn(shape, generator=g, device=DEV, dtype=torch.float32) * scale


def _dense_weights(N, seed, scale=0.05):
    """No exact zeros and nothing tiny, so that only the planted runs rank high."""
    w = _randn((N,), seed, scale)
    return torch.where(w.abs() < 1e-3, torch.full_like(w, 1e-3), w)


def _run_checked(sizes, W, ratio, weights, grads_fn, steps, overlap, leaders=None, expect_single_read=True, seed=7,
                 state_every=1, residual_every=1, pair_select=None):
    """run_parity plus the proof that the case stayed on the single-read path (no pair fell back)."""
    pr = Pruner(sizes, W, ratio, 1e-8, seed)
    orc = oracle.Oracle(sizes, W, ratio, 1e-8, seed)
    pr.set_option("overlap", overlap)
    pr.set_option("speculate", 1)
    # the two ways the single-read path selects from the candidate slots: the chain of launches (0) and the
    # one-launch cluster kernel (1); by default the one the overlap parameter does not pick is used too
    pr.set_option("pair_select", overlap if pair_select is None else pair_select)
    w_host = weights.cpu().numpy()
    update = torch.full((pr.N,), float("nan"), device=DEV)
    failed = 0
    for t in range(steps):
        if leaders is not None:
            pr.set_option("leader_override", leaders[t])
            orc.set_leader_override(leaders[t])
        g = grads_fn(t)
        pr.step(g, weights, update)
        want = orc.step(np.ascontiguousarray(g.cpu().numpy()), w_host)
        if (t + 1) % state_every == 0 or t == steps - 1:
            look = (t + 1) % residual_every == 0 or t == steps - 1
            compare_state(pr, orc, update, want, f"step {t}", check_residual=look)
        else:
            assert_bits_equal(update.cpu().numpy(), want, f"step {t}: update")
        failed += pr.stat("spec_failed")
        update.fill_(float("nan"))
    assert pr.stat("spec_pairs") > 0
    if expect_single_read:
        assert failed == 0, f"{failed} (worker, layer) pairs left the single-read path"
    pr.close()
    orc.close()
    return failed


@pytest.mark.parametrize("overlap", [0, 1])
@pytest.mark.parametrize("start", [8192, 8192 + 100, 4096 - 150, 3 * SEG - 7])
def test_zero_weight_block_of_300(start, overlap):
    # 300 consecutive zero weights: more than 255 and fewer than 512 candidates in one tile, from a segment
    # start, inside a segment, across a tile edge and across a segment edge
    n, W, ratio = 100000, 3, 64.0
    weights = _dense_weights(n, 3)
    weights[start:start + 300] = 0.0
    _run_checked([n], W, ratio, weights, lambda t: _randn((W, n), 11 + t, 1e-3), steps=3, overlap=overlap)


@pytest.mark.parametrize("overlap", [0, 1])
def test_zero_weight_block_across_a_chunk_edge_behind_other_layers(overlap):
    # the layer starts at an offset that is not a multiple of four elements of the tile grid; the run straddles
    # the first chunk edge of the layer (a chunk is 128 tiles) and a second one sits at the layer's ragged tail
    sizes, W, ratio = [300, 20000, CHUNK + 70000], 3, 256.0
    N = sum(sizes)
    weights = _dense_weights(N, 5)
    off = sizes[0] + sizes[1]
    first_chunk_end = ((off // TILE) + 128) * TILE  # chunks hold 128 tiles; tiles follow the flat 4096 grid
    weights[first_chunk_end - 150:first_chunk_end + 150] = 0.0
    weights[N - 280:N] = 0.0
    _run_checked(sizes, W, ratio, weights, lambda t: _randn((W, N), 21 + t, 1e-3), steps=3, overlap=overlap)


@pytest.mark.parametrize("run", [129, 255, 256, 257, 300, 383, 384, 385, 400, 512, 513, 700])
def test_run_lengths(run):
    # every length around the limits of a round (128), of a byte (255/256), of three rounds (384) and of the slot
    # (512); runs of 512 and more overflow the slot and must take the exact fallback
    n, W, ratio = 150000, 2, 256.0
    weights = _dense_weights(n, 9)
    start = 5 * TILE  # from a segment start
    weights[start:start + run] = 0.0
    failed = _run_checked([n], W, ratio, weights, lambda t: _randn((W, n), 31 + t, 1e-3), steps=2, overlap=0,
                          expect_single_read=run <= 400)
    if run >= 513:
        assert failed > 0  # the slot cannot hold the run: this case proves the fallback, not the single-read path


@pytest.mark.parametrize("overlap", [0, 1])
@pytest.mark.parametrize("who", ["leader", "other", "two_others"])
def test_hot_gradient_run_on_one_worker(who, overlap):
    # weights without structure; one worker's gradients are 1000 times larger on a run of 300: on the chosen node
    # (its candidates and the side values of everybody else), on another worker (its own slot only), on two others
    n, W, ratio = 65536, 4, 64.0
    weights = _dense_weights(n, 13)
    leaders = [1, 1, 2, 0]
    hot = {"leader": lambda t: [leaders[t]], "other": lambda t: [(leaders[t] + 1) % W],
           "two_others": lambda t: [(leaders[t] + 1) % W, (leaders[t] + 3) % W]}[who]

    def grads(t):
        g = _randn((W, n), 41 + t, 1e-3)
        for w in hot(t):
            g[w, 700:1000] *= 1000.0  # starts inside a segment, crosses one segment edge
            g[w, 2 * TILE:2 * TILE + 300] *= 1000.0 if t % 2 else 1.0  # every other step a second run, from a tile start
        return g

    _run_checked([n], W, ratio, weights, grads, steps=4, overlap=overlap, leaders=leaders, residual_every=2)


@pytest.mark.parametrize("overlap", [0, 1])
def test_one_tile_full_of_candidates_spread_over_its_segments(overlap):
    # 130 to 500 candidates in one tile, spread over all its segments instead of one run, other tiles sparse
    n, W, ratio = 200000, 3, 128.0
    weights = _dense_weights(n, 17)
    g = torch.Generator(device=DEV)
    g.manual_seed(99)
    for tile, count in ((3, 130), (7, 260), (11, 400), (20, 440)):
        pick = torch.randperm(TILE, generator=g, device=DEV)[:count] + tile * TILE
        weights[pick] = 0.0
    _run_checked([n], W, ratio, weights, lambda t: _randn((W, n), 51 + t, 1e-3), steps=3, overlap=overlap)


@pytest.mark.parametrize("pair_select", [1, 0])
def test_many_dense_tiles_in_a_row(pair_select):
    # 640 tiles; the first eighty hold about 460 candidates each (380 zero weights at random places + the usual 2 %):
    # 37 k candidate keys in the share of ONE CTA of the cluster select, more than the 16 k it keeps in shared memory
    # (the rest is re-read from the slots), and slots of more than 128 entries in every one of those tiles for the chain
    n, W, ratio = 640 * TILE, 2, 64.0
    weights = _dense_weights(n, 23)
    g = torch.Generator(device=DEV)
    g.manual_seed(7)
    for tile in range(80):
        pick = torch.randperm(TILE, generator=g, device=DEV)[:380] + tile * TILE
        weights[pick] = 0.0
    _run_checked([n], W, ratio, weights, lambda t: _randn((W, n), 71 + t, 1e-3), steps=2, overlap=0, pair_select=pair_select)


def test_clustered_runs_with_ties_inside_the_run():
    # the run's importances are all equal (same residual, zero weight): the threshold falls inside the run when the
    # run is longer than k, and the lower indices must win
    n, W, ratio = 80000, 2, 256.0  # k = 313
    weights = _dense_weights(n, 19)
    weights[2 * TILE + 100:2 * TILE + 100 + 450] = 0.0

    def grads(t):
        g = _randn((W, n), 61 + t, 1e-3)
        g[:, 2 * TILE + 100:2 * TILE + 100 + 450] = 0.25
        return g

    _run_checked([n], W, ratio, weights, grads, steps=3, overlap=0, expect_single_read=False)


@pytest.mark.parametrize("seed", range(6))
def test_random_clusters(seed):
    """Seeded random layer lists with random runs of zero weights and hot gradient runs planted at random
    offsets around segment, tile and chunk edges, random chosen nodes and schedules."""
    rng = np.random.default_rng(9000 + seed)
    sizes = [int(rng.choice([20000, 65536, 100000, 150001, CHUNK + 4097])) for _ in range(int(rng.integers(1, 4)))]
    if rng.random() < 0.5:
        sizes.insert(0, int(rng.integers(1, 5000)))
    if sum(sizes) % 4 and rng.random() < 0.6:
        sizes[-1] += 4 - sum(sizes) % 4
    N = sum(sizes)
    W = int(rng.integers(2, 6))
    ratio = float(rng.choice([64.0, 128.0, 256.0]))
    weights = _dense_weights(N, 70 + seed)
    edges = [e for e in (SEG, TILE, CHUNK) if e < N]
    runs = []
    for _ in range(int(rng.integers(1, 5))):
        edge = int(rng.choice(edges)) * int(rng.integers(1, max(2, min(N // int(max(edges)), 8))))
        length = int(rng.choice([140, 256, 257, 300, 384, 385, 450]))
        start = max(0, min(N - length, edge - int(rng.integers(0, length + 1))))
        runs.append((start, length))
        if rng.random() < 0.6:
            weights[start:start + length] = 0.0
    hot_worker = int(rng.integers(0, W))

    def grads(t):
        g = _randn((W, N), 8000 + 50 * seed + t, 1e-3)
        for start, length in runs:
            if (start + t) % 2:
                g[hot_worker, start:start + length] *= 300.0
        return g

    run_parity(sizes, W, ratio, 1e-8, seed=seed, steps=4, weights=weights, grads_fn=grads,
               options={"overlap": int(rng.integers(0, 2)), "speculate": 1}, state_every=int(rng.choice([1, 2])),
               residual_every=int(rng.choice([1, 1000])))
