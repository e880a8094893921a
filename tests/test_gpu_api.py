"""GPU tests of the API contract: determinism, reset / checkpoint round trip, the host-buffer
entry point, option and misuse handling.  Nothing here faults, traps or hangs the device."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from paper_1901_01544_b200 import binding
from paper_1901_01544_b200.binding import Pruner
from parity import assert_bits_equal

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _inputs(W, N, seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    weights = torch.randn(N, generator=g, device=DEV) * 0.05
    grads = [torch.randn((W, N), generator=g, device=DEV) * 1e-3 for _ in range(3)]
    return weights, grads


def test_same_inputs_same_bytes():
    sizes, W = [70000, 512, 33000], 4
    N = sum(sizes)
    weights, grads = _inputs(W, N, 1)
    outs = []
    for rep in range(2):
        pr = Pruner(sizes, W, 32.0, 1e-8, 9)
        o = []
        for g in grads:
            o.append(pr.step(g, weights).clone())
            o += [pr.residual(w) for w in range(W)] + [pr.selection(w)[0] for w in range(W)]
        outs.append(o)
        pr.close()
    for a, b in zip(*outs):
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))


def test_reset_and_checkpoint_roundtrip():
    sizes, W = [50000, 100], 3
    N = sum(sizes)
    weights, grads = _inputs(W, N, 2)
    pr = Pruner(sizes, W, 16.0, 1e-8, 5)
    u0 = pr.step(grads[0], weights).clone()
    u1 = pr.step(grads[1], weights).clone()
    saved = [pr.residual(w) for w in range(W)]
    t_saved = pr.t
    u2 = pr.step(grads[2], weights).clone()
    pr.reset()
    assert pr.t == 0 and pr.leader == -1
    assert all(int(pr.residual(w).abs().max().item() == 0) for w in range(W))
    assert torch.equal(pr.step(grads[0], weights), u0) and torch.equal(pr.step(grads[1], weights), u1)
    # resume from the checkpoint in a fresh context
    pr2 = Pruner(sizes, W, 16.0, 1e-8, 5)
    for w in range(W):
        pr2.set_residual(w, saved[w])
    pr2.set_step(t_saved)
    assert torch.equal(pr2.step(grads[2], weights).view(torch.int32), u2.view(torch.int32))
    assert pr2.leader == binding.iwp_leader_at(5, t_saved, W)
    pr.close()
    pr2.close()


@pytest.mark.parametrize("overlap", [0, 1])
def test_host_buffer_entry_point_matches_oracle(overlap):
    # the host weights change between steps: with the overlapped schedule the other workers' selects of one
    # step may still run while the next call copies new weights into the staging buffer
    sizes, W = [40000, 300, 20000], 4
    N = sum(sizes)
    weights, grads = _inputs(W, N, 3)
    pr = Pruner(sizes, W, 64.0, 1e-8, 0)
    pr.set_option("overlap", overlap)
    orc = oracle.Oracle(sizes, W, 64.0, 1e-8, 0)
    uh = torch.empty(N).pin_memory()
    for t, g in enumerate(grads + grads):
        gh = g.cpu().pin_memory()
        wh = (weights * (1.0 + 0.25 * t)).cpu().pin_memory()
        pr.step_host(gh, wh, uh)
        want = orc.step(gh.numpy(), wh.numpy())
        assert_bits_equal(uh.numpy(), want, "update via host buffers")
    assert pr.sync_status() == 0
    for w in range(W):
        idx, val = pr.selection(w)
        oi, ov = orc.selection(w)
        assert np.array_equal(idx.cpu().numpy().view(np.uint32), oi)
        assert_bits_equal(val.cpu().numpy(), ov, f"worker {w} list values")
    pr.close()


@pytest.mark.parametrize("overlap", [0, 1])
def test_async_host_entry_point_matches_oracle(overlap):
    sizes, W = [40000, 300, 20000], 4
    N = sum(sizes)
    weights, grads = _inputs(W, N, 5)
    pr = Pruner(sizes, W, 64.0, 1e-8, 0)
    pr.set_option("overlap", overlap)
    orc = oracle.Oracle(sizes, W, 64.0, 1e-8, 0)
    steps = 7
    gh = [grads[t % len(grads)].cpu().pin_memory() for t in range(steps)]
    wh = [(weights * (1.0 + 0.25 * t)).cpu().pin_memory() for t in range(steps)]
    uh = [torch.full((N,), float("nan")).pin_memory() for _ in range(steps)]
    for t in range(steps):  # all in flight, two staging sets in turn
        pr.step_host_async(gh[t], wh[t], uh[t])
    pr.host_wait()
    for t in range(steps):
        want = orc.step(gh[t].numpy(), wh[t].numpy())
        assert_bits_equal(uh[t].numpy(), want, f"step {t}: update via the asynchronous host entry point")
    assert pr.sync_status() == 0 and pr.t == steps
    # the synchronous entry point afterwards, on the same context
    pr.step_host(gh[0], wh[0], uh[0])
    assert_bits_equal(uh[0].numpy(), orc.step(gh[0].numpy(), wh[0].numpy()), "synchronous call after asynchronous ones")
    pr.close()


def test_runs_on_a_side_stream():
    sizes, W = [60000], 2
    N = sum(sizes)
    weights, grads = _inputs(W, N, 4)
    ref = Pruner(sizes, W, 32.0, 1e-8, 0)
    want = ref.step(grads[0], weights).clone()
    ref.close()
    s = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        pr = Pruner(sizes, W, 32.0, 1e-8, 0)
        got = pr.step(grads[0], weights)
        assert pr.sync_status() == 0
    s.synchronize()
    assert torch.equal(got, want)
    pr.close()


def test_stream_switch_between_overlapped_steps():
    # steps alternate between two streams while the other workers' selects of the last step may still be
    # running on the library's own streams; every list is checked at the end of each pair of steps
    import oracle

    sizes, W, ratio = [80000, 300, 50000], 4, 16.0
    N = sum(sizes)
    weights, grads = _inputs(W, N, 8)
    pr = Pruner(sizes, W, ratio, 1e-8, 3)
    pr.set_option("overlap", 1)
    orc = oracle.Oracle(sizes, W, ratio, 1e-8, 3)
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    w_host = weights.cpu().numpy()
    for t in range(6):
        s = streams[t % 2]
        g = grads[t % len(grads)]
        with torch.cuda.stream(s):
            pr.use_current_stream()
            got = pr.step(g, weights)
        s.synchronize()
        want = orc.step(np.ascontiguousarray(g.cpu().numpy()), w_host)
        assert_bits_equal(got.cpu().numpy(), want, f"step {t}: update")
        if t % 2 == 1:
            with torch.cuda.stream(s):
                assert pr.sync_status() == 0
                for w in range(W):
                    idx, val = pr.selection(w)
                    oi, ov = orc.selection(w)
                    assert np.array_equal(idx.cpu().numpy().view(np.uint32), oi)
                    assert_bits_equal(val.cpu().numpy(), ov, f"step {t}: worker {w} list values")
    pr.close()
    orc.close()


def test_options_stats_and_misuse():
    pr = Pruner([5000, 20000], 2, 8.0, 1e-8, 0)
    L = binding.lib()
    h = pr._h
    E = binding.IWP_ERR_INVALID
    assert L.iwp_set_option(h, b"no_such_option", 1) == E
    assert L.iwp_set_option(h, b"leader_override", 2) == E and L.iwp_set_option(h, b"leader_override", -2) == E
    assert L.iwp_set_option(h, b"force_scalar", 7) == E
    assert L.iwp_set_option(h, b"leader_override", 1) == 0
    v = C.c_int64()
    assert L.iwp_get_stat(h, b"nope", C.byref(v)) == E
    assert L.iwp_get_residual(h, 2, 0) == E and L.iwp_get_residual(h, -1, 0) == E
    assert L.iwp_get_selection(h, 5, None, None) == E
    assert L.iwp_set_step(h, -1) == E
    assert L.iwp_step(h, None, None, None) == E
    assert pr.t == 0 and pr.stat("launches") == 0
    weights, grads = _inputs(2, 25000, 6)
    pr.step(grads[0], weights)
    assert pr.leader == 1 and pr.t == 1 and pr.stat("launches") > 0 and pr.stat("device_bytes") >= 2 * 25000 * 4
    assert pr.sync_status() == 0
    assert pr.layout() == ([0, 5000], [625, 2500])
    pr.close()
    pr.close()  # idempotent


def test_newer_options_join_and_wire_argument_checks():
    sizes, W = [70000, 300], 3
    N = sum(sizes)
    pr = Pruner(sizes, W, 32.0, 1e-8, 0)
    L = binding.lib()
    h = pr._h
    E = binding.IWP_ERR_INVALID
    for key, bad in ((b"pair_select", 2), (b"pair_select", -2), (b"leader_only_select", 2), (b"reserve_timed_steps", -1),
                     (b"overlap", 2)):
        assert L.iwp_set_option(h, key, bad) == E
    for key, ok in ((b"pair_select", -1), (b"pair_select", 1), (b"leader_only_select", 0), (b"reserve_timed_steps", 4)):
        assert L.iwp_set_option(h, key, ok) == 0
    assert L.iwp_join(None) == E and L.iwp_join(h) == 0
    weights, grads = _inputs(W, N, 12)
    pr.set_option("overlap", 1)
    upd = pr.step(grads[0], weights)
    pr.join()  # work enqueued now is behind every kernel of the step, the late selects included
    done = torch.cuda.Event()
    done.record()
    done.synchronize()
    assert pr.sync_status() == 0 and int(torch.count_nonzero(upd).item()) <= pr.K
    # wire formats: NULL pointers, negative sizes, a mask buffer that is not 4-byte aligned
    idx = pr.selection(pr.leader)[0]
    bits = torch.zeros(binding.iwp_wire_mask_bytes(N) + 4, dtype=torch.uint8, device=DEV)
    assert L.iwp_wire_pack(h, idx.data_ptr(), -1, bits.data_ptr()) == E
    assert L.iwp_wire_pack(h, None, 5, bits.data_ptr()) == E
    assert L.iwp_wire_pack(h, idx.data_ptr(), idx.numel(), bits.data_ptr() + 1) == E
    assert L.iwp_wire_unpack(h, bits.data_ptr() + 2, idx.data_ptr(), idx.numel(), None) == E
    assert L.iwp_wire_unpack(h, bits.data_ptr(), None, 5, None) == E
    assert L.iwp_wire_pack(h, idx.data_ptr(), idx.numel(), bits.data_ptr()) == 0
    n = C.c_int64(-1)
    out = torch.empty_like(idx)
    assert L.iwp_wire_unpack(h, bits.data_ptr(), out.data_ptr(), out.numel(), C.byref(n)) == 0
    assert n.value == idx.numel() and torch.equal(out, idx)  # the list is ascending already
    thr = Pruner(sizes, W, None, 1e-8, 0, thresholds=[1.0, 1.0])
    assert L.iwp_set_option(thr._h, b"leader_only_select", 1) == E  # ratio-mode contexts only
    thr.close()
    pr.close()


def test_single_read_path_is_taken_and_falls_back_when_it_must():
    sizes, W = [300000, 64, 40000], 4
    N = sum(sizes)
    weights, grads = _inputs(W, N, 8)
    pr = Pruner(sizes, W, 64.0, 1e-8, 0)
    orc = oracle.Oracle(sizes, W, 64.0, 1e-8, 0)
    assert pr.stat("spec_pairs") == 2 * W
    for g in grads:
        upd = pr.step(g, weights)
        want = orc.step(g.cpu().numpy(), weights.cpu().numpy())
        assert pr.stat("spec_failed") == 0  # continuous random values: every pair stays on the single-read path
        assert_bits_equal(upd.cpu().numpy(), want, "update")
    # all importances equal: every element reaches the guess, the slots overflow, the exact path takes over
    pr.reset()
    orc.reset()
    g = torch.full((W, N), 0.5, device=DEV)
    wt = torch.ones(N, device=DEV)
    upd = pr.step(g, wt)
    want = orc.step(g.cpu().numpy(), wt.cpu().numpy())
    assert pr.stat("spec_failed") == 2 * W and pr.sync_status() == 0
    assert_bits_equal(upd.cpu().numpy(), want, "update after fallback")
    pr.set_option("speculate", 0)
    assert pr.stat("spec_pairs") == 0
    pr.close()


def test_switching_speculation_off_mid_run_keeps_state_exact():
    sizes, W = [200000, 50], 3
    N = sum(sizes)
    weights, grads = _inputs(W, N, 12)
    pr = Pruner(sizes, W, 64.0, 1e-8, 2)
    orc = oracle.Oracle(sizes, W, 64.0, 1e-8, 2)
    for t, g in enumerate(grads + grads):
        if t == 2:
            pr.set_option("speculate", 0)  # pending lazy zeroing must be applied before the multi-pass path runs
        if t == 4:
            pr.set_option("speculate", 1)
        upd = pr.step(g, weights)
        want = orc.step(g.cpu().numpy(), weights.cpu().numpy())
        assert_bits_equal(upd.cpu().numpy(), want, f"step {t}: update")
    for w in range(W):
        assert_bits_equal(pr.residual(w).cpu().numpy(), orc.residual(w), f"worker {w} residual")
    assert pr.sync_status() == 0
    pr.close()
