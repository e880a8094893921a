"""Shared helper of the GPU parity tests: runs the CUDA library and the CPU oracle on the
same seeded inputs and compares every output bit for bit."""
import numpy as np
import torch

import oracle
from paper_1901_01544_b200.binding import Pruner


def u32(a: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def assert_bits_equal(got: np.ndarray, want: np.ndarray, what: str):
    g, w = u32(got), u32(want)
    if not np.array_equal(g, w):
        bad = np.flatnonzero(g != w)
        i = int(bad[0])
        raise AssertionError(f"{what}: {bad.size} of {g.size} differ; first at {i}: got {got.flat[i]!r} "
                             f"(0x{int(g.flat[i]):08x}) want {want.flat[i]!r} (0x{int(w.flat[i]):08x})")


def compare_state(pr: Pruner, orc: "oracle.Oracle", update_gpu: torch.Tensor, update_cpu: np.ndarray, tag: str,
                  check_mask: bool = True, check_residual: bool = True, leader_list_only: bool = False):
    assert pr.sync_status() == 0, f"{tag}: device status {pr.sync_status()}"
    assert pr.leader == orc.leader, f"{tag}: leader {pr.leader} != {orc.leader}"
    assert_bits_equal(update_gpu.cpu().numpy(), update_cpu, f"{tag}: update")
    for w in range(pr.W):
        if leader_list_only and w != orc.leader:  # option leader_only_select: nobody else makes a list
            if check_residual:
                assert_bits_equal(pr.residual(w).cpu().numpy(), orc.residual(w), f"{tag}: worker {w} residual")
            continue
        idx, val = pr.selection(w)
        oi, ov = orc.selection(w)
        gi = idx.cpu().numpy().view(np.uint32)
        if not np.array_equal(gi, oi):
            bad = np.flatnonzero(gi != oi)
            raise AssertionError(f"{tag}: worker {w} list indices differ at {bad.size} of {gi.size} positions; "
                                 f"first at {int(bad[0])}: got {int(gi[bad[0]])} want {int(oi[bad[0]])}")
        assert_bits_equal(val.cpu().numpy(), ov, f"{tag}: worker {w} list values")
        if check_residual:
            assert_bits_equal(pr.residual(w).cpu().numpy(), orc.residual(w), f"{tag}: worker {w} residual")
    if check_mask:
        assert np.array_equal(pr.mask().cpu().numpy(), orc.mask()), f"{tag}: mask"
        assert np.array_equal(pr.mask_bits().cpu().numpy(), np.packbits(orc.mask(), bitorder="little")), f"{tag}: packed mask"


def run_parity(layer_sizes, W, ratio, eps, seed, steps, weights: torch.Tensor, grads_fn, options=None,
               leader_overrides=None, check_mask=True, threads=0, residual_every=1, momentum=None, state_every=1,
               weights_fn=None, n_leaders=1, per_layer_leaders=False, leader_list_only=False):
    """weights: CUDA tensor [N]; grads_fn(t) -> CUDA tensor [W, N].

    state_every: lists, mask, residuals and the device status are looked at only every that many steps
    and after the last one; in between only the update is compared, which asks the library for nothing,
    so whatever it leaves running past the end of a step keeps running into the next one.
    weights_fn(t) -> CUDA tensor [N]: if given, `weights` is overwritten in place with it right after
    step t - 1 was enqueued, as an optimizer would.

    residual_every: residuals are read back (and compared) only every that many steps and after the
    last one.  Reading them makes the library bring them up to date first, so runs that look only at
    the end exercise the path where the zeroing of sent residuals is left to the next step."""
    pr = Pruner(layer_sizes, W, ratio, eps, seed)
    orc = oracle.Oracle(layer_sizes, W, ratio, eps, seed, threads=threads)
    assert (pr.N, pr.K) == (orc.N, orc.K)
    assert pr.layout() == orc.layout()
    for k, v in (options or {}).items():
        pr.set_option(k, v)
    if momentum is not None:
        pr.set_momentum(momentum)
        orc.set_momentum(momentum)
    if n_leaders > 1:  # several chosen nodes: the index set is the union of their lists
        pr.set_option("n_leaders", n_leaders)
        orc.set_n_leaders(n_leaders)
    if per_layer_leaders:  # every layer draws its own chosen node
        pr.set_option("per_layer_leaders", 1)
        orc.set_per_layer_leaders()
    w_host = weights.cpu().numpy()
    update = torch.full((pr.N,), float("nan"), dtype=torch.float32, device="cuda")
    for t in range(steps):
        if leader_overrides is not None:
            pr.set_option("leader_override", leader_overrides[t])
            orc.set_leader_override(leader_overrides[t])
        g = grads_fn(t)
        if weights_fn is not None:
            weights.copy_(weights_fn(t))
            w_host = weights.cpu().numpy()
        pr.step(g, weights, update)
        upd_cpu = orc.step(np.ascontiguousarray(g.cpu().numpy()), w_host)
        if (t + 1) % state_every != 0 and t != steps - 1:
            assert pr.leader == orc.leader, f"step {t}: leader {pr.leader} != {orc.leader}"
            assert_bits_equal(update.cpu().numpy(), upd_cpu, f"step {t}: update")
            update.fill_(float("nan"))
            continue
        look = (t + 1) % residual_every == 0 or t == steps - 1
        compare_state(pr, orc, update, upd_cpu, f"step {t}", check_mask=check_mask, check_residual=look,
                      leader_list_only=leader_list_only)
        update.fill_(float("nan"))  # the next step must overwrite every element
    pr.close()
    orc.close()
