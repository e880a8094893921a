"""The allocation-free entry point iwp_select_static (for callers that may not allocate device
memory while they run) against the CPU oracle's plain top-k definition and against the
context-based path: same layer, same residual, the list must be identical bit for bit.  Two calls in a row share the library's fixed scratch array, so the
second call also proves that the first left nothing behind that matters.  Collected last on
purpose: a run that stops at the first failure has then already run every other test."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from paper_1901_01544_b200 import binding
from paper_1901_01544_b200.binding import Pruner

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _reference_list(residual, weights, ratio, eps):
    """The list the existing entry points build: a fresh one-worker context whose first step
    accumulates `residual` into zeroed residuals."""
    n = residual.numel()
    pr = Pruner([n], 1, ratio, eps, 0)
    pr.step(residual.view(1, n).contiguous(), weights)
    assert pr.sync_status() == 0
    idx, val = pr.selection(0)
    k = pr.K
    pr.close()
    return k, idx.clone(), val.clone()


def _static_list(residual, weights, ratio, eps):
    n = residual.numel()
    k_max = binding.iwp_keep_count(n, ratio)
    idx = torch.full((k_max,), -1, dtype=torch.int32, device=DEV)
    val = torch.full((k_max,), float("nan"), dtype=torch.float32, device=DEV)
    stream = torch.cuda.current_stream().cuda_stream
    k = binding.iwp_select_static(residual.data_ptr(), weights.data_ptr(), n, ratio, eps, idx.data_ptr(),
                                  val.data_ptr(), stream)
    assert binding.iwp_select_static_status(stream) == 0, "a count check of the select failed on the device"
    torch.cuda.synchronize()
    return k, idx, val


def _assert_matches_oracle(residual, weights, k, eps, idx, val):
    """The plain definition: the k best under (importance descending, index ascending), listed by index."""
    r_host = residual.cpu().numpy()
    want = oracle.select(r_host, weights.cpu().numpy(), k, eps)
    got = idx.cpu().numpy().view(np.uint32)
    assert np.array_equal(got, want), "indices differ from the oracle's top-k"
    assert np.array_equal(val.cpu().numpy().view(np.uint32), r_host[want].view(np.uint32)), "values differ bit-wise"


def test_static_select_matches_context_path_twice_in_a_row():
    g = torch.Generator(device=DEV)
    g.manual_seed(123)
    cases = [(700001, 64.0), (300000, 58.8)]  # the second call is smaller: stale chunk tables must not leak
    for n, ratio in cases:
        weights = torch.randn(n, generator=g, device=DEV) * 0.05
        weights[torch.rand(n, generator=g, device=DEV) < 0.02] = 0.0
        residual = torch.randn(n, generator=g, device=DEV) * 1e-3
        residual[::7] = residual[3]  # repeated values: ties at and around the threshold
        k_ref, idx_ref, val_ref = _reference_list(residual, weights, ratio, 1e-8)
        k, idx, val = _static_list(residual, weights, ratio, 1e-8)
        assert k == k_ref == binding.iwp_keep_count(n, ratio) == oracle.keep_count(n, ratio)
        _assert_matches_oracle(residual, weights, k, 1e-8, idx, val)
        assert torch.equal(idx, idx_ref), "indices differ from the context-based path"
        assert torch.equal(val.view(torch.int32), val_ref.view(torch.int32)), "values differ bit-wise"
        assert torch.all(idx[1:] > idx[:-1])


def test_static_select_unaligned_pointers_and_small_layer():
    g = torch.Generator(device=DEV)
    g.manual_seed(5)
    n = 40001
    wbuf = torch.randn(n + 1, generator=g, device=DEV)
    rbuf = torch.randn(n + 1, generator=g, device=DEV)
    k_ref, idx_ref, val_ref = _reference_list(rbuf[1:].clone(), wbuf[1:].clone(), 16.0, 1e-8)
    k, idx, val = _static_list(rbuf[1:], wbuf[1:], 16.0, 1e-8)  # 4-byte aligned only: scalar access path
    assert k == k_ref and torch.equal(idx, idx_ref) and torch.equal(val.view(torch.int32), val_ref.view(torch.int32))
    _assert_matches_oracle(rbuf[1:], wbuf[1:], k, 1e-8, idx, val)
    # a layer small enough for the context path's one-CTA kernel still gives the same list
    r2, w2 = rbuf[:1000].clone(), wbuf[:1000].clone()
    k_ref, idx_ref, val_ref = _reference_list(r2, w2, 8.0, 1e-8)
    k, idx, val = _static_list(r2, w2, 8.0, 1e-8)
    assert k == k_ref == 125 and torch.equal(idx, idx_ref) and torch.equal(val.view(torch.int32), val_ref.view(torch.int32))
    _assert_matches_oracle(r2, w2, k, 1e-8, idx, val)


def test_static_select_rejects_what_it_cannot_hold():
    L = binding.lib()
    x = torch.zeros(16, device=DEV)
    out_i = torch.zeros(16, dtype=torch.int32, device=DEV)
    E = binding.IWP_ERR_INVALID
    args = lambda n, ratio=2.0, eps=1e-8: (x.data_ptr(), x.data_ptr(), n, ratio, eps, out_i.data_ptr(), x.data_ptr(),
                                            None, None)
    assert L.iwp_select_static(*args((1 << 24) + 1)) == E  # beyond the fixed scratch's maximum
    assert L.iwp_select_static(*args(0)) == E
    assert L.iwp_select_static(*args(16, ratio=0.5)) == E
    assert L.iwp_select_static(*args(16, eps=0.0)) == E
    assert L.iwp_select_static(None, x.data_ptr(), 16, 2.0, 1e-8, out_i.data_ptr(), x.data_ptr(), None, None) == E
    assert "invalid" in binding.iwp_strerror(E)
