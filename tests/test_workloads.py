"""The synthetic input recipes: sizes, determinism and the value structure the
benchmark configurations ask for.  CPU only, on scaled-down size lists."""
import math

import numpy as np
import torch

from paper_1901_01544_b200 import workloads as wl


def test_registry_sizes():
    c = {k: f() for k, f in wl.CONFIGS.items()}
    assert c["single_layer"].N == 1 << 20 and c["single_layer"].W == 4
    assert c["alexnet_w8"].N == 60965224 and len(c["alexnet_w8"].layer_sizes) == 16
    assert c["alexnet_w8"].layer_sizes[:4] == [34848, 96, 307200, 256]
    assert c["resnet50_w8"].N == 25557032 and len(c["resnet50_w8"].layer_sizes) == 161
    assert c["alexnet_w32"].W == 32 and c["alexnet_w32"].ratio == 256.0 and c["alexnet_w32"].steps == 20
    assert c["flat_1g_w4"].N == 1 << 30 and len(c["flat_1g_w4"].layer_sizes) == 96
    sizes = c["resnet50_w8"].layer_sizes
    assert sum(1 for n in sizes if n <= 4096) == 108 and max(sizes) == 2359296
    assert c["flat_1g_w4"].offsets()[1] % 4 != 0  # layer starts are deliberately not 16-byte aligned


def test_single_layer_values():
    c = wl.scaled(wl.single_layer(), [1 << 16], name="c1s")
    w = c.weights()
    assert int((w == 0).sum()) == round(0.01 * (1 << 16))
    assert abs(float(w[w != 0].std()) - 0.05) < 2e-3
    g0, g0b, g1 = c.grads(0), c.grads(0), c.grads(1)
    assert g0.shape == (4, 1 << 16) and torch.equal(g0, g0b) and not torch.equal(g0, g1)
    assert abs(float(g0.std()) - 1e-3) < 5e-5
    assert not torch.equal(g0[0], g0[1])  # independent per worker


def test_tensor_list_values():
    base = wl.alexnet_w8()
    small = [max(8, n // 256) for n in base.layer_sizes]
    c = wl.scaled(base, small, W=2)
    w = c.weights()
    off = c.offsets()
    for j, t in enumerate(c.tensors):
        seg = w[off[j]: off[j] + t.numel]
        if t.kind == "zeros":
            assert torch.all(seg == 0)
        elif t.numel > 1000:
            assert abs(float(seg.std()) / math.sqrt(2.0 / t.fan_in) - 1) < 0.1
    g = c.grads(0)
    j = 10  # w6: fan_in 9216
    seg = g[:, off[j]: off[j] + c.tensors[j].numel]
    assert abs(float(seg.std()) / (0.01 * math.sqrt(2.0 / 9216)) - 1) < 0.05

    r = wl.resnet50_w8()
    cr = wl.scaled(r, [max(4, n // 64) for n in r.layer_sizes], W=2)
    wr = cr.weights()
    o = cr.offsets()
    assert torch.all(wr[o[1]: o[1] + cr.tensors[1].numel] == 1)  # gamma
    assert torch.all(wr[o[2]: o[2] + cr.tensors[2].numel] == 0)  # beta
    gr = cr.grads(3)
    # Laplace(0, b): mean |x| = b, variance 2 b^2
    assert abs(float(gr.abs().mean()) / 1e-4 - 1) < 0.03
    assert abs(float(gr.var()) / 2e-8 - 1) < 0.08


def test_stress_scales_and_heavy_tail():
    base = wl.alexnet_w32()
    c = wl.scaled(base, [max(8, n // 512) for n in base.layer_sizes], W=3, steps=20)
    s0, s1 = wl._c4_scales(c, 0), wl._c4_scales(c, 1)
    assert len(s0) == 8 and all(1e-5 <= s <= 1e-2 for s in s0 + s1) and s0 != s1
    g = c.grads(0)
    off = c.offsets()
    seg = g[:, off[10]: off[10] + c.tensors[10].numel]
    assert abs(float(seg.std()) / s0[5] - 1) < 0.05
    f = wl.scaled(wl.flat_1g_w4(), wl.split_equal(1 << 18, 6), name="c5s")
    gf = f.grads(0)
    x = (gf / 1e-4).double().flatten().numpy()
    # Student-t(3): median |x| = 0.7649, and a far heavier tail than a normal
    assert abs(np.median(np.abs(x)) - 0.7649) < 0.02
    assert (np.abs(x) > 6).mean() > 5e-3
    assert abs(float(f.weights().std()) - 0.02) < 1e-3
