"""The seeded input generators: manifest structure, determinism, distributions, bf16 rounding."""
import math

import numpy as np

from paper_2602_00608_b200 import synth


def test_manifest_counts_and_order():
    m = synth.manifest("sdvae")
    names = [n for n, _, _ in m]
    assert names[0] == "conv_in.weight" and names[-1] == "conv_out.bias"
    assert len(set(names)) == len(names)
    convs3 = [n for n, s, k in m if k == "weight" and len(s) == 4 and s[-1] == 3]
    assert len(convs3) == 33                      # conv_in + 28 block convs + 3 upconvs + conv_out
    assert sum(1 for n in names if n.endswith("shortcut.weight")) == 2
    assert sum(1 for n, s, k in m if k == "gn_gamma") == 30
    shapes = dict((n, s) for n, s, _ in m)
    assert shapes["up2.res0.conv1.weight"] == (256, 512, 3, 3)
    assert shapes["up3.res0.shortcut.weight"] == (128, 256, 1, 1)
    assert shapes["mid.attn.q.weight"] == (512, 512)
    assert shapes["conv_out.weight"] == (3, 128, 3, 3)
    t = dict((n, s) for n, s, _ in synth.manifest("tiny"))
    assert t["up1.upconv.weight"] == (32, 64, 3, 3) and t["conv_out.weight"] == (3, 32, 3, 3)
    assert not any("shortcut" in n or "attn" in n for n in t)


def test_weights_are_seeded_bounded_and_bf16_exact():
    a = synth.make_weights("tiny", 5, "f32")
    b = synth.make_weights("tiny", 5, "f32")
    c = synth.make_weights("tiny", 6, "f32")
    assert all(np.array_equal(a[k], b[k]) for k in a)
    assert not np.array_equal(a["conv_in.weight"], c["conv_in.weight"])
    w = a["mid.res0.conv1.weight"]
    bound = math.sqrt(3.0 / (64 * 9))
    assert np.abs(w).max() <= bound and np.abs(w).max() > 0.98 * bound
    assert abs(w.std() - bound / math.sqrt(3)) < 0.02 * bound      # uniform: std = b/sqrt(3)
    assert np.abs(a["conv_in.bias"]).max() <= 0.01
    g = a["norm_out.weight"]
    assert 0.9 <= g.min() and g.max() <= 1.1
    h = synth.make_weights("tiny", 5, "bf16")
    for k, v in h.items():
        assert np.all((v.view(np.uint32) & 0xFFFF) == 0), k
        assert np.abs(v - a[k]).max() <= np.abs(a[k]).max() * 2 ** -8


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -1.0 - 2 ** -8, 3.0e38, 0.0], np.float32)
    r = synth.round_to_bf16(x)
    # 1+2^-8 is a tie between 1 and 1+2^-7 -> even mantissa (1); 1+3*2^-8 ties to 1+2^-6
    assert r.tolist()[:5] == [1.0, 1.0, 1.0 + 2 ** -7, 1.0 + 2 ** -6, -1.0]
    assert np.array_equal(synth.from_bf16_bits(synth.to_bf16_bits(r)), r)
    y = np.random.default_rng(0).standard_normal(1000).astype(np.float32)
    import torch
    assert np.array_equal(synth.round_to_bf16(y), torch.from_numpy(y).bfloat16().float().numpy())


def test_latent_recipes():
    z = synth.make_latents("normal", 1, 2, 4, 60, 90, "f32")
    assert z.shape == (2, 4, 60, 90) and abs(z.std() - 1) < 0.02 and abs(z.mean()) < 0.02
    zs = synth.make_latents("normal_scaled", 1, 2, 4, 60, 90, "f32")
    np.testing.assert_allclose(zs, z / 0.18215, rtol=1e-6)
    a = synth.make_latents("ar1", 3, 8, 4, 60, 90, "f32").reshape(8, -1).astype(np.float64)
    assert abs(a.std() - 1) < 0.02                                       # stationary unit variance
    r = [np.corrcoef(a[t], a[t + 1])[0, 1] for t in range(7)]
    assert all(abs(x - 0.95) < 0.01 for x in r)                          # lag-1 correlation 0.95
    assert abs(np.corrcoef(a[0], a[2])[0, 1] - 0.95 ** 2) < 0.015
    wl = synth.WORKLOADS[4]
    assert synth.workload_latents(wl).shape == (8, 4, 60, 90)
