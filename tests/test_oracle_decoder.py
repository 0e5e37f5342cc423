"""Pins for the oracle's block and decoder composition (layer order, widths, skip paths,
upsampling, token order).  The layer list comes from the workload definition; the checks are
invariants of that composition plus an independent re-composition from torch CPU library ops
written here, in the test.  No GPU, no product code."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import ref
from paper_2602_00608_b200 import synth


def torch_resblock(x, w, p, G, eps):
    h = F.silu(F.group_norm(x, G, w[f"{p}.norm1.weight"], w[f"{p}.norm1.bias"], eps))
    h = F.conv2d(h, w[f"{p}.conv1.weight"], w[f"{p}.conv1.bias"], padding=1)
    h = F.silu(F.group_norm(h, G, w[f"{p}.norm2.weight"], w[f"{p}.norm2.bias"], eps))
    h = F.conv2d(h, w[f"{p}.conv2.weight"], w[f"{p}.conv2.bias"], padding=1)
    if f"{p}.shortcut.weight" in w:
        x = F.conv2d(x, w[f"{p}.shortcut.weight"], w[f"{p}.shortcut.bias"])
    return x + h


def torch_attn(x, w, p, G, eps):
    n, c, hh, ww = x.shape
    g = F.group_norm(x, G, w[f"{p}.norm.weight"], w[f"{p}.norm.bias"], eps)
    t = g.flatten(2).transpose(1, 2)                                   # [N,T,C], token = i*W + j
    q = t @ w[f"{p}.q.weight"].t() + w[f"{p}.q.bias"]
    k = t @ w[f"{p}.k.weight"].t() + w[f"{p}.k.bias"]
    v = t @ w[f"{p}.v.weight"].t() + w[f"{p}.v.bias"]
    a = torch.softmax(q @ k.transpose(1, 2) / math.sqrt(c), dim=-1) @ v
    o = a @ w[f"{p}.o.weight"].t() + w[f"{p}.o.bias"]
    return x + o.transpose(1, 2).reshape(n, c, hh, ww)


def torch_decode(arch, wnp, z, G, eps):
    w = {k: torch.from_numpy(v).double() for k, v in wnp.items()}
    x = F.conv2d(torch.from_numpy(z).double(), w["conv_in.weight"], w["conv_in.bias"], padding=1)
    up = lambda t: F.interpolate(t, scale_factor=2, mode="nearest")
    if arch == "sdvae":
        x = torch_resblock(x, w, "mid.res0", G, eps)
        x = torch_attn(x, w, "mid.attn", G, eps)
        x = torch_resblock(x, w, "mid.res1", G, eps)
        for i in range(4):
            for j in range(3):
                x = torch_resblock(x, w, f"up{i}.res{j}", G, eps)
            if i < 3:
                x = F.conv2d(up(x), w[f"up{i}.upconv.weight"], w[f"up{i}.upconv.bias"], padding=1)
    else:
        x = torch_resblock(x, w, "mid.res0", G, eps)
        for i in range(3):
            x = F.conv2d(up(x), w[f"up{i}.upconv.weight"], w[f"up{i}.upconv.bias"], padding=1)
            x = torch_resblock(x, w, f"up{i}.res0", G, eps)
    x = F.silu(F.group_norm(x, G, w["norm_out.weight"], w["norm_out.bias"], eps))
    return F.conv2d(x, w["conv_out.weight"], w["conv_out.bias"], padding=1).numpy()


def rel_l2(a, b):
    a, b = a.astype(np.float64), b.astype(np.float64)
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


@pytest.fixture(scope="module")
def tiny():
    wl = synth.WORKLOADS[1]
    return wl, synth.workload_weights(wl), synth.workload_latents(wl)


@pytest.fixture(scope="module")
def sd_small():
    wl = synth.WORKLOADS[2]
    return wl, synth.workload_weights(wl), synth.workload_latents(wl, batch=2, h=4, w=6)


def test_tiny_decoder_matches_torch_recomposition(tiny):
    wl, w, z = tiny
    y = ref.decode(wl.arch, w, z, wl.groups, wl.eps)
    assert y.shape == (1, 3, 64, 64) and y.dtype == np.float32
    assert rel_l2(y, torch_decode(wl.arch, w, z, wl.groups, wl.eps)) < 2e-6


def test_sdvae_decoder_matches_torch_recomposition(sd_small):
    wl, w, z = sd_small
    y = ref.decode(wl.arch, w, z, wl.groups, wl.eps)
    assert y.shape == (2, 3, 32, 48)
    assert rel_l2(y, torch_decode(wl.arch, w, z, wl.groups, wl.eps)) < 2e-6


def test_resblock_with_width_change_uses_1x1_shortcut_on_raw_input():
    wl = synth.WORKLOADS[2]
    w = synth.workload_weights(wl)
    x = np.random.default_rng(3).standard_normal((1, 512, 3, 5)).astype(np.float32)
    y = ref.resblock(x, w, "up2.res0", 32, 1e-6)
    assert y.shape == (1, 256, 3, 5)
    tw = {k: torch.from_numpy(v).double() for k, v in w.items() if k.startswith("up2.res0")}
    assert rel_l2(y, torch_resblock(torch.from_numpy(x).double(), tw, "up2.res0", 32, 1e-6).numpy()) < 1e-6
    # zero the residual branch: what is left is exactly the 1x1 projection of the raw input
    w2 = dict(w)
    w2["up2.res0.conv2.weight"] = np.zeros_like(w["up2.res0.conv2.weight"])
    w2["up2.res0.conv2.bias"] = np.zeros_like(w["up2.res0.conv2.bias"])
    np.testing.assert_allclose(ref.resblock(x, w2, "up2.res0", 32, 1e-6),
                               ref.conv2d(x, w["up2.res0.shortcut.weight"], w["up2.res0.shortcut.bias"]), atol=1e-6)


def test_attention_block_zero_output_projection_is_identity(sd_small):
    wl, w, _ = sd_small
    x = np.random.default_rng(4).standard_normal((1, 512, 3, 4)).astype(np.float32)
    w2 = dict(w)
    w2["mid.attn.o.weight"] = np.zeros_like(w["mid.attn.o.weight"])
    bo = w["mid.attn.o.bias"]
    y = ref.attention_block(x, w2, "mid.attn", 32, 1e-6)
    np.testing.assert_allclose(y, x + bo[None, :, None, None], atol=1e-6)


def test_zero_conv_out_weights_leave_only_the_bias(tiny):
    wl, w, z = tiny
    w2 = dict(w)
    w2["conv_out.weight"] = np.zeros_like(w["conv_out.weight"])
    y = ref.decode(wl.arch, w2, z, wl.groups, wl.eps)
    np.testing.assert_array_equal(y, np.broadcast_to(w["conv_out.bias"][None, :, None, None], y.shape))


def _mirror_kx(w):
    return {k: (v[:, :, :, ::-1].copy() if v.ndim == 4 and v.shape[-1] == 3 else v) for k, v in w.items()}


@pytest.mark.parametrize("which", ["tiny", "sdvae"])
def test_flip_equivariance(which, tiny, sd_small):
    # Mirroring the latent left-right and every 3x3 kernel in kx mirrors the frame: catches an
    # indexing slip in padding, upsampling or the attention's token order.
    wl, w, z = tiny if which == "tiny" else sd_small
    y = ref.decode(wl.arch, w, z, wl.groups, wl.eps)
    yf = ref.decode(wl.arch, _mirror_kx(w), z[:, :, :, ::-1].copy(), wl.groups, wl.eps)
    assert rel_l2(yf[:, :, :, ::-1], y) < 5e-6


def test_batch_independence(sd_small):
    wl, w, z = sd_small
    y = ref.decode(wl.arch, w, z, wl.groups, wl.eps)
    y1 = ref.decode(wl.arch, w, z[1:2], wl.groups, wl.eps)
    np.testing.assert_array_equal(y[1:2], y1)


def test_trace_names_every_block(tiny):
    wl, w, z = tiny
    tr = {}
    ref.decode(wl.arch, w, z, wl.groups, wl.eps, trace=tr)
    assert tr["conv_in"].shape == (1, 64, 8, 8)
    assert tr["up1.upconv"].shape == (1, 32, 32, 32)       # widths 64 -> 64 -> 32 -> 32
    assert tr["up2.res0"].shape == (1, 32, 64, 64)
    assert tr["frames"].shape == (1, 3, 64, 64)


def test_full_shapes_follow_the_eightfold_upsampling():
    for idx, shape in ((3, (480, 720)), (4, (480, 720)), (5, (720, 1280)), (2, (64, 64)), (1, (64, 64))):
        wl = synth.WORKLOADS[idx]
        assert (wl.out_h, wl.out_w) == shape
