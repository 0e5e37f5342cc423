"""Seeded synthetic inputs for the frame decoder: weight manifests, weights and latents.

This module serves both the CPU oracle's tests and the CUDA library's tests and benchmark.  It
holds no decoder arithmetic: it only names the parameter tensors of the two decoder layouts,
draws them (and the latents) from a counter-based generator, and rounds them to the storage
type of the configuration.  Neither the oracle nor the CUDA library is imported here.

The paper measures on gameplay latents of trained models (Section V, experimental setup); the
datasets and weights are not available, so these draws stand in for them: same shapes, same
layer widths, random-initialised parameters.  Decoder cost does not depend on the values.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

ARCH_TINY = "tiny"
ARCH_SDVAE = "sdvae"


@dataclass(frozen=True)
class Workload:
    """One benchmark/parity configuration (index = position in the configuration list, 1-based)."""

    index: int
    name: str
    arch: str            # ARCH_TINY | ARCH_SDVAE
    dtype: str           # "f32" | "bf16": storage type of weights, latents and frames
    batch: int
    latent_h: int
    latent_w: int
    groups: int
    eps: float
    weight_seed: int
    latent_seed: int
    latent_recipe: str   # "normal" | "normal_scaled" | "ar1"
    latent_channels: int = 4
    out_channels: int = 3

    @property
    def out_h(self) -> int:
        return 8 * self.latent_h

    @property
    def out_w(self) -> int:
        return 8 * self.latent_w


WORKLOADS = {
    1: Workload(1, "tiny-f32-64x64", ARCH_TINY, "f32", 1, 8, 8, 8, 1e-6, 1001, 2001, "normal"),
    2: Workload(2, "sdvae-bf16-64x64", ARCH_SDVAE, "bf16", 1, 8, 8, 32, 1e-6, 1002, 2002, "normal"),
    3: Workload(3, "sdvae-bf16-720x480", ARCH_SDVAE, "bf16", 1, 60, 90, 32, 1e-6, 1002, 2003, "normal_scaled"),
    4: Workload(4, "sdvae-bf16-720x480-stream8", ARCH_SDVAE, "bf16", 8, 60, 90, 32, 1e-6, 1002, 2004, "ar1"),
    5: Workload(5, "sdvae-bf16-1280x720-b2", ARCH_SDVAE, "bf16", 2, 90, 160, 32, 1e-6, 1002, 2005, "normal"),
    # beyond the benchmark's list: the paper's second workload shape, the 256x256 platformer frames (Section V,
    # experimental setup; Table III, first row), as a stream of four AR(1) latents of 32x32
    6: Workload(6, "sdvae-bf16-256x256-stream4", ARCH_SDVAE, "bf16", 4, 32, 32, 32, 1e-6, 1002, 2006, "ar1"),
}

SDVAE_LEVEL_CHANNELS = (512, 512, 256, 128)
SDVAE_BLOCKS_PER_LEVEL = 3
TINY_STAGE_CHANNELS = ((64, 64), (64, 32), (32, 32))   # (in, out) of each stage's post-upsample conv


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even) and return them as fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16) << 16
    out = (r & 0xFFFFFFFF).astype(np.uint32).view(np.float32).reshape(a.shape)
    return np.where(np.isfinite(a), out, a)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """The uint16 bit patterns of fp32 values that are already bf16-representable."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """fp32 values of uint16 bf16 bit patterns."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).reshape(b.shape)


def _res_entries(prefix: str, cin: int, cout: int):
    e = [
        (f"{prefix}.norm1.weight", (cin,), "gn_gamma"),
        (f"{prefix}.norm1.bias", (cin,), "gn_beta"),
        (f"{prefix}.conv1.weight", (cout, cin, 3, 3), "weight"),
        (f"{prefix}.conv1.bias", (cout,), "bias"),
        (f"{prefix}.norm2.weight", (cout,), "gn_gamma"),
        (f"{prefix}.norm2.bias", (cout,), "gn_beta"),
        (f"{prefix}.conv2.weight", (cout, cout, 3, 3), "weight"),
        (f"{prefix}.conv2.bias", (cout,), "bias"),
    ]
    if cin != cout:
        e += [
            (f"{prefix}.shortcut.weight", (cout, cin, 1, 1), "weight"),
            (f"{prefix}.shortcut.bias", (cout,), "bias"),
        ]
    return e


def manifest(arch: str, latent_channels: int = 4, out_channels: int = 3):
    """Ordered list of (name, shape, kind) of every parameter tensor of a decoder layout.

    Convolution weights are [Cout, Cin, kh, kw]; the attention projections are [out, in];
    GroupNorm scale/shift and all biases are [C].  The order is also the random draw order.
    """
    m = []
    if arch == ARCH_SDVAE:
        c0 = SDVAE_LEVEL_CHANNELS[0]
        m += [("conv_in.weight", (c0, latent_channels, 3, 3), "weight"), ("conv_in.bias", (c0,), "bias")]
        m += _res_entries("mid.res0", c0, c0)
        m += [("mid.attn.norm.weight", (c0,), "gn_gamma"), ("mid.attn.norm.bias", (c0,), "gn_beta")]
        for p in ("q", "k", "v", "o"):
            m += [(f"mid.attn.{p}.weight", (c0, c0), "weight"), (f"mid.attn.{p}.bias", (c0,), "bias")]
        m += _res_entries("mid.res1", c0, c0)
        prev = c0
        for i, c in enumerate(SDVAE_LEVEL_CHANNELS):
            for j in range(SDVAE_BLOCKS_PER_LEVEL):
                m += _res_entries(f"up{i}.res{j}", prev if j == 0 else c, c)
            prev = c
            if i < len(SDVAE_LEVEL_CHANNELS) - 1:
                m += [(f"up{i}.upconv.weight", (c, c, 3, 3), "weight"), (f"up{i}.upconv.bias", (c,), "bias")]
        m += [("norm_out.weight", (prev,), "gn_gamma"), ("norm_out.bias", (prev,), "gn_beta")]
        m += [("conv_out.weight", (out_channels, prev, 3, 3), "weight"), ("conv_out.bias", (out_channels,), "bias")]
    elif arch == ARCH_TINY:
        c0 = TINY_STAGE_CHANNELS[0][0]
        m += [("conv_in.weight", (c0, latent_channels, 3, 3), "weight"), ("conv_in.bias", (c0,), "bias")]
        m += _res_entries("mid.res0", c0, c0)
        prev = c0
        for i, (cin, cout) in enumerate(TINY_STAGE_CHANNELS):
            assert cin == prev
            m += [(f"up{i}.upconv.weight", (cout, cin, 3, 3), "weight"), (f"up{i}.upconv.bias", (cout,), "bias")]
            m += _res_entries(f"up{i}.res0", cout, cout)
            prev = cout
        m += [("norm_out.weight", (prev,), "gn_gamma"), ("norm_out.bias", (prev,), "gn_beta")]
        m += [("conv_out.weight", (out_channels, prev, 3, 3), "weight"), ("conv_out.bias", (out_channels,), "bias")]
    else:
        raise ValueError(f"unknown arch {arch!r}")
    return m


def make_weights(arch: str, seed: int, dtype: str, gain: float = 1.0, latent_channels: int = 4,
                 out_channels: int = 3) -> dict:
    """Draw every parameter tensor, in manifest order, from Philox(key=seed); fp32 arrays.

    Weights ~ U(-b, b), b = gain*sqrt(3/fan_in), fan_in = Cin*kh*kw (Kaiming-uniform, gain 1);
    biases ~ U(-0.01, 0.01); GroupNorm scale = 1 + U(-0.1, 0.1), shift ~ U(-0.01, 0.01).
    With dtype "bf16" every value is rounded once to bf16 and returned as the fp32 number it
    became, so both consumers see exactly the same numbers.
    """
    rng = np.random.Generator(np.random.Philox(key=seed))
    out = {}
    for name, shape, kind in manifest(arch, latent_channels, out_channels):
        if kind == "weight":
            fan_in = int(np.prod(shape[1:]))
            b = gain * math.sqrt(3.0 / fan_in)
            a = rng.uniform(-b, b, size=shape)
        elif kind == "bias":
            a = rng.uniform(-0.01, 0.01, size=shape)
        elif kind == "gn_gamma":
            a = 1.0 + rng.uniform(-0.1, 0.1, size=shape)
        elif kind == "gn_beta":
            a = rng.uniform(-0.01, 0.01, size=shape)
        else:
            raise AssertionError(kind)
        a = a.astype(np.float32)
        out[name] = round_to_bf16(a) if dtype == "bf16" else a
    return out


def make_latents(recipe: str, seed: int, batch: int, channels: int, h: int, w: int, dtype: str) -> np.ndarray:
    """Latents [batch, channels, h, w] (fp32 array, rounded to the storage dtype).

    "normal": N(0,1).  "normal_scaled": N(0,1)/0.18215 (the caller-side latent scaling of the
    headline workload).  "ar1": frames form a sequence z_0 = e_0, z_t = 0.95 z_{t-1} +
    sqrt(1-0.95^2) e_t, mimicking the temporally redundant latents that the paper's latent
    extrapolation (Algorithm 2) exploits.
    """
    rng = np.random.Generator(np.random.Philox(key=seed))
    e = rng.standard_normal(size=(batch, channels, h, w))
    if recipe == "normal":
        z = e
    elif recipe == "normal_scaled":
        z = e / 0.18215
    elif recipe == "ar1":
        rho = 0.95
        z = np.empty_like(e)
        z[0] = e[0]
        for t in range(1, batch):
            z[t] = rho * z[t - 1] + math.sqrt(1.0 - rho * rho) * e[t]
    else:
        raise ValueError(recipe)
    z = z.astype(np.float32)
    return round_to_bf16(z) if dtype == "bf16" else z


def workload_weights(wl: Workload) -> dict:
    return make_weights(wl.arch, wl.weight_seed, wl.dtype, 1.0, wl.latent_channels, wl.out_channels)


def workload_latents(wl: Workload, batch: int | None = None, h: int | None = None, w: int | None = None) -> np.ndarray:
    return make_latents(wl.latent_recipe, wl.latent_seed, batch or wl.batch, wl.latent_channels,
                        h or wl.latent_h, w or wl.latent_w, wl.dtype)
