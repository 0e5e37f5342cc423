"""End-to-end parity of vd_decode against the oracle on the benchmark configurations, through
the C ABI, on the same seeded inputs."""
import os

import numpy as np
import pytest

from tests.util import BF16_MAX_ABS, BF16_REL_L2, F32_REL_L2, max_abs, rel_l2

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


@pytest.fixture(scope="module")
def env():
    import torch
    from oracle import ref
    from paper_2602_00608_b200 import binding, synth
    return torch, ref, binding, synth


def _decode(env, wl, z, flags=0, max_batch=None):
    torch, ref, vd, synth = env
    wts = synth.workload_weights(wl)
    dec = vd.Decoder(wl.arch, wl.dtype, z.shape[2], z.shape[3], max_batch or z.shape[0], wl.groups, wl.eps, wts, flags)
    zt = torch.from_numpy(z).to("cuda:0", dec.dtype)
    got = dec.decode(zt)
    torch.cuda.synchronize()
    dec.check_status()
    return dec, got, wts


def test_config1_tiny_fp32(env):
    torch, ref, vd, synth = env
    wl = synth.WORKLOADS[1]
    z = synth.workload_latents(wl)
    dec, got, wts = _decode(env, wl, z)
    want = ref.decode(wl.arch, wts, z, wl.groups, wl.eps)
    assert got.shape == (1, 3, 64, 64) and got.dtype == torch.float32
    assert rel_l2(got.cpu().numpy(), want) <= F32_REL_L2


def test_tiny_fp32_odd_size_batch3(env):
    torch, ref, vd, synth = env
    wl = synth.WORKLOADS[1]
    z = synth.workload_latents(wl, batch=3, h=5, w=7)
    dec, got, wts = _decode(env, wl, z)
    want = ref.decode(wl.arch, wts, z, wl.groups, wl.eps)
    assert rel_l2(got.cpu().numpy(), want) <= F32_REL_L2


@pytest.mark.parametrize("flags", [0, 1])
def test_config2_sdvae_bf16_64x64(env, flags):
    torch, ref, vd, synth = env
    wl = synth.WORKLOADS[2]
    z = synth.workload_latents(wl)
    dec, got, wts = _decode(env, wl, z, flags)
    want = ref.decode(wl.arch, wts, z, wl.groups, wl.eps)
    g = got.float().cpu().numpy()
    assert rel_l2(g, want) <= BF16_REL_L2 and max_abs(g, want) <= BF16_MAX_ABS


def test_sdvae_fp32_path_matches_oracle(env):
    # the fp32 FFMA path on the full-width layout (attention and shortcuts included)
    torch, ref, vd, synth = env
    import dataclasses
    wl = dataclasses.replace(synth.WORKLOADS[2], dtype="f32")
    z = synth.workload_latents(wl, batch=2, h=5, w=6)
    dec, got, wts = _decode(env, wl, z)
    want = ref.decode(wl.arch, wts, z, wl.groups, wl.eps)
    assert rel_l2(got.cpu().numpy(), want) <= F32_REL_L2


@pytest.mark.parametrize("flags", [0, 1, 0x10])
def test_sdvae_bf16_ragged_tiles_batch2(env, flags):
    # 20x28 latents: every level's width/height leaves a ragged last tile; two frames
    # (flags: default, FFMA kernels, GroupNorm statistics taken in the convolutions' epilogues)
    torch, ref, vd, synth = env
    wl = synth.WORKLOADS[3]
    z = synth.workload_latents(wl, batch=2, h=20, w=28)
    dec, got, wts = _decode(env, wl, z, flags)
    want = ref.decode(wl.arch, wts, z, wl.groups, wl.eps)
    g = got.float().cpu().numpy()
    assert rel_l2(g, want) <= BF16_REL_L2 and max_abs(g, want) <= BF16_MAX_ABS
    # batch independence and run-to-run determinism
    again = dec.decode(torch.from_numpy(z).to("cuda:0", dec.dtype))
    one = dec.decode(torch.from_numpy(z[1:2]).to("cuda:0", dec.dtype))
    torch.cuda.synchronize()
    assert torch.equal(again, got)
    assert torch.equal(one[0], got[1])


@pytest.mark.parametrize("idx", [3, 4, 5])
def test_full_size_configs_against_sampled_oracle_frames(env, idx):
    """Full-size workloads in the benchmark's launch configuration; the oracle frames were computed
    ahead of time by tests/golden/make_golden.py (oracle only) and sampled at fixed pixels."""
    torch, ref, vd, synth = env
    path = os.path.join(GOLDEN, f"frames_cfg{idx}.npz")
    if not os.path.exists(path):
        pytest.skip(f"{path} not generated")
    gold = np.load(path)
    wl = synth.WORKLOADS[idx]
    z = synth.workload_latents(wl)
    dec, got, wts = _decode(env, wl, z)
    pos = gold["positions"]
    g = got.float().cpu().numpy()
    assert g.shape == (wl.batch, 3, wl.out_h, wl.out_w)
    sampled = g[:, :, pos[:, 0], pos[:, 1]]
    for b in range(wl.batch):
        r, m = rel_l2(sampled[b], gold["values"][b]), max_abs(sampled[b], gold["values"][b])
        assert r <= BF16_REL_L2 and m <= BF16_MAX_ABS, (b, r, m)
        # whole-frame statistics as a property check on the pixels that were not sampled
        std = float(g[b].astype(np.float64).std())
        assert abs(std - gold["stats"][b, 1]) <= 0.01 * gold["stats"][b, 1]
    dec.check_status()


# (measured on one B200, whole frame: rel-L2 2.7e-3 / 5.4e-3 / 5.4e-3, max-abs 1.2e-2 / 2.4e-2 / 2.6e-2 for workloads 3 / 4 / 5)
@pytest.mark.parametrize("idx", [3, 4, 5])
def test_full_size_configs_whole_frame_against_the_oracle(env, idx):
    """The last frame of each full-size workload, complete: every output pixel against the oracle
    frame that tests/golden/make_golden.py --full stored (oracle only), at the bar of the bf16
    path; and the tensor-core path against the FFMA path of the same library on every pixel of
    every frame (the FFMA path is itself checked against the oracle)."""
    torch, ref, vd, synth = env
    path = os.path.join(GOLDEN, f"frame_cfg{idx}_full.npz")
    gold = np.load(path)
    wl = synth.WORKLOADS[idx]
    z = synth.workload_latents(wl)
    dec, got, wts = _decode(env, wl, z)
    b = int(gold["index"])
    assert b == wl.batch - 1
    g = got[b].float().cpu().numpy()
    want = gold["frame"]
    assert g.shape == want.shape == (3, wl.out_h, wl.out_w)
    r, m = rel_l2(g, want), max_abs(g, want)
    print(f"whole-frame parity {wl.name} frame {b}: rel-L2 {r:.3e} max-abs {m:.3e}")
    assert r <= BF16_REL_L2 and m <= BF16_MAX_ABS, (r, m)
    dec.close()
    del dec
    torch.cuda.empty_cache()
    # every pixel of every frame, tcgen05 kernels against the FFMA kernels (same rounding points)
    zs = z[-2:] if wl.batch > 2 else z                      # the FFMA path is slow: two frames are enough
    dec2, got2, _ = _decode(env, wl, zs, flags=vd.VD_FLAG_FORCE_SIMT)
    a = got[-zs.shape[0]:].float()
    d = (a - got2.float())
    r2 = float(d.norm() / got2.float().norm())
    print(f"tcgen05 vs FFMA {wl.name}: rel-L2 {r2:.3e} max-abs {float(d.abs().max()):.3e}")
    # two independently rounded bf16 runs differ by about sqrt(2) x the error of one against fp32 math
    assert r2 <= BF16_REL_L2 and float(d.abs().max()) <= 2 * BF16_MAX_ABS


@pytest.mark.parametrize("flags_name", ["VD_FLAG_FUSED_STATS", "VD_FLAG_UPSAMPLE_9TAP"])
def test_full_size_720x480_whole_frame_with_the_optional_forms(env, flags_name):
    """The selectable forms of the same decoder at full size, every pixel against the stored oracle frame: GroupNorm
    statistics taken in the convolutions' epilogues, and upsampling as nine taps on the 2x grid."""
    torch, ref, vd, synth = env
    gold = np.load(os.path.join(GOLDEN, "frame_cfg3_full.npz"))
    wl = synth.WORKLOADS[3]
    z = synth.workload_latents(wl)
    dec, got, _ = _decode(env, wl, z, flags=getattr(vd, flags_name))
    g = got[int(gold["index"])].float().cpu().numpy()
    r, m = rel_l2(g, gold["frame"]), max_abs(g, gold["frame"])
    print(f"whole-frame parity {wl.name} with {flags_name}: rel-L2 {r:.3e} max-abs {m:.3e}")
    assert r <= BF16_REL_L2 and m <= BF16_MAX_ABS, (r, m)
    dec.check_status()


@pytest.mark.parametrize("h,w,b", [(1, 1, 1), (2, 3, 2), (5, 4, 3), (33, 47, 2)])
def test_sdvae_bf16_degenerate_and_odd_sizes(env, h, w, b):
    """Latents smaller than one tile (every tile of every level ragged, most of each halo outside the image), and a
    larger odd size: the tensor-core path against the FFMA path on every pixel, and against the oracle where
    the oracle finishes in seconds."""
    torch, ref, vd, synth = env
    wl = synth.WORKLOADS[2]
    z = synth.workload_latents(wl, batch=b, h=h, w=w)
    dec, got, wts = _decode(env, wl, z)
    dec2, got2, _ = _decode(env, wl, z, flags=vd.VD_FLAG_FORCE_SIMT)
    assert got.shape == (b, 3, 8 * h, 8 * w)
    if h * w <= 20:
        want = ref.decode(wl.arch, wts, z, wl.groups, wl.eps)
        for gg in (got, got2):
            g = gg.float().cpu().numpy()
            assert rel_l2(g, want) <= BF16_REL_L2 and max_abs(g, want) <= BF16_MAX_ABS
    # two paths that each meet the bound against the exact result differ by at most twice the bound
    d = got.float() - got2.float()
    assert float(d.norm() / got2.float().norm()) <= 2 * BF16_REL_L2 and float(d.abs().max()) <= 2 * BF16_MAX_ABS
    dec.check_status()


def test_fused_statistics_replace_the_norm2_passes(env):
    """VD_FLAG_FUSED_STATS: the second GroupNorm of every ResNet block has no step of its own (its statistics come
    from conv1's epilogue), and the frame stays within the bf16 bound of the default path's frame
    (the oracle comparison of this mode is test_sdvae_bf16_ragged_tiles_batch2[16])."""
    torch, ref, vd, synth = env
    wl = synth.WORKLOADS[2]
    z = synth.workload_latents(wl, batch=1, h=12, w=20)
    dec, got, _ = _decode(env, wl, z)
    dec2, got2, _ = _decode(env, wl, z, flags=vd.VD_FLAG_FUSED_STATS)
    s1, s2 = dec.steps(), dec2.steps()
    gn1 = [s["name"] for s in s1 if s["kind"] == vd.VD_STEP_GN_STATS]
    gn2 = [s["name"] for s in s2 if s["kind"] == vd.VD_STEP_GN_STATS]
    fused = [s["name"] for s in s2 if s.get("stats_fused")]
    assert len(fused) > 0 and len(gn1) - len(gn2) == len(fused)
    assert all(n.endswith("conv1") for n in fused) and not any(n.endswith("norm2") for n in gn2)
    assert not any(s.get("stats_fused") for s in s1)
    d = got.float() - got2.float()
    assert float(d.norm() / got.float().norm()) <= BF16_REL_L2      # (bf16 roundings flip between two correct paths)
    dec2.check_status()


def test_platformer_shape_256x256_stream_against_the_oracle(env):
    """The paper's second workload shape (256x256 frames, latent 32x32), four AR(1) frames in one batch:
    every pixel of the first and last frame against the oracle run in the test."""
    torch, ref, vd, synth = env
    wl = synth.WORKLOADS[6]
    z = synth.workload_latents(wl)
    dec, got, wts = _decode(env, wl, z)
    assert got.shape == (4, 3, 256, 256)
    for b in (0, 3):
        want = ref.decode(wl.arch, wts, z[b:b + 1], wl.groups, wl.eps)[0]
        g = got[b].float().cpu().numpy()
        r, m = rel_l2(g, want), max_abs(g, want)
        print(f"whole-frame parity {wl.name} frame {b}: rel-L2 {r:.3e} max-abs {m:.3e}")
        assert r <= BF16_REL_L2 and m <= BF16_MAX_ABS, (b, r, m)


def test_host_buffer_decode_and_extrapolation(env):
    torch, ref, vd, synth = env
    wl = synth.WORKLOADS[2]
    z = synth.workload_latents(wl, batch=2)
    dec, got, wts = _decode(env, wl, z)
    zh = torch.from_numpy(z).to(dec.dtype).pin_memory()
    fh = torch.empty((2, 3, 64, 64), dtype=dec.dtype).pin_memory()
    dec.decode_host(zh, fh)
    assert torch.equal(fh, got.cpu())
    # Algorithm 2, hit branch: z = z_prev + lambda*v_prev decoded in one call
    v = synth.round_to_bf16((0.1 * np.random.default_rng(1).standard_normal(z.shape)).astype(np.float32))
    lam = 0.5
    z_want, v_want = ref.extrapolate(z, v, lam)
    frames, z_new, v_new = dec.decode_extrapolated(torch.from_numpy(z).to("cuda:0", dec.dtype),
                                                   torch.from_numpy(v).to("cuda:0", dec.dtype), lam)
    torch.cuda.synchronize()
    assert max_abs(z_new.float().cpu().numpy(), z_want) <= 2 ** -8 * np.abs(z_want).max()
    assert max_abs(v_new.float().cpu().numpy(), v_want) <= 2 ** -8 * np.abs(z_want).max()
    want = ref.decode(wl.arch, wts, z_new.float().cpu().numpy(), wl.groups, wl.eps)
    g = frames.float().cpu().numpy()
    assert rel_l2(g, want) <= BF16_REL_L2 and max_abs(g, want) <= BF16_MAX_ABS


def test_decode_argument_errors(env):
    torch, ref, vd, synth = env
    wl = synth.WORKLOADS[1]
    z = synth.workload_latents(wl)
    dec, got, wts = _decode(env, wl, z)
    import ctypes
    l = vd.lib()
    assert l.vd_decode(dec.handle, None, ctypes.c_void_p(got.data_ptr()), 1, None) == vd.VD_ERR_INVALID_ARG
    assert l.vd_decode(dec.handle, ctypes.c_void_p(got.data_ptr()), ctypes.c_void_p(got.data_ptr()), 2, None) == vd.VD_ERR_INVALID_ARG
    assert b"batch" in l.vd_last_error(dec.handle)
    # missing weight / wrong shape / small workspace
    bad = dict(wts)
    del bad["conv_out.bias"]
    with pytest.raises(vd.VdError) as e:
        vd.Decoder(wl.arch, wl.dtype, 8, 8, 1, wl.groups, wl.eps, bad)
    assert e.value.status == vd.VD_ERR_INVALID_ARG and "conv_out.bias" in str(e.value)
    bad = dict(wts)
    bad["conv_in.weight"] = bad["conv_in.weight"][:, :3]
    with pytest.raises(vd.VdError) as e:
        vd.Decoder(wl.arch, wl.dtype, 8, 8, 1, wl.groups, wl.eps, bad)
    assert e.value.status == vd.VD_ERR_INVALID_ARG


@pytest.mark.parametrize("flags", [0, 1])
def test_per_layer_trace_parity(env, flags):
    """Every block output of the decoder against the oracle's named intermediates (localises an
    error to a layer): the decode is stopped after each step and that step's output is read back."""
    torch, ref, vd, synth = env
    wl = synth.WORKLOADS[2]
    z = synth.workload_latents(wl, batch=2, h=12, w=20)
    wts = synth.workload_weights(wl)
    trace = {}
    ref.decode(wl.arch, wts, z, wl.groups, wl.eps, trace=trace)
    dec = vd.Decoder(wl.arch, wl.dtype, 12, 20, 2, wl.groups, wl.eps, wts, flags)
    zt = torch.from_numpy(z).to("cuda:0", dec.dtype)
    checked = 0
    for i, st in enumerate(dec.steps()):
        name = st["name"]
        key = None
        if name in trace:
            key = name                                     # conv_in, upN.upconv, <block>.conv1, mid.attn.core
        elif name.endswith(".conv2") and name[:-6] in trace:
            key = name[:-6]                                # block output (shortcut included)
        elif name == "mid.attn.o":
            key = "mid.attn"
        if key is None or st["out_offset"] < 0:
            continue
        dec.stop_after(i)
        dec.decode(zt)
        torch.cuda.synchronize()
        got = dec.read_step_output(st, 2).cpu().numpy()
        r = rel_l2(got, trace[key])
        assert r <= 8e-3, (name, r)
        checked += 1
    dec.stop_after(-1)
    assert checked >= 30
    if flags == 0:
        impl = {s["name"]: s["impl"] for s in dec.steps()}
        assert impl["up2.res0.conv2"] == 1 and "up2.res0.shortcut" not in impl      # shortcut fused into conv2
        assert impl["conv_out"] == 1 and impl["mid.attn.core"] == 1
