"""Per-kernel parity through the C ABI's operator-level entry points: each fused building block
against the oracle's plain operators on the same seeded inputs, at small/odd shapes that span
several tiles and a ragged tail."""
import math

import numpy as np
import pytest

from tests import util
from tests.util import rel_l2, max_abs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from oracle import ref
    from paper_2602_00608_b200 import binding, synth
    return torch, ref, binding, synth


def _rng(seed):
    return np.random.Generator(np.random.Philox(key=seed))


def _conv_case(env, *, seed, B, H, W, Cin, Cout, k, upsample, prologue, silu, residual, in_bf16, out_bf16, impl,
               bf16_ops=True, out_nchw=False):
    torch, ref, vd, synth = env
    r = _rng(seed)
    x = r.standard_normal((B, Cin, H, W)).astype(np.float32) * 1.5 + 0.3
    w = (r.uniform(-1, 1, (Cout, Cin, k, k)) * math.sqrt(3.0 / (Cin * k * k))).astype(np.float32)
    bias = r.uniform(-0.1, 0.1, Cout).astype(np.float32)
    scale = r.uniform(0.5, 1.5, (B, Cin)).astype(np.float32) if prologue else None
    shift = r.uniform(-0.5, 0.5, (B, Cin)).astype(np.float32) if prologue else None
    OH, OW = (2 * H, 2 * W) if upsample else (H, W)
    res = r.standard_normal((B, Cout, OH, OW)).astype(np.float32) if residual else None
    if in_bf16:
        x = synth.round_to_bf16(x)
    if bf16_ops:
        w = synth.round_to_bf16(w)
    # oracle: plain operators in definition order
    t = x
    if prologue:
        t = t * scale[:, :, None, None] + shift[:, :, None, None]
    if silu:
        t = ref.silu(t)
    if upsample:
        t = ref.upsample2x(t)
    want = ref.conv2d(t, w, bias)
    if residual:
        want = ref.add(want, res)
    dt_in = torch.bfloat16 if in_bf16 else torch.float32
    dev = lambda a: None if a is None else torch.from_numpy(a).cuda()
    y = vd.op_conv2d(util.nchw_to_dev_nhwc(x, dt_in), torch.from_numpy(w).cuda().to(torch.bfloat16 if bf16_ops else torch.float32),
                     dev(bias), dev(scale), dev(shift),
                     None if res is None else util.nchw_to_dev_nhwc(res, torch.float32),
                     upsample=upsample, silu=silu, out_dtype=vd.VD_BF16 if out_bf16 else vd.VD_F32,
                     out_nchw=out_nchw, bf16_operands=bf16_ops, impl=impl)
    torch.cuda.synchronize()
    got = y.float().cpu().numpy() if out_nchw else util.dev_nhwc_to_nchw(y)
    return got, want


SIMT_CASES = [
    dict(B=1, H=9, W=11, Cin=8, Cout=8, k=3, upsample=False, prologue=False, silu=False, residual=False),
    dict(B=2, H=13, W=19, Cin=20, Cout=72, k=3, upsample=False, prologue=True, silu=True, residual=True),
    dict(B=1, H=7, W=9, Cin=16, Cout=40, k=3, upsample=True, prologue=False, silu=False, residual=False),
    dict(B=2, H=10, W=17, Cin=24, Cout=12, k=1, upsample=False, prologue=True, silu=False, residual=True),
    dict(B=1, H=33, W=21, Cin=32, Cout=3, k=3, upsample=False, prologue=True, silu=True, residual=False, out_nchw=True),
    dict(B=1, H=5, W=6, Cin=4, Cout=64, k=3, upsample=False, prologue=False, silu=False, residual=False),
    # thin first-convolution kernel (K = 9 * Cin <= 72, Cout a multiple of 128): pixel count not a multiple of 32,
    # two frames, both supported input widths
    dict(B=2, H=7, W=9, Cin=4, Cout=128, k=3, upsample=False, prologue=False, silu=False, residual=False),
    dict(B=1, H=13, W=5, Cin=8, Cout=256, k=3, upsample=False, prologue=False, silu=False, residual=False),
]


@pytest.mark.parametrize("case", SIMT_CASES)
def test_conv_ffma_fp32_matches_oracle(env, case):
    _, _, vd, _ = env
    got, want = _conv_case(env, seed=11, in_bf16=False, out_bf16=False, impl=vd.VD_IMPL_SIMT, bf16_ops=False, **case)
    assert got.shape == want.shape
    assert rel_l2(got, want) <= 2e-6


@pytest.mark.parametrize("case", SIMT_CASES[:4])
def test_conv_ffma_bf16_operands_matches_oracle(env, case):
    _, _, vd, _ = env
    got, want = _conv_case(env, seed=12, in_bf16=True, out_bf16=True, impl=vd.VD_IMPL_SIMT, bf16_ops=True, **case)
    # one bf16 rounding of the transformed operand (2^-9 relative per element, averaging down in
    # the dot product) and one of the output (2^-9)
    assert rel_l2(got, want) <= 4e-3


def _gn_case(env, seed, B, H, W, C, G, bf16, offset=0.0):
    torch, ref, vd, synth = env
    r = _rng(seed)
    x = (r.standard_normal((B, C, H, W)) * r.uniform(0.5, 3.0, (1, C, 1, 1)) + offset).astype(np.float32)
    if bf16:
        x = synth.round_to_bf16(x)
    gamma = r.uniform(0.9, 1.1, C).astype(np.float32)
    beta = r.uniform(-0.1, 0.1, C).astype(np.float32)
    _, mean, rstd = ref.groupnorm(x, gamma, beta, G, 1e-6, return_stats=True)
    cpg = C // G
    want_scale = gamma[None, :] * np.repeat(rstd, cpg, axis=1)
    want_shift = beta[None, :] - np.repeat(mean, cpg, axis=1) * want_scale
    sc, sh = vd.op_gn_stats(util.nchw_to_dev_nhwc(x, torch.bfloat16 if bf16 else torch.float32),
                            torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda(), G, 1e-6)
    torch.cuda.synchronize()
    return sc.cpu().numpy(), sh.cpu().numpy(), want_scale, want_shift


@pytest.mark.parametrize("B,H,W,C,G,bf16", [
    (1, 8, 8, 32, 8, False), (2, 17, 23, 64, 8, False), (1, 60, 90, 512, 32, False), (2, 31, 45, 256, 32, True),
    (1, 64, 48, 128, 32, True), (1, 1, 1, 128, 32, False), (1, 3, 5, 96, 8, False),
])
def test_gn_stats_match_two_pass_oracle(env, B, H, W, C, G, bf16):
    sc, sh, wsc, wsh = _gn_case(env, 21, B, H, W, C, G, bf16)
    if H * W * (C // G) > 1:
        np.testing.assert_allclose(sc, wsc, rtol=2e-5)
        np.testing.assert_allclose(sh, wsh, rtol=2e-5, atol=2e-5)


@pytest.mark.parametrize("B,H,W,C,G,bf16", [(2, 17, 23, 64, 8, False), (1, 31, 45, 256, 32, True), (1, 9, 5, 128, 32, False)])
def test_gn_stats_with_a_per_channel_offset(env, B, H, W, C, G, bf16):
    """scale * x + shift must normalise x + offset[c] (a bias the tensor's producer left out): against the
    oracle's statistics of the shifted tensor."""
    torch, ref, vd, synth = env
    r = _rng(31)
    x = r.standard_normal((B, C, H, W)).astype(np.float32) * 1.3 + 0.2
    if bf16:
        x = synth.round_to_bf16(x)
    off = r.uniform(-2.0, 2.0, C).astype(np.float32)
    gamma = r.uniform(0.9, 1.1, C).astype(np.float32)
    beta = r.uniform(-0.1, 0.1, C).astype(np.float32)
    want, _, _ = ref.groupnorm(x + off[None, :, None, None], gamma, beta, G, 1e-6, return_stats=True)
    sc, sh = vd.op_gn_stats(util.nchw_to_dev_nhwc(x, torch.bfloat16 if bf16 else torch.float32),
                            torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda(), G, 1e-6,
                            offset=torch.from_numpy(off).cuda())
    torch.cuda.synchronize()
    got = x * sc.cpu().numpy()[:, :, None, None] + sh.cpu().numpy()[:, :, None, None]
    assert rel_l2(got, want) <= 2e-5


def test_gn_stats_survive_a_large_common_offset(env):
    # mean/std = 300: a plain sum-of-squares in fp32 would lose the variance
    sc, sh, wsc, wsh = _gn_case(env, 22, 1, 40, 40, 128, 32, False, offset=300.0)
    np.testing.assert_allclose(sc, wsc, rtol=2e-3)


def test_gn_stats_constant_groups_and_reproducibility(env):
    """Degenerate input (every group constant: variance exactly zero, so rstd = 1/sqrt(eps)), and the
    properties the one-launch kernel promises: the same bits on every call, and a sample's result does
    not depend on the batch it is in."""
    torch, ref, vd, synth = env
    r = _rng(23)
    B, H, W, C, G = 3, 37, 29, 64, 8
    eps = 0.25
    gamma = r.uniform(0.9, 1.1, C).astype(np.float32)
    beta = r.uniform(-0.1, 0.1, C).astype(np.float32)
    const = np.repeat(r.uniform(-5, 5, (B, G)).astype(np.float32), C // G, axis=1)          # [B, C], constant per group
    x = np.broadcast_to(const[:, :, None, None], (B, C, H, W)).copy()
    dev = lambda a_: torch.from_numpy(a_).cuda()
    sc, sh = vd.op_gn_stats(util.nchw_to_dev_nhwc(x, torch.float32), dev(gamma), dev(beta), G, eps)
    torch.cuda.synchronize()
    want_sc = np.broadcast_to(gamma / np.float32(math.sqrt(eps)), (B, C))
    np.testing.assert_allclose(sc.cpu().numpy(), want_sc, rtol=1e-6)
    np.testing.assert_allclose(sh.cpu().numpy(), beta - const * want_sc, rtol=1e-5, atol=1e-6)

    y = (r.standard_normal((B, C, H, W)) * 2.0 + 0.7).astype(np.float32)
    yd = util.nchw_to_dev_nhwc(y, torch.float32)
    a1 = vd.op_gn_stats(yd, dev(gamma), dev(beta), G, 1e-6)
    a2 = vd.op_gn_stats(yd, dev(gamma), dev(beta), G, 1e-6)
    one = vd.op_gn_stats(yd[1:2].contiguous(), dev(gamma), dev(beta), G, 1e-6)
    torch.cuda.synchronize()
    assert torch.equal(a1[0], a2[0]) and torch.equal(a1[1], a2[1])
    assert torch.equal(a1[0][1:2], one[0]) and torch.equal(a1[1][1:2], one[1])


def _attn_case(env, seed, B, T, C, bf16, impl):
    torch, ref, vd, synth = env
    r = _rng(seed)
    qkv = r.standard_normal((B, T, 3 * C)).astype(np.float32)
    qkv[:, :, :C] *= 2.0
    if bf16:
        qkv = synth.round_to_bf16(qkv)
    q, k, v = (np.ascontiguousarray(qkv[:, :, i * C:(i + 1) * C].transpose(0, 2, 1)) for i in range(3))
    scale = 1.0 / math.sqrt(C)
    want = ref.attention_core(q, k, v, scale).transpose(0, 2, 1)
    got = vd.op_attention(torch.from_numpy(qkv).cuda().to(torch.bfloat16 if bf16 else torch.float32), C, scale, impl)
    torch.cuda.synchronize()
    return got.float().cpu().numpy(), want


@pytest.mark.parametrize("B,T,C", [(1, 64, 512), (2, 77, 64), (1, 300, 512), (1, 1, 32)])
def test_attention_ffma_matches_oracle(env, B, T, C):
    _, _, vd, _ = env
    got, want = _attn_case(env, 31, B, T, C, False, vd.VD_IMPL_SIMT)
    assert rel_l2(got, want) <= 5e-6


# ------------------------------------------------------------------ tensor-core convolution
def test_conv_tc_identity_kernel_reproduces_the_operand(env):
    """Centre-tap identity weights: the output is the bf16 operand itself, bit for bit; any slip
    in the shared-memory operand layout, the tap views or the accumulator read-back shows here."""
    torch, ref, vd, synth = env
    B, H, W, C = 1, 21, 13, 128
    x = synth.round_to_bf16(_rng(5).standard_normal((B, C, H, W)).astype(np.float32))
    w = np.zeros((C, C, 3, 3), np.float32)
    w[np.arange(C), np.arange(C), 1, 1] = 1.0
    y = vd.op_conv2d(util.nchw_to_dev_nhwc(x, torch.bfloat16), torch.from_numpy(w).cuda().bfloat16(),
                     out_dtype=vd.VD_F32, bf16_operands=True, impl=vd.VD_IMPL_TC)
    torch.cuda.synchronize()
    assert np.array_equal(util.dev_nhwc_to_nchw(y), x)


@pytest.mark.parametrize("ky,kx", [(0, 0), (0, 2), (2, 1), (1, 0)])
def test_conv_tc_single_tap_shifts(env, ky, kx):
    torch, ref, vd, synth = env
    B, H, W, C = 1, 18, 11, 64
    x = synth.round_to_bf16(_rng(6).standard_normal((B, C, H, W)).astype(np.float32))
    w = np.zeros((128, C, 3, 3), np.float32)
    w[np.arange(C), np.arange(C), ky, kx] = 1.0          # output channels 64..127 stay zero
    y = vd.op_conv2d(util.nchw_to_dev_nhwc(x, torch.bfloat16), torch.from_numpy(w).cuda().bfloat16(),
                     out_dtype=vd.VD_F32, bf16_operands=True, impl=vd.VD_IMPL_TC)
    torch.cuda.synchronize()
    got = util.dev_nhwc_to_nchw(y)
    want = ref.conv2d(x, w)
    assert np.array_equal(got, want)


TC_CASES = [
    dict(B=1, H=16, W=8, Cin=64, Cout=128, k=3, upsample=False, prologue=False, silu=False, residual=False, in_bf16=True, out_bf16=False),
    dict(B=2, H=19, W=27, Cin=128, Cout=128, k=3, upsample=False, prologue=True, silu=True, residual=True, in_bf16=False, out_bf16=False),
    dict(B=1, H=33, W=20, Cin=256, Cout=256, k=3, upsample=False, prologue=True, silu=True, residual=False, in_bf16=True, out_bf16=True),
    dict(B=1, H=9, W=13, Cin=128, Cout=256, k=3, upsample=True, prologue=False, silu=False, residual=False, in_bf16=False, out_bf16=False),
    dict(B=2, H=10, W=17, Cin=256, Cout=128, k=1, upsample=False, prologue=False, silu=False, residual=False, in_bf16=False, out_bf16=False),
    dict(B=1, H=12, W=10, Cin=512, Cout=1536, k=1, upsample=False, prologue=True, silu=False, residual=False, in_bf16=False, out_bf16=True),
    dict(B=1, H=8, W=9, Cin=512, Cout=512, k=1, upsample=False, prologue=False, silu=False, residual=True, in_bf16=True, out_bf16=False),
    dict(B=1, H=17, W=16, Cin=512, Cout=512, k=3, upsample=False, prologue=True, silu=True, residual=True, in_bf16=True, out_bf16=False),
    dict(B=2, H=37, W=21, Cin=128, Cout=3, k=3, upsample=False, prologue=True, silu=True, residual=False, in_bf16=False, out_bf16=True, out_nchw=True),
    dict(B=3, H=50, W=70, Cin=128, Cout=128, k=3, upsample=False, prologue=True, silu=True, residual=True, in_bf16=True, out_bf16=False),
    # upsampling layers with 256-channel blocks run as two-CTA pairs: an odd number of tiles per channel block
    # (the peer CTA of the last pair has no tile), two channel blocks, two frames
    dict(B=1, H=17, W=9, Cin=64, Cout=256, k=3, upsample=True, prologue=False, silu=False, residual=False, in_bf16=False, out_bf16=False),
    dict(B=2, H=12, W=11, Cin=128, Cout=512, k=3, upsample=True, prologue=True, silu=True, residual=False, in_bf16=False, out_bf16=True),
]


# Phase-collapsed upsampling convolution (upsample=2): per output parity a 2x2 convolution of the source with
# pre-summed weights.  Ragged source tiles, an odd number of tiles per channel block (the peer CTA of the
# last pair has none), several channel blocks and frames, 1..8 input chunks, every dtype combination.
PHASE_CASES = [
    dict(B=1, H=9, W=13, Cin=128, Cout=256, k=3, upsample=2, prologue=False, silu=False, residual=False, in_bf16=False, out_bf16=False),
    dict(B=1, H=16, W=24, Cin=64, Cout=128, k=3, upsample=2, prologue=False, silu=False, residual=False, in_bf16=True, out_bf16=False),
    dict(B=2, H=12, W=11, Cin=128, Cout=512, k=3, upsample=2, prologue=True, silu=True, residual=False, in_bf16=False, out_bf16=True),
    dict(B=3, H=20, W=30, Cin=512, Cout=128, k=3, upsample=2, prologue=False, silu=False, residual=False, in_bf16=False, out_bf16=False),
    dict(B=2, H=33, W=17, Cin=256, Cout=256, k=3, upsample=2, prologue=True, silu=False, residual=False, in_bf16=True, out_bf16=True),
    dict(B=1, H=1, W=1, Cin=64, Cout=128, k=3, upsample=2, prologue=False, silu=False, residual=False, in_bf16=False, out_bf16=False),
]


@pytest.mark.parametrize("case", PHASE_CASES)
def test_conv_tc_phase_collapsed_upsample_matches_oracle(env, case):
    _, _, vd, _ = env
    got, want = _conv_case(env, seed=47, impl=vd.VD_IMPL_TC, bf16_ops=True, **case)
    assert got.shape == want.shape
    # both operands of this form are fp16 (2^-12 relative per rounding, activations and pre-summed
    # weights alike): an eighth of the bf16 forms' error; a bf16 output adds its own 2^-9 rounding
    tol = 4e-3 if case["out_bf16"] else 6e-4
    assert rel_l2(got, want) <= tol
    # against the 9-tap folded form of the same kernel family: same operands, weights summed after
    # instead of before the rounding
    got9, _ = _conv_case(env, seed=47, impl=vd.VD_IMPL_TC, bf16_ops=True, **dict(case, upsample=1))
    assert rel_l2(got, got9) <= (4.5e-3 if case["out_bf16"] else 2.5e-3)


@pytest.mark.parametrize("ky,kx", [(ky, kx) for ky in range(3) for kx in range(3)])
def test_conv_tc_phase_collapsed_single_taps_are_exact(env, ky, kx):
    """A single 3x3 tap with identity channels: every pre-summed weight is 0 or 1, so the output is
    the shifted, upsampled bf16 operand bit for bit.  Pins the tap sets of the four parities, the
    parity of the output coordinates and the zero ring, tap by tap."""
    torch, ref, vd, synth = env
    B, H, W, C = 2, 19, 10, 64
    x = synth.round_to_bf16(_rng(7).standard_normal((B, C, H, W)).astype(np.float32))
    x[np.abs(x) < 2.0 ** -10] = 0.0       # the kernel's operands are fp16: bf16 values this small would not convert exactly
    w = np.zeros((128, C, 3, 3), np.float32)
    w[np.arange(C), np.arange(C), ky, kx] = 1.0
    y = vd.op_conv2d(util.nchw_to_dev_nhwc(x, torch.bfloat16), torch.from_numpy(w).cuda().bfloat16(),
                     upsample=2, out_dtype=vd.VD_F32, bf16_operands=True, impl=vd.VD_IMPL_TC)
    torch.cuda.synchronize()
    got = util.dev_nhwc_to_nchw(y)
    want = ref.conv2d(ref.upsample2x(x), w)
    assert got.shape == want.shape == (B, 128, 2 * H, 2 * W)
    assert np.array_equal(got, want)


def test_conv_tc_phase_collapsed_all_ones_counts_taps(env):
    """All-ones input and weights: every output is (number of in-image taps) x Cin: 9 Cin inside,
    6 Cin on the edges, 4 Cin in the corners of the UPSAMPLED image (sums of small integers are
    exact in bf16 weights and fp32 accumulation)."""
    torch, ref, vd, synth = env
    H, W, C = 5, 7, 64
    x = np.ones((1, C, H, W), np.float32)
    w = np.ones((128, C, 3, 3), np.float32)
    y = vd.op_conv2d(util.nchw_to_dev_nhwc(x, torch.bfloat16), torch.from_numpy(w).cuda().bfloat16(),
                     upsample=2, out_dtype=vd.VD_F32, bf16_operands=True, impl=vd.VD_IMPL_TC)
    torch.cuda.synchronize()
    got = util.dev_nhwc_to_nchw(y)[0, 0]
    cnt_y = np.full(2 * H, 3.0); cnt_y[[0, -1]] = 2.0
    cnt_x = np.full(2 * W, 3.0); cnt_x[[0, -1]] = 2.0
    assert np.array_equal(got, np.outer(cnt_y, cnt_x) * C)


@pytest.mark.parametrize("case", TC_CASES)
def test_conv_tc_matches_oracle(env, case):
    _, _, vd, _ = env
    got, want = _conv_case(env, seed=41, impl=vd.VD_IMPL_TC, bf16_ops=True, **case)
    assert got.shape == want.shape
    # operand rounded once to bf16 (2^-9 relative, averaging down over the dot product); a bf16
    # output adds one more rounding of the result
    tol = 4e-3 if case["out_bf16"] else 2.5e-3
    assert rel_l2(got, want) <= tol
    # and the two GPU implementations agree far more closely than either does with fp32 math.
    # With SiLU in the prologue the tensor-core kernel uses the hardware tanh (relative error
    # 2^-11, an eighth of a bf16 rounding step), which moves a small fraction of the operands
    # across a bf16 rounding boundary; without it the operands are bitwise the same.
    got2, _ = _conv_case(env, seed=41, impl=vd.VD_IMPL_SIMT, bf16_ops=True, **case)
    assert rel_l2(got, got2) <= (4e-3 if case["out_bf16"] else (2e-4 if case["silu"] else 2e-5))


STAT_CASES = [
    # B, H, W, Cin, Cout, k, G, prologue  (channels per group 4, 8, 16; one- and two-tile items, CTA pairs, ragged edges)
    (1, 16, 8, 64, 128, 3, 32, False),
    (2, 19, 13, 64, 128, 3, 32, False),
    (1, 37, 29, 128, 256, 3, 32, False),
    (3, 9, 21, 64, 512, 3, 32, False),
    (1, 60, 90, 64, 512, 1, 32, False),
    (2, 33, 17, 64, 128, 3, 8, False),
    (1, 23, 31, 128, 256, 3, 32, True),
]


@pytest.mark.parametrize("B,H,W,Cin,Cout,k,G,prologue", STAT_CASES)
def test_conv_tc_epilogue_statistics_match_oracle(env, B, H, W, Cin, Cout, k, G, prologue):
    """The GroupNorm statistics a convolution's epilogue takes of its own output against the oracle's two-pass
    statistics of the oracle's convolution.  Without a prologue the bf16 operands are exact on both sides, so the
    values differ by fp32 accumulation only and the bound is tight."""
    torch, ref, vd, synth = env
    r = _rng(77 + Cout + H)
    x = synth.round_to_bf16(r.standard_normal((B, Cin, H, W)).astype(np.float32) * 1.5 + 0.3)
    w = synth.round_to_bf16((r.uniform(-1, 1, (Cout, Cin, k, k)) * math.sqrt(3.0 / (Cin * k * k))).astype(np.float32))
    bias = r.uniform(-0.5, 0.5, Cout).astype(np.float32)
    gamma = r.uniform(0.9, 1.1, Cout).astype(np.float32)
    beta = r.uniform(-0.1, 0.1, Cout).astype(np.float32)
    scale = r.uniform(0.5, 1.5, (B, Cin)).astype(np.float32) if prologue else None
    shift = r.uniform(-0.5, 0.5, (B, Cin)).astype(np.float32) if prologue else None
    t = x
    if prologue:
        t = ref.silu(t * scale[:, :, None, None] + shift[:, :, None, None])
    want = ref.conv2d(t, w, bias)
    _, mean, rstd = ref.groupnorm(want, gamma, beta, G, 1e-6, return_stats=True)
    cpg = Cout // G
    want_scale = gamma[None, :] * np.repeat(rstd, cpg, axis=1)
    want_shift = beta[None, :] - np.repeat(mean, cpg, axis=1) * want_scale
    dev = lambda a: None if a is None else torch.from_numpy(a).cuda()
    y, sc, sh = vd.op_conv2d_stats(util.nchw_to_dev_nhwc(x, torch.bfloat16), torch.from_numpy(w).cuda().to(torch.bfloat16),
                                   dev(gamma), dev(beta), G, 1e-6, dev(bias), dev(scale), dev(shift), silu=prologue)
    y2, sc2, sh2 = vd.op_conv2d_stats(util.nchw_to_dev_nhwc(x, torch.bfloat16), torch.from_numpy(w).cuda().to(torch.bfloat16),
                                      dev(gamma), dev(beta), G, 1e-6, dev(bias), dev(scale), dev(shift), silu=prologue)
    torch.cuda.synchronize()
    got = util.dev_nhwc_to_nchw(y)
    assert rel_l2(got, want) <= 1e-2
    tol = 3e-3 if prologue else 1e-4
    np.testing.assert_allclose(sc.cpu().numpy(), want_scale, rtol=tol)
    np.testing.assert_allclose(sh.cpu().numpy(), want_shift, rtol=tol, atol=tol)
    assert torch.equal(sc, sc2) and torch.equal(sh, sh2) and torch.equal(y, y2)      # fixed summation order


def test_conv_tc_epilogue_statistics_unsupported_layers_say_so(env):
    torch, ref, vd, synth = env
    x = torch.zeros((1, 8, 8, 64), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((128, 64, 3, 3), dtype=torch.bfloat16, device="cuda")
    g = torch.ones(128, device="cuda")
    with pytest.raises(vd.VdError) as e:
        vd.op_conv2d_stats(x, w, g, g, 64, 1e-6)          # two channels per group
    assert e.value.status == vd.VD_ERR_UNSUPPORTED
    with pytest.raises(vd.VdError) as e:
        vd.op_conv2d_stats(x, w, g, g, 32, 1e-6, impl=vd.VD_IMPL_SIMT)
    assert e.value.status == vd.VD_ERR_UNSUPPORTED


def test_conv_tc_real_layer_shape_sampled(env):
    """A full-size layer (128->128 at 480x720, the most common launch of the headline workload):
    sampled windows of the output against the oracle run on crops of the same seeded input."""
    torch, ref, vd, synth = env
    r = _rng(43)
    H, W, C = 480, 720, 128
    x = synth.round_to_bf16(r.standard_normal((1, C, H, W)).astype(np.float32))
    w = synth.round_to_bf16((r.uniform(-1, 1, (C, C, 3, 3)) * math.sqrt(3.0 / (C * 9))).astype(np.float32))
    bias = r.uniform(-0.1, 0.1, C).astype(np.float32)
    y = vd.op_conv2d(util.nchw_to_dev_nhwc(x, torch.bfloat16), torch.from_numpy(w).cuda().bfloat16(),
                     torch.from_numpy(bias).cuda(), out_dtype=vd.VD_F32, bf16_operands=True, impl=vd.VD_IMPL_TC)
    torch.cuda.synchronize()
    got = util.dev_nhwc_to_nchw(y)
    for (i0, j0) in [(0, 0), (0, W - 8), (H - 8, 0), (H - 8, W - 8), (236, 356), (15, 7), (400, 100)]:
        # crop with a one-pixel ring where the image has one; the ring's outputs are discarded
        a0, a1, b0, b1 = max(i0 - 1, 0), min(i0 + 9, H), max(j0 - 1, 0), min(j0 + 9, W)
        want = ref.conv2d(x[:, :, a0:a1, b0:b1], w, bias)[:, :, i0 - a0:i0 - a0 + 8, j0 - b0:j0 - b0 + 8]
        assert rel_l2(got[:, :, i0:i0 + 8, j0:j0 + 8], want) <= 1e-4, (i0, j0)


# ------------------------------------------------------------------ tensor-core attention
@pytest.mark.parametrize("B,T", [(1, 64), (1, 128), (2, 300), (1, 1000), (1, 129)])
def test_attention_tc_matches_oracle(env, B, T):
    _, _, vd, _ = env
    got, want = _attn_case(env, 51, B, T, 512, True, vd.VD_IMPL_TC)
    # bf16 probabilities and bf16 output: two roundings of 2^-9 relative
    assert rel_l2(got, want) <= 6e-3
    got2, _ = _attn_case(env, 51, B, T, 512, True, vd.VD_IMPL_SIMT)
    assert rel_l2(got, got2) <= 6e-3


def test_attention_tc_growing_scores_trigger_rescaling(env):
    """Keys ordered so that the row maximum keeps growing by more than the rescaling threshold from
    one key tile to the next: exercises the accumulator rescale path against the oracle."""
    torch, ref, vd, synth = env
    T, C = 640, 512
    r = _rng(52)
    q = r.standard_normal((1, T, C)).astype(np.float32)
    k = r.standard_normal((1, T, C)).astype(np.float32) * 0.05
    ramp = (np.arange(T) // 128).astype(np.float32)[None, :, None]         # + one step per key tile
    k = k + ramp * 0.6 * np.sign(q.mean(axis=1, keepdims=True))             # scores grow with the tile index
    q = q + 0.5 * np.sign(q.mean(axis=1, keepdims=True))
    v = r.standard_normal((1, T, C)).astype(np.float32)
    qkv = synth.round_to_bf16(np.concatenate([q, k, v], axis=2))
    scale = 1.0 / math.sqrt(C)
    qq, kk, vv = (np.ascontiguousarray(qkv[:, :, i * C:(i + 1) * C].transpose(0, 2, 1)) for i in range(3))
    want, probs = ref.attention_core(qq, kk, vv, scale, return_probs=True)
    s = np.einsum("ct,cu->tu", qq[0].astype(np.float64), kk[0].astype(np.float64)) * scale
    tile_max = np.stack([s[:, i:i + 128].max(axis=1) for i in range(0, T, 128)], axis=1)
    assert np.median(np.diff(tile_max, axis=1)) * 1.4427 > 8.0              # really beyond the threshold
    got = vd.op_attention(torch.from_numpy(qkv).cuda().bfloat16(), C, scale, vd.VD_IMPL_TC)
    torch.cuda.synchronize()
    assert rel_l2(got.float().cpu().numpy(), want.transpose(0, 2, 1)) <= 6e-3
