"""Pins for the oracle's operators: closed forms, invariants, brute force on tiny inputs and
library routines, chosen so that a dropped term, a wrong sign or index, or a transposed
operand in oracle/vd_ref.c fails at least one of them.  No GPU, no product code."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import ref

RNG = np.random.default_rng(7)


def rnd(*shape):
    return RNG.standard_normal(shape).astype(np.float32)


# ------------------------------------------------------------------ conv2d
def test_conv_identity_kernel_is_exact():
    x = rnd(2, 5, 7, 9)
    w = np.zeros((5, 5, 3, 3), np.float32)
    for c in range(5):
        w[c, c, 1, 1] = 1.0
    assert np.array_equal(ref.conv2d(x, w), x)


@pytest.mark.parametrize("ky,kx", [(a, b) for a in range(3) for b in range(3)])
def test_conv_single_tap_is_a_shift_with_zero_border(ky, kx):
    # tap (ky,kx) reads x[i+ky-1, j+kx-1]: cross-correlation, not convolution
    x = rnd(1, 1, 6, 8)
    w = np.zeros((1, 1, 3, 3), np.float32)
    w[0, 0, ky, kx] = 1.0
    y = ref.conv2d(x, w)
    exp = np.zeros_like(x)
    for i in range(6):
        for j in range(8):
            ii, jj = i + ky - 1, j + kx - 1
            if 0 <= ii < 6 and 0 <= jj < 8:
                exp[0, 0, i, j] = x[0, 0, ii, jj]
    assert np.array_equal(y, exp)


def test_conv_all_ones_counts_taps():
    cin = 3
    y = ref.conv2d(np.ones((1, cin, 5, 6), np.float32), np.ones((2, cin, 3, 3), np.float32))
    assert np.all(y[:, :, 1:-1, 1:-1] == 9 * cin)
    assert np.all(y[:, :, 0, 1:-1] == 6 * cin) and np.all(y[:, :, 1:-1, 0] == 6 * cin)
    assert y[0, 0, 0, 0] == 4 * cin and y[0, 1, -1, -1] == 4 * cin


def test_conv_brute_force_seven_loops():
    x, w, b = rnd(2, 3, 4, 5), rnd(4, 3, 3, 3), rnd(4)
    exp = np.zeros((2, 4, 4, 5), np.float64)
    for j in range(5):                      # deliberately a different loop order
        for kx in range(3):
            for i in range(4):
                for ky in range(3):
                    ii, jj = i + ky - 1, j + kx - 1
                    if not (0 <= ii < 4 and 0 <= jj < 5):
                        continue
                    for n in range(2):
                        for o in range(4):
                            for c in range(3):
                                exp[n, o, i, j] += float(w[o, c, ky, kx]) * float(x[n, c, ii, jj])
    exp += b.astype(np.float64)[None, :, None, None]
    np.testing.assert_allclose(ref.conv2d(x, w, b), exp, rtol=0, atol=2e-6)


@pytest.mark.parametrize("k", [1, 3])
def test_conv_matches_library(k):
    x, w, b = rnd(2, 6, 9, 11), rnd(5, 6, k, k), rnd(5)
    exp = F.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(), torch.from_numpy(b).double(),
                   padding=k // 2).numpy()
    np.testing.assert_allclose(ref.conv2d(x, w, b), exp, rtol=0, atol=3e-6)


def test_conv1x1_is_a_per_pixel_matrix_product():
    x, w, b = rnd(1, 6, 4, 3), rnd(5, 6, 1, 1), rnd(5)
    exp = np.einsum("oc,nchw->nohw", w[:, :, 0, 0].astype(np.float64), x.astype(np.float64)) + b[None, :, None, None]
    np.testing.assert_allclose(ref.conv2d(x, w, b), exp, rtol=0, atol=2e-6)


def test_conv_no_bias_and_bad_kernel():
    x, w = rnd(1, 2, 3, 3), rnd(2, 2, 3, 3)
    np.testing.assert_allclose(ref.conv2d(x, w) + 0.5, ref.conv2d(x, w, np.full(2, 0.5, np.float32)), atol=1e-6)
    with pytest.raises(ValueError):
        ref.conv2d(x, rnd(2, 2, 5, 5))


# ------------------------------------------------------------------ groupnorm
def test_groupnorm_zero_mean_unit_variance_per_group():
    x = rnd(2, 8, 5, 7) * 3.0 + 1.5
    y = ref.groupnorm(x, None, None, 4, 1e-6).astype(np.float64).reshape(2, 4, -1)
    xg = x.astype(np.float64).reshape(2, 4, -1)
    var = xg.var(axis=2)
    np.testing.assert_allclose(y.mean(axis=2), 0.0, atol=1e-6)
    np.testing.assert_allclose(y.var(axis=2), var / (var + 1e-6), rtol=1e-5)


def test_groupnorm_constant_input_returns_beta():
    x = np.full((1, 4, 3, 3), 2.5, np.float32)
    beta = np.array([0.1, -0.2, 0.3, 0.4], np.float32)
    y = ref.groupnorm(x, np.array([2, 3, 4, 5], np.float32), beta, 2, 1e-6)
    np.testing.assert_allclose(y, np.broadcast_to(beta[None, :, None, None], y.shape), atol=1e-6)


def test_groupnorm_invariant_to_positive_affine_of_input():
    x = rnd(1, 6, 4, 4)
    g, b = rnd(6), rnd(6)
    # eps breaks exact scale invariance; use a scale that makes var >> eps either way
    np.testing.assert_allclose(ref.groupnorm(3.0 * x + 7.0, g, b, 3, 1e-6), ref.groupnorm(x, g, b, 3, 1e-6),
                               atol=2e-5)


def test_groupnorm_groups_are_contiguous_channel_blocks_and_per_sample():
    x = rnd(2, 4, 3, 3)
    x[:, 2:] *= 100.0          # second group on another scale: mixing channels across groups would show
    x[1] += 5.0                # second sample offset: batch statistics would show
    y = ref.groupnorm(x, None, None, 2, 1e-6)
    for n in range(2):
        for g in range(2):
            blk = y[n, 2 * g:2 * g + 2].astype(np.float64)
            assert abs(blk.mean()) < 1e-6 and abs(blk.var() - 1.0) < 1e-4
    np.testing.assert_array_equal(y[1:2], ref.groupnorm(x[1:2], None, None, 2, 1e-6))


def test_groupnorm_eps_is_inside_the_square_root():
    x = (rnd(1, 2, 4, 4) * 1e-3).astype(np.float32)
    eps = 0.25   # exactly representable in fp32
    y, mean, rstd = ref.groupnorm(x, None, None, 1, eps, return_stats=True)
    var = x.astype(np.float64).var()
    assert abs(rstd[0, 0] - 1.0 / math.sqrt(var + eps)) < 1e-9
    assert abs(mean[0, 0] - x.astype(np.float64).mean()) < 1e-12


def test_groupnorm_matches_library():
    x, g, b = rnd(2, 12, 5, 6), rnd(12), rnd(12)
    exp = F.group_norm(torch.from_numpy(x).double(), 4, torch.from_numpy(g).double(), torch.from_numpy(b).double(),
                       1e-6).numpy()
    np.testing.assert_allclose(ref.groupnorm(x, g, b, 4, 1e-6), exp, atol=2e-6)


def test_groupnorm_rejects_indivisible_groups():
    with pytest.raises(ValueError):
        ref.groupnorm(rnd(1, 6, 2, 2), None, None, 4, 1e-6)


# ------------------------------------------------------------------ silu
def test_silu_closed_forms():
    assert ref.silu(np.zeros(3, np.float32)).tolist() == [0.0, 0.0, 0.0]
    x = np.linspace(-8, 8, 1001).astype(np.float32)
    np.testing.assert_allclose(ref.silu(x) - ref.silu(-x), x, atol=1e-6)       # silu(x) - silu(-x) = x
    xs = np.linspace(-3, 0, 30001).astype(np.float32)
    ys = ref.silu(xs)
    k = int(np.argmin(ys))
    assert abs(ys[k] - (-0.27846)) < 1e-4 and abs(xs[k] - (-1.27846)) < 1e-3  # the single minimum
    np.testing.assert_allclose(ref.silu(x), F.silu(torch.from_numpy(x).double()).numpy(), atol=1e-6)
    assert abs(ref.silu(np.array([20.0], np.float32))[0] - 20.0) < 1e-6


# ------------------------------------------------------------------ upsample (+conv)
def test_upsample_replicates_each_pixel_into_a_2x2_block():
    x = rnd(2, 3, 4, 5)
    y = ref.upsample2x(x)
    assert y.shape == (2, 3, 8, 10)
    for a in range(2):
        for b in range(2):
            assert np.array_equal(y[:, :, a::2, b::2], x)


def test_upsample_then_conv_matches_brute_force():
    x, w, b = rnd(1, 2, 3, 4), rnd(3, 2, 3, 3), rnd(3)
    H2, W2 = 6, 8
    exp = np.zeros((1, 3, H2, W2), np.float64)
    for o in range(3):
        for i in range(H2):
            for j in range(W2):
                s = float(b[o])
                for c in range(2):
                    for ky in range(3):
                        for kx in range(3):
                            ii, jj = i + ky - 1, j + kx - 1
                            if 0 <= ii < H2 and 0 <= jj < W2:     # zero padding lives on the upsampled grid
                                s += float(w[o, c, ky, kx]) * float(x[0, c, ii // 2, jj // 2])
                exp[0, o, i, j] = s
    np.testing.assert_allclose(ref.conv2d(ref.upsample2x(x), w, b), exp, atol=2e-6)


def test_upsample_then_conv_equals_phase_collapsed_2x2_convs():
    # Independent derivation: for output parity (a,b) the 3x3 taps collapse onto a 2x2 source
    # neighbourhood with summed weights (rows: parity 0 -> {ky=0: i-1, ky=1,2: i}; parity 1 -> {ky=0,1: i, ky=2: i+1}).
    x, w = rnd(1, 2, 4, 5).astype(np.float64), rnd(2, 2, 3, 3).astype(np.float64)
    y = ref.conv2d(ref.upsample2x(x.astype(np.float32)), w.astype(np.float32)).astype(np.float64)
    xp = np.pad(x, ((0, 0), (0, 0), (1, 1), (1, 1)))
    rows = {0: [(-1, [0]), (0, [1, 2])], 1: [(0, [0, 1]), (1, [2])]}
    for a in range(2):
        for b in range(2):
            exp = np.zeros((1, 2, 4, 5))
            for di, kys in rows[a]:
                for dj, kxs in rows[b]:
                    wsum = sum(w[:, :, ky, kx] for ky in kys for kx in kxs)          # [o,c]
                    src = xp[:, :, 1 + di:1 + di + 4, 1 + dj:1 + dj + 5]
                    exp += np.einsum("oc,nchw->nohw", wsum, src)
            np.testing.assert_allclose(y[:, :, a::2, b::2], exp, atol=1e-5)


# ------------------------------------------------------------------ attention core
def test_attention_rows_sum_to_one_and_match_library():
    q, k, v = rnd(2, 8, 10), rnd(2, 8, 10), rnd(2, 8, 10)
    scale = 1.0 / math.sqrt(8)
    o, p = ref.attention_core(q, k, v, scale, return_probs=True)
    np.testing.assert_allclose(p.sum(axis=2), 1.0, atol=1e-12)
    tq, tk, tv = (torch.from_numpy(t).double().transpose(1, 2) for t in (q, k, v))      # [N,T,C]
    exp = F.scaled_dot_product_attention(tq, tk, tv, scale=scale).transpose(1, 2).numpy()
    np.testing.assert_allclose(o, exp, atol=2e-6)


def test_attention_zero_queries_average_the_values():
    k, v = rnd(1, 4, 7), rnd(1, 4, 7)
    o = ref.attention_core(np.zeros((1, 4, 7), np.float32), k, v, 0.5)
    np.testing.assert_allclose(o, np.broadcast_to(v.mean(axis=2, keepdims=True), o.shape), atol=1e-6)


def test_attention_constant_values_pass_through():
    q, k = rnd(1, 4, 6), rnd(1, 4, 6)
    v = np.broadcast_to(rnd(1, 4, 1), (1, 4, 6)).copy()
    np.testing.assert_allclose(ref.attention_core(q, k, v, 0.5), v, atol=1e-6)


def test_attention_is_query_indexed_not_key_indexed():
    # one-hot keys: a large score for (t, u=pi(t)) must route value pi(t) to output t (catches a transposed score matrix)
    T, C = 5, 5
    pi = np.array([2, 0, 4, 1, 3])
    q = np.zeros((1, C, T), np.float32)
    k = np.zeros((1, C, T), np.float32)
    for t in range(T):
        q[0, pi[t], t] = 50.0     # query t points along axis pi(t)
        k[0, t, t] = 1.0          # key u is the unit vector along axis u
    v = rnd(1, 3, T)
    q3 = q; k3 = k
    o = ref.attention_core(q3, k3, np.concatenate([v, np.zeros((1, C - 3, T), np.float32)], axis=1), 1.0)
    np.testing.assert_allclose(o[:, :3], v[:, :, pi], atol=1e-5)


def test_attention_token_permutation_equivariance_and_large_scores():
    q, k, v = rnd(1, 6, 9) * 30, rnd(1, 6, 9) * 30, rnd(1, 6, 9)      # scores of order 1e3: needs the row-max subtraction
    o = ref.attention_core(q, k, v, 1.0)
    assert np.all(np.isfinite(o))
    perm = RNG.permutation(9)
    np.testing.assert_allclose(ref.attention_core(q[:, :, perm], k, v, 1.0), o[:, :, perm], atol=1e-6)
    np.testing.assert_allclose(ref.attention_core(q, k[:, :, perm], v[:, :, perm], 1.0), o, atol=1e-5)


# ------------------------------------------------------------------ misc
def test_add_and_extrapolate():
    a, b = rnd(10), rnd(10)
    assert np.array_equal(ref.add(a, b), a + b)
    z0, v0 = rnd(2, 4, 3, 3), rnd(2, 4, 3, 3)
    z1, v1 = ref.extrapolate(z0, v0, 1.0)                     # Eq. 10 with a unit step: z + v, and v is reproduced
    np.testing.assert_allclose(z1, z0 + v0, atol=1e-6)
    np.testing.assert_allclose(v1, v0, atol=1e-6)
    z2, v2 = ref.extrapolate(z0, v0, 0.0)
    assert np.array_equal(z2, z0) and np.all(v2 == 0)


def test_results_do_not_depend_on_thread_count():
    x, w = rnd(1, 8, 9, 9), rnd(8, 8, 3, 3)
    n = ref.num_threads()
    y_many = ref.conv2d(x, w)
    ref.set_num_threads(1)
    try:
        assert np.array_equal(ref.conv2d(x, w), y_many)
    finally:
        ref.set_num_threads(n)


def test_pack_u8_fixed_points_saturation_and_layout():
    # -1 -> 0, 0 -> 128 (127.5 ties to even), 1 -> 255; anything outside saturates; NaN -> 0
    x = np.array([-1.0, 0.0, 1.0, -7.0, 3.0, np.nan, -1e30, 1e30], np.float32).reshape(1, 1, 2, 4)
    assert ref.pack_u8(x).ravel().tolist() == [0, 128, 255, 0, 255, 0, 0, 255]
    # channel interleaving: [N,C,H,W] -> [N,H,W,C]
    y = np.stack([np.full((2, 3), -1.0), np.zeros((2, 3)), np.ones((2, 3))]).astype(np.float32)[None]
    q = ref.pack_u8(y)
    assert q.shape == (1, 2, 3, 3) and (q[0, :, :, 0] == 0).all() and (q[0, :, :, 1] == 128).all() and (q[0, :, :, 2] == 255).all()


def test_pack_u8_is_the_exact_rounding_away_from_boundaries_and_monotone():
    from fractions import Fraction
    r = np.random.Generator(np.random.Philox(key=71))
    x = np.sort(np.concatenate([r.uniform(-1.2, 1.2, 4000), np.linspace(-1, 1, 511)]).astype(np.float32))
    q = ref.pack_u8(x.reshape(1, 1, 1, -1)).ravel().astype(int)
    assert (np.diff(q) >= 0).all()                                     # monotone
    checked = 0
    for xv, qv in zip(x.tolist(), q.tolist()):
        t = Fraction(xv) * Fraction(255, 2) + Fraction(255, 2)         # exact x * 127.5 + 127.5
        t = min(max(t, Fraction(0)), Fraction(255))
        lo = int(t)                                                    # floor (t >= 0)
        frac = t - lo
        if abs(frac - Fraction(1, 2)) > Fraction(1, 10000):            # away from a rounding boundary: one answer
            assert qv == (lo if frac < Fraction(1, 2) else lo + 1), (xv, qv)
            checked += 1
    assert checked > 4000
    # every level is reached exactly at its centre x = (2k - 255) / 255
    k = np.arange(256)
    centres = ((2.0 * k - 255.0) / 255.0).astype(np.float32)
    assert (ref.pack_u8(centres.reshape(1, 1, 1, -1)).ravel() == k).all()
