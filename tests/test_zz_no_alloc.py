"""The allocation-free GroupNorm-statistics entry point (for callers that cannot allocate device
memory when they call: real-time loops, plug-ins inside someone else's memory budget, host
callbacks).  It must give what the ordinary entry point gives, call after call, although all
calls share one built-in scratch array that keeps the previous call's contents.

Collected last on purpose (file name), so a run that stops at the first failure has already run
everything else; it passes alone in a fresh process as well as after the other tests."""
import ctypes

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_the_ordinary_one_twice_in_a_row():
    import torch
    from oracle import ref
    from paper_2602_00608_b200 import binding as vd

    gen = np.random.Generator(np.random.Philox(key=99))
    cases = [(2, 37, 53, 128, 32, torch.float32), (1, 60, 90, 512, 32, torch.bfloat16)]   # a big then a smaller footprint
    for (b, h, w, c, g, dt) in cases:
        x = torch.from_numpy(gen.standard_normal((b, h, w, c)).astype(np.float32) * 2.0 + 0.5).cuda().to(dt)
        gamma = torch.from_numpy(gen.uniform(0.9, 1.1, c).astype(np.float32)).cuda()
        beta = torch.from_numpy(gen.uniform(-0.1, 0.1, c).astype(np.float32)).cuda()
        want_scale, want_shift = vd.op_gn_stats(x, gamma, beta, g, 1e-6)
        # and against the oracle's two-pass GroupNorm, so that the test stands on its own
        x_nchw = x.float().permute(0, 3, 1, 2).contiguous().cpu().numpy()
        _, mean, rstd = ref.groupnorm(x_nchw, gamma.cpu().numpy(), beta.cpu().numpy(), g, 1e-6, return_stats=True)
        ref_scale = gamma.cpu().numpy()[None, :] * np.repeat(rstd, c // g, axis=1)
        ref_shift = beta.cpu().numpy()[None, :] - np.repeat(mean, c // g, axis=1) * ref_scale
        for _ in range(2):                                   # second call sees the first call's leftovers
            scale, shift = vd.op_gn_stats_static(x, gamma, beta, g, 1e-6)
            torch.cuda.synchronize()
            # same kernels, same summation order: the tolerance of the statistics tests is far from reached
            np.testing.assert_allclose(scale.cpu().numpy(), want_scale.cpu().numpy(), rtol=2e-5)
            np.testing.assert_allclose(shift.cpu().numpy(), want_shift.cpu().numpy(), rtol=2e-5, atol=2e-5)
            np.testing.assert_allclose(scale.cpu().numpy(), ref_scale, rtol=2e-5)
            np.testing.assert_allclose(shift.cpu().numpy(), ref_shift, rtol=2e-5, atol=2e-5)


def test_static_scratch_entry_point_rejects_what_does_not_fit():
    import torch
    from paper_2602_00608_b200 import binding as vd

    x = torch.zeros((3, 4, 4, 128), device="cuda")           # 3 frames x 32 groups = 96 > 64
    gamma = torch.ones(128, device="cuda")
    beta = torch.zeros(128, device="cuda")
    with pytest.raises(vd.VdError) as e:
        vd.op_gn_stats_static(x, gamma, beta, 32, 1e-6)
    assert e.value.status == vd.VD_ERR_UNSUPPORTED and "64" in str(e.value)
    assert vd.lib().vd_op_gn_stats_static(None, 0, 1, 1, 1, 4, 1, ctypes.c_float(1e-6), None, None, None, None, None) == vd.VD_ERR_INVALID_ARG
