"""The output side of the decode step (Algorithm 1, Q_out.push(I_t); Table II, data transport):
display-packed uint8 frames written by the last convolution's epilogue, and the streaming
host-buffer entry point that hides the copies behind the decodes."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from oracle import ref
    from paper_2602_00608_b200 import binding, synth
    return torch, ref, binding, synth


def _bf16_neighbours(f32: np.ndarray):
    """For bf16-representable fp32 values F: the ends of the interval of reals that round to F,
    [F - ulp/2, F + ulp/2], computed exactly in float64."""
    bits = f32.view(np.uint32)
    up = ((bits + np.uint32(0x10000)) & np.uint32(0xFFFF0000)).view(np.float32).astype(np.float64)
    dn = ((bits - np.uint32(0x10000)) & np.uint32(0xFFFF0000)).view(np.float32).astype(np.float64)
    f = f32.astype(np.float64)
    hi_nb = np.where(f >= 0, up, dn)      # next bf16 value away from / towards zero depending on sign
    lo_nb = np.where(f >= 0, dn, up)
    hi = np.maximum(hi_nb, lo_nb)
    lo = np.minimum(hi_nb, lo_nb)
    return (f + lo) / 2, (f + hi) / 2


@pytest.mark.parametrize("idx,flags", [(1, 0), (2, 0), (2, 1)])
def test_u8_frames_are_the_packed_float_frames(env, idx, flags):
    """Integer work, compared bit for bit: the uint8 frame is pack_u8 (oracle) of the value the same decode
    produces before its output cast.  fp32 configuration: that value IS the float frame, so the two must
    be equal everywhere.  bf16 configuration: the float frame F is that value rounded to bf16, so the value
    lies in [F - ulp/2, F + ulp/2] and, pack_u8 being monotone, the uint8 must lie between the packings of
    the interval's ends (equal to pack_u8(F) unless a quantisation boundary falls inside the interval)."""
    torch, ref, vd, synth = env
    wl = synth.WORKLOADS[idx]
    z = synth.workload_latents(wl, batch=2, h=7, w=9) * 0.35       # scaled so that the frames straddle [-1, 1]
    if wl.dtype == "bf16":
        z = synth.round_to_bf16(z.astype(np.float32))
    wts = synth.workload_weights(wl)
    dec_f = vd.Decoder(wl.arch, wl.dtype, 7, 9, 2, wl.groups, wl.eps, wts, flags)
    dec_q = vd.Decoder(wl.arch, wl.dtype, 7, 9, 2, wl.groups, wl.eps, wts, flags | vd.VD_FLAG_OUT_U8)
    zt = torch.from_numpy(z).to("cuda:0", dec_f.dtype)
    f = dec_f.decode(zt).float().cpu().numpy()
    q = dec_q.decode(zt)
    torch.cuda.synchronize()
    dec_q.check_status()
    assert q.dtype == torch.uint8 and tuple(q.shape) == (2, 56, 72, 3)
    q = q.cpu().numpy()
    assert (f < -1).any() and (f > 1).any()                        # both saturating ends are exercised
    if wl.dtype == "f32":
        assert np.array_equal(q, ref.pack_u8(f))
    else:
        lo, hi = _bf16_neighbours(f)
        q_lo, q_hi = ref.pack_u8(lo.astype(np.float32)), ref.pack_u8(hi.astype(np.float32))
        assert (q >= q_lo).all() and (q <= q_hi).all()
        assert (q == ref.pack_u8(f)).mean() > 0.9              # a bf16 ulp near 1 is half a level: some values do straddle
    # and against the oracle's own frame: a few levels at most (3e-2 of the float bar is 3.8 levels)
    want = ref.pack_u8(ref.decode(wl.arch, wts, z, wl.groups, wl.eps))
    tol = 1 if wl.dtype == "f32" else 4
    assert np.abs(q.astype(int) - want.astype(int)).max() <= tol


@pytest.mark.parametrize("u8", [False, True])
def test_host_stream_equals_frame_by_frame_decodes(env, u8):
    """Five frames, two per decode (the last step is a single frame): the frames the streaming entry point
    leaves in host memory are bit for bit those of plain device decodes of the same latents."""
    torch, ref, vd, synth = env
    wl = synth.WORKLOADS[2]
    n = 5
    z = synth.workload_latents(wl, batch=n)
    wts = synth.workload_weights(wl)
    dec = vd.Decoder(wl.arch, wl.dtype, 8, 8, 2, wl.groups, wl.eps, wts, vd.VD_FLAG_OUT_U8 if u8 else 0)
    zt = torch.from_numpy(z).to(dec.dtype)
    want = torch.cat([dec.decode(zt[i:i + 2].cuda()).cpu() for i in range(0, n, 2)])
    zh = zt.pin_memory()
    fh = torch.zeros((n,) + dec.out_shape, dtype=dec.out_dtype).pin_memory()
    for _ in range(2):                                             # a second call reuses the pipeline
        fh.zero_()
        dec.decode_host_stream(zh, fh, batch=2)
        assert torch.equal(fh, want)
    dec.check_status()
    # one frame per step, and the plain host entry point
    fh.zero_()
    dec.decode_host_stream(zh, fh, batch=1)
    one = torch.cat([dec.decode(zt[i:i + 1].cuda()).cpu() for i in range(n)])
    assert torch.equal(fh, one)
    f2 = torch.zeros((2,) + dec.out_shape, dtype=dec.out_dtype).pin_memory()
    dec.decode_host(zh[:2].clone().pin_memory(), f2)
    assert torch.equal(f2, want[:2])
    with pytest.raises(vd.VdError):
        dec.decode_host_stream(zh, fh, batch=3)                    # larger than max_batch
