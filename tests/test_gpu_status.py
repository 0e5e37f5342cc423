"""The device-timeout path end to end: a status word that a kernel (or, here, the host) sets is
reported by vd_get_status as VD_ERR_DEVICE_TIMEOUT with the code and block in vd_last_error, stays
set until vd_clear_status, and a bounded wait that really runs out on the GPU returns normally and
leaves the context and the handle usable.  Nothing here faults, traps or hangs the GPU: the wait
has a limit of about 0.1 ms and the kernel returns when it is reached."""
import numpy as np
import pytest

from tests.util import F32_REL_L2, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dec_env():
    import torch
    from oracle import ref
    from paper_2602_00608_b200 import binding as vd, synth
    wl = synth.WORKLOADS[1]
    wts = synth.workload_weights(wl)
    z = synth.workload_latents(wl)
    dec = vd.Decoder(wl.arch, wl.dtype, 8, 8, 1, wl.groups, wl.eps, wts)
    want = ref.decode(wl.arch, wts, z, wl.groups, wl.eps)
    return torch, vd, dec, torch.from_numpy(z).to("cuda:0", dec.dtype), want


def test_status_word_planted_by_the_host_is_reported_and_cleared(dec_env):
    torch, vd, dec, z, want = dec_env
    dec.check_status()
    word = dec.status_word()
    word[0] = 0xC0DE0001 - (1 << 32)         # int32 view of the convolution's code
    word[1] = 37
    word[2] = 256
    torch.cuda.synchronize()
    with pytest.raises(vd.VdError) as e:
        dec.check_status()
    assert e.value.status == vd.VD_ERR_DEVICE_TIMEOUT
    assert "0xc0de0001" in str(e.value) and "block 37" in str(e.value) and "convolution" in str(e.value)
    # sticky until cleared
    assert vd.lib().vd_get_status(dec.handle) == vd.VD_ERR_DEVICE_TIMEOUT
    dec.clear_status()
    torch.cuda.synchronize()
    dec.check_status()
    assert int(word[0].item()) == 0


def test_a_wait_that_runs_out_on_the_gpu_is_latched_and_the_handle_stays_usable(dec_env):
    torch, vd, dec, z, want = dec_env
    dec.check_status()
    dec.wait_probe(200_000)                  # ~0.1 ms at 1.9 GHz, then the kernel gives up and returns
    torch.cuda.synchronize()
    with pytest.raises(vd.VdError) as e:
        dec.check_status()
    assert e.value.status == vd.VD_ERR_DEVICE_TIMEOUT and "0xc0de0003" in str(e.value) and "wait probe" in str(e.value)
    # the first failure is kept: a second probe does not overwrite the record
    dec.wait_probe(100_000)
    torch.cuda.synchronize()
    assert int(dec.status_word()[2].item()) == 200_000
    dec.clear_status()
    got = dec.decode(z)
    torch.cuda.synchronize()
    dec.check_status()
    assert rel_l2(got.cpu().numpy(), want) <= F32_REL_L2
    with pytest.raises(vd.VdError):
        dec.wait_probe(10)                   # limit below the accepted range: rejected on the host


def test_clear_and_probe_reject_null_handles(dec_env):
    torch, vd, dec, z, want = dec_env
    assert vd.lib().vd_clear_status(None, None) == vd.VD_ERR_INVALID_ARG
    assert vd.lib().vd_debug_wait_probe(None, 100000, None) == vd.VD_ERR_INVALID_ARG
    assert vd.lib().vd_debug_status_offset(dec.handle, None) == vd.VD_ERR_INVALID_ARG


@pytest.mark.parametrize("idx,flags", [(1, 0), (2, 0), (2, 1), (2, 4)])
def test_workspace_guards_survive_decodes_and_catch_a_planted_overrun(idx, flags):
    """Every workspace region of a handle created with VD_FLAG_CANARY is followed by a guard pattern: odd-sized,
    batched decodes on every kernel path leave all guards intact, and a byte planted from the host is reported."""
    import torch
    from paper_2602_00608_b200 import binding as vd, synth
    wl = synth.WORKLOADS[idx]
    wts = synth.workload_weights(wl)
    h, w, b = 11, 13, 3
    dec = vd.Decoder(wl.arch, wl.dtype, h, w, b, wl.groups, wl.eps, wts, flags | vd.VD_FLAG_CANARY)
    plain = vd.Decoder(wl.arch, wl.dtype, h, w, b, wl.groups, wl.eps, wts, flags)
    z = torch.from_numpy(synth.workload_latents(wl, batch=b, h=h, w=w)).to("cuda:0", dec.dtype)
    got = dec.decode(z)
    dec.decode(z[:2].contiguous())
    n = dec.check_canaries()
    assert n > 50
    assert torch.equal(got, plain.decode(z))                 # the guards change the layout, not the result
    assert plain.check_canaries() == 0
    # plant an overrun: the workspace ends with the guard of its last region; overwrite that guard's last byte
    off = int(vd.query_workspace(dec.cfg))
    dec.workspace[off - 1] = 0
    with pytest.raises(vd.VdError) as e:
        dec.check_canaries()
    assert e.value.status == vd.VD_ERR_WORKSPACE and "guard" in str(e.value)
