"""The C-ABI boundary without a GPU: the library loads, exports every symbol the header
declares, and rejects bad arguments on the host before touching a device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def vd():
    import __graft_entry__  # noqa: F401  (repository root is on sys.path via conftest)
    from paper_2602_00608_b200 import build
    build.build()
    from paper_2602_00608_b200 import binding
    return binding


def declared_symbols():
    text = "".join(open(os.path.join(ROOT, "include", f)).read() for f in sorted(os.listdir(os.path.join(ROOT, "include"))))
    return sorted(set(re.findall(r"VD_API\s+[\w\s\*]+?\b(vd_\w+)\s*\(", text)))


def test_header_and_binding_list_the_same_entry_points(vd):
    assert declared_symbols() == sorted(vd.EXPORTED)


def test_library_exports_every_declared_symbol(vd):
    l = ctypes.CDLL(vd.LIB_PATH)
    for name in declared_symbols():
        assert hasattr(l, name), name


def test_struct_sizes_match_the_header_layout(vd):
    assert ctypes.sizeof(vd.VdConfig) == 44
    assert ctypes.sizeof(vd.VdTensor) == 56
    assert ctypes.sizeof(vd.VdConvDesc) == 56
    assert ctypes.sizeof(vd.VdStepInfo) == 64 + 12 * 4 + 8 + 3 * 8 + 24 + 8


def test_query_workspace_is_host_only_and_scales_with_batch(vd):
    c1 = vd.make_config("sdvae", "bf16", 60, 90, 1, 32, 1e-6)
    c8 = vd.make_config("sdvae", "bf16", 60, 90, 8, 32, 1e-6)
    b1, b8 = vd.query_workspace(c1), vd.query_workspace(c8)
    assert 0.8e9 < b1 < 2.5e9          # two fp32 stream buffers of 345600 x 256 dominate
    assert 6 * b1 < b8 < 8.01 * b1
    t = vd.query_workspace(vd.make_config("tiny", "f32", 8, 8, 1, 8, 1e-6))
    assert t < 8e6


@pytest.mark.parametrize("mutate,status", [
    (lambda c: setattr(c, "struct_size", 12), -1),
    (lambda c: setattr(c, "arch", 7), -1),
    (lambda c: setattr(c, "dtype", 3), -1),
    (lambda c: setattr(c, "latent_h", 0), -1),
    (lambda c: setattr(c, "max_batch", 0), -1),
    (lambda c: setattr(c, "norm_groups", 48), -1),
    (lambda c: setattr(c, "norm_groups", 64), -1),      # 128/64 = 2 channels per group: not a multiple of 4
    (lambda c: setattr(c, "norm_eps", 0.0), -1),
    (lambda c: setattr(c, "flags", 0x80), -1),
    (lambda c: setattr(c, "latent_channels", 8), -2),
])
def test_bad_configs_are_rejected(vd, mutate, status):
    c = vd.make_config("sdvae", "bf16", 8, 8, 1, 32, 1e-6)
    mutate(c)
    with pytest.raises(vd.VdError) as e:
        vd.query_workspace(c)
    assert e.value.status == status
    assert str(e.value)


def test_null_arguments_are_rejected_without_a_device(vd):
    l = vd.lib()
    assert l.vd_query_workspace(None, None) == vd.VD_ERR_INVALID_ARG
    c = vd.make_config("tiny", "f32", 8, 8, 1, 8, 1e-6)
    assert l.vd_query_workspace(ctypes.byref(c), None) == vd.VD_ERR_INVALID_ARG
    h = ctypes.c_void_p()
    assert l.vd_create(ctypes.byref(c), None, 0, None, 0, None, ctypes.byref(h)) == vd.VD_ERR_INVALID_ARG
    assert not h.value
    t = (vd.VdTensor * 1)()
    assert l.vd_create(ctypes.byref(c), t, 1, None, 0, None, ctypes.byref(h)) == vd.VD_ERR_INVALID_ARG
    assert l.vd_create(ctypes.byref(c), t, 1, ctypes.c_void_p(128), 1 << 20, None, ctypes.byref(h)) == vd.VD_ERR_INVALID_ARG  # misaligned
    assert l.vd_decode(None, None, None, 1, None) == vd.VD_ERR_INVALID_ARG
    assert l.vd_destroy(None) == vd.VD_ERR_INVALID_ARG
    assert l.vd_get_status(None) == vd.VD_ERR_INVALID_ARG
    assert l.vd_num_steps(None, None) == vd.VD_ERR_INVALID_ARG
    assert l.vd_op_conv2d(None, None, None, None, None, None, None, None, None) == vd.VD_ERR_INVALID_ARG
    assert l.vd_op_gn_stats(None, 0, 1, 1, 1, 4, 1, 1e-6, None, None, None, None, None, None, None) == vd.VD_ERR_INVALID_ARG
    assert l.vd_op_attention(None, None, None, None, 0, 1, 1, 32, 32, 32, 1.0, 0, None, None) == vd.VD_ERR_INVALID_ARG
    assert l.vd_gn_scratch_bytes(0, 32) == 0
    assert b"NULL" in l.vd_last_error(None) or l.vd_last_error(None)


def test_conv_descriptor_validation(vd):
    l = vd.lib()
    n = ctypes.c_size_t()
    d = vd.conv_desc(1, 8, 8, 64, 64, 3, False, True, vd.VD_BF16, vd.VD_BF16, False, True, vd.VD_IMPL_SIMT)
    assert l.vd_conv_packed_weight_bytes(ctypes.byref(d), ctypes.byref(n)) == 0 and n.value == 9 * 64 * 64 * 4
    d.ksize = 5
    assert l.vd_conv_packed_weight_bytes(ctypes.byref(d), ctypes.byref(n)) == vd.VD_ERR_INVALID_ARG
    d.ksize = 3
    d.impl = 9
    assert l.vd_conv_packed_weight_bytes(ctypes.byref(d), ctypes.byref(n)) == vd.VD_ERR_INVALID_ARG
