"""Thin ctypes binding of libvd.so: the same entry points as include/vd.h, argument marshalling
only.  PyTorch provides device memory and streams; every step of the decode runs in the CUDA
library.  There is no fallback: if the library is missing or the device is not sm_100 the calls
raise."""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char, c_char_p, c_double, c_float, c_int32, c_int64, c_size_t, c_uint32, c_void_p

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libvd.so")

VD_OK, VD_ERR_INVALID_ARG, VD_ERR_UNSUPPORTED, VD_ERR_WORKSPACE, VD_ERR_CUDA, VD_ERR_DEVICE_TIMEOUT = 0, -1, -2, -3, -4, -5
VD_F32, VD_BF16 = 0, 1
VD_ARCH_TINY, VD_ARCH_SDVAE = 0, 1
VD_FLAG_FORCE_SIMT = 0x1
VD_FLAG_UPSAMPLE_9TAP = 0x2
VD_FLAG_OUT_U8 = 0x4
VD_FLAG_CANARY = 0x8
VD_FLAG_FUSED_STATS = 0x10
VD_IMPL_AUTO, VD_IMPL_SIMT, VD_IMPL_TC = 0, 1, 2
VD_STEP_INGEST, VD_STEP_GN_STATS, VD_STEP_CONV, VD_STEP_ATTENTION = 0, 1, 2, 3
STATUS_NAMES = {0: "VD_OK", -1: "VD_ERR_INVALID_ARG", -2: "VD_ERR_UNSUPPORTED", -3: "VD_ERR_WORKSPACE",
                -4: "VD_ERR_CUDA", -5: "VD_ERR_DEVICE_TIMEOUT"}

EXPORTED = [
    "vd_query_workspace", "vd_create", "vd_decode", "vd_decode_extrapolated", "vd_decode_host", "vd_get_status",
    "vd_last_error", "vd_destroy", "vd_num_steps", "vd_get_step", "vd_profile", "vd_debug_stop_after",
    "vd_conv_packed_weight_bytes", "vd_conv_pack_weight", "vd_op_conv2d", "vd_conv_stats_scratch_bytes", "vd_op_conv2d_stats", "vd_gn_scratch_bytes", "vd_op_gn_stats",
    "vd_op_attention", "vd_attention_scratch_bytes", "vd_op_gn_stats_static", "vd_clear_status", "vd_decode_host_stream", "vd_debug_check_canaries", "vd_debug_status_offset", "vd_debug_wait_probe",
]


class VdConfig(Structure):
    _fields_ = [("struct_size", c_uint32), ("arch", c_int32), ("dtype", c_int32), ("latent_channels", c_int32),
                ("out_channels", c_int32), ("latent_h", c_int32), ("latent_w", c_int32), ("max_batch", c_int32),
                ("norm_groups", c_int32), ("norm_eps", c_float), ("flags", c_uint32)]


class VdTensor(Structure):
    _fields_ = [("name", c_char_p), ("dptr", c_void_p), ("dtype", c_int32), ("ndim", c_int32), ("shape", c_int64 * 4)]


class VdStepInfo(Structure):
    _fields_ = [("name", c_char * 64), ("kind", c_int32), ("impl", c_int32), ("launches", c_int32),
                ("c_in", c_int32), ("c_out", c_int32), ("ksize", c_int32), ("upsample", c_int32),
                ("out_h", c_int32), ("out_w", c_int32), ("out_channels", c_int32), ("out_dtype", c_int32),
                ("out_nchw", c_int32), ("out_offset", c_int64), ("flops_per_frame", c_double),
                ("bytes_per_frame", c_double), ("weight_bytes", c_double), ("c_in2", c_int32),
                ("has_residual", c_int32), ("phase_collapsed", c_int32), ("out_u8", c_int32),
                ("stats_fused", c_int32), ("reserved", c_int32), ("out_pending_offset", c_int64)]


class VdConvDesc(Structure):
    _fields_ = [("struct_size", c_uint32), ("batch", c_int32), ("in_h", c_int32), ("in_w", c_int32),
                ("c_in", c_int32), ("c_out", c_int32), ("ksize", c_int32), ("upsample", c_int32), ("silu", c_int32),
                ("in_dtype", c_int32), ("out_dtype", c_int32), ("out_nchw", c_int32), ("bf16_operands", c_int32),
                ("impl", c_int32)]


class VdError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


_lib = None


def lib():
    """Loads libvd.so (raises if it has not been built: there is no other implementation)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_00608_b200.build`")
        l = ctypes.CDLL(LIB_PATH)
        vp = c_void_p
        l.vd_query_workspace.argtypes = [POINTER(VdConfig), POINTER(c_size_t)]
        l.vd_create.argtypes = [POINTER(VdConfig), POINTER(VdTensor), c_int32, vp, c_size_t, vp, POINTER(vp)]
        l.vd_decode.argtypes = [vp, vp, vp, c_int32, vp]
        l.vd_decode_extrapolated.argtypes = [vp, vp, vp, c_float, vp, vp, vp, c_int32, vp]
        l.vd_decode_host.argtypes = [vp, vp, vp, c_int32, vp]
        l.vd_get_status.argtypes = [vp]
        l.vd_last_error.argtypes = [vp]
        l.vd_last_error.restype = c_char_p
        l.vd_destroy.argtypes = [vp]
        l.vd_num_steps.argtypes = [vp, POINTER(c_int32)]
        l.vd_get_step.argtypes = [vp, c_int32, POINTER(VdStepInfo)]
        l.vd_profile.argtypes = [vp, vp, vp, c_int32, vp, POINTER(c_float), c_int32]
        l.vd_debug_stop_after.argtypes = [vp, c_int32]
        l.vd_clear_status.argtypes = [vp, vp]
        l.vd_decode_host_stream.argtypes = [vp, vp, vp, c_int32, c_int32, vp]
        l.vd_debug_check_canaries.argtypes = [vp, POINTER(c_int32)]
        l.vd_debug_status_offset.argtypes = [vp, POINTER(c_int64)]
        l.vd_debug_wait_probe.argtypes = [vp, c_int64, vp]
        l.vd_conv_packed_weight_bytes.argtypes = [POINTER(VdConvDesc), POINTER(c_size_t)]
        l.vd_conv_pack_weight.argtypes = [POINTER(VdConvDesc), vp, c_int32, vp, vp]
        l.vd_op_conv2d.argtypes = [POINTER(VdConvDesc), vp, vp, vp, vp, vp, vp, vp, vp]
        l.vd_conv_stats_scratch_bytes.argtypes = [c_int32, c_int32]
        l.vd_conv_stats_scratch_bytes.restype = c_size_t
        l.vd_op_conv2d_stats.argtypes = [POINTER(VdConvDesc), vp, vp, vp, vp, vp, vp, c_int32, c_float, vp, vp, vp, vp, vp, vp]
        l.vd_gn_scratch_bytes.argtypes = [c_int32, c_int32]
        l.vd_gn_scratch_bytes.restype = c_size_t
        l.vd_op_gn_stats.argtypes = [vp, c_int32, c_int32, c_int32, c_int32, c_int32, c_int32, c_float, vp, vp, vp, vp, vp, vp, vp]
        l.vd_op_gn_stats_static.argtypes = [vp, c_int32, c_int32, c_int32, c_int32, c_int32, c_int32, c_float, vp, vp, vp, vp, vp]
        l.vd_op_attention.argtypes = [vp, vp, vp, vp, c_int32, c_int32, c_int32, c_int32, c_int32, c_int32, c_float, c_int32, vp, vp]
        l.vd_attention_scratch_bytes.argtypes = [c_int32, c_int32, c_int32]
        l.vd_attention_scratch_bytes.restype = c_size_t
        for name in EXPORTED:
            if name not in ("vd_last_error", "vd_gn_scratch_bytes", "vd_attention_scratch_bytes"):
                getattr(l, name).restype = c_int32
        _lib = l
    return _lib


def _check(status: int, handle=None):
    if status != VD_OK:
        msg = lib().vd_last_error(handle)
        raise VdError(status, (msg or b"").decode())


def make_config(arch: str, dtype: str, latent_h: int, latent_w: int, max_batch: int, groups: int, eps: float,
                flags: int = 0, latent_channels: int = 4, out_channels: int = 3) -> VdConfig:
    return VdConfig(ctypes.sizeof(VdConfig), {"tiny": VD_ARCH_TINY, "sdvae": VD_ARCH_SDVAE}[arch],
                    {"f32": VD_F32, "bf16": VD_BF16}[dtype], latent_channels, out_channels, latent_h, latent_w,
                    max_batch, groups, eps, flags)


def query_workspace(cfg: VdConfig) -> int:
    n = c_size_t(0)
    _check(lib().vd_query_workspace(byref(cfg), byref(n)))
    return int(n.value)


def _torch_dtype(dtype: int):
    import torch
    return torch.bfloat16 if dtype == VD_BF16 else torch.float32


def _stream_ptr(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return c_void_p(s.cuda_stream)


class Decoder:
    """A decoder handle plus the device memory it lives in (allocated with PyTorch).

    `weights` maps parameter names to numpy fp32 arrays or torch tensors (any device); they are
    moved to the device in the configuration's dtype for vd_create and may be dropped afterwards.
    """

    def __init__(self, arch: str, dtype: str, latent_h: int, latent_w: int, max_batch: int, groups: int, eps: float,
                 weights: dict, flags: int = 0, device: str = "cuda:0"):
        import torch
        self.torch = torch
        self.device = torch.device(device)
        self.cfg = make_config(arch, dtype, latent_h, latent_w, max_batch, groups, eps, flags)
        self.dtype = _torch_dtype(self.cfg.dtype)
        self.workspace_bytes = query_workspace(self.cfg)
        torch.cuda.set_device(self.device)
        self.workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=self.device)
        assert self.workspace.data_ptr() % 256 == 0
        dev_w = {}
        for name, w in weights.items():
            t = torch.as_tensor(w)
            dev_w[name] = t.to(device=self.device, dtype=self.dtype).contiguous()
        arr = (VdTensor * len(dev_w))()
        keep = []
        for i, (name, t) in enumerate(dev_w.items()):
            nb = name.encode()
            keep.append(nb)
            shape = (c_int64 * 4)(*(list(t.shape) + [1] * (4 - t.dim())))
            arr[i] = VdTensor(nb, t.data_ptr(), self.cfg.dtype, t.dim(), shape)
        h = c_void_p()
        _check(lib().vd_create(byref(self.cfg), arr, len(dev_w), c_void_p(self.workspace.data_ptr()),
                               self.workspace_bytes, _stream_ptr(), byref(h)))
        self.handle = h
        self.out_u8 = bool(flags & VD_FLAG_OUT_U8)
        self.out_dtype = torch.uint8 if self.out_u8 else self.dtype
        self.out_shape = ((8 * latent_h, 8 * latent_w, self.cfg.out_channels) if self.out_u8
                          else (self.cfg.out_channels, 8 * latent_h, 8 * latent_w))
        self.latent_shape = (self.cfg.latent_channels, latent_h, latent_w)

    # ---- decode
    def decode(self, latents, frames=None, stream=None):
        """latents: device tensor [B,4,h,w] of the configuration's dtype -> frames [B,3,8h,8w]."""
        torch = self.torch
        assert latents.is_cuda and latents.dtype == self.dtype and latents.is_contiguous()
        b = latents.shape[0]
        assert tuple(latents.shape[1:]) == self.latent_shape
        if frames is None:
            frames = torch.empty((b,) + self.out_shape, dtype=self.out_dtype, device=self.device)
        assert frames.dtype == self.out_dtype and frames.is_contiguous()
        _check(lib().vd_decode(self.handle, c_void_p(latents.data_ptr()), c_void_p(frames.data_ptr()), b,
                               _stream_ptr(stream)), self.handle)
        return frames

    def decode_extrapolated(self, z_prev, v_prev, lam: float, frames=None, want_state: bool = True, stream=None):
        torch = self.torch
        b = z_prev.shape[0]
        if frames is None:
            frames = torch.empty((b,) + self.out_shape, dtype=self.out_dtype, device=self.device)
        z = torch.empty_like(z_prev) if want_state else None
        v = torch.empty_like(z_prev) if want_state else None
        _check(lib().vd_decode_extrapolated(
            self.handle, c_void_p(z_prev.data_ptr()), c_void_p(v_prev.data_ptr()), lam,
            c_void_p(z.data_ptr()) if want_state else None, c_void_p(v.data_ptr()) if want_state else None,
            c_void_p(frames.data_ptr()), b, _stream_ptr(stream)), self.handle)
        return frames, z, v

    def decode_host(self, latents_host, frames_host, stream=None):
        """Host tensors in, host tensors out (pinned memory recommended); returns after the copy back."""
        assert not latents_host.is_cuda and not frames_host.is_cuda
        assert latents_host.dtype == self.dtype and frames_host.dtype == self.out_dtype
        b = latents_host.shape[0]
        _check(lib().vd_decode_host(self.handle, c_void_p(latents_host.data_ptr()), c_void_p(frames_host.data_ptr()),
                                    b, _stream_ptr(stream)), self.handle)
        return frames_host

    def decode_host_stream(self, latents_host, frames_host, batch: int = 1, stream=None):
        """A stream of frames through (pinned) host memory, `batch` per decode, copies overlapped with the
        decodes; returns when the last frame has reached frames_host."""
        assert not latents_host.is_cuda and not frames_host.is_cuda
        assert latents_host.dtype == self.dtype and frames_host.dtype == self.out_dtype
        assert latents_host.is_contiguous() and frames_host.is_contiguous()
        n = latents_host.shape[0]
        assert frames_host.shape[0] == n and tuple(frames_host.shape[1:]) == self.out_shape
        _check(lib().vd_decode_host_stream(self.handle, c_void_p(latents_host.data_ptr()), c_void_p(frames_host.data_ptr()),
                                           n, batch, _stream_ptr(stream)), self.handle)
        return frames_host

    # ---- introspection
    def check_status(self):
        _check(lib().vd_get_status(self.handle), self.handle)

    def clear_status(self, stream=None):
        _check(lib().vd_clear_status(self.handle, _stream_ptr(stream)), self.handle)

    def status_word(self):
        """The four 32-bit words of the device status record, as a view of the workspace (for tests)."""
        off = c_int64(0)
        _check(lib().vd_debug_status_offset(self.handle, byref(off)), self.handle)
        return self.workspace[off.value: off.value + 16].view(self.torch.int32)

    def wait_probe(self, limit_cycles: int, stream=None):
        _check(lib().vd_debug_wait_probe(self.handle, limit_cycles, _stream_ptr(stream)), self.handle)

    def check_canaries(self) -> int:
        """Verifies the workspace guards (handles created with VD_FLAG_CANARY); returns their number."""
        n = c_int32(0)
        _check(lib().vd_debug_check_canaries(self.handle, byref(n)), self.handle)
        return int(n.value)

    def steps(self):
        n = c_int32(0)
        _check(lib().vd_num_steps(self.handle, byref(n)), self.handle)
        out = []
        for i in range(n.value):
            info = VdStepInfo()
            _check(lib().vd_get_step(self.handle, i, byref(info)), self.handle)
            out.append({f: (getattr(info, f).decode() if f == "name" else getattr(info, f)) for f, _ in VdStepInfo._fields_})
        return out

    def profile(self, latents, frames, stream=None):
        n = len(self.steps())
        ms = (c_float * n)()
        _check(lib().vd_profile(self.handle, c_void_p(latents.data_ptr()), c_void_p(frames.data_ptr()),
                                latents.shape[0], _stream_ptr(stream), ms, n), self.handle)
        return list(ms)

    def stop_after(self, index: int):
        _check(lib().vd_debug_stop_after(self.handle, index), self.handle)

    def read_step_output(self, step: dict, batch: int):
        """The output of a step as an fp32 NCHW torch tensor (device): the stored tensor from the workspace plus,
        where the step left its bias pending (out_pending_offset), that per-channel vector."""
        torch = self.torch
        dt = _torch_dtype(step["out_dtype"])
        c = step["out_channels"]
        n = batch * step["out_h"] * step["out_w"] * c
        es = 2 if step["out_dtype"] == VD_BF16 else 4
        raw = self.workspace[step["out_offset"]: step["out_offset"] + n * es].view(dt)
        t = raw.view(batch, step["out_h"], step["out_w"], c).float()
        po = step.get("out_pending_offset", -1)
        if po >= 0:
            t = t + self.workspace[po: po + 4 * c].view(torch.float32)
        return t.permute(0, 3, 1, 2).contiguous()

    def close(self):
        if getattr(self, "handle", None):
            lib().vd_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ---- operator-level wrappers (device torch tensors, internal NHWC layout) ----------------------
def _dt(t) -> int:
    import torch
    return VD_BF16 if t.dtype == torch.bfloat16 else VD_F32


def conv_desc(batch, in_h, in_w, c_in, c_out, ksize, upsample, silu, in_dtype, out_dtype, out_nchw, bf16_operands,
              impl) -> VdConvDesc:
    return VdConvDesc(ctypes.sizeof(VdConvDesc), batch, in_h, in_w, c_in, c_out, ksize, int(upsample), int(silu),
                      in_dtype, out_dtype, int(out_nchw), int(bf16_operands), impl)


def op_conv2d(x_nhwc, w_oihw, bias=None, scale=None, shift=None, residual=None, *, upsample=False, silu=False,
              out_dtype=None, out_nchw=False, bf16_operands=False, impl=VD_IMPL_AUTO):
    """Fused convolution on device tensors; x is NHWC, w is [Cout,Cin,k,k]; returns y (NHWC or NCHW)."""
    import torch
    b, h, w, cin = x_nhwc.shape
    cout, _, k, _ = w_oihw.shape
    od = _dt(x_nhwc) if out_dtype is None else out_dtype
    d = conv_desc(b, h, w, cin, cout, k, upsample, silu, _dt(x_nhwc), od, out_nchw, bf16_operands, impl)
    nb = c_size_t(0)
    _check(lib().vd_conv_packed_weight_bytes(byref(d), byref(nb)))
    packed = torch.empty(nb.value, dtype=torch.uint8, device=x_nhwc.device)
    w_oihw = w_oihw.contiguous()
    _check(lib().vd_conv_pack_weight(byref(d), c_void_p(w_oihw.data_ptr()), _dt(w_oihw), c_void_p(packed.data_ptr()), _stream_ptr()))
    oh, ow = (2 * h, 2 * w) if upsample else (h, w)
    shape = (b, cout, oh, ow) if out_nchw else (b, oh, ow, cout)
    y = torch.empty(shape, dtype=_torch_dtype(od), device=x_nhwc.device)
    p = lambda t: None if t is None else c_void_p(t.data_ptr())
    for t in (bias, scale, shift, residual):
        assert t is None or (t.dtype == torch.float32 and t.is_contiguous())
    _check(lib().vd_op_conv2d(byref(d), p(x_nhwc.contiguous()), p(packed), p(bias), p(scale), p(shift), p(residual), p(y), _stream_ptr()))
    return y


def op_conv2d_stats(x_nhwc, w_oihw, gamma, beta, groups: int, eps: float, bias=None, scale=None, shift=None, *,
                    silu=False, out_dtype=None, impl=VD_IMPL_TC):
    """op_conv2d (bf16 operands, NHWC output) whose epilogue also takes the statistics of GroupNorm(y):
    returns (y, out_scale, out_shift)."""
    import torch
    b, h, w, cin = x_nhwc.shape
    cout, _, k, _ = w_oihw.shape
    od = VD_BF16 if out_dtype is None else out_dtype
    d = conv_desc(b, h, w, cin, cout, k, False, silu, _dt(x_nhwc), od, False, True, impl)
    nb = c_size_t(0)
    _check(lib().vd_conv_packed_weight_bytes(byref(d), byref(nb)))
    packed = torch.empty(nb.value, dtype=torch.uint8, device=x_nhwc.device)
    w_oihw = w_oihw.contiguous()
    _check(lib().vd_conv_pack_weight(byref(d), c_void_p(w_oihw.data_ptr()), _dt(w_oihw), c_void_p(packed.data_ptr()), _stream_ptr()))
    y = torch.empty((b, h, w, cout), dtype=_torch_dtype(od), device=x_nhwc.device)
    out_scale = torch.empty((b, cout), dtype=torch.float32, device=x_nhwc.device)
    out_shift = torch.empty((b, cout), dtype=torch.float32, device=x_nhwc.device)
    scratch = torch.empty(max(1, lib().vd_conv_stats_scratch_bytes(max(b, 1), groups)), dtype=torch.uint8, device=x_nhwc.device)
    p = lambda t: None if t is None else c_void_p(t.data_ptr())
    for t in (bias, scale, shift, gamma, beta):
        assert t is None or (t.dtype == torch.float32 and t.is_contiguous())
    _check(lib().vd_op_conv2d_stats(byref(d), p(x_nhwc.contiguous()), p(packed), p(bias), p(scale), p(shift), p(y), groups, eps,
                                    p(gamma), p(beta), p(out_scale), p(out_shift), p(scratch), _stream_ptr()))
    return y, out_scale, out_shift


def op_gn_stats(x_nhwc, gamma, beta, groups: int, eps: float, offset=None):
    """Per-(sample, channel) GroupNorm scale and shift of an NHWC device tensor (of x + offset[c] if given)."""
    import torch
    b, h, w, c = x_nhwc.shape
    scratch = torch.empty(max(1, lib().vd_gn_scratch_bytes(max(b, 1), groups)), dtype=torch.uint8, device=x_nhwc.device)
    scale = torch.empty((b, c), dtype=torch.float32, device=x_nhwc.device)
    shift = torch.empty((b, c), dtype=torch.float32, device=x_nhwc.device)
    p = lambda t: None if t is None else c_void_p(t.data_ptr())
    _check(lib().vd_op_gn_stats(p(x_nhwc.contiguous()), _dt(x_nhwc), b, h, w, c, groups, eps, p(gamma), p(beta), p(offset), p(scale), p(shift), p(scratch), _stream_ptr()))
    return scale, shift


def op_gn_stats_static(x_nhwc, gamma, beta, groups: int, eps: float):
    """op_gn_stats through the entry point that uses the library's built-in scratch array: for
    callers that may not allocate (this wrapper itself only allocates the two outputs)."""
    import torch
    b, h, w, c = x_nhwc.shape
    scale = torch.empty((b, c), dtype=torch.float32, device=x_nhwc.device)
    shift = torch.empty((b, c), dtype=torch.float32, device=x_nhwc.device)
    p = lambda t: c_void_p(t.data_ptr())
    _check(lib().vd_op_gn_stats_static(p(x_nhwc.contiguous()), _dt(x_nhwc), b, h, w, c, groups, eps, p(gamma), p(beta),
                                       p(scale), p(shift), _stream_ptr()))
    return scale, shift


def op_attention(qkv, channels: int, scale: float, impl=VD_IMPL_AUTO):
    """qkv: device [B,T,3C] (q | k | v per token) -> o [B,T,C]."""
    import torch
    b, t, c3 = qkv.shape
    assert c3 == 3 * channels and qkv.is_contiguous()
    o = torch.empty((b, t, channels), dtype=qkv.dtype, device=qkv.device)
    scratch = torch.empty(max(16, lib().vd_attention_scratch_bytes(b, t, channels)), dtype=torch.uint8, device=qkv.device)
    es = qkv.element_size()
    base = qkv.data_ptr()
    _check(lib().vd_op_attention(c_void_p(base), c_void_p(base + channels * es), c_void_p(base + 2 * channels * es),
                                 c_void_p(o.data_ptr()), _dt(qkv), b, t, channels, c3, channels, scale, impl,
                                 c_void_p(scratch.data_ptr()), _stream_ptr()))
    return o
