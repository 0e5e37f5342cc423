"""Python face of the oracle: loads (building if needed) the plain C operators of `vd_ref.c`
and composes them into the decoder exactly as the workload definition lists its layers.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path imports this module, and this module
imports nothing from the CUDA library.  All tensors are fp32 NCHW numpy arrays.

The paper gives the operator chain of a decoder stage, Upsample -> Conv2d -> GroupNorm -> SiLU
(Section IV-B.1), and states the problem as latent in, frame out (Algorithm 1, the VAE decode
step); the layer list itself comes from the benchmark's configuration text:
  * "sdvae": conv_in 4->512; mid = ResNet(512), single-head attention(512), ResNet(512);
    four levels with channels 512, 512, 256, 128, three ResNet blocks each (1x1 shortcut where
    the width changes), nearest-2x upsample + conv3x3 after each of the first three levels;
    GroupNorm, SiLU, conv_out 128->3.
  * "tiny": conv_in 4->64; one ResNet block at 64; three stages of [nearest-2x upsample,
    conv3x3, one ResNet block] with widths 64->64->32->32; GroupNorm, SiLU, conv_out 32->3.
A ResNet block is x -> shortcut(x) + conv2(silu(gn2(conv1(silu(gn1(x)))))).
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vd_ref.c")
_LIB_PATH = os.path.join(_HERE, "libvd_ref.so")
_lock = threading.Lock()
_lib = None

_f32p = ctypes.POINTER(ctypes.c_float)
_f64p = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile vd_ref.c with gcc into libvd_ref.so beside it (if missing or stale)."""
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(_SRC)):
        return _LIB_PATH
    tmp = _LIB_PATH + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O3", "-fopenmp", "-fPIC", "-shared", "-fvisibility=hidden", "-std=c11",
           "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def lib():
    global _lib
    with _lock:
        if _lib is None:
            l = ctypes.CDLL(build())
            i, f, lg = ctypes.c_int, ctypes.c_float, ctypes.c_long
            l.vd_ref_num_threads.restype = i
            l.vd_ref_set_num_threads.argtypes = [i]
            l.vd_ref_conv2d.argtypes = [_f32p, _f32p, _f32p, _f32p, i, i, i, i, i, i]
            l.vd_ref_groupnorm.argtypes = [_f32p, _f32p, _f32p, _f32p, i, i, i, i, i, f, _f64p, _f64p]
            l.vd_ref_silu.argtypes = [_f32p, _f32p, lg]
            l.vd_ref_upsample2x.argtypes = [_f32p, _f32p, i, i, i, i]
            l.vd_ref_add.argtypes = [_f32p, _f32p, _f32p, lg]
            l.vd_ref_attention_core.argtypes = [_f32p, _f32p, _f32p, _f32p, i, i, i, f, _f64p]
            l.vd_ref_extrapolate.argtypes = [_f32p, _f32p, f, _f32p, _f32p, lg]
            l.vd_ref_pack_u8.argtypes = [_f32p, ctypes.POINTER(ctypes.c_ubyte), i, i, i, i]
            _lib = l
    return _lib


def num_threads() -> int:
    return int(lib().vd_ref_num_threads())


def set_num_threads(n: int) -> None:
    lib().vd_ref_set_num_threads(int(n))


def _c(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _p(a):
    return None if a is None else a.ctypes.data_as(_f32p)


def _ok(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"oracle: {what} rejected its arguments")


def conv2d(x, w, b=None):
    """Zero-padded stride-1 cross-correlation, kernel 1x1 or 3x3 (Conv2d of Section IV-A)."""
    x, w = _c(x), _c(w)
    b = None if b is None else _c(b)
    n, cin, h, wd = x.shape
    cout, cin2, kh, kw = w.shape
    assert cin == cin2 and kh == kw
    y = np.empty((n, cout, h, wd), dtype=np.float32)
    _ok(lib().vd_ref_conv2d(_p(x), _p(w), _p(b), _p(y), n, cin, h, wd, cout, kh), "conv2d")
    return y


def groupnorm(x, gamma, beta, groups: int, eps: float, return_stats: bool = False):
    """Two-pass GroupNorm with biased variance, per sample (GroupNorm of Section IV-A)."""
    x = _c(x)
    gamma = None if gamma is None else _c(gamma)
    beta = None if beta is None else _c(beta)
    n, c, h, w = x.shape
    y = np.empty_like(x)
    mean = np.empty((n, groups), dtype=np.float64)
    rstd = np.empty((n, groups), dtype=np.float64)
    _ok(lib().vd_ref_groupnorm(_p(x), _p(gamma), _p(beta), _p(y), n, c, h, w, groups, eps,
                               mean.ctypes.data_as(_f64p), rstd.ctypes.data_as(_f64p)), "groupnorm")
    return (y, mean, rstd) if return_stats else y


def silu(x):
    x = _c(x)
    y = np.empty_like(x)
    _ok(lib().vd_ref_silu(_p(x), _p(y), x.size), "silu")
    return y


def upsample2x(x):
    x = _c(x)
    n, c, h, w = x.shape
    y = np.empty((n, c, 2 * h, 2 * w), dtype=np.float32)
    _ok(lib().vd_ref_upsample2x(_p(x), _p(y), n, c, h, w), "upsample2x")
    return y


def add(a, b):
    a, b = _c(a), _c(b)
    assert a.shape == b.shape
    y = np.empty_like(a)
    _ok(lib().vd_ref_add(_p(a), _p(b), _p(y), a.size), "add")
    return y


def attention_core(q, k, v, scale: float, return_probs: bool = False):
    """softmax(scale * q^T k) v over tokens; q, k, v are [N, C, T]."""
    q, k, v = _c(q), _c(k), _c(v)
    n, c, t = q.shape
    o = np.empty_like(q)
    probs = np.empty((n, t, t), dtype=np.float64) if return_probs else None
    pp = probs.ctypes.data_as(_f64p) if return_probs else None
    _ok(lib().vd_ref_attention_core(_p(q), _p(k), _p(v), _p(o), n, c, t, scale, pp), "attention_core")
    return (o, probs) if return_probs else o


def extrapolate(z_prev, v_prev, lam: float):
    """Hit branch of Algorithm 2 / Eq. 10: z = z_prev + lam*v_prev and the new motion vector z - z_prev."""
    z_prev, v_prev = _c(z_prev), _c(v_prev)
    z = np.empty_like(z_prev)
    v = np.empty_like(z_prev)
    _ok(lib().vd_ref_extrapolate(_p(z_prev), _p(v_prev), lam, _p(z), _p(v), z_prev.size), "extrapolate")
    return z, v


def pack_u8(x):
    """Display packing of frames for transport (output side of Algorithm 1's decode step): NCHW fp32 in
    [-1, 1] -> NHWC uint8, q = rint(clamp(fma(x, 127.5, 127.5), 0, 255)) in fp32, ties to even."""
    x = _c(x)
    n, c, h, w = x.shape
    q = np.empty((n, h, w, c), np.uint8)
    _ok(lib().vd_ref_pack_u8(_p(x), q.ctypes.data_as(ctypes.POINTER(ctypes.c_ubyte)), n, c, h, w), "pack_u8")
    return q


# ---------------------------------------------------------------------------------------------
# Blocks and the decoder, composed from the operators above in the order the layers are listed.
# ---------------------------------------------------------------------------------------------

def _note(trace, name, value):
    if trace is not None:
        trace[name] = value


def resblock(x, wts: dict, prefix: str, groups: int, eps: float, trace=None):
    """x -> shortcut(x) + conv2(silu(gn2(conv1(silu(gn1(x)))))); 1x1 shortcut iff the width changes."""
    h = silu(groupnorm(x, wts[f"{prefix}.norm1.weight"], wts[f"{prefix}.norm1.bias"], groups, eps))
    h = conv2d(h, wts[f"{prefix}.conv1.weight"], wts[f"{prefix}.conv1.bias"])
    _note(trace, f"{prefix}.conv1", h)
    h = silu(groupnorm(h, wts[f"{prefix}.norm2.weight"], wts[f"{prefix}.norm2.bias"], groups, eps))
    h = conv2d(h, wts[f"{prefix}.conv2.weight"], wts[f"{prefix}.conv2.bias"])
    if f"{prefix}.shortcut.weight" in wts:
        x = conv2d(x, wts[f"{prefix}.shortcut.weight"], wts[f"{prefix}.shortcut.bias"])
    y = add(x, h)
    _note(trace, prefix, y)
    return y


def attention_block(x, wts: dict, prefix: str, groups: int, eps: float, trace=None):
    """x + Wo * softmax((Wq g)(Wk g)^T / sqrt(C)) (Wv g) + bo with g = gn(x) (no SiLU), one head,
    tokens = pixels in row-major order."""
    n, c, h, w = x.shape
    g = groupnorm(x, wts[f"{prefix}.norm.weight"], wts[f"{prefix}.norm.bias"], groups, eps)

    def proj(name, t):
        wt = _c(wts[f"{prefix}.{name}.weight"]).reshape(c, c, 1, 1)
        return conv2d(t, wt, wts[f"{prefix}.{name}.bias"])

    q, k, v = proj("q", g), proj("k", g), proj("v", g)
    o = attention_core(q.reshape(n, c, h * w), k.reshape(n, c, h * w), v.reshape(n, c, h * w),
                       1.0 / math.sqrt(c)).reshape(n, c, h, w)
    _note(trace, f"{prefix}.core", o)
    y = add(x, proj("o", o))
    _note(trace, prefix, y)
    return y


def decode(arch: str, wts: dict, latents, groups: int, eps: float, trace=None):
    """Latents [N,4,h,w] -> frames [N,3,8h,8w] through the named decoder layout."""
    x = conv2d(latents, wts["conv_in.weight"], wts["conv_in.bias"])
    _note(trace, "conv_in", x)
    if arch == "sdvae":
        x = resblock(x, wts, "mid.res0", groups, eps, trace)
        x = attention_block(x, wts, "mid.attn", groups, eps, trace)
        x = resblock(x, wts, "mid.res1", groups, eps, trace)
        for i in range(4):
            for j in range(3):
                x = resblock(x, wts, f"up{i}.res{j}", groups, eps, trace)
            if i < 3:
                x = conv2d(upsample2x(x), wts[f"up{i}.upconv.weight"], wts[f"up{i}.upconv.bias"])
                _note(trace, f"up{i}.upconv", x)
    elif arch == "tiny":
        x = resblock(x, wts, "mid.res0", groups, eps, trace)
        for i in range(3):
            x = conv2d(upsample2x(x), wts[f"up{i}.upconv.weight"], wts[f"up{i}.upconv.bias"])
            _note(trace, f"up{i}.upconv", x)
            x = resblock(x, wts, f"up{i}.res0", groups, eps, trace)
    else:
        raise ValueError(f"unknown arch {arch!r}")
    x = silu(groupnorm(x, wts["norm_out.weight"], wts["norm_out.bias"], groups, eps))
    y = conv2d(x, wts["conv_out.weight"], wts["conv_out.bias"])
    _note(trace, "frames", y)
    return y
