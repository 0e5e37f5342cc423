"""Micro-benchmark of one fused convolution layer through the C ABI (vd_op_conv2d), for profiling a
single kernel on a small case.

    python bench_layer.py --h 240 --w 360 --cin 256 --cout 256 [--in-f32]
        [--out-f32] [--residual] [--prologue] [--upsample] [--k 3] [--iters 5] [--batch 1]

Prints one JSON line with the mean device time (CUDA events on the launching stream) and the
achieved TFLOP/s (algorithmic flops 2*k*k*Cin*Cout*H*W*B) and GB/s (input + residual + output).
"""
from __future__ import annotations

import argparse
import ctypes
import json

import torch

import os
import sys

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
from paper_2602_00608_b200 import binding as vd  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--h", type=int, default=240)
    ap.add_argument("--w", type=int, default=360)
    ap.add_argument("--cin", type=int, default=256)
    ap.add_argument("--cout", type=int, default=256)
    ap.add_argument("--k", type=int, default=3)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--in-f32", action="store_true")
    ap.add_argument("--out-f32", action="store_true")
    ap.add_argument("--residual", action="store_true")
    ap.add_argument("--prologue", action="store_true")
    ap.add_argument("--upsample", action="store_true")
    ap.add_argument("--phase", action="store_true", help="with --upsample: the phase-collapsed form (upsample=2)")
    ap.add_argument("--nchw", action="store_true")
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=2)
    ap.add_argument("--impl", type=int, default=vd.VD_IMPL_TC)
    ap.add_argument("--no-bias", action="store_true", help="no bias in the epilogue (the build the decoder runs where a layer's bias is pending)")
    a = ap.parse_args()

    g = torch.Generator(device="cuda").manual_seed(1)
    in_dt = torch.float32 if a.in_f32 else torch.bfloat16
    x = torch.randn((a.batch, a.h, a.w, a.cin), generator=g, device="cuda", dtype=torch.float32).to(in_dt)
    wt = (torch.rand((a.cout, a.cin, a.k, a.k), generator=g, device="cuda") - 0.5).to(torch.bfloat16)
    bias = None if a.no_bias else torch.zeros(a.cout, device="cuda")   # None: the build the decoder runs where the bias is pending
    oh, ow = (2 * a.h, 2 * a.w) if a.upsample else (a.h, a.w)
    res = torch.randn((a.batch, oh, ow, a.cout), generator=g, device="cuda") if a.residual else None
    scale = torch.ones((a.batch, a.cin), device="cuda") if a.prologue else None
    shift = torch.zeros((a.batch, a.cin), device="cuda") if a.prologue else None
    od = vd.VD_F32 if a.out_f32 else vd.VD_BF16

    d = vd.conv_desc(a.batch, a.h, a.w, a.cin, a.cout, a.k, (2 if a.phase else 1) if a.upsample else 0, a.prologue, vd._dt(x), od, a.nchw, True, a.impl)
    nb = ctypes.c_size_t(0)
    vd._check(vd.lib().vd_conv_packed_weight_bytes(ctypes.byref(d), ctypes.byref(nb)))
    packed = torch.empty(nb.value, dtype=torch.uint8, device="cuda")
    vd._check(vd.lib().vd_conv_pack_weight(ctypes.byref(d), ctypes.c_void_p(wt.data_ptr()), vd.VD_BF16,
                                           ctypes.c_void_p(packed.data_ptr()), vd._stream_ptr()))
    shape = (a.batch, a.cout, oh, ow) if a.nchw else (a.batch, oh, ow, a.cout)
    y = torch.empty(shape, dtype=torch.float32 if a.out_f32 else torch.bfloat16, device="cuda")
    p = lambda t: None if t is None else ctypes.c_void_p(t.data_ptr())

    def run():
        vd._check(vd.lib().vd_op_conv2d(ctypes.byref(d), p(x), p(packed), p(bias), p(scale), p(shift), p(res), p(y),
                                        vd._stream_ptr()))

    for _ in range(a.warmup):
        run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.iters
    flops = 2.0 * a.k * a.k * a.cin * a.cout * oh * ow * a.batch
    byts = x.numel() * x.element_size() + y.numel() * y.element_size() + (res.numel() * 4 if res is not None else 0)
    print(json.dumps({"ms": ms, "tflops": flops / ms / 1e9, "gbs": byts / ms / 1e6, "args": vars(a)}))


if __name__ == "__main__":
    main()
