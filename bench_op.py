"""Micro-benchmark of the two other operators of the decoder through the C ABI, for profiling a single
kernel on a small case:

    python bench_op.py gn --h 480 --w 720 --c 128 [--f32] [--iters 5]
    python bench_op.py attn --tokens 5400 --c 512 [--iters 5]

gn:   GroupNorm statistics (vd_op_gn_stats) of an NHWC tensor, 32 groups; prints the mean device time and the
      achieved GB/s (algorithmic bytes: one read of the tensor).
attn: single-head attention core (vd_op_attention) over `tokens` tokens; prints the mean device time and
      the achieved TFLOP/s (algorithmic flops 4*T*T*C).
Times are CUDA events on the launching stream around `iters` back-to-back calls.
"""
from __future__ import annotations

import argparse
import json

import torch

import os
import sys

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
from paper_2602_00608_b200 import binding as vd  # noqa: E402


def _time(fn, iters, warmup):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["gn", "attn"])
    ap.add_argument("--h", type=int, default=480)
    ap.add_argument("--w", type=int, default=720)
    ap.add_argument("--c", type=int, default=128)
    ap.add_argument("--tokens", type=int, default=5400)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--f32", action="store_true")
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=2)
    a = ap.parse_args()
    g = torch.Generator(device="cuda").manual_seed(1)
    if a.op == "gn":
        dt = torch.float32 if a.f32 else torch.bfloat16
        x = torch.randn((a.batch, a.h, a.w, a.c), generator=g, device="cuda").to(dt)
        gamma, beta = torch.ones(a.c, device="cuda"), torch.zeros(a.c, device="cuda")
        ms = _time(lambda: vd.op_gn_stats(x, gamma, beta, 32, 1e-6), a.iters, a.warmup)
        byts = x.numel() * x.element_size()
        print(json.dumps({"op": "gn_stats", "ms": ms, "gbs": byts / ms / 1e6, "mbytes": byts / 1e6, "args": vars(a)}))
    else:
        qkv = torch.randn((a.batch, a.tokens, 3 * a.c), generator=g, device="cuda").to(torch.bfloat16)
        ms = _time(lambda: vd.op_attention(qkv, a.c, a.c ** -0.5, vd.VD_IMPL_TC), a.iters, a.warmup)
        flops = 4.0 * a.tokens * a.tokens * a.c * a.batch
        print(json.dumps({"op": "attention", "ms": ms, "tflops": flops / ms / 1e9, "args": vars(a)}))


if __name__ == "__main__":
    main()
