"""Runs one kernel of the library a few times on synthetic data, for profiling under ncu.

    python -m paper_1910_06188_b200.profile_cases attention --B 64 --S 384 --heads 16 --reps 3
    python -m paper_1910_06188_b200.profile_cases layernorm --rows 24576 --H 1024
"""
from __future__ import annotations

import argparse

import torch

from . import binding as q8


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["attention", "layernorm"])
    ap.add_argument("--B", type=int, default=64)
    ap.add_argument("--S", type=int, default=384)
    ap.add_argument("--heads", type=int, default=16)
    ap.add_argument("--rows", type=int, default=24576)
    ap.add_argument("--H", type=int, default=1024)
    ap.add_argument("--reps", type=int, default=3)
    a = ap.parse_args()
    g = torch.Generator(device="cuda").manual_seed(1)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if a.case == "attention":
        qkv = torch.randn((a.B * a.S, 3 * a.heads * 64), device="cuda", generator=g)
        ctx = torch.empty((a.B * a.S, a.heads * 64), device="cuda")
        fn = lambda: q8.q8_attention(qkv, a.B, a.S, a.heads, ctx=ctx)
        work = 4.0 * a.B * a.heads * a.S * a.S * 64
    else:
        x = torch.randn((a.rows, a.H), device="cuda", generator=g)
        r = torch.randn((a.rows, a.H), device="cuda", generator=g)
        out = torch.empty_like(x)
        fn = lambda: q8.q8_add_layernorm(x, r, out=out)
        work = 12.0 * a.rows * a.H
    fn()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(a.reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.reps
    unit = "TFLOP/s" if a.case == "attention" else "TB/s"
    print(f"{a.case}: {ms * 1e3:.1f} us per call, {work / (ms * 1e-3) / 1e12:.2f} {unit}")


if __name__ == "__main__":
    main()
