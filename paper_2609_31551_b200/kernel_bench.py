"""Micro-benchmarks of the single-kernel entry points (CUDA events on the launching stream).

    python -m paper_2609_31551_b200.kernel_bench gemm --M 18464 --N 4096 --K 1024 --act 1
    python -m paper_2609_31551_b200.kernel_bench norm --rows 18464 --d 1024 --kind 0
    python -m paper_2609_31551_b200.kernel_bench attention --lens 577x32 --heads 16 --head-dim 64

Prints one JSON line per run: milliseconds per launch and TFLOP/s (GEMM, attention) or GB/s (norm)."""
from __future__ import annotations
import argparse
import json
import numpy as np
import torch

from . import binding as B


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


def bench_gemm(a):
    g = torch.Generator(device="cuda").manual_seed(1)
    A = torch.randn(a.M, a.K, device="cuda", generator=g).bfloat16()
    W = (torch.randn(a.N, a.K, device="cuda", generator=g) * 0.05).bfloat16()
    b = torch.randn(a.N, device="cuda", generator=g).bfloat16()
    out = torch.empty((a.M, a.N // 2 if a.act == 2 else a.N), dtype=torch.float32 if a.fp32 else torch.bfloat16, device="cuda")
    if a.fp32:
        out.zero_()
    resid = out if a.fp32 else None
    ms = _time(lambda: B.kernel_gemm(A, W, b, act=a.act, out_fp32=a.fp32, resid=resid, sm_budget=a.sm_budget, out=out),
               a.iters, a.warmup)
    return {"kernel": "gemm", "M": a.M, "N": a.N, "K": a.K, "act": a.act, "fp32_resid": a.fp32, "sm_budget": a.sm_budget,
            "ms": ms, "tflops": 2.0 * a.M * a.N * a.K / ms / 1e9}


def bench_norm(a):
    x = torch.randn(a.rows, a.d, device="cuda")
    g = torch.ones(a.d, device="cuda").bfloat16()
    b = torch.zeros(a.d, device="cuda").bfloat16()
    ms = _time(lambda: B.kernel_norm(x, g, b, a.kind, 1e-5, sm_budget=a.sm_budget), a.iters, a.warmup)
    return {"kernel": "norm", "rows": a.rows, "d": a.d, "kind": a.kind, "sm_budget": a.sm_budget, "ms": ms,
            "gbs": a.rows * a.d * 6 / ms / 1e6}


def bench_attention(a):
    lens = []
    for part in a.lens.split(","):
        if "x" in part:
            s, n = part.split("x")
            lens += [int(s)] * int(n)
        else:
            lens.append(int(part))
    T, d = sum(lens), a.heads * a.head_dim
    qkv = torch.randn(T, 3 * d, device="cuda").bfloat16()
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    ms = _time(lambda: B.kernel_attention(qkv, cu, a.heads, a.head_dim, sm_budget=a.sm_budget, impl=a.impl), a.iters, a.warmup)
    return {"kernel": "attention", "lens": a.lens, "heads": a.heads, "head_dim": a.head_dim, "impl": a.impl,
            "sm_budget": a.sm_budget, "ms": ms, "tflops": 4.0 * d * sum(s * s for s in lens) / ms / 1e9}


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="which", required=True)
    for name in ("gemm", "norm", "attention"):
        sp = sub.add_parser(name)
        sp.add_argument("--iters", type=int, default=20)
        sp.add_argument("--warmup", type=int, default=3)
        sp.add_argument("--sm-budget", type=int, default=0)
        if name == "gemm":
            sp.add_argument("--M", type=int, default=18464); sp.add_argument("--N", type=int, default=4096)
            sp.add_argument("--K", type=int, default=1024); sp.add_argument("--act", type=int, default=0)
            sp.add_argument("--fp32", action="store_true")
        elif name == "norm":
            sp.add_argument("--rows", type=int, default=18464); sp.add_argument("--d", type=int, default=1024)
            sp.add_argument("--kind", type=int, default=0)
        else:
            sp.add_argument("--lens", default="577x32"); sp.add_argument("--heads", type=int, default=16)
            sp.add_argument("--head-dim", type=int, default=64); sp.add_argument("--impl", type=int, default=0)
    a = ap.parse_args()
    res = {"gemm": bench_gemm, "norm": bench_norm, "attention": bench_attention}[a.which](a)
    print(json.dumps(res))


if __name__ == "__main__":
    main()
