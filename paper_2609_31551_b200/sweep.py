"""Throughput sweep of the encoder over micro-batch size and sm_budget (the table of the headline metric).

    python -m paper_2609_31551_b200.sweep --config c1 --micro-batches 1,2,4,8,16,32,64 --budgets 37,74,111,148

One JSON line per point: tokens/s, items/s, TFLOP/s and the fraction of the measured bf16 peaks; inputs are the
seeded synthetic workloads of eas_synth, resident in HBM; W warm-up steps, K timed steps between CUDA events."""
from __future__ import annotations
import argparse
import json
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402  (FLOP model, workload recipe, measured peaks)
import eas_synth as S  # noqa: E402
from . import binding as B  # noqa: E402


def run_point(enc, cfg, shapes, seed, budget, steps, warmup):
    items = S.make_items(cfg, shapes, seed)
    data, offsets = B.pack_items(items)
    cu = np.concatenate([[0], np.cumsum([S.tokens_per_item(cfg, s) for s in shapes])]).astype(np.int32)
    cu_dev = torch.from_numpy(cu).cuda()
    f = bench.flops_of(cfg, shapes)
    out = torch.empty((f["out_rows"], cfg["d_out"]), dtype=torch.bfloat16, device="cuda")
    for _ in range(warmup):
        enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev, sm_budget=budget, out=out)
    enc.status()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev, sm_budget=budget, out=out)
    e1.record()
    torch.cuda.synchronize()
    enc.status()
    ms = e0.elapsed_time(e1) / steps
    return ms, f


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="c1")
    ap.add_argument("--micro-batches", default="1,2,4,8,16,32,64")
    ap.add_argument("--budgets", default="37,74,111,148")
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--max-tokens", type=int, default=400000, help="skip points with more encoder tokens than this")
    a = ap.parse_args()
    peaks = bench.measured_peaks()
    cfg = S.get_config(a.config)
    w = S.make_weights(cfg)
    enc = B.Encoder(cfg, B.weights_to_device(w))
    del w
    for mb in [int(x) for x in a.micro_batches.split(",")]:
        _, shapes, seed = bench.workload(a.config, mb)
        T = sum(S.tokens_per_item(cfg, s) for s in shapes)
        if T > a.max_tokens:
            print(json.dumps({"config": a.config, "micro_batch": mb, "skipped": f"{T} tokens > --max-tokens"}))
            continue
        for budget in [int(x) for x in a.budgets.split(",")]:
            ms, f = run_point(enc, cfg, shapes, seed, budget, a.steps, a.warmup)
            tf = f["total"] / ms / 1e9
            print(json.dumps({"config": a.config, "micro_batch": mb, "sm_budget": budget, "tokens": f["tokens"],
                              "sum_s2": f["sum_s2"], "ms_per_step": round(ms, 4),
                              "tokens_per_s": round(f["tokens"] / ms * 1e3, 1), "items_per_s": round(mb / ms * 1e3, 2),
                              "tflops": round(tf, 1), "attn_flop_share": round(f["attention"] / f["total"], 3),
                              "frac_burst": round(tf / peaks["burst"], 4), "frac_sustained": round(tf / peaks["sustained"], 4),
                              "peaks": peaks["source"]}), flush=True)


if __name__ == "__main__":
    main()
