#!/usr/bin/env python
"""Benchmark of the Encode-stage forward pass (one step = one micro-batch through the whole encoder).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c1] [--micro-batch 32] [--sm-budget 0]
    python bench.py --impl reference ...      # times the CPU fp64 oracle on a bounded sample

Prints ONE JSON line.  `value` is encoder tokens/s with inputs resident in HBM; `e2e` is the same metric
through the C ABI with host buffers (pinned host -> device copy of the pixels and device -> host copy of the
embeddings inside the timed region, double-buffered on copy streams); `roofline` is the dominant kernel class
(the GEMMs) timed with CUDA events inside the library; `cpu_baseline` is the oracle on this machine's host cores.
Multi-GPU: replicas only (items are independent, the path has no collective); each rank encodes its own
micro-batches and the job value is the sum of tokens over the slowest rank's time."""
from __future__ import annotations
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import eas_synth as S  # noqa: E402


from paper_2609_31551_b200.measure import (ClockSampler, Point, flops_of, gemm_flops_by_class, measured_peaks,  # noqa: E402
                                           time_point, workload)

# The points of the headline metric (tokens/s and items/s against micro-batch and sm_budget) that the default run
# measures besides the main one, grouped by configuration so that every encoder is built once:
# (config, [(micro-batch, [sm budgets])]).  0 = all SMs.
SWEEP = [
    ("c1", [(1, [0]), (16, [0]), (64, [0]), (32, [37, 74, 111])]),
    ("c3", [(1, [0, 37, 74, 111]), (2, [0])]),
    ("c2", [(16, [0])]),
    ("c4", [(16, [37, 74, 111, 0])]),
]


def other_rooflines(cfg, shapes, f, acc, n_prof, peaks):
    """The two other kernel classes of a step against their own roofs (start-to-start times, so launch gaps count):
    attention against the bf16 tensor peaks (its exponentials, not the tensor pipe, pace it), and the norm kernels
    against the measured HBM copy rate with 6 algorithmic bytes per element (fp32 in, bf16 out)."""
    out = []
    if 5 in acc and acc[5][0] > 0:
        t = acc[5][0] / n_prof * 1e-3
        tf = f["attention"] / t / 1e12
        out.append({"kernel": "attn_tc_kernel", "bound": "tensor", "achieved": tf, "peak": peaks["burst"], "unit": "TFLOP/s",
                    "frac": tf / peaks["burst"], "frac_burst": tf / peaks["burst"], "frac_sustained": tf / peaks["sustained"],
                    "launches_per_step": acc[5][1] // n_prof})
    if 3 in acc and acc[3][0] > 0:
        t = acc[3][0] / n_prof * 1e-3
        n_norm = acc[3][1] // n_prof
        gbs = 6.0 * f["tokens"] * cfg["d_model"] * n_norm / t / 1e9
        out.append({"kernel": "norm_kernel", "bound": "hbm", "achieved": gbs, "peak": peaks["hbm"], "unit": "GB/s",
                    "frac": gbs / peaks["hbm"], "launches_per_step": n_norm,
                    "note": "6 bytes per element and launch; head and embed norms touch fewer rows, so this is an upper bound on bytes"})
    return out


def gemm_algorithmic_bytes(cfg, shapes):
    """Algorithmic HBM bytes of all GEMM launches of one forward pass: every operand read once, every output written
    once (bf16 activations and weights; the fp32 residual stream is read and written by proj and fc2; the embedding
    reads the patch operand and writes fp32)."""
    d, I, L = cfg["d_model"], cfg["d_mlp"], cfg["n_layers"]
    f = flops_of(cfg, shapes)
    T = f["tokens"]
    up_n = (2 if cfg["mlp"] == 1 else 1) * I
    per_layer = (2 * T * d + 2 * 3 * d * d + 2 * T * 3 * d) + (2 * T * d + 2 * d * d + 8 * T * d) \
        + (2 * T * d + 2 * up_n * d + 2 * T * I) + (2 * T * I + 2 * d * I + 8 * T * d)
    total = L * per_layer
    if cfg["family"] == 2:
        total += sum(2 * s[0] * cfg["in_channels"] + 2 * s[0] * d + 2 * s[0] * d + 4 * ((s[0] + 1) // 2) * d for s in shapes)
        total += 2 * 3 * cfg["in_channels"] * d + 2 * 3 * d * d
    else:
        k = S.configs.embed_k(cfg)
        total += (T * k * 2) + 2 * k * d + 4 * T * d
    if cfg["head"]:
        kin = 4 * d if cfg["head"] == 2 else d
        r, hh, do = f["out_rows"], cfg["d_head_hidden"], cfg["d_out"]
        total += 2 * r * kin + 2 * kin * hh + 2 * r * hh + 2 * r * hh + 2 * hh * do + 2 * r * do
    return total


def profile_traffic(config, micro_batch):
    """DRAM bytes per GEMM launch (read + write, averaged over the GEMM launches of one forward pass) from the ncu
    launch list of this workload, if a summary of it is committed under profiles/: the summary carries a line
    `gemm_dram_bytes_per_launch = <bytes>`.  None when there is no capture of this workload."""
    path = os.path.join(ROOT, "profiles", f"launches_{config}_mb{micro_batch}.md")
    try:
        with open(path) as fh:
            for ln in fh:
                if ln.strip().startswith("gemm_dram_bytes_per_launch"):
                    return float(ln.split("=")[1].split()[0]), os.path.relpath(path, ROOT)
    except (OSError, ValueError, IndexError):
        pass
    return None, None


def run_sweep(main_enc, main_cfg_name, sampler):
    """The sweep of the default run: every point timed for at least 10 steps and at least 1 s of device time, each with
    the clock record of its own timed region."""
    import gc
    import torch
    import paper_2609_31551_b200 as P
    points = []
    for cfg_name, plan in SWEEP:
        if cfg_name == main_cfg_name:
            enc, w = main_enc, None
        else:
            cfg = S.get_config(cfg_name)
            w = S.make_weights(cfg)
            enc = P.Encoder(cfg, P.weights_to_device(w))
            del w
        for mb, budgets in plan:
            cfg, shapes, seed = workload(cfg_name, mb)
            pt = Point(enc, cfg, shapes, seed)
            for b in budgets:
                r = time_point(pt, b, sampler, min_steps=10, min_seconds=1.0)
                points.append(dict(config=cfg_name, micro_batch=mb, sm_budget=b if b else "all", sum_s2=pt.f["sum_s2"], **r))
            del pt
        if enc is not main_enc:
            enc.close()
            del enc
        gc.collect()
        torch.cuda.empty_cache()
    return points


def config_of(args, n_items, tokens, world):
    """The `config` object of a line: the same for both arms (the reference arm times the oracle on this workload)."""
    return {"workload": f"{args.config} micro-batch {args.micro_batch}", "items_per_step": n_items,
            "tokens_per_step": tokens, "sm_budget": args.sm_budget if args.sm_budget else "all",
            "l2": "working set (weights + activations) larger than L2; no flush",
            "parallelism": "replicas" if world > 1 else "single",
            "launch": ("cuda graph replay" if args.graph else "one launch per kernel") + (", split K" if args.split_k else "")}


# ------------------------------------------------------------------ reference arm: the oracle on host cores
def run_reference(args):
    import torch
    from oracle import encoder_oracle as O
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg, shapes, seed = workload(args.config, args.micro_batch)
    sample_shapes = shapes[:1]          # bounded sample: the first item of the micro-batch
    w = S.make_weights(cfg)
    items = S.make_items(cfg, sample_shapes, seed)
    f = flops_of(cfg, sample_shapes)
    for _ in range(args.warmup):
        O.encode_microbatch(cfg, w, items)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        O.encode_microbatch(cfg, w, items)
    dt = (time.perf_counter() - t0) / args.steps
    val = f["tokens"] / dt
    line = {"impl": "reference", "metric": "encoder_tokens_per_sec", "value": val, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(args, len(shapes), sum(S.tokens_per_item(cfg, s) for s in shapes),
                                int(os.environ.get("WORLD_SIZE", "1"))),
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": torch.get_num_threads(), "kind": "oracle",
                             "sample": f"each step encodes 1 item ({f['tokens']} tokens) of the {args.config} micro-batch "
                                       "on the host cores (bounded sample)"},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------ CUDA arm
def run_cuda(args):
    import torch
    import paper_2609_31551_b200 as P
    from paper_2609_31551_b200 import replicas as R

    world, rank, local_rank = R.world()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the encoder has no CPU fallback")
    torch.cuda.set_device(local_rank)
    R.init("nccl", torch.device("cuda", local_rank))

    cfg, shapes, seed = workload(args.config, args.micro_batch, seed_shift=R.rank_seed_shift(rank))
    w = S.make_weights(cfg)
    enc = P.Encoder(cfg, P.weights_to_device(w))
    items = S.make_items(cfg, shapes, seed)
    data, offsets = P.pack_items(items)
    cu = np.concatenate([[0], np.cumsum([S.tokens_per_item(cfg, s) for s in shapes])]).astype(np.int32)
    cu_dev = torch.from_numpy(cu).cuda()
    f = flops_of(cfg, shapes)
    T = f["tokens"]
    budget = args.sm_budget
    if args.split_k:
        enc.set_split_k(True)          # before any workspace is sized
    if args.norm_fold:
        enc.set_norm_fold(True)
    if args.graph:
        # the launch-overhead path: captured forward passes need a stream of their own
        torch.cuda.set_stream(torch.cuda.Stream())
        enc.set_graph_mode(True)
    stream = torch.cuda.current_stream()
    out = torch.empty((f["out_rows"], cfg["d_out"]), dtype=torch.bfloat16, device="cuda")

    def step():
        enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev, sm_budget=budget, out=out)

    def barrier():
        torch.cuda.synchronize()
        R.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    enc.status()

    # ---- value: inputs resident in HBM
    sampler = ClockSampler(local_rank).start()
    time.sleep(0.3)                    # the sampler's first line
    barrier()
    mark0 = sampler.mark()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    enc.status()
    launches = enc.last_launch_count() * args.steps

    # ---- e2e: host buffers, copies inside the timed region, double-buffered
    host_in = torch.empty(data.numel(), dtype=torch.bfloat16, pin_memory=True)
    host_in.copy_(data.cpu())
    host_out = [torch.empty(out.shape, dtype=torch.bfloat16, pin_memory=True) for _ in range(2)]
    dev_in = [torch.empty_like(data) for _ in range(2)]
    dev_out = [torch.empty_like(out) for _ in range(2)]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_done = [torch.cuda.Event() for _ in range(2)]
    ev_free_in = [torch.cuda.Event() for _ in range(2)]
    ev_free_out = [torch.cuda.Event() for _ in range(2)]

    def e2e_loop(n):
        for i in range(n):
            b = i & 1
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_free_in[b])
                dev_in[b].copy_(host_in, non_blocking=True)
                ev_in[b].record(s_in)
            stream.wait_event(ev_in[b])
            if i >= 2:
                stream.wait_event(ev_free_out[b])
            enc.encode_microbatch(dev_in[b], shapes, offsets, cu, cu_seqlens_dev=cu_dev, sm_budget=budget, out=dev_out[b])
            ev_done[b].record(stream)
            ev_free_in[b].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[b])
                host_out[b].copy_(dev_out[b], non_blocking=True)
                ev_free_out[b].record(s_out)

    e2e_loop(2)
    barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    e2e_loop(args.steps)
    s_out.wait_stream(stream)
    t1.record(s_out)
    barrier()
    ms_e2e = t0.elapsed_time(t1)
    clocks = sampler.summary(mark0, sampler.mark())      # the two timed regions (resident and end-to-end)
    h2d = data.numel() * 2
    d2h = out.numel() * 2

    # ---- per-kernel-class timing (separate pass over the same workload, events inside the library)
    enc.enable_timing(True)
    acc = {}
    n_prof = max(5, min(args.steps, 20))
    mark1 = sampler.mark()
    for _ in range(n_prof):
        step()
        cls, kms = enc.timing_read()
        for c_, m_ in zip(cls.tolist(), kms.tolist()):
            a = acc.setdefault(c_, [0.0, 0])
            a[0] += m_; a[1] += 1
    enc.enable_timing(False)
    torch.cuda.synchronize()
    clocks_prof = sampler.summary(mark1, sampler.mark())

    (ms, ms_e2e), (total_tokens, launches, total_items, total_flops) = R.combine(
        [ms, ms_e2e], [float(T), float(launches), float(len(shapes)), float(f["total"])], device="cuda")
    launches = int(launches)

    if rank == 0:
        peaks = measured_peaks()
        gf = gemm_flops_by_class(cfg, shapes)
        gemm_ids = [2, 4, 6, 7, 8, 9]
        gemm_ms = sum(acc[c_][0] for c_ in gemm_ids if c_ in acc) / n_prof
        gemm_launch = sum(acc[c_][1] for c_ in gemm_ids if c_ in acc) / n_prof
        gemm_fl = sum(gf[c_] for c_ in gemm_ids)
        achieved = gemm_fl / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
        traffic, traffic_src = profile_traffic(args.config, args.micro_batch) if not budget else (None, None)
        gemm_bytes = gemm_algorithmic_bytes(cfg, shapes)
        names = {0: "prep", 1: "embed_gather", 2: "gemm_embed", 3: "norm", 4: "gemm_qkv", 5: "attention", 6: "gemm_proj",
                 7: "gemm_fc1", 8: "gemm_fc2", 9: "gemm_head"}
        breakdown = {}
        for c_, (tm, cnt) in sorted(acc.items()):
            ent = {"ms_per_step": round(tm / n_prof, 4), "launches_per_step": cnt // n_prof}
            if c_ in gf and tm > 0:
                ent["tflops"] = round(gf[c_] / (tm / n_prof * 1e-3) / 1e12, 1)
            breakdown[names.get(c_, str(c_))] = ent
        step_ms = ms / args.steps
        line = {
            "metric": "encoder_tokens_per_sec", "value": total_tokens * args.steps / (ms * 1e-3), "unit": "tokens/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": step_ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_of(args, len(shapes), T, world),
            "items_per_sec": total_items * args.steps / (ms * 1e-3),
            "tflops": total_flops / (step_ms * 1e-3) / 1e12,
            "frac_of_bf16_peak": {"burst_measured": f["total"] / (step_ms * 1e-3) / 1e12 / peaks["burst"],
                                  "sustained_measured": f["total"] / (step_ms * 1e-3) / 1e12 / peaks["sustained"],
                                  "source": peaks["source"]},
            "e2e": {"value": total_tokens * args.steps / (ms_e2e * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": launches,
            "clocks": clocks,
            "roofline": {"bound": "tensor", "kernel": "gemm_kernel (all GEMM launches of a step)", "achieved": achieved,
                         "peak": peaks["burst"], "unit": "TFLOP/s", "frac": achieved / peaks["burst"],
                         "peak_kind": f"burst bf16, {peaks['source']}",
                         "frac_burst": achieved / peaks["burst"], "frac_sustained": achieved / peaks["sustained"],
                         "peak_sustained": peaks["sustained"],
                         "traffic": traffic, "traffic_source": traffic_src,
                         "algorithmic_bytes_per_launch": gemm_bytes / max(gemm_launch, 1),
                         "launches_per_step": gemm_launch, "avg_launch_ms": gemm_ms / max(gemm_launch, 1),
                         "timed_steps": n_prof, "clocks": clocks_prof},
            "roofline_other": other_rooflines(cfg, shapes, f, acc, n_prof, peaks),
            "kernel_breakdown": breakdown,
        }
        default_point = args.config == "c1" and args.micro_batch == 32 and not budget and not args.graph and not args.split_k
        if world == 1 and default_point and not args.no_sweep:
            line["sweep"] = run_sweep(enc, args.config, sampler)
            line["sweep_note"] = ("each point: 3 warm-up steps, then >= 10 steps and >= 1 s of device time between CUDA "
                                  "events, inputs resident, with the clock record of its own timed region; fractions are "
                                  "of the measured burst / sustained bf16 peaks")
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(cfg, w, shapes, seed)
        sampler.stop()
        print(json.dumps(line))
    else:
        sampler.stop()
    R.finish()


def cpu_baseline(cfg, w, shapes, seed):
    """The oracle, as it stands, on one item of the workload (a bounded sample of the same step)."""
    import torch
    from oracle import encoder_oracle as O
    items = S.make_items(cfg, shapes[:1], seed)
    f1 = flops_of(cfg, shapes[:1])
    t0 = time.perf_counter()
    n = 0
    while True:
        O.encode_microbatch(cfg, w, items)
        n += 1
        if time.perf_counter() - t0 > 10.0 or n >= 8:
            break
    dt = (time.perf_counter() - t0) / n
    return {"value": f1["tokens"] / dt, "unit": "tokens/s", "cores": torch.get_num_threads(), "kind": "oracle",
            "sample": f"{n} x 1 item ({f1['tokens']} tokens, {f1['total'] / 1e9:.0f} GFLOP fp64) of the step's micro-batch",
            "gflops": f1["total"] / dt / 1e9}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--config", default="c1", choices=["c0", "c1", "c2", "c3", "c4"])
    ap.add_argument("--micro-batch", type=int, default=32)
    ap.add_argument("--sm-budget", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true",
                    help="skip the micro-batch x sm_budget sweep that the default run (c1, micro-batch 32, 1 GPU) appends")
    ap.add_argument("--split-k", action="store_true",
                    help="split the K loop of the residual GEMMs when a micro-batch has fewer tiles than SMs (latency path)")
    ap.add_argument("--norm-fold", action="store_true",
                    help="fold the blocks' normalisations into the GEMMs around them instead of one kernel per norm1 / norm2")
    ap.add_argument("--graph", action="store_true",
                    help="replay captured forward passes (CUDA graphs): the launch-overhead path for small micro-batches")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
