"""Measurement helpers shared by bench.py and sweep.py: the FLOP model of a forward pass, the workload recipe, the
measured peaks, a clock / throttle-reason sampler, and the timing of one (config, micro-batch, sm_budget) point.
Nothing here computes any part of the forward pass."""
from __future__ import annotations
import json
import math
import os
import statistics
import subprocess
import threading

import numpy as np

import eas_synth as S

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


# ------------------------------------------------------------------ algorithmic work (real tokens only)
def flops_of(cfg, shapes):
    """Algorithmic FLOPs of one forward pass: 2*M*N*K per linear map, 4*d*S^2 per item and layer for attention."""
    d, I, L = cfg["d_model"], cfg["d_mlp"], cfg["n_layers"]
    seqs = [S.tokens_per_item(cfg, s) for s in shapes]
    T = sum(seqs)
    mlp = (6 if cfg["mlp"] == 1 else 4) * d * I
    lin = L * T * (8 * d * d + mlp)
    attn = L * 4 * d * sum(s * s for s in seqs)
    if cfg["family"] == 2:
        emb = sum(2 * s[0] * 3 * cfg["in_channels"] * d + 2 * ((s[0] + 1) // 2) * 3 * d * d for s in shapes)
    else:
        emb = 2 * (T - (len(shapes) if cfg["has_cls"] else 0)) * S.configs.embed_k(cfg) * d
    head = 0
    out_rows = sum(S.out_tokens_per_item(cfg, s) for s in shapes)
    if cfg["head"] == 1:
        head = 2 * out_rows * (d * cfg["d_head_hidden"] + cfg["d_head_hidden"] * cfg["d_out"])
    elif cfg["head"] == 2:
        head = 2 * out_rows * (4 * d * cfg["d_head_hidden"] + cfg["d_head_hidden"] * cfg["d_out"])
    return dict(total=lin + attn + emb + head, linear=lin + emb + head, attention=attn, tokens=T, out_rows=out_rows,
                sum_s2=sum(s * s for s in seqs))


def gemm_flops_by_class(cfg, shapes):
    """Algorithmic FLOPs per kernel class of the GEMMs and attention (keys = EAS_KC_* ids)."""
    d, I, L = cfg["d_model"], cfg["d_mlp"], cfg["n_layers"]
    f = flops_of(cfg, shapes)
    T = f["tokens"]
    up = (4 if cfg["mlp"] == 1 else 2) * d * I
    emb = f["linear"] - L * T * (8 * d * d + (6 if cfg["mlp"] == 1 else 4) * d * I)
    head = 0
    if cfg["head"]:
        kin = 4 * d if cfg["head"] == 2 else d
        head = 2 * f["out_rows"] * (kin * cfg["d_head_hidden"] + cfg["d_head_hidden"] * cfg["d_out"])
    return {2: emb - head, 4: L * T * 6 * d * d, 6: L * T * 2 * d * d, 7: L * T * up, 8: L * T * 2 * d * I, 9: head,
            5: f["attention"]}


def workload(cfg_name, mb, seed_shift=0):
    """The seeded synthetic workload of a (config, micro-batch) point: (config, item shapes, input seed)."""
    cfg = S.get_config(cfg_name)
    ci = S.configs.CONFIG_INDEX[cfg_name]
    lg = int(np.log2(max(mb, 1)))
    shapes = S.draw_item_shapes(cfg, mb, 3000 + 100 * ci + lg + seed_shift)
    return cfg, shapes, 2000 + 100 * ci + lg + seed_shift


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm=p["hbm_gbs"], burst=p["bf16_tflops"], sustained=p["bf16_tflops_sustained"], source="measured")
    return dict(hbm=6650.0, burst=1590.0, sustained=1400.0, source="fallback")


# ------------------------------------------------------------------ clocks during a timed region
class ClockSampler:
    """Samples SM clock, power and throttle reasons with nvidia-smi while a timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index: int, period_ms: int = 100):
        self.gpu = gpu_index
        self.period_ms = period_ms
        self.proc = None
        self.lines = []
        self.lock = threading.Lock()

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", str(self.period_ms)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            with self.lock:
                self.lines.append(line.strip())

    def mark(self) -> int:
        """Index of the next sample: summary(mark_a, mark_b) covers what was sampled between two marks."""
        with self.lock:
            return len(self.lines)

    def summary(self, lo: int = 0, hi: int | None = None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        with self.lock:
            lines = list(self.lines[lo:hi])
        sm, mx, reasons, pw = [], [], set(), []
        for ln in lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); pw.append(float(parts[2]))
            except ValueError:
                continue
            for nm, val in zip(self.NAMES, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}

    def stop(self):
        if self.proc is None:
            return self.summary()
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        return self.summary()


# ------------------------------------------------------------------ one point of the metric
class Point:
    """A (config, micro-batch) workload resident on the device, ready to be stepped at any sm_budget."""

    def __init__(self, enc, cfg, shapes, seed):
        import torch
        from . import binding as B
        self.enc, self.cfg, self.shapes = enc, cfg, shapes
        items = S.make_items(cfg, shapes, seed)
        self.data, self.offsets = B.pack_items(items)
        self.cu = np.concatenate([[0], np.cumsum([S.tokens_per_item(cfg, s) for s in shapes])]).astype(np.int32)
        self.cu_dev = torch.from_numpy(self.cu).cuda()
        self.f = flops_of(cfg, shapes)
        self.out = torch.empty((self.f["out_rows"], cfg["d_out"]), dtype=torch.bfloat16, device="cuda")

    def step(self, budget=0):
        self.enc.encode_microbatch(self.data, self.shapes, self.offsets, self.cu, cu_seqlens_dev=self.cu_dev,
                                   sm_budget=budget, out=self.out)


def time_point(point: Point, budget: int, sampler: ClockSampler | None, min_steps: int = 10, min_seconds: float = 1.0,
               warmup: int = 3, max_steps: int = 2000):
    """Times `point` at `budget` SMs: `warmup` untimed steps, then at least `min_steps` steps and at least
    `min_seconds` of device time between two CUDA events on the launching stream.  The clock record covers the timed
    region only.  Returns a dict (ms_per_step, steps, tokens/s, items/s, TFLOP/s, fractions of the measured peaks,
    clocks)."""
    import torch
    stream = torch.cuda.current_stream()
    for _ in range(max(warmup, 3)):
        point.step(budget)
    point.enc.status()
    # a short calibration pass decides how many steps make up min_seconds
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    c0.record(stream)
    for _ in range(2):
        point.step(budget)
    c1.record(stream)
    torch.cuda.synchronize()
    est_ms = max(c0.elapsed_time(c1) / 2, 1e-3)
    steps = int(min(max_steps, max(min_steps, math.ceil(min_seconds * 1e3 / est_ms))))
    lo = sampler.mark() if sampler is not None else 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(steps):
        point.step(budget)
    e1.record(stream)
    torch.cuda.synchronize()
    hi = sampler.mark() if sampler is not None else 0
    point.enc.status()
    ms = e0.elapsed_time(e1) / steps
    f, peaks = point.f, measured_peaks()
    tf = f["total"] / ms / 1e9
    res = {"ms_per_step": round(ms, 4), "steps": steps, "tokens": f["tokens"], "items": len(point.shapes),
           "tokens_per_s": round(f["tokens"] / ms * 1e3, 1), "items_per_s": round(len(point.shapes) / ms * 1e3, 2),
           "tflops": round(tf, 1), "frac_burst": round(tf / peaks["burst"], 4),
           "frac_sustained": round(tf / peaks["sustained"], 4), "attn_flop_share": round(f["attention"] / f["total"], 3)}
    if sampler is not None:
        res["clocks"] = sampler.summary(lo, hi)
    return res
