"""Drives the encoder the way the paper's Encode worker does: arrivals -> Poisson-gap micro-batcher (Section 3.2) ->
SM share from the lookup table (Section 3.4) -> eas_encode_microbatch -> deficit-counter routing with per-destination
envelope plan (Section 3.3).  Also the two start-up profiling steps: encode capacity C_E (Stage 1 of HAS: double B until
throughput saturates) and the SM table (latency sweep over SM levels x batch sizes, 20 % rule).

    python -m paper_2609_31551_b200.serve_sim --config c1 --rate 400 --requests 2000 --batch-bound 16

Device time comes from CUDA events around each forward pass; the queueing around it is simulated on that measured service
time (one encode worker, no host sleep), so the run is fast and deterministic for a seed."""
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

import eas_synth as S  # noqa: E402
from . import binding as B  # noqa: E402
from . import serving as SV  # noqa: E402


class EncodeWorker:
    """One encoder handle plus cached per-batch-size inputs; measures the device time of a forward pass."""

    def __init__(self, config: str, split_k: bool = False):
        self.cfg = S.get_config(config)
        self.enc = B.Encoder(self.cfg, B.weights_to_device(S.make_weights(self.cfg)))
        if split_k:                      # latency path for the small micro-batches of a lightly loaded worker
            self.enc.set_split_k(True)
        self._inputs = {}

    def _batch(self, n: int):
        if n not in self._inputs:
            shapes = S.draw_item_shapes(self.cfg, n, 3000 + n)
            items = S.make_items(self.cfg, shapes, 2000 + n)
            data, offsets = B.pack_items(items)
            cu = np.concatenate([[0], np.cumsum([S.tokens_per_item(self.cfg, s) for s in shapes])]).astype(np.int32)
            rows = [S.out_tokens_per_item(self.cfg, s) for s in shapes]
            self._inputs[n] = (data, shapes, offsets, cu, torch.from_numpy(cu).cuda(), rows)
        return self._inputs[n]

    def latency_ms(self, n: int, sm_budget: int = 0, reps: int = 3) -> float:
        data, shapes, offsets, cu, cu_dev, _ = self._batch(n)
        self.enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev, sm_budget=sm_budget)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            self.enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev, sm_budget=sm_budget)
        e1.record()
        torch.cuda.synchronize()
        self.enc.status()
        return e0.elapsed_time(e1) / reps

    def out_rows(self, n: int):
        return self._batch(n)[5]


def profile_encode_capacity(worker: EncodeWorker, max_batch: int = 64, saturation: float = 0.05):
    """C_E: double B until items/s improves by less than `saturation`.  Returns (C_E items/s, B at saturation, curve)."""
    curve, best, b = [], 0.0, 1
    while b <= max_batch:
        thr = b / worker.latency_ms(b) * 1e3
        curve.append((b, thr))
        if best > 0 and thr < best * (1 + saturation):
            return max(best, thr), b, curve
        best = max(best, thr)
        b *= 2
    return best, b // 2, curve


def build_sm_table(worker: EncodeWorker, sm_total: int, batches, levels=(0.1, 0.3, 0.5, 0.7, 0.9), tolerance: float = 0.2):
    """The paper's start-up sweep: encode-only latency at 5 SM levels x batch sizes, kept when within 20 % of exclusive."""
    sm_counts = [max(2, int(sm_total * f) // 2 * 2) for f in levels]
    excl = [worker.latency_ms(b, 0) for b in batches]
    lat = [[worker.latency_ms(b, sm) for b in batches] for sm in sm_counts]
    return SV.sm_table_build(sm_counts, list(batches), lat, excl, tolerance), sm_counts, lat, excl


def simulate(worker: EncodeWorker, rate: float, n_requests: int, batch_bound: int, offload: float, table=None,
             arrival_cv: float = 1.0, seed: int = 1, p: float = 0.6, max_age: float = 1.0, n_remote: int = 2):
    """One encode worker under synthetic arrivals (Poisson, or Gamma with the given coefficient of variation)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    shape = 1.0 / (arrival_cv ** 2)
    arrivals = np.cumsum(rng.gamma(shape, 1.0 / (rate * shape), size=n_requests))
    batches = SV.run_batcher(arrivals.tolist(), batch_bound, rate, p, max_age)
    num, den = SV.router_fraction(offload, 1000)
    decisions = SV.route(num, den, n_requests)
    lat_cache, free_at, done, sizes, budgets, req = {}, 0.0, [], [], [], 0
    remote_rr, transfers = 0, 0
    for when, size in batches:
        sm = SV.sm_table_lookup(table, size) if table is not None else 0
        key = (size, sm)
        if key not in lat_cache:
            lat_cache[key] = worker.latency_ms(size, sm) * 1e-3
        start = max(when, free_at)
        free_at = start + lat_cache[key]
        # destinations: 0 = the co-resident local prefill worker, 1.. = remote prefill workers (round-robin)
        dest = []
        for i in range(size):
            if decisions[req + i]:
                dest.append(1 + remote_rr % n_remote)
                remote_rr += 1
            else:
                dest.append(0)
        _, dest_rows = SV.envelope_plan(dest, worker.out_rows(size), 1 + n_remote)
        transfers += sum(1 for r in dest_rows if r > 0)
        done += [free_at - arrivals[req + i] for i in range(size)]
        req += size
        sizes.append(size)
        budgets.append(sm)
    done = np.asarray(done)
    return {"requests": n_requests, "rate": rate, "batch_bound": batch_bound, "gap_s": SV.kappa(batch_bound, p) / rate,
            "dispatches": len(batches), "mean_batch": float(np.mean(sizes)), "full_batches": float(np.mean(np.asarray(sizes) == batch_bound)),
            "throughput": n_requests / max(free_at - arrivals[0], 1e-9), "encode_latency_mean_s": float(done.mean()),
            "encode_latency_p99_s": float(np.quantile(done, 0.99)), "remote_fraction": float(np.mean(decisions)),
            "transfers": transfers, "mean_sm_budget": float(np.mean(budgets)) if table is not None else None}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="c1")
    ap.add_argument("--rate", type=float, default=400.0)
    ap.add_argument("--requests", type=int, default=2000)
    ap.add_argument("--batch-bound", type=int, default=16)
    ap.add_argument("--offload", type=float, default=0.7)
    ap.add_argument("--arrival-cv", type=float, default=1.0)
    ap.add_argument("--no-table", action="store_true")
    ap.add_argument("--split-k", action="store_true", help="latency path: split K in micro-batches with few tiles")
    a = ap.parse_args()
    w = EncodeWorker(a.config, split_k=a.split_k)
    sm_total = torch.cuda.get_device_properties(0).multi_processor_count
    ce, b_sat, curve = profile_encode_capacity(w)
    print(json.dumps({"capacity_items_per_s": ce, "saturation_batch": b_sat, "curve": curve}))
    table = None
    if not a.no_table:
        batches = [b for b in (1, 2, 4, 8, 16, 32, 64) if b <= a.batch_bound]
        table, sm_counts, lat, excl = build_sm_table(w, sm_total, batches)
        print(json.dumps({"sm_levels": sm_counts, "max_batch": [table.max_batch[i] for i in range(table.n_levels)],
                          "latency_ms": lat, "exclusive_ms": excl}))
    print(json.dumps(simulate(w, a.rate, a.requests, a.batch_bound, a.offload, table, a.arrival_cv)))


if __name__ == "__main__":
    main()
