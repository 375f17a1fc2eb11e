"""Throughput sweep of the encoder over micro-batch size and sm_budget (the table of the headline metric).

    python -m paper_2609_31551_b200.sweep --config c1 --micro-batches 1,2,4,8,16,32,64 --budgets 37,74,111,148

One JSON line per point.  Every point is measured `--repeats` times (default 3), each repeat being at least
`--min-steps` steps and `--min-seconds` of device time between CUDA events after 3 warm-up steps, with inputs (the
seeded synthetic workloads of eas_synth) resident in HBM and the SM clock / throttle reasons sampled during the
repeat.  The line gives the median repeat, the range over repeats, tokens/s, items/s, TFLOP/s and the fractions of the
measured bf16 peaks; a repeat whose clock record shows a thermal or hardware slowdown is flagged."""
from __future__ import annotations
import argparse
import json
import os
import statistics
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import eas_synth as S  # noqa: E402
from . import binding as B  # noqa: E402
from . import measure as M  # noqa: E402

BAD_REASONS = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="c1")
    ap.add_argument("--micro-batches", default="1,2,4,8,16,32,64")
    ap.add_argument("--budgets", default="37,74,111,148")
    ap.add_argument("--repeats", type=int, default=3)
    ap.add_argument("--min-steps", type=int, default=10)
    ap.add_argument("--min-seconds", type=float, default=0.5)
    ap.add_argument("--max-tokens", type=int, default=400000, help="skip points with more encoder tokens than this")
    a = ap.parse_args()
    import torch
    peaks = M.measured_peaks()
    cfg = S.get_config(a.config)
    w = S.make_weights(cfg)
    enc = B.Encoder(cfg, B.weights_to_device(w))
    del w
    sampler = M.ClockSampler(torch.cuda.current_device()).start()
    for mb in [int(x) for x in a.micro_batches.split(",")]:
        _, shapes, seed = M.workload(a.config, mb)
        T = sum(S.tokens_per_item(cfg, s) for s in shapes)
        if T > a.max_tokens:
            print(json.dumps({"config": a.config, "micro_batch": mb, "skipped": f"{T} tokens > --max-tokens"}))
            continue
        pt = M.Point(enc, cfg, shapes, seed)
        for budget in [int(x) for x in a.budgets.split(",")]:
            runs = [M.time_point(pt, budget, sampler, min_steps=a.min_steps, min_seconds=a.min_seconds) for _ in range(a.repeats)]
            runs.sort(key=lambda r: r["ms_per_step"])
            med = runs[len(runs) // 2]
            reasons = sorted(set(x for r in runs for x in r["clocks"]["reasons"]))
            mhz = [r["clocks"]["sm_mhz"] for r in runs if r["clocks"].get("sm_mhz")]
            line = dict(config=a.config, micro_batch=mb, sm_budget=budget, sum_s2=pt.f["sum_s2"], **med)
            line.update(repeats=len(runs), ms_min=runs[0]["ms_per_step"], ms_max=runs[-1]["ms_per_step"],
                        sm_mhz_median=statistics.median(mhz) if mhz else None, reasons=reasons,
                        rejected=bool(BAD_REASONS & set(reasons)), peaks=peaks["source"])
            line.pop("clocks", None)
            print(json.dumps(line), flush=True)
        del pt
    sampler.stop()


if __name__ == "__main__":
    main()
