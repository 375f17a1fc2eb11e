"""Co-residency of the Encode stage with a "local prefill" neighbour on one GPU (Section 3.4).

The paper gives the encoder a share of the SMs and the co-located prefill worker the rest, and picks the share from a
table so that encoding is slowed by at most 20 %.  Here the share is the `sm_budget` argument of every call: the
encoder's persistent kernels launch `sm_budget` CTAs (each fills an SM: its shared-memory request excludes a second
one), and a neighbour that launches `sm_total - sm_budget` CTAs of the same kind fits beside it, so the two never
queue behind one another for SMs.  What they still share is L2 and HBM.  This module measures that remaining
interference: encode latency at budget N alone, then with a stream of large GEMMs (the synthetic prefill: a
compute-bound bf16 matrix product, like the projections of a language-model prefill step) running on the other
SMs, and the neighbour's own slow-down.

    python -m paper_2609_31551_b200.coresidency --config c1 --micro-batch 8

The neighbour's kernels never wait for the encoder's or the reverse: they are independent launches on two streams."""
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


class PrefillNeighbour:
    """A stream of out = A W^T products (M x N x K, bf16) on `sm_budget` SMs of its own stream."""

    def __init__(self, m: int = 4096, n: int = 8192, k: int = 8192):
        g = torch.Generator(device="cuda").manual_seed(7)
        self.a = (torch.randn(m, k, device="cuda", generator=g) * 0.05).bfloat16()
        self.w = (torch.randn(n, k, device="cuda", generator=g) * 0.05).bfloat16()
        self.bias = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
        self.out = torch.empty(m, n, dtype=torch.bfloat16, device="cuda")
        self.status = torch.zeros(4, dtype=torch.int32, device="cuda")
        self.flops = 2.0 * m * n * k
        self.stream = torch.cuda.Stream()

    def enqueue(self, count: int, sm_budget: int):
        for _ in range(count):
            B.kernel_gemm(self.a, self.w, self.bias, sm_budget=sm_budget, stream=self.stream, out=self.out, status=self.status)


def _encode_ms(enc, batch, sm_budget, reps, stream):
    data, shapes, offsets, cu, cu_dev, out, ws = batch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(reps):
        enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev, sm_budget=sm_budget, out=out, workspace=ws,
                              stream=stream)
    e1.record(stream)
    return e0, e1


def measure(config: str, micro_batch: int, levels=(0.3, 0.5, 0.7), reps: int = 5, neighbour_shape=(4096, 8192, 8192),
            partition: str = "grid"):
    """-> list of dicts, one per SM level: encode latency alone / beside the neighbour, and the neighbour's rate.

    partition = "grid": both sides bound their SM use by their grid sizes (`sm_budget`) on ordinary streams.
    partition = "green": eas_sm_partition splits the SMs into two driver-enforced sets (green contexts) and each side
    runs on its set's stream; the level is rounded up to the driver's granularity."""
    cfg = S.get_config(config)
    enc = B.Encoder(cfg, B.weights_to_device(S.make_weights(cfg)))
    shapes = S.draw_item_shapes(cfg, micro_batch, 3000 + micro_batch)
    items = S.make_items(cfg, shapes, 2000 + micro_batch)
    data, offsets = B.pack_items(items)
    cu = np.concatenate([[0], np.cumsum([S.tokens_per_item(cfg, s) for s in shapes])]).astype(np.int32)
    cu_dev = torch.from_numpy(cu).cuda()
    out = torch.empty((enc.out_rows(cu), cfg["d_out"]), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(enc.workspace_bytes(int(cu[-1]), len(shapes)) + 1024, dtype=torch.uint8, device="cuda")
    batch = (data, shapes, offsets, cu, cu_dev, out, ws)
    sm_total = torch.cuda.get_device_properties(0).multi_processor_count
    nb = PrefillNeighbour(*neighbour_shape)
    enc_stream = torch.cuda.Stream()
    torch.cuda.synchronize()

    def encode_alone(budget, stream=None):
        stream = stream or enc_stream
        best = float("inf")
        for _ in range(3):              # the first passes also bring the clocks up after an idle stretch: keep the best
            e0, e1 = _encode_ms(enc, batch, budget, reps, stream)
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1) / reps)
        return best

    def neighbour_alone(budget, count):
        nb.enqueue(2, budget)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(nb.stream)
        nb.enqueue(count, budget)
        e1.record(nb.stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / count

    rows = []
    exclusive = encode_alone(0)
    plain_streams = (enc_stream, nb.stream)
    for f in levels:
        n_enc = max(2, int(sm_total * f) // 2 * 2)
        n_nb = sm_total - n_enc
        part = None
        if partition == "green":
            part = B.SmPartition(n_enc)
            n_enc, n_nb = part.sm_count(0), part.sm_count(1)
            enc_stream, nb.stream = part.stream(0), part.stream(1)
        alone = encode_alone(n_enc, enc_stream)
        nb_ms = neighbour_alone(n_nb, 4)
        # enough neighbour launches to cover the encoder's timed region with margin on both sides
        count = int(np.ceil((reps + 2) * alone / nb_ms)) + 4
        n0, n1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0.record(nb.stream)
        nb.enqueue(count, n_nb)
        n1.record(nb.stream)
        enc_stream.wait_event(n0)                                            # start beside the neighbour's first product
        _encode_ms(enc, batch, n_enc, 1, enc_stream)
        e0, e1 = _encode_ms(enc, batch, n_enc, reps, enc_stream)
        torch.cuda.synchronize()
        enc.status(enc_stream)
        beside = e0.elapsed_time(e1) / reps
        nb_beside = n0.elapsed_time(n1) / count
        if part is not None:
            enc_stream, nb.stream = plain_streams
            part.close()
        rows.append({"partition": partition, "sm_encode": n_enc, "sm_neighbour": n_nb, "encode_ms_exclusive": exclusive, "encode_ms_alone": alone,
                     "encode_ms_beside_neighbour": beside, "inflation": beside / alone,
                     "vs_exclusive": beside / exclusive,
                     "neighbour_tflops_alone": nb.flops / (nb_ms * 1e-3) / 1e12,
                     "neighbour_tflops_beside_encoder": nb.flops / (nb_beside * 1e-3) / 1e12})
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="c1")
    ap.add_argument("--micro-batch", type=int, default=8)
    ap.add_argument("--levels", default="0.3,0.5,0.7")
    ap.add_argument("--partition", default="grid", choices=("grid", "green"))
    a = ap.parse_args()
    for r in measure(a.config, a.micro_batch, tuple(float(x) for x in a.levels.split(",")), partition=a.partition):
        print(json.dumps(r))


if __name__ == "__main__":
    main()
