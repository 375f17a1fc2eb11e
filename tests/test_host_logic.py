"""CPU-only checks: the C ABI library loads and exports every symbol the header declares, host-side
argument validation answers without a GPU, the generators and the replica bookkeeping behave."""
import ctypes
import os
import re
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

import eas_synth as S

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_31551_b200.build import build_library
    build_library()
    import paper_2609_31551_b200 as P
    return P.load_library()


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "eas_encoder.h")).read()
    declared = set(re.findall(r"\b(eas_[a-z_0-9]+)\s*\(", header))
    declared -= {"eas_status"}
    assert len(declared) >= 15
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in include/eas_encoder.h but not exported"
    from paper_2609_31551_b200.binding import EXPORTED_SYMBOLS
    assert declared == set(EXPORTED_SYMBOLS)
    header2 = open(os.path.join(ROOT, "include", "eas_serving.h")).read()
    declared2 = set(re.findall(r"\b(eas_[a-z_0-9]+)\s*\(", header2))
    from paper_2609_31551_b200.serving import SERVING_SYMBOLS
    assert declared2 == set(SERVING_SYMBOLS)
    for name in sorted(declared2):
        assert hasattr(lib, name), f"{name} is declared in include/eas_serving.h but not exported"


def test_arena_size_and_config_validation_run_on_the_host(lib):
    from paper_2609_31551_b200.binding import arch_struct
    for name in ("c0", "c1", "c2", "c3", "c4"):
        cfg = S.get_config(name)
        n = lib.eas_encoder_weight_arena_bytes(ctypes.byref(arch_struct(cfg)))
        assert n > 0
    # RoPE models re-lay every qkv matrix and every gate/up pair into the arena
    c2 = S.get_config("c2")
    d, I, L = c2["d_model"], c2["d_mlp"], c2["n_layers"]
    n = lib.eas_encoder_weight_arena_bytes(ctypes.byref(arch_struct(c2)))
    assert n >= L * (3 * d * d + 2 * I * d) * 2
    bad = S.get_config("c0", n_heads=3)        # 256 % 3 != 0
    assert lib.eas_encoder_weight_arena_bytes(ctypes.byref(arch_struct(bad))) == 0
    assert b"n_heads" in lib.eas_last_error()
    bad = S.get_config("c0", n_heads=2)        # head_dim 128 unsupported
    assert lib.eas_encoder_weight_arena_bytes(ctypes.byref(arch_struct(bad))) == 0


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_create_fails_loudly_without_a_gpu(lib):
    from paper_2609_31551_b200.binding import arch_struct, Weights, Tensor
    cfg = S.get_config("c0")
    arena_bytes = lib.eas_encoder_weight_arena_bytes(ctypes.byref(arch_struct(cfg)))
    t = (Tensor * 1)()
    t[0].name = b"x"
    t[0].dev_ptr = 16
    w = Weights(t, 1, ctypes.c_void_p(1024), arena_bytes)
    h = ctypes.c_void_p()
    st = lib.eas_encoder_create(ctypes.byref(arch_struct(cfg)), ctypes.byref(w), ctypes.byref(h))
    assert st != 0 and not h.value
    assert len(lib.eas_last_error()) > 0


def test_generators_are_seeded_and_bf16_exact():
    cfg = S.get_config("c0")
    a, b = S.make_weights(cfg), S.make_weights(cfg)
    assert all(np.array_equal(a[k], b[k]) for k in a)
    for v in a.values():
        assert np.array_equal(S.round_to_bf16(v), v)
    sharp = S.make_weights(cfg, profile="sharp")
    d = cfg["d_model"]
    assert np.allclose(sharp["blk0.qkv.w"][: 2 * d], S.round_to_bf16(2 * a["blk0.qkv.w"][: 2 * d]))
    assert np.array_equal(sharp["blk0.qkv.w"][2 * d:], a["blk0.qkv.w"][2 * d:])
    shapes = S.draw_item_shapes(S.get_config("c2"), 64, 3206)
    assert all(h % 28 == 0 and w % 28 == 0 and 224 <= h <= 1344 and 224 <= w <= 1344 for _, h, w in shapes)
    assert len({s for s in shapes}) > 30
    clips = S.draw_item_shapes(S.get_config("c3"), 32, 3303)
    assert {f for f, _, _ in clips} <= {16, 32, 64}
    assert S.tokens_per_item(S.get_config("c3"), (64, 448, 448)) == 32768
    assert S.tokens_per_item(S.get_config("c1"), (1, 336, 336)) == 577
    assert S.out_tokens_per_item(S.get_config("c1"), (1, 336, 336)) == 576
    assert S.tokens_per_item(S.get_config("c4"), (3000, 128, 1)) == 1500


def test_bench_flop_model_matches_the_per_item_totals():
    sys.path.insert(0, ROOT)
    import bench
    c1 = S.get_config("c1")
    f = bench.flops_of(c1, [(1, 336, 336)])
    assert abs(f["total"] / 1e9 - 406) < 3             # 406 GFLOP per image
    c4 = S.get_config("c4")
    assert abs(bench.flops_of(c4, [(3000, 128, 1)])["total"] / 1e12 - 2.27) < 0.03
    c3 = S.get_config("c3")
    assert abs(bench.flops_of(c3, [(16, 448, 448)])["total"] / 1e12 - 24.9) < 0.3
    by_class = bench.gemm_flops_by_class(c1, [(1, 336, 336)] * 3)
    assert abs(sum(by_class.values()) - bench.flops_of(c1, [(1, 336, 336)] * 3)["total"]) < 1e-6 * sum(by_class.values())


def _replica_worker(rank, world_size, port, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world_size), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    from paper_2609_31551_b200 import replicas as R
    R.init("gloo")
    R.barrier()
    ms, sums = R.combine([10.0 + rank, 5.0 - rank], [100.0 * (rank + 1), 7.0])
    q.put((rank, ms, sums, R.rank_seed_shift(rank)))
    R.finish()


def test_replica_bookkeeping_world_size_2_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_replica_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, sums, shift in res:
        assert ms == [11.0, 5.0]            # slowest rank per measurement
        assert sums == [300.0, 14.0]        # work adds up over replicas
        assert shift == 1000 * rank         # every replica draws its own micro-batches


def test_flop_model_against_closed_forms():
    """The benchmark's algorithmic FLOP count against the per-item figures that follow from the layer shapes:
    c1 704 MFLOP per token (406 GFLOP per 336x336 image), c4 2.27 TFLOP per 3000-frame clip; attention is 4 d S^2 per
    item and layer; nothing is counted for padding."""
    from paper_2609_31551_b200 import measure as M
    c1 = S.get_config("c1")
    f = M.flops_of(c1, [(1, 336, 336)])
    assert f["tokens"] == 577 and f["out_rows"] == 576
    assert abs(f["total"] / 1e9 - 406) < 2
    lin = 24 * 577 * (8 * 1024 * 1024 + 4 * 1024 * 4096)
    assert f["attention"] == 24 * 4 * 1024 * 577 * 577
    assert f["linear"] == lin + 2 * 576 * 588 * 1024 + 2 * 576 * (1024 * 4096 + 4096 * 4096)
    two = M.flops_of(c1, [(1, 336, 336)] * 2)
    assert two["total"] == 2 * f["total"]                       # items never interact
    c4 = S.get_config("c4")
    f4 = M.flops_of(c4, [(3000, 128, 1)])
    assert f4["tokens"] == 1500 and abs(f4["total"] / 1e12 - 2.27) < 0.02
    assert M.flops_of(c4, [(2999, 128, 1)])["tokens"] == 1500    # odd frame counts: ceil(n / 2) tokens
    c3 = S.get_config("c3")
    f3 = M.flops_of(c3, [(16, 448, 448)])
    assert f3["tokens"] == 8192 and abs(f3["total"] / 1e12 - 24.9) < 0.2
    by = M.gemm_flops_by_class(c1, [(1, 336, 336)])
    assert sum(by.values()) == f["total"]


def test_reference_arm_prints_the_contract_line():
    """`bench.py --impl reference` (the oracle on host cores) prints one JSON line with the keys the benchmark contract
    names and the same `config` object the CUDA arm prints for the same arguments."""
    import json
    import subprocess
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "c0",
                          "--micro-batch", "4", "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in line, key
    assert line["impl"] == "reference" and line["dtype"] == "f64" and line["vs_baseline"] is None
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    import argparse
    import bench
    args = argparse.Namespace(config="c0", micro_batch=4, sm_budget=0, graph=False, split_k=False)
    assert line["config"] == bench.config_of(args, 4, 784, 1)
