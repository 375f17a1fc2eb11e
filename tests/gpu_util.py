"""Helpers for the GPU parity tests: run the CUDA encoder through the C ABI binding and the fp64
oracle on the same seeded inputs, and compare per output embedding (row)."""
import json
import os

import numpy as np
import torch

import eas_synth as S

REL_TOL = 1e-2     # max over output rows of ||gpu - ref||_2 / ||ref||_2
ABS_TOL = 5e-2     # max |gpu - ref| over all output elements


def item_shape(cfg, it):
    if cfg["family"] == 2:
        return (it.shape[0], it.shape[1], 1)
    if it.ndim == 4:
        return (it.shape[0], it.shape[2], it.shape[3])
    return (1, it.shape[1], it.shape[2])


def cu_seqlens_of(cfg, items):
    cu = [0]
    for it in items:
        cu.append(cu[-1] + S.tokens_per_item(cfg, item_shape(cfg, it)))
    return np.asarray(cu, dtype=np.int32)


def run_gpu(enc, cfg, items, sm_budget=0):
    """-> float64 ndarray [out_rows, d_out] from the CUDA path (synchronised, device status checked)."""
    import paper_2609_31551_b200 as P
    data, offsets = P.pack_items(items)
    shapes = [item_shape(cfg, it) for it in items]
    cu = cu_seqlens_of(cfg, items)
    out = enc.encode_microbatch(data, shapes, offsets, cu, sm_budget=sm_budget)
    enc.status()
    return out.float().cpu().numpy().astype(np.float64), out


def errors(gpu, ref):
    diff = gpu - ref
    row_rel = np.linalg.norm(diff, axis=1) / np.maximum(np.linalg.norm(ref, axis=1), 1e-30)
    return float(row_rel.max()), float(np.abs(diff).max())


def assert_parity(gpu, ref, what=""):
    assert gpu.shape == ref.shape, (gpu.shape, ref.shape)
    assert np.isfinite(gpu).all(), f"{what}: non-finite GPU output"
    rel, mabs = errors(gpu, ref)
    assert rel <= REL_TOL and mabs <= ABS_TOL, f"{what}: row-rel {rel:.3e} (tol {REL_TOL}), max-abs {mabs:.3e} (tol {ABS_TOL})"
    return rel, mabs


MARGIN_LOG = os.environ.get("EAS_PARITY_LOG",
                            os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "gpurun_out",
                                         "parity_margins.jsonl"))


def record_margin(case, profile, seed, rel, mabs, **extra):
    """Appends one line (case, weight profile, input seed, row-relative error, max-abs error) to the margin log, so
    that a test run leaves the measured distance to the tolerances on record.  Never fails a test."""
    try:
        os.makedirs(os.path.dirname(MARGIN_LOG), exist_ok=True)
        with open(MARGIN_LOG, "a") as f:
            f.write(json.dumps(dict(case=case, profile=profile, seed=seed, row_rel=rel, max_abs=mabs,
                                    rel_tol=REL_TOL, abs_tol=ABS_TOL, **extra)) + "\n")
    except OSError:
        pass
