"""Multi-GPU runs are independent replicas: items of a micro-batch never interact and the forward pass has no
exchange step, so ranks share nothing on the data path.  torch.distributed is used only to line the ranks up
and to combine their measurements (slowest rank's time, summed work)."""
from __future__ import annotations
import os
import torch
import torch.distributed as dist


def world():
    return int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0"))


def init(backend: str, device=None):
    ws, _, _ = world()
    if ws > 1 and not dist.is_initialized():
        if device is not None:
            dist.init_process_group(backend, device_id=device)
        else:
            dist.init_process_group(backend)


def rank_seed_shift(rank: int) -> int:
    """Each replica draws its own micro-batches."""
    return 1000 * rank


def combine(ms_list, sums_list, device="cpu"):
    """ms_list: per-rank durations -> max over ranks; sums_list: per-rank work counters -> sum over ranks."""
    ws, _, _ = world()
    ms = torch.tensor(list(ms_list), dtype=torch.float64, device=device)
    sm = torch.tensor(list(sums_list), dtype=torch.float64, device=device)
    if ws > 1:
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
        dist.all_reduce(sm, op=dist.ReduceOp.SUM)
    return ms.tolist(), sm.tolist()


def barrier():
    ws, _, _ = world()
    if ws > 1:
        dist.barrier()


def finish():
    if dist.is_initialized():
        dist.destroy_process_group()
