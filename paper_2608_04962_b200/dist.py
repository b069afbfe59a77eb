"""Multi-process plumbing of the benchmark: one process per GPU, no data-path collective.

The hot path shards by sequence (every step is independent per sequence; weights are
replicated), so ranks only meet to bracket the timed region and to aggregate the result:
time = max over ranks, units = sum over ranks.
"""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def launch_plan(gpus: int, env=None):
    """What ``--gpus N`` asks of this process.  ("run", None): go ahead as the rank the environment says (a launcher
    started N ranks, or N == 1 and there is no launcher).  ("spawn", None): N > 1 and no launcher: the caller
    starts N ranks itself.  ("refuse", message): a launcher started a different number of ranks than N."""
    env = os.environ if env is None else env
    ws = env.get("WORLD_SIZE")
    if ws is None:
        return ("run", None) if gpus <= 1 else ("spawn", None)
    if int(ws) != int(gpus):
        return ("refuse", f"--gpus {gpus} but the launcher started WORLD_SIZE={ws} ranks: start "
                          f"--nproc-per-node {gpus}, or drop the launcher and let bench.py start its ranks")
    return ("run", None)


def init(backend: str) -> bool:
    """Joins the process group when launched with more than one rank.  Returns True if joined."""
    rank, _, world = env_world()
    if world <= 1:
        return False
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29500")
    dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return True


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def aggregate(elapsed_ms: float, units: float, device="cpu") -> Tuple[float, float]:
    """(max elapsed over ranks, total units over ranks)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(elapsed_ms), float(units)
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def finish():
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
