"""Host-side logic of running the verify step on several GPUs: independent replicas, no data-path collective.

Sequences are independent (Section 3.2 verifies one tree per sequence), so N GPUs means N processes that each
verify their own seeded batch.  The only communication is a barrier around the timed region and the maximum of
the per-rank timings; throughput is what all ranks processed divided by that maximum.  Nothing here touches a
GPU: the functions work on any ``torch.distributed`` backend (``nccl`` in the benchmark, ``gloo`` in the CPU
tests).
"""
from __future__ import annotations

import os
from dataclasses import replace
from typing import Sequence, Tuple

import torch
import torch.distributed as dist


def env_rank_world() -> Tuple[int, int, int]:
    """(rank, world size, local rank) from the launcher's environment; (0, 1, 0) without a launcher."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def rank_config(cfg, rank: int):
    """The workload of one rank: the same shapes, another seed family (its config_id moves by 20 per rank), so
    that every replica verifies different trees, logits and caches."""
    return cfg if rank == 0 else replace(cfg, config_id=cfg.config_id + 20 * rank)


def max_over_ranks(values: Sequence[float], device="cpu") -> list:
    """Element-wise maximum of a short list of timings over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def barrier() -> None:
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def aggregate_nodes_per_second(nodes_per_rank: int, world: int, ms_per_step_max: float) -> float:
    """Whole-job throughput: every rank verifies `nodes_per_rank` tree nodes per step (weak scaling) and the job
    is as slow as its slowest rank."""
    return nodes_per_rank * world / (ms_per_step_max * 1e-3)
