"""The N > 1 path of the benchmark is independent replicas: this checks its host logic with two gloo ranks on CPU
(seed families per rank, barrier, maximum of the timings over ranks, whole-job throughput)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2506_14158_b200 import replicas
from paper_2506_14158_b200 import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert replicas.env_rank_world() == (rank, world, rank)
        cfg = replicas.rank_config(W.CONFIGS["c1"], rank)
        parent = W.make_trees(cfg)
        x = W.make_accept_inputs(cfg, parent, 1.0, token_mode="topk")
        replicas.barrier()
        mine = [10.0 + rank, 5.0 - rank, 1.0]            # per-rank "timings"
        got = replicas.max_over_ranks(mine)
        out[rank] = dict(max=got, logits_sum=float(np.asarray(x["logits"], dtype=np.float64).sum()),
                         config_id=cfg.config_id, shape=tuple(x["logits"].shape))
        replicas.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_run_independent_replicas():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    # the maximum over ranks is the same everywhere and element-wise
    assert r0["max"] == r1["max"] == [11.0, 5.0, 1.0]
    # same shapes, different data: another seed family per rank
    assert r0["shape"] == r1["shape"] and r0["config_id"] != r1["config_id"]
    assert r0["logits_sum"] != r1["logits_sum"]
    # whole-job throughput: all ranks' nodes over the slowest rank's time
    assert replicas.aggregate_nodes_per_second(26, 2, 0.5) == 26 * 2 / 0.5e-3


def test_single_process_is_the_identity():
    assert replicas.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    replicas.barrier()
    assert replicas.rank_config(W.CONFIGS["c2"], 0) is W.CONFIGS["c2"]
