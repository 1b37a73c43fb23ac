"""The N > 1 path of the benchmark (independent replicas) on two CPU ranks with the gloo backend."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_03079_b200 import replicas
from paper_2609_03079_b200 import workload as wl


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        replicas.barrier()
        spec = wl.SPECS["tiny"]
        toks = wl.make_tokens(spec, 4, stream=replicas.stream_of_rank(rank))
        local_ms = 10.0 + 5.0 * rank      # rank 1 is the slow one
        local_units = 100 + rank           # and decodes one more token
        ms, units = replicas.aggregate(local_ms, local_units, torch.device("cpu"))
        tps = replicas.throughput(local_ms, local_units, torch.device("cpu"))
        out[rank] = (ms, units, tps, float(toks.sum()))
    finally:
        dist.destroy_process_group()


def test_two_replicas_aggregate_max_time_and_sum_units():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        ms, units, tps, _ = res[rank]
        assert ms == 15.0 and units == 201           # slowest rank, all units
        assert abs(tps - 201 / 0.015) < 1e-6
    assert res[0][3] != res[1][3]                     # each replica decodes its own token stream


def test_single_process_is_identity():
    assert replicas.aggregate(3.5, 7, torch.device("cpu")) == (3.5, 7)
    assert replicas.stream_of_rank(3) == 3
