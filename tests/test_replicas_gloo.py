"""The N > 1 path of the benchmark is N independent replicas; its only cross-rank logic (barrier, slowest
rank's time, bytes summed) is exercised here with two gloo ranks on CPU."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2604_05887_b200 import replicas
    import hkv_inputs as hi
    # every rank builds its own small workload from its own seed
    L = hi.tiny(seed=replicas.replica_seed(7, rank), B=1, C=64, chunk_size=8, w=4, Hq=4, Hkv=2, d=16)
    replicas.barrier()
    ms, byt, w = replicas.aggregate_step(10.0 + 5.0 * rank, 1000 * (rank + 1))
    out[rank] = (ms, byt, w, int(L.k.sum()))
    replicas.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_aggregate_like_the_benchmark():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][:3] == (15.0, 3000, 2) and res[1][:3] == (15.0, 3000, 2)     # max time, summed bytes, world size
    assert res[0][3] != res[1][3]                                             # different seeds, different data


def test_single_process_needs_no_process_group():
    from paper_2604_05887_b200 import replicas
    assert replicas.aggregate_step(3.5, 42) == (3.5, 42, 1)
    replicas.barrier()
    assert replicas.replica_seed(2, 3) == 3002
