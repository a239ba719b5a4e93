"""The N>1 path of the benchmark (replicas only): world-size-2 gloo ranks on CPU check the
whole-job aggregation (sum of units over ranks / slowest rank's time) and the per-rank seeds."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2510_07535_b200 import replicas, workloads as W


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dev = torch.device("cpu")
    # rank r "processed" (r+1)*100 units in (r+1)*0.5 s
    units, sec = replicas.aggregate((rank + 1) * 100.0, (rank + 1) * 0.5, dev)
    thr = replicas.throughput((rank + 1) * 100.0, (rank + 1) * 0.5, dev)
    spec = W.config_spec(0, ctx_div=64, vocab=64)
    spec.seed = replicas.replica_seed(spec.seed, rank)
    wl = W.generate(spec, threads=1)
    ret[rank] = (units, sec, thr, int(wl.q.astype(np.int64).sum()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation():
    world = 2
    port = _free_port()
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, port, ret), nprocs=world, join=True)
    for r in range(world):
        units, sec, thr, _ = ret[r]
        assert units == 300.0 and sec == 1.0 and thr == 300.0
    assert ret[0][3] != ret[1][3]          # replicas draw different inputs


def test_single_process_passthrough():
    assert replicas.aggregate(5.0, 2.0, torch.device("cpu")) == (5.0, 2.0)
    assert replicas.replica_seed(7, 0) == 7 and replicas.replica_seed(7, 3) == 3007
