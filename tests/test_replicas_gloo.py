"""The N > 1 path on CPU: two gloo ranks, each with its own shard of samples, combine their timings."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
import moqe_workloads as wl


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2508_09204_b200 import replicas
    w = wl.get("llama7b_decode")
    seed = replicas.shard_seed(wl.BASE_SEED, rank)
    ids = oracle.route(wl.router_logits(w, seed))                 # this rank's shard: its own routing
    replicas.barrier()
    ms = replicas.max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"))
    out[rank] = (ids.tolist(), ms, replicas.whole_job_value(sum(w.sample_rows), world, ms))
    dist.destroy_process_group()


def test_two_replicas_over_gloo():
    world, port = 2, 29500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    assert r0[0] != r1[0]                       # different shards of samples
    assert r0[1] == r1[1] == 15.0               # the slowest rank's time, on every rank
    assert r0[2] == r1[2] == 2 * 16 / 15.0e-3   # whole-job tokens/s


def test_single_process_is_identity():
    from paper_2508_09204_b200 import replicas
    assert replicas.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    assert replicas.shard_seed(7, 0) == 7 and replicas.shard_seed(7, 3) == 3007
    assert replicas.whole_job_value(16, 1, 0.25) == 64000.0
