"""The multi-GPU story is "replicas only": every rank runs an independent copy of the round and
only the timing is reduced (max over ranks). This checks that reduction with two CPU ranks
over gloo."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 10.0 + 5.0 * rank                   # rank 1 is the slower replica
    ms = bench.max_over_ranks(ms_local, world, device="cpu")
    value = bench.job_throughput(ms, steps=20, world=world)
    out[rank] = (ms, value, bench.replica_seed(3, rank))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_whole_job_throughput():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0                       # max over ranks, on every rank
    assert abs(res[0][1] - world * 20 / 15e-3) < 1e-6           # rounds/s of the whole job
    assert res[0][2] != res[1][2]                               # replicas draw different inputs


def test_single_rank_needs_no_process_group():
    assert bench.max_over_ranks(7.5, 1, device="cpu") == 7.5
    assert bench.job_throughput(10.0, steps=10, world=1) == 1000.0
