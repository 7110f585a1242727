"""The N > 1 host logic of bench.py on CPU: two gloo ranks on 127.0.0.1 draw different sequences
(weak scaling: every rank owns its own) and agree on the maximum of their timings."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    par, layers, ver, exp = bench.build_workload(rank, 1)
    mx = bench.max_over_ranks(torch, [1.0 + rank, 10.0 - rank, 5.0], "cpu")
    dist.barrier()
    out[rank] = (mx, par.tolist(), int(layers[0].q[0, 0, 0]), int(ver.tok[1]))
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_by_sequence_and_reduce_max():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    assert r0[0] == r1[0] == [2.0, 10.0, 5.0]          # max over ranks, same on both
    assert r0[1:] != r1[1:]                            # different sequences per rank
    assert len(r0[1]) == len(r1[1]) == 60              # same shape (weak scaling)


def test_max_over_ranks_without_process_group_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(torch, [3.0, 1.5], "cpu") == [3.0, 1.5]
