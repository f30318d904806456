"""The N > 1 path of bench.py on CPU: two gloo ranks, each a replica with its own step time; the job's
value must use the slowest rank's time and count every rank's bytes (the path shards by replicas, so
there is no data-path collective to test - only this aggregation and the seeds differing per rank)."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = [0.10, 0.25][rank]
        slow = bench.max_over_ranks(ms, device="cpu")
        out[rank] = (slow, bench.whole_job_value(3.0e8, slow, world))
    finally:
        dist.destroy_process_group()


def test_two_rank_aggregation():
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
        res = dict(out)
    assert res[0] == res[1]
    slow, value = res[0]
    assert slow == 0.25
    assert value == 2 * 3.0e8 / 0.25e-3 / 1e9


def test_replicas_use_different_seeds():
    import bench
    from paper_2609_38121_b200 import workloads as W
    a = dict(W.CONFIGS["cfg0"])
    b = dict(a)
    b["seed"] += 1000                      # what bench.Session does for rank 1
    ka = W.LayerWorkload(a).calibration()[0]
    kb = W.LayerWorkload(b).calibration()[0]
    assert ka.shape == kb.shape and not np.array_equal(ka, kb)
    assert bench.max_over_ranks(0.5) == 0.5  # outside torch.distributed: identity
