"""Multi-GPU host logic on CPU: two gloo ranks stand in for two replicas."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp

from paper_2605_13319_b200 import replicas, synth


def test_partition_is_complete_balanced_and_deterministic():
    lens, _, _ = synth.ragged_requests(0, 32)
    for n in (1, 2, 4, 8):
        parts = replicas.partition_requests(lens, n)
        assert sorted(i for p in parts for i in p) == list(range(32))
        loads = [int(sum(int(lens[i]) for i in p)) for p in parts]
        assert max(loads) - min(loads) <= int(max(lens))          # longest-first greedy bound
        assert parts == replicas.partition_requests(lens, n)
    assert replicas.partition_requests([5, 5, 5], 2) == [[0, 2], [1]]


def _rank_main(rank, world, port, q):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r "measured" (10 + r) ms for the device-resident region, (20 - r) ms end to end, and (100 + r) tokens
    times, counts = replicas.reduce_replicas([10.0 + rank, 20.0 - rank], [100.0 + rank, 7.0])
    q.put((rank, times, counts))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_max_time_and_summed_tokens():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    for rank, times, counts in got:
        assert times == [11.0, 20.0]          # max over ranks
        assert counts == [201.0, 14.0]        # sum over ranks


def test_single_process_is_passed_through():
    assert replicas.reduce_replicas([3.0], [5.0]) == ([3.0], [5.0])
    assert np.isclose(sum(map(len, replicas.partition_requests([1, 2, 3], 3))), 3)
