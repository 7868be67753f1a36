"""Host logic of multi-GPU runs.  The verify pass does not shard inside a request (every layer depends on the
previous one); across requests it is embarrassingly parallel (paper App. I: one cloud model serves independent
edges).  So N GPUs run N independent replicas -- full weights each, the KV of their own requests -- with no
collective on the data path; the only exchange is the timing scalars below."""
from __future__ import annotations

from typing import Sequence


def partition_requests(prefix_lengths: Sequence[int], n_ranks: int) -> list[list[int]]:
    """Assign requests to ranks so that the summed prefix lengths (the K/V bytes a rank streams per pass) are
    balanced: longest first, each to the rank that is lightest so far (ties: lowest rank).  Deterministic.
    Returns, per rank, the request indices in increasing order."""
    if n_ranks < 1:
        raise ValueError("n_ranks must be positive")
    load = [0] * n_ranks
    out: list[list[int]] = [[] for _ in range(n_ranks)]
    order = sorted(range(len(prefix_lengths)), key=lambda i: (-int(prefix_lengths[i]), i))
    for i in order:
        r = min(range(n_ranks), key=lambda j: (load[j], j))
        out[r].append(i)
        load[r] += int(prefix_lengths[i])
    return [sorted(x) for x in out]


def reduce_replicas(times_ms: Sequence[float], counts: Sequence[float], device=None):
    """Whole-job figures of a replica run: every time is the MAX over ranks (the job ends when the slowest
    replica does), every count the SUM over ranks.  Uses the default process group (NCCL on GPUs, gloo in the
    CPU tests); returns the inputs unchanged when no group is initialised."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(t) for t in times_ms], [float(c) for c in counts]
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    n = torch.tensor(list(counts), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.cpu()], [float(x) for x in n.cpu()]
