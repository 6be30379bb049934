"""Multi-GPU throughput = independent replicas.  A batch-1 speculative loop is a chain of dependent passes;
independent sequences shard trivially: rank r of W takes the global sequences r, r+W, ...  A sequence's
global number selects its prompt and its seed (and, for batches, its Philox sequence index through
`sps_set_sequence_index0`), so what a sequence generates does not depend on which rank ran it; there is no
collective on the data path, and the job's time is the maximum over ranks.  (Sharding ONE sequence over
GPUs is tensor parallelism: `tensor_parallel.py`.)"""
from __future__ import annotations


def shard_sequences(n_sequences: int, rank: int, world: int) -> list[int]:
    """Global indices of the sequences rank `rank` generates."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("bad rank / world size")
    return list(range(rank, n_sequences, world))


def job_time_and_tokens(local_seconds: float, local_tokens: int, dist=None, device=None):
    """(max over ranks of the time, sum over ranks of the tokens); `dist` = torch.distributed or None."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(local_seconds), int(local_tokens)
    import torch
    t = torch.tensor([local_seconds], dtype=torch.float64, device=device)
    n = torch.tensor([local_tokens], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t[0]), int(n[0])
