"""Multi-GPU bookkeeping.  The compression path shards with no exchange step: every (layer,
sequence, KV head) is independent, so ranks only agree on how the work is split and on one
clock.  Nothing here touches K/V data."""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch


def shard_sequences(seq_lens: Sequence[int], rank: int, world: int) -> List[int]:
    """Indices of the sequences rank `rank` compresses when one batch is split over `world` ranks:
    longest first, each to the rank with the least tokens so far (every rank computes the same split)."""
    order = sorted(range(len(seq_lens)), key=lambda i: (-seq_lens[i], i))
    load = [0] * world
    mine: List[int] = []
    for i in order:
        r = min(range(world), key=lambda q: (load[q], q))
        load[r] += seq_lens[i]
        if r == rank:
            mine.append(i)
    return sorted(mine)


def job_throughput(tokens_local: int, ms_local: float, device: str = "cpu") -> Tuple[float, float, int]:
    """Whole-job (tokens per second, milliseconds, tokens): tokens summed over ranks, time = slowest rank.
    Works without a process group (single rank) and with gloo (CPU tensors) or nccl (CUDA tensors)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return tokens_local / (ms_local * 1e-3), ms_local, tokens_local
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    n = torch.tensor([tokens_local], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    ms, tokens = float(t.item()), int(n.item())
    return tokens / (ms * 1e-3), ms, tokens
