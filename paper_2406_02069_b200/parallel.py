"""Multi-GPU plumbing.

The compression path shards with no exchange step: every (layer, sequence, KV head) is independent, so
for ordinary batches ranks only agree on how the work is split and on one clock (`shard_sequences`,
`job_throughput`).

Only a context whose K does not fit one GPU needs communication.  `compress_layer_sharded` runs one layer
with the keys of every sequence split into contiguous ranges over the ranks: the library's shard calls do
all arithmetic, this module moves the two small exchange payloads (row normalisers, score ranges) and the
kept rows with torch.distributed collectives."""
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


def split_keys(seq_len: int, alpha: int, world: int) -> List[Tuple[int, int]]:
    """(begin, keys) of each rank's contiguous key range of one sequence: near-equal ranges; the last one
    holds the alpha window keys and at least one prefix key.  Every rank computes the same split."""
    if seq_len < alpha + 1:
        raise ValueError("sequence shorter than the window plus one prefix key")
    if seq_len - (alpha + 1) < world - 1:
        raise ValueError("sequence too short to give every rank a key")
    base, extra = divmod(seq_len, world)
    keys = [base + (1 if r < extra else 0) for r in range(world)]
    short = alpha + 1 - keys[-1]                 # the last range must reach back over the window + 1
    r = world - 2
    while short > 0 and r >= 0:
        take = min(short, keys[r] - 1)
        keys[r] -= take
        keys[-1] += take
        short -= take
        r -= 1
    out, begin = [], 0
    for kcount in keys:
        out.append((begin, kcount))
        begin += kcount
    return out


class TorchExchange:
    """The two collectives the sharded layer needs, over torch.distributed.  With nccl the payloads stay on
    the GPUs; with gloo, CUDA payloads are staged through host memory (a debugging path: it lets the ranks
    of a test share one GPU, since they then meet only on the host)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self.via_host = dist.get_backend(group) == "gloo"

    def all_gather(self, t: torch.Tensor) -> torch.Tensor:
        src = t.contiguous()
        if self.via_host and src.is_cuda:
            src = src.cpu()
        parts = [torch.empty_like(src) for _ in range(self.world)]
        self.dist.all_gather(parts, src, group=self.group)
        return torch.stack(parts).to(t.device)

    def sum_bits(self, t: torch.Tensor) -> None:
        """In-place integer sum of the raw bits: exact when every element is non-zero on one rank only."""
        view = t.view(torch.int32) if t.element_size() * t.shape[-1] % 4 == 0 else t.view(torch.int16)
        if self.via_host and view.is_cuda:
            host = view.cpu()
            self.dist.all_reduce(host, op=self.dist.ReduceOp.SUM, group=self.group)
            view.copy_(host)
        else:
            self.dist.all_reduce(view, op=self.dist.ReduceOp.SUM, group=self.group)


def compress_layer_sharded(cfg, layer: int, q_win: torch.Tensor, k_shard: torch.Tensor, v_shard: torch.Tensor,
                           seq_lens: Sequence[int], k_out: torch.Tensor, v_out: torch.Tensor, indices: torch.Tensor,
                           scores: torch.Tensor, workspace: torch.Tensor, exchange, ops=None, stream=None) -> None:
    """One layer with every sequence's keys split over the ranks of `exchange` by `split_keys`.

    q_win [batch][H_q][alpha][d] is the same on every rank; k_shard / v_shard [batch][H_kv][keys_max][d] hold
    this rank's key range of each sequence.  On return every rank holds the layer's packed compact cache
    (k_out, v_out), its index list and the full score rows scores [batch][H_kv][>= max prefix].
    `ops` is the kernel binding (tests may pass a stand-in with the same functions).
    With `stream` given, the whole layer (the kernels, torch's copies and fills, and the collectives, which
    follow torch's current stream) runs on that stream.
    """
    if stream is not None and q_win.is_cuda:
        with torch.cuda.stream(stream):
            return compress_layer_sharded(cfg, layer, q_win, k_shard, v_shard, seq_lens, k_out, v_out, indices,
                                          scores, workspace, exchange, ops=ops, stream=None)
    if ops is None:
        from . import binding as ops
    world, rank = exchange.world, exchange.rank
    alpha, batch = cfg.window, len(seq_lens)
    splits = [split_keys(n, alpha, world) for n in seq_lens]            # [batch][world] (begin, keys)
    begin = [splits[b][rank][0] for b in range(batch)]
    keys = [splits[b][rank][1] for b in range(batch)]
    wkeys = [alpha if rank == world - 1 else 0 for _ in range(batch)]
    k_layer = ops.layer_budgets(cfg)[layer]
    dev = q_win.device

    # 1-2. partial normalisers of the window rows -> all-gather -> full normalisers
    part = torch.empty((batch, cfg.num_q_heads, alpha), dtype=torch.float32, device=dev)
    ops.shard_window_lse(cfg, q_win, k_shard, keys, wkeys, part, workspace, stream=stream)
    parts = exchange.all_gather(part)
    lse = torch.empty_like(part)
    ops.merge_lse(parts, lse, stream=stream)

    # 3. scores of this rank's prefix keys -> all-gather (padded to the longest range) -> full score rows
    pad = max(splits[b][r][1] for b in range(batch) for r in range(world))
    local = torch.zeros((batch, cfg.num_kv_heads, pad), dtype=torch.float32, device=dev)
    ops.shard_scores(cfg, q_win, k_shard, lse, keys, wkeys, local, workspace, stream=stream)
    gathered = exchange.all_gather(local)
    for b in range(batch):
        for r in range(world):
            b0, cnt = splits[b][r]
            cnt -= alpha if r == world - 1 else 0
            scores[b, :, b0:b0 + cnt] = gathered[r, b, :, :cnt]

    # 4. the same selection on every rank
    ops.select_topk(cfg, scores, seq_lens, k_layer, indices, workspace, stream=stream)

    # 5. every rank copies the rows it owns; the integer sum leaves each row's bits from its one owner
    k_out.zero_()
    v_out.zero_()
    ops.shard_gather(cfg, k_shard, v_shard, indices, seq_lens, k_layer, begin, keys, k_out, v_out, stream=stream)
    exchange.sum_bits(k_out)
    exchange.sum_bits(v_out)
