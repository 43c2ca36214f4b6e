"""World-size-2 checks of the multi-rank bookkeeping on CPU (gloo): split of a ragged batch, one clock."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2406_02069_b200 import parallel, workloads


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lens = workloads.MISTRAL_RAGGED.seq_lens()
    mine = parallel.shard_sequences(lens, rank, world)
    tokens = sum(lens[i] for i in mine)
    ms = 10.0 + 5.0 * rank                                   # rank 1 is the slow one
    value, ms_job, total = parallel.job_throughput(tokens, ms)
    out[rank] = (mine, tokens, value, ms_job, total)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_split_the_batch_and_share_one_clock():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    lens = workloads.MISTRAL_RAGGED.seq_lens()
    a, b = res[0], res[1]
    assert sorted(a[0] + b[0]) == list(range(len(lens)))     # every sequence exactly once
    assert a[1] + b[1] == sum(lens) == a[4] == b[4]
    assert abs(a[1] - b[1]) <= max(lens)                     # balanced to within one sequence
    assert a[3] == b[3] == 15.0                              # slowest rank's time on both
    assert a[2] == b[2] == sum(lens) / 15.0e-3               # whole-job tokens / that time


def test_single_rank_needs_no_process_group():
    value, ms, tokens = parallel.job_throughput(1000, 2.0)
    assert (value, ms, tokens) == (500000.0, 2.0, 1000)
    assert parallel.shard_sequences([5, 9, 7], 0, 1) == [0, 1, 2]
