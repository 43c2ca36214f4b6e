"""GPU parity for the sequence-sharded layer: the keys of each sequence split into contiguous ranges.

With one GPU the ranks are emulated one after another through the library's shard calls (their kernels never
wait on one another: the exchanges happen between launches), and once more as two processes that share the
GPU and meet only on the host (gloo)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
import paper_2406_02069_b200 as pkv
from paper_2406_02069_b200 import binding, parallel, workloads
from helpers import assert_indices_match, assert_scores_close, packed_rows

pytestmark = pytest.mark.gpu
DEV = "cuda"


def shard_views(x, lens, alpha, world, rank):
    """This rank's K/V ranges, padded to its longest range, plus (begin, keys, window_keys) per sequence."""
    splits = [parallel.split_keys(n, alpha, world) for n in lens]
    begin = [splits[b][rank][0] for b in range(len(lens))]
    keys = [splits[b][rank][1] for b in range(len(lens))]
    pad = max(keys)
    ks = torch.zeros(len(lens), x.k.shape[1], pad, x.k.shape[3], dtype=x.k.dtype, device=x.k.device)
    vs = torch.zeros_like(ks)
    for b in range(len(lens)):
        ks[b, :, : keys[b]] = x.k[b, :, begin[b]: begin[b] + keys[b]]
        vs[b, :, : keys[b]] = x.v[b, :, begin[b]: begin[b] + keys[b]]
    wkeys = [alpha if rank == world - 1 else 0] * len(lens)
    return ks, vs, begin, keys, wkeys


CASES = [
    (workloads.TINY, None, 2),
    (workloads.scaled(workloads.LLAMA3_8B, num_layers=2, seq_len=5037, name="llama3_8b_5k"), None, 4),
    (workloads.scaled(workloads.LLAMA3_70B, num_layers=3, seq_len=3011, name="llama3_70b_3k"), None, 3),
    (workloads.scaled(workloads.MISTRAL_RAGGED, num_layers=2, batch=3, name="mistral_b3"), "ragged", 2),
    (workloads.scaled(workloads.LLAMA2_7B, num_layers=2, seq_len=600, name="llama2_600", dtype="fp32"), None, 8),
]


@pytest.mark.parametrize("w,ragged,world", CASES, ids=lambda x: getattr(x, "name", str(x)))
def test_emulated_ranks_reproduce_the_unsharded_layer(w, ragged, world):
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    if ragged:
        lens = [300 + (n % 1777) for n in lens]
    alpha, batch = w.window, len(lens)
    layer = w.num_layers - 1
    kl = pkv.layer_budgets(cfg)[layer]
    x = workloads.make_layer(w, layer, device=DEV, seq_lens=lens)
    ws = pkv.new_workspace(cfg, batch, max(lens), DEV)
    rows = pkv.total_rows(cfg, kl, lens)
    shards = [shard_views(x, lens, alpha, world, r) for r in range(world)]

    # 1. partial normalisers on every rank; 2. the exchange and the merge
    parts = torch.empty(world, batch, w.num_q_heads, alpha, dtype=torch.float32, device=DEV)
    for r, (ks, vs, begin, keys, wkeys) in enumerate(shards):
        pkv.binding.shard_window_lse(cfg, x.q_win, ks, keys, wkeys, parts[r], ws)
    lse = torch.empty(batch, w.num_q_heads, alpha, dtype=torch.float32, device=DEV)
    pkv.binding.merge_lse(parts, lse)
    pkv.check_status(ws)
    qc, kc = x.q_win.cpu(), x.k.cpu()
    want_lse = np.stack([oracle.window_lse(qc[b], kc[b, :, :n]) for b, n in enumerate(lens)])
    np.testing.assert_allclose(lse.cpu().numpy(), want_lse, rtol=0, atol=2e-4)

    # 3. every rank scores its range; the ranges are laid side by side
    scores = torch.full((batch, w.num_kv_heads, max(lens)), -1.0, dtype=torch.float32, device=DEV)
    for r, (ks, vs, begin, keys, wkeys) in enumerate(shards):
        local = torch.full((batch, w.num_kv_heads, max(keys) + 3), -2.0, dtype=torch.float32, device=DEV)
        pkv.binding.shard_scores(cfg, x.q_win, ks, lse, keys, wkeys, local, ws)
        for b in range(batch):
            cnt = keys[b] - wkeys[b]
            scores[b, :, begin[b]: begin[b] + cnt] = local[b, :, :cnt]
            assert (local[b, :, cnt:] == -2.0).all()                  # nothing written past the range's prefix
    pkv.check_status(ws)

    # 4. selection on the full rows; 5. every rank gathers what it owns
    idx = torch.empty(rows, dtype=torch.int32, device=DEV)
    pkv.select_topk(cfg, scores, lens, kl, idx, ws)
    k_sum = torch.zeros(rows, w.head_dim, dtype=torch.int32 if x.k.element_size() == 4 else torch.int16, device=DEV)
    v_sum = torch.zeros_like(k_sum)
    owners = torch.zeros(rows, dtype=torch.int32, device=DEV)
    for r, (ks, vs, begin, keys, wkeys) in enumerate(shards):
        k_out = torch.zeros(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
        v_out = torch.zeros_like(k_out)
        pkv.binding.shard_gather(cfg, ks, vs, idx, lens, kl, begin, keys, k_out, v_out)
        k_sum += k_out.view(k_sum.dtype)
        v_sum += v_out.view(v_sum.dtype)
        owners += (k_out != 0).any(dim=1).int()
    pkv.check_status(ws)
    assert int(owners.max()) == 1                                     # each row written by one rank
    k_all, v_all = k_sum.view(x.k.dtype), v_sum.view(x.k.dtype)

    # against the oracle on the unsharded tensors
    ref = oracle.compress_batch(qc, kc, x.v.cpu(), lens, pool_kernel=w.pool_kernel, avg_budget=w.avg_budget,
                                k_layer=kl)
    got_scores, got_idx = scores.cpu().numpy(), idx.cpu().numpy()
    for b, n in enumerate(lens):
        assert_scores_close(got_scores[b, :, : n - alpha], ref["scores"][b], "%s seq %d" % (w.name, b))
    identical = 0
    for b, h, sl in packed_rows(ref["counts"], w.num_kv_heads):
        identical += bool(assert_indices_match(got_idx[sl], ref["indices"][sl], ref["scores"][b][h], w.pool_kernel,
                                               alpha, "%s b %d h %d" % (w.name, b, h)))
        sel = idx[sl].long()
        assert torch.equal(k_all[sl], x.k[b, h, sel]) and torch.equal(v_all[sl], x.v[b, h, sel])
    assert identical >= 0.95 * len(ref["counts"]) * w.num_kv_heads


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spmd_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = workloads.scaled(workloads.LLAMA3_8B, num_layers=2, seq_len=4001, name="llama3_8b_4k")
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    layer = 1
    kl = pkv.layer_budgets(cfg)[layer]
    x = workloads.make_layer(w, layer, device=DEV)                    # same seed on both ranks
    ks, vs, begin, keys, wkeys = shard_views(x, lens, w.window, world, rank)
    rows = pkv.total_rows(cfg, kl, lens)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    k_out = torch.empty(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
    v_out = torch.empty_like(k_out)
    idx = torch.empty(rows, dtype=torch.int32, device=DEV)
    scores = torch.zeros(len(lens), w.num_kv_heads, max(lens), dtype=torch.float32, device=DEV)
    parallel.compress_layer_sharded(cfg, layer, x.q_win, ks, vs, lens, k_out, v_out, idx, scores, ws,
                                    parallel.TorchExchange())
    pkv.check_status(ws)
    # the unsharded call on the same GPU
    k_one = torch.empty_like(k_out)
    v_one = torch.empty_like(v_out)
    idx_one = torch.empty_like(idx)
    pkv.compress_layer(cfg, layer, x.q_win, x.k, x.v, lens, k_one, v_one, idx_one, ws)
    pkv.check_status(ws)
    same = torch.equal(idx, idx_one)
    count = rows // w.num_kv_heads                                    # one sequence: row = head * count + r
    flat = x.k[0].reshape(-1, w.head_dim)                             # [H_kv * n][d]
    src = (torch.arange(rows, device=DEV) // count) * lens[0] + idx.long()
    rows_ok = bool(torch.equal(k_out, flat[src]))
    cache_equal = bool(torch.equal(k_out, k_one) and torch.equal(v_out, v_one)) if same else None
    out[rank] = (idx.cpu().numpy().tolist(), idx_one.cpu().numpy().tolist(), rows_ok, cache_equal)
    dist.barrier()
    dist.destroy_process_group()


def test_two_processes_sharing_the_gpu_run_the_sharded_layer():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_spmd_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0]                                     # both ranks hold the same list
    for r in range(world):
        sharded, single, rows_ok, cache_equal = res[r]
        assert rows_ok                                                # gathered rows are the listed rows
        if cache_equal is not None:
            assert cache_equal                                        # and equal the unsharded cache bit for bit
        # sharding only changes the summation order of the normalisers: the lists agree, or differ in a few
        # entries at the selection threshold
        assert len(set(sharded) ^ set(single)) <= 0.01 * len(single) or sharded == single
