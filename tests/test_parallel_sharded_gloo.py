"""World-size-2 and -3 runs of the sequence-sharded layer's plumbing on CPU (gloo).

No kernel can run here, so the ranks get a stand-in for the kernel binding, written in plain double-precision
torch below; what is under test is the orchestration: the key split, which payloads are exchanged, how the
score ranges are laid side by side, and the owner-wise merge of the gathered rows.  The outcome must be the
oracle's result on the unsharded tensors.
"""
import math
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2406_02069_b200 import parallel, workloads


class Cfg:
    def __init__(self, w):
        self.w, self.window = w, w.window
        self.num_q_heads, self.num_kv_heads = w.num_q_heads, w.num_kv_heads


class TorchOps:
    """The binding's shard calls restated with torch ops (float64), for CPU tensors."""

    def layer_budgets(self, cfg):
        w = cfg.w
        return oracle.layer_budgets(w.num_layers, w.avg_budget, w.window, w.beta)

    def _logits(self, cfg, q_win, k_shard, b, keys, wkeys):
        w = cfg.w
        q = q_win[b].double()                                           # [H_q][alpha][d]
        k = k_shard[b, :, :keys].double().repeat_interleave(w.group, dim=0)
        logits = torch.einsum("hjd,hid->hji", q, k) / math.sqrt(w.head_dim)
        prefix = keys - wkeys
        i = torch.arange(keys).view(1, 1, -1)
        j = torch.arange(w.window).view(1, -1, 1)
        return logits.masked_fill(i > prefix + j, float("-inf")), prefix

    def shard_window_lse(self, cfg, q_win, k_shard, keys, wkeys, lse_out, workspace, stream=None):
        for b in range(len(keys)):
            logits, _ = self._logits(cfg, q_win, k_shard, b, keys[b], wkeys[b])
            lse_out[b] = torch.logsumexp(logits, dim=-1).float()

    def merge_lse(self, parts, out, stream=None):
        out.copy_(torch.logsumexp(parts.double(), dim=0).float())

    def shard_scores(self, cfg, q_win, k_shard, lse, keys, wkeys, scores, workspace, stream=None):
        w = cfg.w
        for b in range(len(keys)):
            logits, prefix = self._logits(cfg, q_win, k_shard, b, keys[b], wkeys[b])
            a = torch.exp(logits - lse[b].double().unsqueeze(-1))       # [H_q][alpha][keys]
            s = a.sum(dim=1).view(w.num_kv_heads, w.group, -1).mean(dim=1)
            scores[b, :, :prefix] = s[:, :prefix].float()

    def select_topk(self, cfg, scores, seq_lens, k_layer, indices, workspace, stream=None):
        w, off = cfg.w, 0
        for b, n in enumerate(seq_lens):
            c = oracle.kept_count(w.avg_budget, w.window, k_layer, n)
            for h in range(w.num_kv_heads):
                if n <= w.avg_budget:
                    row = np.arange(n)
                else:
                    pooled = oracle.pool_max(scores[b, h, : n - w.window].numpy(), w.pool_kernel)
                    row = np.concatenate([oracle.select_topk(pooled, k_layer), np.arange(n - w.window, n)])
                indices[off: off + c] = torch.from_numpy(row.astype(np.int32))
                off += c

    def shard_gather(self, cfg, k_shard, v_shard, indices, seq_lens, k_layer, begin, keys, k_out, v_out, stream=None):
        w, off = cfg.w, 0
        for b, n in enumerate(seq_lens):
            c = oracle.kept_count(w.avg_budget, w.window, k_layer, n)
            for h in range(w.num_kv_heads):
                for r in range(c):
                    local = int(indices[off + r]) - begin[b]
                    if 0 <= local < keys[b]:
                        k_out[off + r] = k_shard[b, h, local]
                        v_out[off + r] = v_shard[b, h, local]
                off += c


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _case():
    w = workloads.scaled(workloads.MISTRAL_RAGGED, num_layers=2, batch=2, name="mistral_b2_cpu", window=8,
                         avg_budget=64)
    return w, [301, 517]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.set_num_threads(1)
    w, lens = _case()
    x = workloads.make_layer(w, 0, seq_lens=lens)
    cfg = Cfg(w)
    splits = [parallel.split_keys(n, w.window, world) for n in lens]
    keys = [splits[b][rank][1] for b in range(len(lens))]
    ks = torch.zeros(len(lens), w.num_kv_heads, max(keys), w.head_dim, dtype=x.k.dtype)
    vs = torch.zeros_like(ks)
    for b in range(len(lens)):
        b0 = splits[b][rank][0]
        ks[b, :, : keys[b]] = x.k[b, :, b0: b0 + keys[b]]
        vs[b, :, : keys[b]] = x.v[b, :, b0: b0 + keys[b]]
    kl = oracle.layer_budgets(w.num_layers, w.avg_budget, w.window, w.beta)[0]
    rows = sum(w.num_kv_heads * oracle.kept_count(w.avg_budget, w.window, kl, n) for n in lens)
    k_out = torch.full((rows, w.head_dim), 7.0, dtype=x.k.dtype)           # must be zeroed by the call
    v_out = torch.full_like(k_out, 7.0)
    idx = torch.empty(rows, dtype=torch.int32)
    scores = torch.zeros(len(lens), w.num_kv_heads, max(lens))
    parallel.compress_layer_sharded(cfg, 0, x.q_win, ks, vs, lens, k_out, v_out, idx, scores, None,
                                    parallel.TorchExchange(), ops=TorchOps())
    out[rank] = (idx.numpy().copy(), k_out.float().numpy().copy(), v_out.float().numpy().copy(), scores.numpy().copy())
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_plumbing_reproduces_the_unsharded_oracle(world):
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    w, lens = _case()
    x = workloads.make_layer(w, 0, seq_lens=lens)
    kl = oracle.layer_budgets(w.num_layers, w.avg_budget, w.window, w.beta)[0]
    ref = oracle.compress_batch(x.q_win, x.k, x.v, lens, pool_kernel=w.pool_kernel, avg_budget=w.avg_budget, k_layer=kl)
    for r in range(world):
        idx, k_out, v_out, scores = res[r]
        for b, n in enumerate(lens):
            np.testing.assert_allclose(scores[b, :, : n - w.window], ref["scores"][b], rtol=1e-5, atol=1e-9)
        assert np.array_equal(idx, ref["indices"])
        assert np.array_equal(k_out, ref["k_out"].float().numpy()) and np.array_equal(v_out, ref["v_out"].float().numpy())


def test_key_split_properties():
    for n, alpha, world in [(100, 8, 4), (20, 8, 4), (12, 8, 4), (131072, 32, 8), (4097, 32, 3), (33, 32, 1)]:
        parts = parallel.split_keys(n, alpha, world)
        assert len(parts) == world and parts[0][0] == 0
        assert all(parts[r][0] + parts[r][1] == parts[r + 1][0] for r in range(world - 1))   # contiguous
        assert parts[-1][0] + parts[-1][1] == n
        assert all(k >= 1 for _, k in parts) and parts[-1][1] >= alpha + 1
        if n // world >= alpha + 1:
            assert max(k for _, k in parts) - min(k for _, k in parts) <= 1                  # balanced
    with pytest.raises(ValueError):
        parallel.split_keys(11, 8, 4)
    with pytest.raises(ValueError):
        parallel.split_keys(8, 8, 1)
