"""Seeded random configurations through the fused layer call, each against the oracle: shapes, types, pools,
budgets and ragged batches that no hand-written case lists."""
import numpy as np
import pytest
import torch

import oracle
import paper_2406_02069_b200 as pkv
from helpers import assert_indices_match, assert_scores_close, packed_rows

pytestmark = pytest.mark.gpu
DEV = "cuda"
TORCH = {"bf16": torch.bfloat16, "fp16": torch.float16, "fp32": torch.float32}


def draw(seed):
    rng = np.random.default_rng(1000 + seed)
    dtype = ["bf16", "fp16", "fp32"][int(rng.integers(0, 3))]
    d = int(rng.choice([64, 128]))
    hkv = int(rng.integers(1, 5))
    group = int(rng.choice([1, 2, 4, 8]))
    alpha = int(rng.choice([1, 4, 8, 16, 32, 48]))
    batch = int(rng.integers(1, 4))
    lens = [int(rng.integers(alpha + 1, 2600)) for _ in range(batch)]
    m = int(rng.choice([1, 2, 5, 12]))
    return dict(dtype=dtype, d=d, hkv=hkv, group=group, alpha=alpha, lens=lens, m=m,
                layer=int(rng.integers(0, m)), pool=int(rng.choice([1, 3, 5, 7, 9])),
                kind=["max", "avg"][int(rng.integers(0, 2))], budget=int(rng.integers(alpha, alpha + 700)),
                beta=float(rng.choice([1.0, 3.5, 20.0])), gain=float(rng.choice([0.5, 1.0, 2.5])), seed=seed)


@pytest.mark.parametrize("seed", range(36))
def test_random_configuration_matches_oracle(seed):
    c = draw(seed)
    hq, alpha, d, lens = c["hkv"] * c["group"], c["alpha"], c["d"], c["lens"]
    cfg = pkv.make_config(num_layers=c["m"], num_q_heads=hq, num_kv_heads=c["hkv"], head_dim=d, window=alpha,
                          pool_kernel=c["pool"], dtype=c["dtype"], avg_budget=c["budget"], beta=c["beta"],
                          pool_kind={"max": 0, "avg": 1}[c["kind"]])
    budgets = pkv.layer_budgets(cfg)
    assert budgets == oracle.layer_budgets(c["m"], c["budget"], alpha, c["beta"])
    kl = budgets[c["layer"]]
    g = torch.Generator().manual_seed(c["seed"])
    n_max = max(lens)
    q = (torch.randn(len(lens), hq, alpha, d, generator=g) * c["gain"]).to(TORCH[c["dtype"]])
    k = torch.randn(len(lens), c["hkv"], n_max, d, generator=g)
    k[:, :, 0] *= 2.0                                                  # one dominant key
    k = k.to(TORCH[c["dtype"]])
    v = torch.randn(len(lens), c["hkv"], n_max, d, generator=g).to(TORCH[c["dtype"]])
    ws = pkv.new_workspace(cfg, len(lens), n_max, DEV)
    rows = pkv.total_rows(cfg, kl, lens)
    k_out = torch.empty(rows, d, dtype=k.dtype, device=DEV)
    v_out = torch.empty_like(k_out)
    idx = torch.empty(rows, dtype=torch.int32, device=DEV)
    scores = torch.full((len(lens), c["hkv"], n_max), -1.0, dtype=torch.float32, device=DEV)
    kd, vd = k.to(DEV), v.to(DEV)
    pkv.compress_layer(cfg, c["layer"], q.to(DEV), kd, vd, lens, k_out, v_out, idx, ws, scores=scores)
    pkv.check_status(ws)
    ref = oracle.compress_batch(q, k, v, lens, pool_kernel=c["pool"], avg_budget=c["budget"], k_layer=kl,
                                pool_kind=c["kind"])
    got_scores, got_idx = scores.cpu().numpy(), idx.cpu().numpy()
    assert ref["indices"].shape[0] == rows
    for b, n in enumerate(lens):
        assert_scores_close(got_scores[b, :, : n - alpha], ref["scores"][b], "%r seq %d" % (c, b))
        assert (got_scores[b, :, n - alpha:] == -1.0).all()
    for b, h, sl in packed_rows(ref["counts"], c["hkv"]):
        assert_indices_match(got_idx[sl], ref["indices"][sl], ref["scores"][b][h], c["pool"], alpha,
                             "%r b %d h %d" % (c, b, h), pool_kind=c["kind"])
        sel = idx[sl].long()
        assert torch.equal(k_out[sl], kd[b, h, sel]) and torch.equal(v_out[sl], vd[b, h, sel])
