"""GPU parity for the variants reached through the configuration alone: binary16 inputs, the mean pool,
other window sizes and pyramid slopes (the appendix's alpha and beta sweeps), a uniform split (beta = 1)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2406_02069_b200 as pkv
from paper_2406_02069_b200 import workloads
from helpers import assert_indices_match, assert_scores_close, packed_rows

pytestmark = pytest.mark.gpu
DEV = "cuda"


def check_layer(w, layer, lens, min_identical=0.95):
    """One layer through the fused call against the oracle: kept lists (exact, or within tolerance at the
    threshold), gathered rows bit for bit."""
    cfg = pkv.config_of(w)
    budgets = pkv.layer_budgets(cfg)
    assert budgets == oracle.layer_budgets(w.num_layers, w.avg_budget, w.window, w.beta, schedule=w.schedule)
    kl = budgets[layer]
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    x = workloads.make_layer(w, layer, device=DEV, seq_lens=lens)
    rows = pkv.total_rows(cfg, kl, lens)
    k_out = torch.empty(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
    v_out = torch.empty_like(k_out)
    idx = torch.empty(rows, dtype=torch.int32, device=DEV)
    scores = torch.full((len(lens), w.num_kv_heads, max(lens)), -1.0, dtype=torch.float32, device=DEV)
    pkv.compress_layer(cfg, layer, x.q_win, x.k, x.v, lens, k_out, v_out, idx, ws, scores=scores)
    pkv.check_status(ws)
    ref = oracle.compress_batch(x.q_win.cpu(), x.k.cpu(), x.v.cpu(), lens, pool_kernel=w.pool_kernel,
                                avg_budget=w.avg_budget, k_layer=kl, pool_kind=w.pool_kind)
    got_scores, got_idx = scores.cpu().numpy(), idx.cpu().numpy()
    for b, n in enumerate(lens):
        assert_scores_close(got_scores[b, :, : n - w.window], ref["scores"][b], "%s seq %d" % (w.name, b))
    identical = 0
    for b, h, sl in packed_rows(ref["counts"], w.num_kv_heads):
        same = assert_indices_match(got_idx[sl], ref["indices"][sl], ref["scores"][b][h], w.pool_kernel, w.window,
                                    "%s layer %d b %d h %d" % (w.name, layer, b, h), pool_kind=w.pool_kind)
        identical += bool(same)
        sel = idx[sl].long()
        assert torch.equal(k_out[sl], x.k[b, h, sel]) and torch.equal(v_out[sl], x.v[b, h, sel])
        if same:
            assert torch.equal(k_out[sl].cpu(), ref["k_out"][sl]) and torch.equal(v_out[sl].cpu(), ref["v_out"][sl])
    total = len(ref["counts"]) * w.num_kv_heads
    assert identical >= min_identical * total, "only %d of %d index lists identical" % (identical, total)
    return x, idx, k_out, v_out, ref


# ----------------------------------------------------------------------------- binary16 inputs
@pytest.mark.parametrize("hq,hkv,alpha,d,lens", [
    (12, 4, 8, 64, [129, 1000, 136]),     # tensor-core path, head_dim 64, ragged
    (8, 2, 48, 128, [2000, 333]),         # two row blocks
    (16, 2, 32, 128, [1500]),             # R = 256
    (20, 2, 32, 128, [700]),              # R = 320: fp32-pipe kernels
])
def test_scores_fp16_shapes(hq, hkv, alpha, d, lens):
    cfg = pkv.make_config(num_layers=1, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, window=alpha, pool_kernel=3,
                          dtype="fp16", avg_budget=alpha, beta=1.0)
    g = torch.Generator(device="cpu").manual_seed(hq * 100 + alpha + 1)
    n_max = max(lens)
    # values with more mantissa bits than bfloat16 holds, so a kernel that read them as bf16 would be far off
    q = (torch.randn(len(lens), hq, alpha, d, generator=g) * 1.5).to(torch.float16)
    k = torch.randn(len(lens), hkv, n_max, d, generator=g).to(torch.float16)
    k[:, :, 0] *= 3.0
    ws = pkv.new_workspace(cfg, len(lens), n_max, DEV)
    scores = torch.full((len(lens), hkv, n_max), -1.0, dtype=torch.float32, device=DEV)
    pkv.score_window(cfg, q.to(DEV), k.to(DEV), lens, scores, ws)
    pkv.check_status(ws)
    got = scores.cpu().numpy()
    for b, n in enumerate(lens):
        want, _ = oracle.window_scores(q[b], k[b, :, :n])
        assert_scores_close(got[b, :, : n - alpha], want, "seq %d" % b)
        assert (got[b, :, n - alpha:] == -1.0).all()


@pytest.mark.parametrize("base,kw", [
    (workloads.LLAMA3_8B, dict(num_layers=2, seq_len=5037)),
    (workloads.MISTRAL_RAGGED, dict(num_layers=2, batch=3)),
], ids=["llama3_8b_5k_fp16", "mistral_b3_fp16"])
def test_fp16_layer_matches_oracle(base, kw):
    w = workloads.scaled(base, name=base.name + "_fp16", dtype="fp16", **kw)
    lens = w.seq_lens()
    if w.batch > 1:
        lens = [300 + (n % 1777) for n in lens]
    for layer in range(w.num_layers):
        x, idx, k_out, v_out, ref = check_layer(w, layer, lens)
        assert k_out.dtype == torch.float16
    # decode over the fp16 compact cache of the last layer
    cfg = pkv.config_of(w)
    kl = pkv.layer_budgets(cfg)[w.num_layers - 1]
    g = torch.Generator(device="cpu").manual_seed(5)
    q_new = torch.randn(len(lens), w.num_q_heads, w.head_dim, generator=g).to(torch.float16)
    out = torch.empty(len(lens), w.num_q_heads, w.head_dim, dtype=torch.float32, device=DEV)
    pkv.decode_attention(cfg, q_new.to(DEV), k_out, v_out, lens, kl, out)
    torch.cuda.synchronize()
    kc, vc, got = k_out.cpu(), v_out.cpu(), out.cpu().numpy()
    counts = [pkv.kept_count(cfg, kl, n) for n in lens]
    for b, h, sl in packed_rows(counts, w.num_kv_heads):
        for gq in range(w.group):
            hq = h * w.group + gq
            want = oracle.decode_attention(q_new[b, hq], kc[sl], vc[sl])
            np.testing.assert_allclose(got[b, hq], want, rtol=2e-3, atol=2e-4)


# ----------------------------------------------------------------------------- mean pool
@pytest.mark.parametrize("P,k,w", [(1, 1, 1), (5, 2, 7), (33, 32, 3), (100, 250, 5), (1000, 37, 7), (4064, 188, 7),
                                   (8193, 500, 7), (4000, 900, 7), (2500, 2000, 5), (40000, 937, 5), (131040, 188, 7), (140000, 64, 7), (3000, 40, 35), (300000 + 3, 500, 7)])
def test_avg_pool_select_is_bit_exact_on_oracle_scores(P, k, w):
    """The mean pool's rounding is part of its definition, so the lists must be identical."""
    alpha, hkv, batch = 4, 3, 2
    rng = np.random.default_rng(P * 11 + k)
    levels = rng.integers(0, 50, size=(batch, hkv, P)).astype(np.float32) / 64.0
    levels[0, 0] = rng.random(P).astype(np.float32)                 # sums that do round
    levels[0, 1] = (rng.random(P) * 1e-4).astype(np.float32)        # the small magnitudes long contexts give
    if P > 10:
        levels[1, 1] = 0.25                                         # all equal: edges lower than the interior
    cfg = pkv.make_config(num_layers=1, num_q_heads=hkv, num_kv_heads=hkv, head_dim=64, window=alpha, pool_kernel=w,
                          dtype="fp32", avg_budget=alpha + k, beta=1.0, pool_kind=1)
    lens = [P + alpha] * batch
    ws = pkv.new_workspace(cfg, batch, P + alpha, DEV)
    scores = torch.from_numpy(levels).to(DEV)
    c = pkv.kept_count(cfg, k, P + alpha)
    idx = torch.full((batch * hkv * c,), -7, dtype=torch.int32, device=DEV)
    pkv.select_topk(cfg, scores, lens, k, idx, ws)
    pkv.check_status(ws)
    got = idx.cpu().numpy()
    for b, h, rows in packed_rows([c] * batch, hkv):
        if P + alpha <= alpha + k:
            want = np.arange(P + alpha)
        else:
            want = np.concatenate([oracle.select_topk(oracle.pool_avg(levels[b, h], w), k), np.arange(P, P + alpha)])
        np.testing.assert_array_equal(got[rows], want.astype(np.int32), err_msg="b=%d h=%d" % (b, h))


@pytest.mark.parametrize("base,kw", [
    (workloads.TINY, dict()),
    (workloads.LLAMA3_8B, dict(num_layers=2, seq_len=5037)),
    (workloads.LLAMA3_70B, dict(num_layers=3, seq_len=3011)),
], ids=["tiny_avg", "llama3_8b_5k_avg", "llama3_70b_3k_avg"])
def test_avg_pool_layer_matches_oracle(base, kw):
    w = workloads.scaled(base, name=base.name + "_avg", pool_kind="avg", **kw)
    for layer in range(w.num_layers):
        check_layer(w, layer, w.seq_lens())


# ----------------------------------------------------------------------------- alpha and beta sweeps
@pytest.mark.parametrize("alpha", [8, 16, 24, 40, 48])
def test_window_sizes_of_the_alpha_sweep(alpha):
    """Llama-3-8B head layout at a 128-entry budget, as in the appendix's study of alpha."""
    w = workloads.scaled(workloads.LLAMA3_8B, num_layers=4, seq_len=3000 + alpha, name="alpha_%d" % alpha,
                         window=alpha, avg_budget=128)
    for layer in (0, 3):
        check_layer(w, layer, w.seq_lens())


@pytest.mark.parametrize("beta", [1.0, 14.0, 16.0, 18.0])
def test_pyramid_slopes_of_the_beta_sweep(beta):
    """beta = 1 is the uniform split (every layer the same budget); 14..18 are the appendix's values."""
    w = workloads.scaled(workloads.LLAMA3_8B, num_layers=4, seq_len=2500, name="beta_%g" % beta, window=8,
                         avg_budget=128, beta=beta)
    budgets = pkv.layer_budgets(pkv.config_of(w))
    if beta == 1.0:
        assert budgets == [120] * 4
    else:
        assert budgets[0] > budgets[-1] and sum(budgets) == 4 * 120
    for layer in (0, 3):
        check_layer(w, layer, w.seq_lens())


# ----------------------------------------------------------------------------- retrieval-shaped sweep
@pytest.mark.parametrize("seq_len,depth,budget", [(1024, 0.1, 64), (4096, 0.9, 96), (8192, 0.5, 128),
                                                  (8192, 0.0, 64), (3000, 1.0, 128)])
def test_needle_sweep_cells_match_oracle(seq_len, depth, budget):
    """Cells of the context-length x depth x cache-size grid (Mistral-7B heads): same lists as the oracle, and
    the planted block is kept wherever the layer's budget has room for it."""
    w = workloads.needle_case(seq_len, depth, budget)
    budgets = pkv.layer_budgets(pkv.config_of(w))
    room = w.needle_block + w.n_sink + 2 * (w.pool_kernel - 1)
    for layer in (0, 12, 31):
        x, idx, k_out, v_out, ref = check_layer(w, layer, w.seq_lens())
        needle = set(x.planted[0][w.n_sink:])
        if budgets[layer] >= room:
            got = idx.cpu().numpy()
            for b, h, sl in packed_rows(ref["counts"], w.num_kv_heads):
                assert needle <= set(got[sl].tolist()), "needle evicted in layer %d head %d" % (layer, h)


# ----------------------------------------------------------------------------- geometric decay of the budgets
@pytest.mark.parametrize("layer", [0, 3, 7])
def test_geometric_schedule_through_the_fused_call(layer):
    """The appendix's geometric allocation: the same kernels with another budget per layer (the lowest layer keeps
    far more rows than under Eq. 1, the upper ones fewer)."""
    w = workloads.scaled(workloads.LLAMA3_8B, num_layers=8, seq_len=5000 + 17, avg_budget=256, schedule="geometric",
                         name="llama3_8b_geometric")
    geo = pkv.layer_budgets(pkv.config_of(w))
    lin = oracle.layer_budgets(w.num_layers, w.avg_budget, w.window, w.beta)
    assert geo[0] > lin[0] and geo[3] < lin[3] and sum(geo) == sum(lin)
    check_layer(w, layer, w.seq_lens())
