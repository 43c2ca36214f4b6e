"""GPU parity of the kernel that is the prefill attention of the last alpha queries and emits the window scores
from inside it (Section 4.1, Section 4.2.2 Eq. 2-3): attention output and scores against the oracle, the kept
lists of the fused layer call against the oracle too.

Tolerance of the attention output.  The kernel rounds each probability p_i to the inputs' 16-bit type before it
multiplies V (relative error at most 2^-9 for bfloat16, 2^-12 for binary16) and forms p_i with the same
approximations as the scores (2e-3 relative).  With out_c = sum_i p_i v_ic the error is therefore at most
(2^-9 + 2e-3) * sum_i p_i |v_ic| < 4e-3 * A_c, where A_c is the attention output over |V|, which the oracle computes.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2406_02069_b200 as pkv
from paper_2406_02069_b200 import binding, workloads
from helpers import assert_indices_match, assert_scores_close, packed_rows

pytestmark = pytest.mark.gpu
DEV = "cuda"
OUT_RTOL = 4e-3      # of A_c, see above
OUT_ATOL = 1e-6


def make_inputs(hq, hkv, alpha, lens, dtype, seed, pad_value=None):
    g = torch.Generator(device="cpu").manual_seed(seed)
    n_max, d = max(lens), 128
    q = (torch.randn(len(lens), hq, alpha, d, generator=g) * 1.2).to(dtype)
    k = torch.randn(len(lens), hkv, n_max, d, generator=g).to(dtype)
    v = torch.randn(len(lens), hkv, n_max, d, generator=g).to(dtype)
    k[:, :, 0] *= 3.0                                   # a sink
    for b, n in enumerate(lens):                        # a few keys aligned with the window queries
        for j, pos in enumerate(range(n // 3, n, max(1, n // 5))):
            k[b, :, pos] = (q[b, :: hq // hkv, j % alpha].float() * 0.9).to(dtype)
        if pad_value is not None and n < n_max:
            k[b, :, n:] = pad_value
            v[b, :, n:] = pad_value
    return q, k, v


def check_attention(got_out, q, k, v, lens, alpha, hq, hkv, sample=None):
    """sample: None = every query head, else the (KV head, member of its group) pairs to check."""
    G = hq // hkv
    for b, n in enumerate(lens):
        pos = np.arange(n)
        for h in range(hkv):
            kb, vb = k[b, h, :n], v[b, h, :n]
            for g in range(G):
                if sample is not None and (h, g) not in sample:
                    continue
                want = oracle.window_attention(q[b, h * G + g], kb, vb, pos, n)
                bound = oracle.window_attention(q[b, h * G + g], kb, vb.abs(), pos, n)
                err = np.abs(got_out[b, h * G + g].astype(np.float64) - want)
                worst = (err / (OUT_RTOL * bound + OUT_ATOL)).max()
                assert worst <= 1.0, "seq %d query head %d: %.3f of the tolerance" % (b, h * G + g, worst)


@pytest.mark.parametrize("hq,hkv,alpha,lens,dtype", [
    (16, 2, 32, [1500], torch.bfloat16),               # R = 256: two units per K tile, scores exchanged between groups
    (8, 2, 32, [700, 129, 1290], torch.bfloat16),      # R = 128, ragged batch, tails of every kind
    (4, 4, 32, [1000, 40], torch.bfloat16),            # R = 32 (no grouping): P x V padded to a 64-row block
    (6, 2, 16, [390], torch.bfloat16),                 # R = 48 -> 64 columns
    (12, 4, 8, [257, 2100], torch.float16),            # binary16, R = 24 -> 32 columns
    (16, 2, 16, [2049], torch.float16),                # binary16, R = 128
    (24, 4, 40, [3000, 777], torch.bfloat16),          # alpha = 40, R = 240 -> 256 columns, many CTAs per head
], ids=["r256", "r128_ragged", "r32", "r48", "fp16_r24", "fp16_r128", "r240"])
def test_window_attention_and_scores_match_the_oracle(hq, hkv, alpha, lens, dtype):
    cfg = pkv.make_config(num_layers=1, num_q_heads=hq, num_kv_heads=hkv, head_dim=128, window=alpha, pool_kernel=7,
                          dtype="fp16" if dtype == torch.float16 else "bf16", avg_budget=alpha, beta=1.0)
    q, k, v = make_inputs(hq, hkv, alpha, lens, dtype, seed=hq * 1000 + alpha)
    n_max = max(lens)
    ws = pkv.new_workspace(cfg, len(lens), n_max, DEV)
    scores = torch.full((len(lens), hkv, n_max), -1.0, dtype=torch.float32, device=DEV)
    out = torch.full((len(lens), hq, alpha, 128), float("nan"), dtype=torch.float32, device=DEV)
    pkv.attend_window(cfg, q.to(DEV), k.to(DEV), v.to(DEV), lens, out, scores, ws)
    pkv.check_status(ws)
    got_scores, got_out = scores.cpu().numpy(), out.cpu().numpy()
    assert np.isfinite(got_out).all()
    for b, n in enumerate(lens):
        want, _ = oracle.window_scores(q[b], k[b, :, :n])
        assert_scores_close(got_scores[b, :, : n - alpha], want, "seq %d" % b)
        assert (got_scores[b, :, n - alpha:] == -1.0).all()
    check_attention(got_out, q, k, v, lens, alpha, hq, hkv)


def test_rows_behind_a_sequence_are_never_used():
    """In a ragged batch the tensors hold rows behind the shorter sequences.  Whatever they contain (here NaN in K
    and V), outputs are finite and equal to those of a run with zeros there."""
    hq, hkv, alpha, lens = 8, 2, 32, [1100, 333, 640]
    cfg = pkv.make_config(num_layers=1, num_q_heads=hq, num_kv_heads=hkv, head_dim=128, window=alpha, pool_kernel=7,
                          dtype="bf16", avg_budget=alpha, beta=1.0)
    results = []
    for pad in (0.0, float("nan")):
        q, k, v = make_inputs(hq, hkv, alpha, lens, torch.bfloat16, seed=11, pad_value=pad)
        ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
        scores = torch.zeros((len(lens), hkv, max(lens)), dtype=torch.float32, device=DEV)
        out = torch.zeros((len(lens), hq, alpha, 128), dtype=torch.float32, device=DEV)
        pkv.attend_window(cfg, q.to(DEV), k.to(DEV), v.to(DEV), lens, out, scores, ws)
        pkv.check_status(ws)
        results.append((scores.cpu(), out.cpu()))
    assert torch.isfinite(results[1][1]).all() and torch.isfinite(results[1][0]).all()
    assert torch.equal(results[0][0], results[1][0]) and torch.equal(results[0][1], results[1][1])


@pytest.mark.parametrize("base,kw", [
    (workloads.LLAMA3_8B, dict(num_layers=2, seq_len=5037)),
    (workloads.LLAMA3_70B, dict(num_layers=2, seq_len=4200)),
    (workloads.MISTRAL_RAGGED, dict(num_layers=2, batch=3)),
], ids=["llama3_8b_5k", "llama3_70b_4k", "mistral_b3"])
def test_fused_layer_call_matches_the_oracle(base, kw):
    """The layer call that also returns the window rows' attention: kept lists and gathered rows against the oracle
    as for the plain call, attention output against the oracle."""
    w = workloads.scaled(base, name=base.name + "_attend", **kw)
    lens = w.seq_lens()
    if w.batch > 1:
        lens = [300 + (n % 1777) for n in lens]
    cfg = pkv.config_of(w)
    budgets = pkv.layer_budgets(cfg)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    for layer in range(w.num_layers):
        kl = budgets[layer]
        x = workloads.make_layer(w, layer, device=DEV, seq_lens=lens)
        rows = pkv.total_rows(cfg, kl, lens)
        k_out = torch.empty(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
        v_out = torch.empty_like(k_out)
        idx = torch.empty(rows, dtype=torch.int32, device=DEV)
        out = torch.empty(len(lens), w.num_q_heads, w.window, w.head_dim, dtype=torch.float32, device=DEV)
        pkv.attend_compress_layer(cfg, layer, x.q_win, x.k, x.v, lens, out, k_out, v_out, idx, ws)
        pkv.check_status(ws)
        ref = oracle.compress_batch(x.q_win.cpu(), x.k.cpu(), x.v.cpu(), lens, pool_kernel=w.pool_kernel,
                                    avg_budget=w.avg_budget, k_layer=kl, pool_kind=w.pool_kind)
        got_idx = idx.cpu().numpy()
        for b, h, sl in packed_rows(ref["counts"], w.num_kv_heads):
            assert_indices_match(got_idx[sl], ref["indices"][sl], ref["scores"][b][h], w.pool_kernel, w.window,
                                 "%s layer %d b %d h %d" % (w.name, layer, b, h), pool_kind=w.pool_kind)
            sel = idx[sl].long()
            assert torch.equal(k_out[sl], x.k[b, h, sel]) and torch.equal(v_out[sl], x.v[b, h, sel])
        check_attention(out.cpu().numpy(), x.q_win.cpu(), x.k.cpu(), x.v.cpu(), lens, w.window, w.num_q_heads,
                        w.num_kv_heads)


@pytest.mark.parametrize("w,layer,sample", [
    (workloads.LLAMA3_70B, 79, {(0, 0), (3, 5), (7, 7)}),
    (workloads.LLAMA2_7B, 0, {(0, 0), (13, 0), (31, 0)}),
    (workloads.MISTRAL_RAGGED, 0, {(0, 0), (2, 3), (7, 1)}),
], ids=lambda x: getattr(x, "name", None))
def test_full_size_layer_with_attention(w, layer, sample):
    """The configurations at their full sizes, in the launch shapes `bench.py --mode attend` times: every score and
    every kept list of the layer against the oracle, the attention output of sampled query heads."""
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    kl = pkv.layer_budgets(cfg)[layer]
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    x = workloads.make_layer(w, layer, device=DEV)
    rows = pkv.total_rows(cfg, kl, lens)
    k_out = torch.empty(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
    v_out = torch.empty_like(k_out)
    idx = torch.empty(rows, dtype=torch.int32, device=DEV)
    scores = torch.full((len(lens), w.num_kv_heads, max(lens)), -1.0, dtype=torch.float32, device=DEV)
    out = torch.empty(len(lens), w.num_q_heads, w.window, w.head_dim, dtype=torch.float32, device=DEV)
    pkv.attend_compress_layer(cfg, layer, x.q_win, x.k, x.v, lens, out, k_out, v_out, idx, ws, scores=scores)
    pkv.check_status(ws)
    qc, kc, vc = x.q_win.cpu(), x.k.cpu(), x.v.cpu()
    ref = oracle.compress_batch(qc, kc, vc, lens, pool_kernel=w.pool_kernel, avg_budget=w.avg_budget, k_layer=kl)
    got_scores, got_idx = scores.cpu().numpy(), idx.cpu().numpy()
    for b, n in enumerate(lens):
        assert_scores_close(got_scores[b, :, : n - w.window], ref["scores"][b], "%s seq %d" % (w.name, b))
    for b, h, sl in packed_rows(ref["counts"], w.num_kv_heads):
        assert_indices_match(got_idx[sl], ref["indices"][sl], ref["scores"][b][h], w.pool_kernel, w.window,
                             "%s b %d h %d" % (w.name, b, h))
        sel = idx[sl].long()
        assert torch.equal(k_out[sl], x.k[b, h, sel]) and torch.equal(v_out[sl], x.v[b, h, sel])
    check_attention(out.cpu().numpy(), qc, kc, vc, lens, w.window, w.num_q_heads, w.num_kv_heads, sample=sample)


def test_shapes_the_kernel_does_not_take_are_refused():
    cfg = pkv.make_config(num_layers=1, num_q_heads=4, num_kv_heads=2, head_dim=64, window=8, pool_kernel=5,
                          dtype="bf16", avg_budget=8, beta=1.0)
    q = torch.zeros(1, 4, 8, 64, dtype=torch.bfloat16, device=DEV)
    k = torch.zeros(1, 2, 100, 64, dtype=torch.bfloat16, device=DEV)
    ws = pkv.new_workspace(cfg, 1, 100, DEV)
    scores = torch.zeros(1, 2, 100, dtype=torch.float32, device=DEV)
    out = torch.zeros(1, 4, 8, 64, dtype=torch.float32, device=DEV)
    with pytest.raises(pkv.PkvError) as err:
        pkv.attend_window(cfg, q, k, k, [100], out, scores, ws)
    assert err.value.status == 2      # PKV_ERR_UNSUPPORTED: head_dim 64


def test_a_wait_that_runs_out_in_the_attention_kernel_is_reported():
    """One K tile of one CTA of the window-attention kernel is never loaded and the bound of the waits is lowered to
    about a millisecond: the kernel winds down by itself (every role leaves, accumulator memory released), the status
    word says so, and the next ordinary call on the same workspace gives what a fresh workspace gives."""
    hq, hkv, alpha, lens = 16, 2, 32, [5000]
    cfg = pkv.make_config(num_layers=1, num_q_heads=hq, num_kv_heads=hkv, head_dim=128, window=alpha, pool_kernel=7,
                          dtype="bf16", avg_budget=alpha, beta=1.0)
    q, k, v = (t.to(DEV) for t in make_inputs(hq, hkv, alpha, lens, torch.bfloat16, seed=3))
    ws = pkv.new_workspace(cfg, 1, max(lens), DEV)
    scores = torch.zeros(1, hkv, max(lens), dtype=torch.float32, device=DEV)
    out = torch.zeros(1, hq, alpha, 128, dtype=torch.float32, device=DEV)
    try:
        binding.test_hooks(wait_clocks=1 << 21, withhold_attend_tile=True)
        pkv.attend_window(cfg, q, k, v, lens, out, scores, ws)
        with pytest.raises(pkv.PkvError) as e:
            pkv.check_status(ws)
        assert e.value.status == binding.PKV_ERR_DEVICE_STATUS and "0x2" in str(e.value)
    finally:
        binding.test_hooks(0, False)
    ws[:256].zero_()
    again_s, again_o = torch.zeros_like(scores), torch.zeros_like(out)
    pkv.attend_window(cfg, q, k, v, lens, again_o, again_s, ws)
    pkv.check_status(ws)
    fresh_ws = pkv.new_workspace(cfg, 1, max(lens), DEV)
    fresh_s, fresh_o = torch.zeros_like(scores), torch.zeros_like(out)
    pkv.attend_window(cfg, q, k, v, lens, fresh_o, fresh_s, fresh_ws)
    pkv.check_status(fresh_ws)
    assert torch.equal(again_s, fresh_s) and torch.equal(again_o, fresh_o)
    check_attention(again_o.cpu().numpy(), q.cpu(), k.cpu(), v.cpu(), lens, alpha, hq, hkv)
