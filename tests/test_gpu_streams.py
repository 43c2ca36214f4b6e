"""The layers of a model are independent, so the whole-model driver may spread them over several CUDA streams (a
workspace per stream).  Results must not depend on it: every layer's kept list and gathered rows are compared bit
for bit with the single-stream run, on the tensor-core sweeps, the single-sweep kernel for short contexts and a
ragged batch, with the call made from a stream of the caller's own."""
import pytest
import torch

import paper_2406_02069_b200 as pkv
from paper_2406_02069_b200 import streaming, workloads

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("base,kw,count", [
    (workloads.LLAMA3_8B, dict(num_layers=7, seq_len=6000 + 11), 3),
    (workloads.LLAMA2_7B, dict(num_layers=6, seq_len=4096), 4),
    (workloads.MISTRAL_RAGGED, dict(num_layers=5, batch=3), 2),
    (workloads.LLAMA3_70B, dict(num_layers=4, seq_len=9000), 8),      # more streams than layers
], ids=["llama3_8b", "llama2_7b_resident", "mistral_ragged", "llama3_70b"])
def test_layers_on_several_streams_give_the_single_stream_result(base, kw, count):
    w = workloads.scaled(base, name=base.name + "_streams", **kw)
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    if w.batch > 1:
        lens = [500 + (n % 3000) for n in lens]
    layers = [workloads.make_layer(w, l, device=DEV, seq_lens=lens) for l in range(w.num_layers)]
    ref = streaming.LayerOutputs(cfg, lens, w.torch_dtype(), DEV)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    streaming.compress_model(cfg, layers, lens, ref, ws)
    pkv.check_status(ws)
    got = streaming.LayerOutputs(cfg, lens, w.torch_dtype(), DEV)
    for t in got.k + got.v:
        t.zero_()
    for t in got.idx:
        t.fill_(-1)
    ls = streaming.LayerStreams(cfg, lens, count, DEV)
    mine = torch.cuda.Stream()
    mine.wait_stream(torch.cuda.current_stream())      # the fills above
    for _ in range(2):                                  # twice: the second pass reuses every workspace
        streaming.compress_model(cfg, layers, lens, got, None, stream=mine, layer_streams=ls)
    # the caller's stream is ordered behind all layer streams: reading through it needs no other synchronisation
    with torch.cuda.stream(mine):
        copies = [(a.cpu(), b.cpu(), c.cpu()) for a, b, c in zip(got.k, got.v, got.idx)]
    mine.synchronize()
    ls.check_status()
    for l, (k, v, i) in enumerate(copies):
        assert torch.equal(i, ref.idx[l].cpu()), "layer %d: kept list" % l
        assert torch.equal(k, ref.k[l].cpu()) and torch.equal(v, ref.v[l].cpu()), "layer %d: rows" % l


def test_a_step_on_several_streams_can_be_captured_in_one_cuda_graph():
    """Fork and join are events, so a whole step on several streams is one graph; replaying it gives the same cache."""
    w = workloads.scaled(workloads.LLAMA3_8B, name="llama3_8b_streams_graph", num_layers=5, seq_len=4000 + 3)
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    layers = [workloads.make_layer(w, l, device=DEV) for l in range(w.num_layers)]
    ref = streaming.LayerOutputs(cfg, lens, w.torch_dtype(), DEV)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    streaming.compress_model(cfg, layers, lens, ref, ws)
    pkv.check_status(ws)
    got = streaming.LayerOutputs(cfg, lens, w.torch_dtype(), DEV)
    ls = streaming.LayerStreams(cfg, lens, 3, DEV)
    streaming.compress_model(cfg, layers, lens, got, None, layer_streams=ls)      # warms every first-use path
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            streaming.compress_model(cfg, layers, lens, got, None, layer_streams=ls)
    for t in got.k + got.v:
        t.zero_()
    for t in got.idx:
        t.fill_(-1)
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    ls.check_status()
    for l in range(w.num_layers):
        assert torch.equal(got.idx[l], ref.idx[l]) and torch.equal(got.k[l], ref.k[l]) and torch.equal(got.v[l], ref.v[l])


@pytest.mark.parametrize("sweep_ctas", [1, 37, 74, 1024])
def test_a_share_of_the_sms_for_the_sweeps_changes_nothing_but_rounding(sweep_ctas):
    """pkv_config.sweep_ctas caps the CTAs of the persistent score sweeps (a caller's way to let two layers' sweeps run
    side by side).  Whatever the cap, down to a single CTA that walks every head, the scores stay within the
    tolerance of the oracle and the kept lists match it; the window-attention call honours the cap too."""
    import numpy as np
    import oracle
    from helpers import assert_indices_match, assert_scores_close, packed_rows
    w = workloads.scaled(workloads.MISTRAL_RAGGED, name="mistral_sweep_ctas", num_layers=2, batch=3)
    lens = [300 + (n % 1500) for n in w.seq_lens()]
    cfg = pkv.config_of(w, sweep_ctas=sweep_ctas)
    assert cfg.sweep_ctas == sweep_ctas
    layer = 1
    kl = pkv.layer_budgets(cfg)[layer]
    x = workloads.make_layer(w, layer, device=DEV, seq_lens=lens)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    rows = pkv.total_rows(cfg, kl, lens)
    k_out = torch.empty(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
    v_out = torch.empty_like(k_out)
    idx = torch.empty(rows, dtype=torch.int32, device=DEV)
    scores = torch.zeros(len(lens), w.num_kv_heads, max(lens), dtype=torch.float32, device=DEV)
    pkv.compress_layer(cfg, layer, x.q_win, x.k, x.v, lens, k_out, v_out, idx, ws, scores=scores)
    pkv.check_status(ws)
    ref = oracle.compress_batch(x.q_win.cpu(), x.k.cpu(), x.v.cpu(), lens, pool_kernel=w.pool_kernel,
                                avg_budget=w.avg_budget, k_layer=kl)
    got_scores, got_idx = scores.cpu().numpy(), idx.cpu().numpy()
    for b, n in enumerate(lens):
        assert_scores_close(got_scores[b, :, : n - w.window], ref["scores"][b], "seq %d" % b)
    for b, h, sl in packed_rows(ref["counts"], w.num_kv_heads):
        assert_indices_match(got_idx[sl], ref["indices"][sl], ref["scores"][b][h], w.pool_kernel, w.window,
                             "b %d h %d" % (b, h))
    # the fused attention call under the same cap
    out = torch.empty(len(lens), w.num_q_heads, w.window, w.head_dim, dtype=torch.float32, device=DEV)
    scores2 = torch.zeros_like(scores)
    pkv.attend_window(cfg, x.q_win, x.k, x.v, lens, out, scores2, ws)
    pkv.check_status(ws)
    got2 = scores2.cpu().numpy()
    for b, n in enumerate(lens):
        assert_scores_close(got2[b, :, : n - w.window], ref["scores"][b], "attend seq %d" % b)
    assert np.isfinite(out.cpu().numpy()).all()


def test_a_cap_above_the_limit_is_refused():
    w = workloads.scaled(workloads.LLAMA3_8B, name="cap", num_layers=1, seq_len=500)
    cfg = pkv.config_of(w, sweep_ctas=1025)
    with pytest.raises(pkv.PkvError) as err:
        pkv.layer_budgets(cfg)
    assert err.value.status == 1      # PKV_ERR_INVALID_ARG
