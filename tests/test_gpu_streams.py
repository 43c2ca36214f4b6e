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
