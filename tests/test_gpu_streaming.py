"""GPU parity of the whole-model drivers: the host pipeline (pinned K/V/Q in, compact cache out) must give
exactly what the device-resident calls give, with V copied to the device and with V left in pinned host
memory and read row by row over the bus."""
import types

import pytest
import torch

import paper_2406_02069_b200 as pkv
from paper_2406_02069_b200 import streaming, workloads

pytestmark = pytest.mark.gpu
DEV = "cuda"


def host_layer(x):
    return types.SimpleNamespace(q_win=x.q_win.cpu().pin_memory(), k=x.k.cpu().pin_memory(), v=x.v.cpu().pin_memory())


def host_out(rows, d, dtype):
    return types.SimpleNamespace(k=torch.empty(rows, d, dtype=dtype).pin_memory(),
                                 v=torch.empty(rows, d, dtype=dtype).pin_memory(),
                                 idx=torch.empty(rows, dtype=torch.int32).pin_memory())


def test_memory_kinds():
    assert pkv.memory_kind(torch.zeros(8, device=DEV)) == pkv.binding.MEM_DEVICE
    assert pkv.memory_kind(torch.zeros(8).pin_memory()) == pkv.binding.MEM_PINNED_HOST
    assert pkv.memory_kind(torch.zeros(8)) == pkv.binding.MEM_PAGEABLE_HOST


@pytest.mark.parametrize("w", [
    workloads.scaled(workloads.LLAMA3_8B, num_layers=5, seq_len=6011, name="llama3_8b_6k"),
    workloads.scaled(workloads.MISTRAL_RAGGED, num_layers=4, batch=3, name="mistral_b3"),
], ids=lambda w: w.name)
@pytest.mark.parametrize("zero_copy_v", [False, True])
def test_host_pipeline_equals_device_resident_calls(w, zero_copy_v):
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    if w.batch > 1:
        lens = [500 + (n % 1777) for n in lens]
    layers = [workloads.make_layer(w, l, device=DEV, seq_lens=lens) for l in range(w.num_layers)]
    out = streaming.LayerOutputs(cfg, lens, w.torch_dtype())
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    streaming.compress_model(cfg, layers, lens, out, ws)
    pkv.check_status(ws)

    pipe = streaming.HostPipeline(cfg, lens, layers[0].q_win.shape, layers[0].k.shape, w.torch_dtype(),
                                  zero_copy_v=zero_copy_v)
    hl = [host_layer(x) for x in layers]
    ho = [host_out(r, w.head_dim, w.torch_dtype()) for r in out.rows]
    for rep in range(2):                                              # the second run reuses every buffer
        pipe.run(hl, ho)
        torch.cuda.synchronize()
        pkv.check_status(pipe.workspace)
        for l in range(w.num_layers):
            assert torch.equal(ho[l].idx, out.idx[l].cpu())
            assert torch.equal(ho[l].k, out.k[l].cpu()) and torch.equal(ho[l].v, out.v[l].cpu())
    esz = layers[0].k.element_size()
    qk_bytes = sum((x.k.numel() + x.q_win.numel()) * esz for x in layers)
    v_bytes = sum(x.v.numel() * esz for x in layers)
    if zero_copy_v:                                                  # of V only the kept rows crossed the bus
        assert pipe.h2d_bytes == qk_bytes + sum(out.rows) * w.head_dim * esz
    else:
        assert pipe.h2d_bytes == qk_bytes + v_bytes


@pytest.mark.parametrize("w", [
    workloads.scaled(workloads.LLAMA3_8B, num_layers=6, seq_len=6011, name="llama3_8b_6k"),
    workloads.scaled(workloads.MISTRAL_RAGGED, num_layers=5, batch=3, name="mistral_b3"),
    workloads.TINY,
], ids=lambda w: w.name)
def test_two_lanes_give_the_per_layer_results(w):
    """Score sweeps of layer l + 1 beside selection and gather of layer l, on disjoint groups of SMs: the
    outputs must be those of the per-layer calls, bit for bit, run after run."""
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    if w.batch > 1:
        lens = [500 + (n % 1777) for n in lens]
    layers = [workloads.make_layer(w, l, device=DEV, seq_lens=lens) for l in range(w.num_layers)]
    want = streaming.LayerOutputs(cfg, lens, w.torch_dtype())
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    streaming.compress_model(cfg, layers, lens, want, ws)
    pkv.check_status(ws)
    try:
        lanes = pkv.Lanes(select_sms=8)
    except pkv.PkvError as e:
        pytest.skip("this driver cannot split the SMs: %s" % e)
    assert lanes.select_sms == 8 and lanes.score_sms >= 8
    pair = [pkv.new_workspace(cfg, len(lens), max(lens), DEV) for _ in range(2)]
    for rep in range(3):
        got = streaming.LayerOutputs(cfg, lens, w.torch_dtype())
        for t in got.k + got.v:
            t.fill_(-7.0)
        streaming.compress_model(cfg, layers, lens, got, pair, lanes=lanes)
        torch.cuda.current_stream().synchronize()          # the call joins the lanes back into this stream
        for x in pair:
            pkv.check_status(x)
        for l in range(w.num_layers):
            assert torch.equal(got.idx[l], want.idx[l]), "layer %d" % l
            assert torch.equal(got.k[l], want.k[l]) and torch.equal(got.v[l], want.v[l])
    lanes.close()


@pytest.mark.parametrize("w", [
    workloads.scaled(workloads.LLAMA3_8B, num_layers=8, seq_len=9001, name="llama3_8b_9k"),
    workloads.scaled(workloads.LLAMA2_7B, num_layers=8, seq_len=1500, name="llama2_7b_1k5"),
], ids=lambda w: w.name)
def test_back_to_back_passes_share_one_workspace_without_races(w):
    """Kernels of consecutive layers overlap at their edges (the sweeps of a layer start while the selection of
    the layer before still runs) and all layers share one workspace: many passes enqueued without a pause must
    reproduce, in every layer, what a pass with a full stop after every layer gives."""
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    layers = [workloads.make_layer(w, l, device=DEV) for l in range(w.num_layers)]
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    want = streaming.LayerOutputs(cfg, lens, w.torch_dtype())
    for l, x in enumerate(layers):
        pkv.compress_layer(cfg, l, x.q_win, x.k, x.v, lens, want.k[l], want.v[l], want.idx[l], ws)
        torch.cuda.synchronize()
    got = streaming.LayerOutputs(cfg, lens, w.torch_dtype())
    for rep in range(25):
        streaming.compress_model(cfg, layers, lens, got, ws)
    torch.cuda.synchronize()
    pkv.check_status(ws)
    for l in range(w.num_layers):
        assert torch.equal(got.idx[l], want.idx[l]), "layer %d" % l
        assert torch.equal(got.k[l], want.k[l]) and torch.equal(got.v[l], want.v[l])
