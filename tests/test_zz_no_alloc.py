"""The workspace-free scoring call (pyramidkv_score_window_static).

Some users of the library may not allocate device memory where they call it: an
operator inside a serving engine that owns the whole memory pool, or code that is
handed nothing but its input and output tensors.  For them the library carries its
own fixed 8 MiB of scratch.  This file checks, through the C boundary, that the
call gives the same scores as the ordinary workspace-taking call, twice in a row
(the built-in array is shared by all calls and keeps the previous call's contents),
that those scores are the oracle's, that the largest graded shape fits, and that a
problem too large for the array is refused up front.

The file name sorts last on purpose, so a run that stops at the first failure has
already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2406_02069_b200 as pkv
from paper_2406_02069_b200 import binding, workloads
from helpers import assert_scores_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


def scores_both_ways(w, layer, lens):
    cfg = pkv.config_of(w)
    x = workloads.make_layer(w, layer, device=DEV, seq_lens=lens)
    ld = max(lens) - w.window
    want = torch.zeros(len(lens), w.num_kv_heads, ld, dtype=torch.float32, device=DEV)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    pkv.score_window(cfg, x.q_win, x.k, lens, want, ws)
    pkv.check_status(ws)
    got = torch.zeros_like(want)
    pkv.score_window_static(cfg, x.q_win, x.k, lens, got)
    pkv.check_status_static()                                   # synchronises; the array's own status word is clean
    return got.cpu().numpy(), want.cpu().numpy()


def test_static_scratch_scores_equal_workspace_scores_twice_in_a_row():
    # two different shapes back to back: the second call finds the first one's leftovers in the array
    first = workloads.scaled(workloads.LLAMA3_8B, num_layers=2, seq_len=6000 + 13, name="static_a")
    second = workloads.scaled(workloads.MISTRAL_RAGGED, num_layers=2, batch=3, name="static_b")
    for w, layer, lens in ((first, 0, first.seq_lens()), (second, 1, [1500, 777, 2049]), (first, 1, first.seq_lens())):
        got, want = scores_both_ways(w, layer, lens)
        for b, n in enumerate(lens):
            P = n - w.window
            assert_scores_close(got[b, :, :P], want[b, :, :P], "static vs workspace, %s seq %d" % (w.name, b))
            assert np.isfinite(got[b, :, :P]).all() and got[b, :, :P].max() > 0


@pytest.mark.parametrize("w", [workloads.scaled(workloads.LLAMA3_8B, num_layers=2, seq_len=3000 + 41, name="static_bf16"),
                               workloads.TINY], ids=lambda w: w.name)
def test_static_scratch_scores_are_the_oracles(w):
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    x = workloads.make_layer(w, 1, device=DEV)
    got = torch.zeros(len(lens), w.num_kv_heads, max(lens) - w.window, dtype=torch.float32, device=DEV)
    pkv.score_window_static(cfg, x.q_win, x.k, lens, got)
    pkv.check_status_static()
    for b, n in enumerate(lens):
        want, _ = oracle.window_scores(x.q_win[b].cpu(), x.k[b, :, :n].cpu())
        assert_scores_close(got[b, :, : n - w.window].cpu().numpy(), want, "static vs oracle, %s seq %d" % (w.name, b))


def test_the_128k_eight_head_256_row_shape_fits_the_built_in_scratch():
    """One layer of the long-context configuration (131072 keys, 8 KV heads, 8 x 32 window rows, 16-bit inputs):
    the tensor-core sweeps need a few megabytes of scratch whatever the context length."""
    w = workloads.scaled(workloads.LLAMA3_70B, num_layers=2, name="llama3_70b_one_layer")
    got, want = scores_both_ways(w, 0, w.seq_lens())
    P = w.seq_lens()[0] - w.window
    assert_scores_close(got[0, :, :P], want[0, :, :P], "static vs workspace, 128k")
    assert np.isfinite(got).all() and got.max() > 0


def test_problem_larger_than_the_built_in_scratch_is_refused():
    """fp32 inputs go through the fp32-pipe kernels, which keep statistics per 128-key chunk: 33000 keys x 8 heads
    x 256 rows need a little over 8 MiB.  Every tensor is as large as the call says, so a refusal that came too
    late would still only touch valid memory."""
    w = workloads.scaled(workloads.LLAMA3_70B, name="llama3_70b_fp32_33k", dtype="fp32", num_layers=1, seq_len=33000)
    cfg = pkv.config_of(w)
    x = workloads.make_layer(w, 0, device=DEV)
    scores = torch.zeros(1, w.num_kv_heads, 33000, dtype=torch.float32, device=DEV)
    with pytest.raises(pkv.PkvError) as e:                          # refused before any kernel is enqueued
        pkv.score_window_static(cfg, x.q_win, x.k, [33000], scores)
    assert e.value.status == binding.PKV_ERR_STATIC_SCRATCH
    assert "built-in scratch" in str(e.value)
    pkv.check_status_static()
    assert float(scores.abs().max()) == 0.0                         # nothing ran
