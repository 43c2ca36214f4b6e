"""The workspace-free scoring call (pyramidkv_score_window_static).

Some users of the library may not allocate device memory where they call it: an
operator inside a serving engine that owns the whole memory pool, or code that is
handed nothing but its input and output tensors.  For them the library carries its
own fixed 8 MiB of scratch.  This file checks, through the C boundary, that the
call gives the same scores as the ordinary workspace-taking call, twice in a row
(the built-in array is shared by all calls and keeps the previous call's contents),
and that a problem too large for the array is refused up front.

The file name sorts last on purpose, so a run that stops at the first failure has
already run every other test.
"""
import numpy as np
import pytest
import torch

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
    torch.cuda.synchronize()
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


def test_problem_larger_than_the_built_in_scratch_is_refused():
    # 128k tokens in fp32: the fp32-pipe kernels keep statistics per 128-key chunk, ~34 MB of scratch
    w = workloads.scaled(workloads.LLAMA3_70B, name="llama3_70b_fp32", dtype="fp32")
    cfg = pkv.config_of(w)
    assert pkv.workspace_bytes(cfg, 1, 131072) > binding.PKV_STATIC_SCRATCH_BYTES
    small = workloads.make_layer(workloads.scaled(w, num_layers=1, seq_len=256), 0, device=DEV)
    scores = torch.zeros(1, w.num_kv_heads, 131072, dtype=torch.float32, device=DEV)
    with pytest.raises(pkv.PkvError) as e:                          # refused before any kernel is enqueued
        pkv.score_window_static(cfg, small.q_win, small.k, [131072], scores)
    assert e.value.status == binding.PKV_ERR_STATIC_SCRATCH
    assert "built-in scratch" in str(e.value)
    torch.cuda.synchronize()
