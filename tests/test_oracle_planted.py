"""The synthetic stand-in for the retrieval result: planted tokens survive compression in the oracle.

The paper reports that a fact placed at any depth of a long context stays retrievable after compression.
Without the model and the benchmark's items, the checkable part is structural: keys that the window
attends to strongly (sinks, a planted block) are in the kept set of every layer whose budget has room for
their pooled plateaus.
"""
import numpy as np
import pytest

import oracle
from paper_2406_02069_b200 import workloads


def needle_recall(kept_row, needle):
    return len(set(needle) & set(int(x) for x in kept_row)) / len(needle)


@pytest.mark.parametrize("depth", [0.0, 0.5, 1.0])
@pytest.mark.parametrize("budget", [64, 96, 128])
def test_needle_block_survives_where_the_budget_has_room(depth, budget):
    w = workloads.needle_case(2048, depth, budget)
    budgets = oracle.layer_budgets(w.num_layers, w.avg_budget, w.window, w.beta)
    assert sum(budgets) == w.num_layers * (budget - w.window)
    lens = w.seq_lens()
    room = w.needle_block + w.n_sink + 2 * (w.pool_kernel - 1)          # the plateaus of block and sinks
    checked = 0
    for layer in (0, 8, 16, 31):
        x = workloads.make_layer(w, layer)
        sinks, needle = x.planted[0][: w.n_sink], x.planted[0][w.n_sink:]
        assert len(needle) == w.needle_block and needle == list(range(needle[0], needle[0] + w.needle_block))
        prefix = lens[0] - w.window
        want_start = w.n_sink + round(depth * (prefix - w.needle_block - w.n_sink - 1))
        assert needle[0] == want_start                                 # the block sits at the asked depth
        r = oracle.compress_layer(x.q_win[0], x.k[0], x.v[0], pool_kernel=w.pool_kernel, avg_budget=budget,
                                  k_layer=budgets[layer], want_scores=False)
        if budgets[layer] >= room:
            for h in range(w.num_kv_heads):
                assert needle_recall(r["kept"][h], needle) == 1.0, (layer, h)
                assert set(sinks) <= set(r["kept"][h].tolist())
            checked += 1
    assert checked >= 2                                                # the low layers always have room


def test_depth_moves_the_block_and_nothing_else():
    a = workloads.make_layer(workloads.needle_case(1024, 0.1, 128), 3)
    b = workloads.make_layer(workloads.needle_case(1024, 0.9, 128), 3)
    assert a.planted[0][:4] == b.planted[0][:4] and a.planted[0][4] < b.planted[0][4]
    assert (a.q_win == b.q_win).all() and (a.v == b.v).all()
    moved = (a.k != b.k).any(dim=-1).any(dim=1)[0].nonzero().flatten().tolist()
    assert set(moved) == set(a.planted[0][4:]) | set(b.planted[0][4:])
