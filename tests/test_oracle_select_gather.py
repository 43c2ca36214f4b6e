"""Pins for the oracle's pooling, top-k selection, window retention and gather."""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- pooling
@pytest.mark.parametrize("P,w", [(1, 1), (1, 5), (2, 7), (3, 3), (17, 5), (100, 7), (64, 1), (9, 9), (5, 11)])
def test_pool_equals_library_max_pool(P, w):
    rng = np.random.default_rng(P * 31 + w)
    x = rng.random(P).astype(np.float32)
    got = oracle.pool_max(x, w)
    want = torch.nn.functional.max_pool1d(torch.from_numpy(x).view(1, 1, P), kernel_size=w, stride=1,
                                          padding=(w - 1) // 2).view(-1).numpy()
    np.testing.assert_array_equal(got, want)
    assert (got >= x).all()
    if w == 1:
        np.testing.assert_array_equal(got, x)


def test_pool_rejects_even_width():
    with pytest.raises(ValueError):
        oracle.pool_max(np.zeros(8, dtype=np.float32), 4)


def test_pool_spreads_one_spike_over_w_positions():
    x = np.zeros(40, dtype=np.float32)
    x[20] = 1.0
    got = oracle.pool_max(x, 7)
    assert list(np.nonzero(got)[0]) == list(range(17, 24))
    x[:] = 0.25
    np.testing.assert_array_equal(oracle.pool_max(x, 7), x)


# ----------------------------------------------------------------------------- mean pool (variant)
@pytest.mark.parametrize("P,w", [(1, 1), (1, 5), (2, 7), (3, 3), (17, 5), (100, 7), (64, 1), (9, 9), (5, 11)])
def test_avg_pool_equals_library_avg_pool(P, w):
    rng = np.random.default_rng(P * 37 + w)
    x = rng.random(P).astype(np.float32)
    got = oracle.pool_avg(x, w)
    want = torch.nn.functional.avg_pool1d(torch.from_numpy(x).double().view(1, 1, P), kernel_size=w, stride=1,
                                          padding=(w - 1) // 2).view(-1).numpy()     # zeros outside, divided by w
    np.testing.assert_allclose(got, want, rtol=(w + 1) * 2.0 ** -24, atol=0)
    if w == 1:
        np.testing.assert_array_equal(got, x)


@pytest.mark.parametrize("w", [3, 5, 7, 11])
def test_avg_pool_is_exact_on_small_integers(w):
    # Integer inputs make every partial sum exact, so only the final division rounds: the result must be the
    # float nearest to the rational sum / w.
    rng = np.random.default_rng(w)
    P = 50
    x = rng.integers(0, 9, P).astype(np.float32)
    got = oracle.pool_avg(x, w)
    r = (w - 1) // 2
    for i in range(P):
        total = int(sum(x[max(0, i - r): min(P, i + r + 1)]))
        assert got[i] == np.float32(total / w), (i, total)


def test_avg_pool_divides_by_full_width_at_the_edges():
    x = np.zeros(30, dtype=np.float32)
    x[0] = 7.0                                              # at the left edge: 4 windows of width 7 contain it
    got = oracle.pool_avg(x, 7)
    np.testing.assert_array_equal(got[:4], np.ones(4, dtype=np.float32))
    assert not got[4:].any()
    x[:] = 0
    x[15] = 7.0                                             # interior spike: spread over 7 positions, mass kept
    got = oracle.pool_avg(x, 7)
    assert list(np.nonzero(got)[0]) == list(range(12, 19)) and got.sum() == 7.0


def test_avg_and_max_pool_choose_differently():
    s = np.zeros(60, dtype=np.float32)
    s[10] = 1.0                                             # a lone spike
    s[30:37] = 0.5                                          # a plateau as wide as the pool
    assert list(oracle.select_topk(oracle.pool_max(s, 7), 1)) == [7]       # spike wins, left-most of its ties
    assert list(oracle.select_topk(oracle.pool_avg(s, 7), 1)) == [33]      # plateau centre wins (0.5 > 1/7)


def test_layer_with_avg_pool_is_pool_then_select():
    g = torch.Generator().manual_seed(21)
    q = torch.randn(4, 8, 64, generator=g)
    k = torch.randn(2, 300, 64, generator=g)
    v = torch.randn(2, 300, 64, generator=g)
    r = oracle.compress_layer(q, k, v, pool_kernel=5, avg_budget=64, k_layer=40, pool_kind="avg")
    for h in range(2):
        want = oracle.select_topk(oracle.pool_avg(r["scores"][h], 5), 40)
        assert list(r["kept"][h][:40]) == list(want)
        assert list(r["kept"][h][40:]) == list(range(292, 300))
        assert torch.equal(r["k_out"][h], k[h][torch.from_numpy(r["kept"][h]).long()])
    m = oracle.compress_layer(q, k, v, pool_kernel=5, avg_budget=64, k_layer=40)
    assert not np.array_equal(m["kept"], r["kept"])          # the two pools do select different rows here


# ----------------------------------------------------------------------------- selection
def brute_force_select(p, k):
    order = sorted(range(len(p)), key=lambda i: (-float(p[i]), i))
    return sorted(order[: max(0, min(k, len(p)))])


@pytest.mark.parametrize("seed", range(12))
def test_select_equals_full_sort_with_ties(seed):
    rng = np.random.default_rng(seed)
    P = int(rng.integers(1, 60))
    levels = int(rng.integers(1, 6))                       # few distinct values: ties everywhere
    p = (rng.integers(0, levels, P) / 4.0).astype(np.float32)
    for k in (0, 1, P // 3, P - 1, P, P + 5):
        got = oracle.select_topk(p, k)
        assert list(got) == brute_force_select(p, k)
        assert all(a < b for a, b in zip(got, got[1:]))     # ascending, no duplicates


@pytest.mark.parametrize("seed", range(6))
def test_select_equals_library_topk_when_boundary_is_strict(seed):
    rng = np.random.default_rng(100 + seed)
    P, k = 500, 37
    p = rng.permutation(P).astype(np.float32)              # all distinct
    got = oracle.select_topk(p, k)
    want = torch.topk(torch.from_numpy(p), k).indices.sort().values.numpy()
    np.testing.assert_array_equal(got, want)


def test_select_maximises_kept_attention_for_pool_width_one():
    """With no pooling the top-k set keeps the most attention any k-subset can (attention recall)."""
    rng = np.random.default_rng(7)
    for P, k in [(8, 3), (12, 5), (14, 1), (10, 9)]:
        s = rng.random(P).astype(np.float32)
        got = oracle.select_topk(oracle.pool_max(s, 1), k)
        best = max(sum(float(s[i]) for i in c) for c in itertools.combinations(range(P), k))
        assert abs(sum(float(s[i]) for i in got) - best) < 1e-6


def test_tie_break_takes_leftmost_at_threshold():
    p = np.array([0.5, 0.9, 0.5, 0.5, 0.9, 0.5], dtype=np.float32)
    assert list(oracle.select_topk(p, 3)) == [0, 1, 4]
    assert list(oracle.select_topk(p, 4)) == [0, 1, 2, 4]
    assert list(oracle.select_topk(p, 2)) == [1, 4]
    assert list(oracle.select_topk(p, 1)) == [1]


# ----------------------------------------------------------------------------- whole layer
def draw(hq, hkv, alpha, n, d, seed, dtype=torch.float32):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(hq, alpha, d, generator=g).to(dtype)
    k = torch.randn(hkv, n, d, generator=g).to(dtype)
    v = torch.randn(hkv, n, d, generator=g).to(dtype)
    return q, k, v


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_layer_is_scores_pool_select_window_gather(dtype):
    hq, hkv, alpha, n, d, w, B, kl = 4, 2, 8, 200, 32, 5, 64, 40
    q, k, v = draw(hq, hkv, alpha, n, d, seed=1, dtype=dtype)
    r = oracle.compress_layer(q, k, v, pool_kernel=w, avg_budget=B, k_layer=kl)
    P = n - alpha
    assert r["count"] == kl + alpha
    s, _ = oracle.window_scores(q, k)
    np.testing.assert_array_equal(r["scores"], s)
    for h in range(hkv):
        pooled = torch.nn.functional.max_pool1d(torch.from_numpy(s[h]).view(1, 1, P), w, 1, (w - 1) // 2).view(-1).numpy()
        want = brute_force_select(pooled, kl) + list(range(P, n))
        assert list(r["kept"][h]) == want
        # the instruction tokens close every list
        assert list(r["kept"][h][-alpha:]) == list(range(P, n))
        idx = torch.tensor(want)
        assert torch.equal(r["k_out"][h], k[h, idx])        # gather == fancy indexing, bit for bit
        assert torch.equal(r["v_out"][h], v[h, idx])


def test_budget_at_least_context_keeps_everything_and_attention_is_unchanged():
    hq, hkv, alpha, n, d, w = 4, 2, 8, 60, 16, 5
    q, k, v = draw(hq, hkv, alpha, n, d, seed=2)
    for B in (60, 64, 500):
        r = oracle.compress_layer(q, k, v, pool_kernel=w, avg_budget=B, k_layer=3)
        assert r["count"] == n
        for h in range(hkv):
            assert list(r["kept"][h]) == list(range(n))
        assert torch.equal(r["k_out"], k) and torch.equal(r["v_out"], v)
    # attention of the window queries over the compact cache == over the full cache
    group = hq // hkv
    for hq_i in range(hq):
        h = hq_i // group
        full = oracle.window_attention(q[hq_i], k[h], v[h], np.arange(n), n)
        comp = oracle.window_attention(q[hq_i], r["k_out"][h], r["v_out"][h], r["kept"][h], n)
        np.testing.assert_array_equal(full, comp)
        # and the attention routine itself agrees with the library softmax
        logits = (q[hq_i].double() @ k[h].double().T) / np.sqrt(d)
        mask = torch.arange(n).view(1, n) > torch.arange(n - alpha, n).view(alpha, 1)
        want = torch.softmax(logits.masked_fill(mask, float("-inf")), dim=-1) @ v[h].double()
        np.testing.assert_allclose(full, want.numpy(), rtol=1e-10, atol=1e-12)


def test_budget_larger_than_prefix_keeps_whole_prefix():
    hq, hkv, alpha, n, d = 2, 2, 4, 50, 8
    q, k, v = draw(hq, hkv, alpha, n, d, seed=3)
    r = oracle.compress_layer(q, k, v, pool_kernel=3, avg_budget=40, k_layer=70)
    assert r["count"] == n
    for h in range(hkv):
        assert list(r["kept"][h]) == list(range(n))


def test_dropping_rows_changes_attention_only_by_the_dropped_mass():
    """Attention over a compressed cache is the full attention renormalised over the kept rows."""
    hq, hkv, alpha, n, d = 2, 1, 4, 80, 16
    q, k, v = draw(hq, hkv, alpha, n, d, seed=5)
    r = oracle.compress_layer(q, k, v, pool_kernel=1, avg_budget=24, k_layer=20)
    kept = r["kept"][0]
    comp = oracle.window_attention(q[0], r["k_out"][0], r["v_out"][0], kept, n)
    logits = (q[0].double() @ k[0].double().T) / np.sqrt(d)
    mask = torch.arange(n).view(1, n) > torch.arange(n - alpha, n).view(alpha, 1)
    dropped = torch.ones(n, dtype=torch.bool)
    dropped[torch.from_numpy(kept).long()] = False
    logits = logits.masked_fill(mask | dropped.view(1, n), float("-inf"))
    want = torch.softmax(logits, dim=-1) @ v[0].double()
    np.testing.assert_allclose(comp, want.numpy(), rtol=1e-10, atol=1e-12)


def test_ragged_batch_packing():
    hq, hkv, alpha, d, w, B, kl = 4, 2, 4, 8, 3, 16, 9
    lens = [40, 23, 12, 31]                                 # 12 <= B: kept whole
    g = torch.Generator().manual_seed(12)
    n_max = max(lens)
    q = torch.randn(len(lens), hq, alpha, d, generator=g)
    k = torch.randn(len(lens), hkv, n_max, d, generator=g)
    v = torch.randn(len(lens), hkv, n_max, d, generator=g)
    out = oracle.compress_batch(q, k, v, lens, pool_kernel=w, avg_budget=B, k_layer=kl)
    assert out["counts"] == [13, 13, 12, 13]
    off = 0
    for b, n in enumerate(lens):
        c = out["counts"][b]
        single = oracle.compress_layer(q[b], k[b, :, :n], v[b, :, :n], pool_kernel=w, avg_budget=B, k_layer=kl)
        for h in range(hkv):
            rows = slice(off + h * c, off + (h + 1) * c)
            np.testing.assert_array_equal(out["indices"][rows], single["kept"][h])
            assert torch.equal(out["k_out"][rows], k[b, h, torch.from_numpy(single["kept"][h]).long()])
        off += hkv * c
    assert out["k_out"].shape[0] == off


def test_kept_positions_follow_the_papers_position_example():
    """Appendix on rotary embeddings: kept positions ascend and end with the last prompt token."""
    with open(os.path.join(GOLDEN, "rope_positions.txt")) as f:
        printed = [int(x) for line in f if not line.startswith("#") for x in line.split()]
    assert printed == sorted(printed)
    n = printed[-1] + 1                                     # positions 0 .. 4012
    hq, hkv, alpha, d = 1, 1, 1, 8
    g = torch.Generator().manual_seed(0)
    q = torch.randn(hq, alpha, d, generator=g)
    k = 0.01 * torch.randn(hkv, n, d, generator=g)
    v = torch.randn(hkv, n, d, generator=g)
    u = q[0, 0] / q[0, 0].norm()
    for p in printed[:-1]:
        k[0, p] += 20.0 * u                                 # make exactly the printed prefix positions stand out
    r = oracle.compress_layer(q, k, v, pool_kernel=1, avg_budget=len(printed), k_layer=len(printed) - 1)
    assert list(r["kept"][0]) == printed


# ----------------------------------------------------------------------------- consumers of the compact cache
def test_decode_attention_is_library_softmax_attention():
    g = torch.Generator().manual_seed(9)
    d, c = 32, 57
    q = torch.randn(d, generator=g)
    k = torch.randn(c, d, generator=g)
    v = torch.randn(c, d, generator=g)
    got = oracle.decode_attention(q, k, v)
    want = torch.softmax((k.double() @ q.double()) / np.sqrt(d), dim=0) @ v.double()
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-12, atol=1e-13)
    # a single cached row returns that row's value; permuting the cache changes nothing
    np.testing.assert_allclose(oracle.decode_attention(q, k[:1], v[:1]), v[0].double().numpy(), rtol=1e-12)
    perm = torch.randperm(c, generator=g)
    np.testing.assert_allclose(oracle.decode_attention(q, k[perm], v[perm]), got, rtol=1e-10, atol=1e-12)


def test_attention_recall_definition_and_monotonicity():
    """Recall = kept share of the window rows' attention, from the full attention matrix (library softmax)."""
    hq, hkv, alpha, n, d = 4, 2, 4, 90, 16
    q, k, v = draw(hq, hkv, alpha, n, d, seed=17)
    P = n - alpha
    group = hq // hkv
    logits = torch.einsum("gjd,gnd->gjn", q.double(), k.double().repeat_interleave(group, dim=0)) / np.sqrt(d)
    mask = torch.arange(n).view(1, 1, n) > torch.arange(P, n).view(1, alpha, 1)
    att = torch.softmax(logits.masked_fill(mask, float("-inf")), dim=-1)            # [H_q][alpha][n]
    prev = None
    for kl in (5, 20, 60, P):
        r = oracle.compress_layer(q, k, v, pool_kernel=1, avg_budget=alpha + kl, k_layer=kl)
        vals = []
        for h in range(hkv):
            kept = torch.from_numpy(r["kept"][h]).long()
            want = att[h * group:(h + 1) * group][:, :, kept].sum(dim=-1).mean().item()   # mean over heads and rows
            got = oracle.attention_recall(r["scores"][h], alpha, r["kept"][h])
            assert abs(got - want) < 1e-6
            vals.append(got)
        if prev is not None:
            assert all(a >= b - 1e-9 for a, b in zip(vals, prev))                     # more budget, more recall
        prev = vals
    assert all(abs(x - 1.0) < 1e-6 for x in prev)                                     # nothing evicted
