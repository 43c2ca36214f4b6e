"""GPU parity: every C-ABI call against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
import paper_2406_02069_b200 as pkv
from paper_2406_02069_b200 import binding, workloads
from helpers import assert_indices_match, assert_scores_close, packed_rows

pytestmark = pytest.mark.gpu
DEV = "cuda"

# Cases the oracle finishes in seconds; each spans several key tiles and a ragged tail.
SCALED = [
    workloads.TINY,
    workloads.scaled(workloads.LLAMA2_7B, num_layers=2, seq_len=4096, name="llama2_7b_full_len"),
    workloads.scaled(workloads.LLAMA3_8B, num_layers=2, seq_len=5000 + 37, name="llama3_8b_5k"),
    workloads.scaled(workloads.LLAMA3_70B, num_layers=3, seq_len=3000 + 11, name="llama3_70b_3k"),
    workloads.scaled(workloads.MISTRAL_RAGGED, num_layers=2, batch=3, name="mistral_b3"),
    workloads.scaled(workloads.with_budget(workloads.MISTRAL_RAGGED, 2048), num_layers=1, batch=2, name="mistral_b2_2048"),
]


def small_lens(w):
    """Shrink the ragged workload's lengths so the oracle stays fast, keeping them uneven."""
    lens = w.seq_lens()
    if w.name.startswith("mistral"):
        lens = [300 + (n % 1777) for n in lens]
    return lens


def run_scores(w, cfg, x, lens):
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    ld = max(lens) - w.window + 5
    scores = torch.full((len(lens), w.num_kv_heads, ld), -1.0, dtype=torch.float32, device=DEV)
    pkv.score_window(cfg, x.q_win, x.k, lens, scores, ws)
    pkv.check_status(ws)
    return scores


@pytest.mark.parametrize("w", SCALED, ids=lambda w: w.name)
def test_scores_match_oracle(w):
    cfg = pkv.config_of(w)
    lens = small_lens(w)
    for layer in range(w.num_layers):
        x = workloads.make_layer(w, layer, device=DEV, seq_lens=lens)
        scores = run_scores(w, cfg, x, lens).cpu().numpy()
        qc, kc = x.q_win.cpu(), x.k.cpu()
        for b, n in enumerate(lens):
            want, mass = oracle.window_scores(qc[b], kc[b, :, :n])
            got = scores[b, :, : n - w.window]
            assert_scores_close(got, want, "%s layer %d seq %d" % (w.name, layer, b))
            # mass invariant on the GPU result too: prefix scores + window mass = alpha
            np.testing.assert_allclose(got.astype(np.float64).sum(axis=1) + mass, w.window, rtol=1e-3)
            assert (scores[b, :, n - w.window:] == -1.0).all()        # nothing written past the prefix


@pytest.mark.parametrize("hq,hkv,alpha,d,lens", [
    (3, 3, 8, 64, [700]),                 # R = 8, head_dim 64
    (12, 4, 8, 64, [129, 1000, 136]),     # R = 24, ragged, one sequence barely longer than a tile
    (8, 2, 48, 128, [2000, 333]),         # R = 192: two row blocks, padded
    (16, 2, 32, 128, [1500]),             # R = 256
    (4, 4, 1, 128, [300]),                # alpha = 1
    (8, 1, 16, 128, [16 + 1, 16 + 128, 16 + 129]),   # prefix of 1, of one tile, of one tile + 1
    (1, 1, 256, 128, [900]),              # R = 256 from one head: the widest window the tensor-core path takes
    (2, 2, 128, 64, [700, 300]),          # R = 128 exactly, head_dim 64
    (16, 1, 16, 128, [1000]),             # G = 16
    (64, 2, 8, 128, [777]),               # G = 32, R = 256
    (4, 2, 24, 128, [60 + i * 37 for i in range(64)]),   # the largest batch, short ragged sequences
])
def test_scores_bf16_shapes(hq, hkv, alpha, d, lens):
    """Tensor-core score path over window sizes, group sizes, head dims and ragged tails."""
    cfg = pkv.make_config(num_layers=1, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, window=alpha, pool_kernel=3,
                          dtype="bf16", avg_budget=alpha, beta=1.0)
    g = torch.Generator(device="cpu").manual_seed(hq * 100 + alpha)
    n_max = max(lens)
    q = (torch.randn(len(lens), hq, alpha, d, generator=g) * 1.5).to(torch.bfloat16)
    k = torch.randn(len(lens), hkv, n_max, d, generator=g).to(torch.bfloat16)
    k[:, :, 0] *= 3.0
    ws = pkv.new_workspace(cfg, len(lens), n_max, DEV)
    scores = torch.full((len(lens), hkv, n_max), -1.0, dtype=torch.float32, device=DEV)
    for rep in range(2):                                            # second run reuses the workspace
        pkv.score_window(cfg, q.to(DEV), k.to(DEV), lens, scores, ws)
        pkv.check_status(ws)
    got = scores.cpu().numpy()
    for b, n in enumerate(lens):
        want, _ = oracle.window_scores(q[b], k[b, :, :n])
        assert_scores_close(got[b, :, : n - alpha], want, "seq %d" % b)
        assert (got[b, :, n - alpha:] == -1.0).all()


@pytest.mark.parametrize("w", [SCALED[0], SCALED[2], SCALED[3], SCALED[4]], ids=lambda w: w.name)
def test_single_sweep_with_prefill_lse_matches_oracle(w):
    """Hand-off mode: the window rows' log-sum-exp comes from outside (here: from the oracle)."""
    cfg = pkv.config_of(w)
    lens = small_lens(w)
    budgets = pkv.layer_budgets(cfg)
    layer = w.num_layers - 1
    x = workloads.make_layer(w, layer, device=DEV, seq_lens=lens)
    qc, kc = x.q_win.cpu(), x.k.cpu()
    lse = np.stack([oracle.window_lse(qc[b], kc[b, :, :n]) for b, n in enumerate(lens)]).astype(np.float32)
    lse_dev = torch.from_numpy(lse).to(DEV)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    scores = torch.full((len(lens), w.num_kv_heads, max(lens)), -1.0, dtype=torch.float32, device=DEV)
    pkv.score_window(cfg, x.q_win, x.k, lens, scores, ws, window_lse=lse_dev)
    pkv.check_status(ws)
    got = scores.cpu().numpy()
    for b, n in enumerate(lens):
        want, _ = oracle.window_scores(qc[b], kc[b, :, :n])
        assert_scores_close(got[b, :, : n - w.window], want, "%s seq %d" % (w.name, b))
    # the whole layer through the same mode equals the self-contained call
    kl = budgets[layer]
    rows = pkv.total_rows(cfg, kl, lens)
    outs = []
    for use_lse in (False, True):
        k_out = torch.empty(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
        v_out = torch.empty_like(k_out)
        idx = torch.empty(rows, dtype=torch.int32, device=DEV)
        pkv.compress_layer(cfg, layer, x.q_win, x.k, x.v, lens, k_out, v_out, idx, ws,
                           window_lse=lse_dev if use_lse else None)
        pkv.check_status(ws)
        outs.append((idx.cpu().numpy(), k_out.cpu(), v_out.cpu()))
    counts = [pkv.kept_count(cfg, kl, n) for n in lens]
    heads = [np.array_equal(outs[0][0][sl], outs[1][0][sl]) for _, _, sl in packed_rows(counts, w.num_kv_heads)]
    assert np.mean(heads) >= 0.95, "only %d of %d heads keep the same list in both modes" % (sum(heads), len(heads))
    if all(heads):
        assert torch.equal(outs[0][1], outs[1][1]) and torch.equal(outs[0][2], outs[1][2])


@pytest.mark.parametrize("P,k,w", [(1, 1, 1), (5, 2, 7), (33, 32, 3), (100, 0, 5), (100, 100, 5), (100, 250, 5),
                                   (1000, 37, 7), (4064, 188, 7), (8193, 500, 7), (20000, 4, 7), (40000, 937, 7),
                                   (131040, 188, 7), (4000, 900, 7), (2500, 2000, 5), (4096, 513, 7), (70001, 2016, 1), (131073 + 4, 188, 7), (262144 + 5, 300, 7),
                                   (1048576 + 77, 2016, 7)])
def test_select_is_bit_exact_on_oracle_scores(P, k, w):
    """Selection alone: same scores in, identical index lists out, ties included."""
    alpha, hkv, batch = 4, 3, 2
    rng = np.random.default_rng(P * 7 + k)
    # few distinct levels plus pooling plateaus: ties at the threshold are the normal case
    levels = rng.integers(0, 50, size=(batch, hkv, P)).astype(np.float32) / 64.0
    levels[0, 0] = rng.random(P).astype(np.float32)                 # one head with distinct values
    if P > 10:
        levels[1, 1] = 0.25                                         # one head all equal
    cfg = pkv.make_config(num_layers=1, num_q_heads=hkv, num_kv_heads=hkv, head_dim=64, window=alpha, pool_kernel=w,
                          dtype="fp32", avg_budget=alpha + k, beta=1.0)
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
            want = np.concatenate([oracle.select_topk(oracle.pool_max(levels[b, h], w), k), np.arange(P, P + alpha)])
        np.testing.assert_array_equal(got[rows], want.astype(np.int32), err_msg="b=%d h=%d" % (b, h))


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("fp32", 64), ("bf16", 64), ("fp32", 128)])
def test_gather_is_bit_exact(dtype, d):
    hkv, alpha, B, kl = 3, 4, 40, 21
    lens = [300, 77, 30, 129]                                        # 30 <= B: kept whole
    cfg = pkv.make_config(num_layers=1, num_q_heads=hkv, num_kv_heads=hkv, head_dim=d, window=alpha, pool_kernel=3,
                          dtype=dtype, avg_budget=B, beta=1.0)
    g = torch.Generator(device="cpu").manual_seed(5)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    n_max = max(lens)
    # non-contiguous views: token stride wider than d, as a fused QKV buffer would give
    kbuf = torch.randn(len(lens), hkv, n_max, 2 * d, generator=g).to(tdt).to(DEV)
    k, v = kbuf[..., :d], kbuf[..., d:]
    counts = [pkv.kept_count(cfg, kl, n) for n in lens]
    rows = sum(c * hkv for c in counts)
    idx_np = np.zeros(rows, dtype=np.int32)
    rng = np.random.default_rng(1)
    for b, h, sl in packed_rows(counts, hkv):
        idx_np[sl] = np.sort(rng.choice(lens[b], size=counts[b], replace=False))
    idx = torch.from_numpy(idx_np).to(DEV)
    k_out = torch.zeros(rows, d, dtype=tdt, device=DEV)
    v_out = torch.zeros(rows, d, dtype=tdt, device=DEV)
    pkv.gather_compact(cfg, k, v, idx, lens, kl, k_out, v_out)
    torch.cuda.synchronize()
    for b, h, sl in packed_rows(counts, hkv):
        sel = torch.from_numpy(idx_np[sl]).long().to(DEV)
        assert torch.equal(k_out[sl], k[b, h, sel]) and torch.equal(v_out[sl], v[b, h, sel])
    # K only
    k_only = torch.zeros_like(k_out)
    pkv.gather_compact(cfg, k, None, idx, lens, kl, k_only, None)
    torch.cuda.synchronize()
    assert torch.equal(k_only, k_out)


@pytest.mark.parametrize("w", SCALED, ids=lambda w: w.name)
def test_compress_layer_matches_oracle(w):
    cfg = pkv.config_of(w)
    lens = small_lens(w)
    budgets = pkv.layer_budgets(cfg)
    assert budgets == oracle.layer_budgets(w.num_layers, w.avg_budget, w.window, w.beta)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    for layer in range(w.num_layers):
        kl = budgets[layer]
        x = workloads.make_layer(w, layer, device=DEV, seq_lens=lens)
        rows = pkv.total_rows(cfg, kl, lens)
        k_out = torch.empty(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
        v_out = torch.empty_like(k_out)
        idx = torch.empty(rows, dtype=torch.int32, device=DEV)
        pkv.compress_layer(cfg, layer, x.q_win, x.k, x.v, lens, k_out, v_out, idx, ws)   # scores in the workspace
        pkv.check_status(ws)
        ref = oracle.compress_batch(x.q_win.cpu(), x.k.cpu(), x.v.cpu(), lens, pool_kernel=w.pool_kernel,
                                    avg_budget=w.avg_budget, k_layer=kl)
        assert ref["indices"].shape[0] == rows
        got_idx = idx.cpu().numpy()
        identical = 0
        for b, h, sl in packed_rows(ref["counts"], w.num_kv_heads):
            same = assert_indices_match(got_idx[sl], ref["indices"][sl], ref["scores"][b][h], w.pool_kernel, w.window,
                                        "%s layer %d b %d h %d" % (w.name, layer, b, h))
            identical += bool(same)
            # gathered rows must be the rows the GPU's own index list names, bit for bit
            sel = idx[sl].long()
            assert torch.equal(k_out[sl], x.k[b, h, sel]) and torch.equal(v_out[sl], x.v[b, h, sel])
            if same:
                assert torch.equal(k_out[sl].cpu(), ref["k_out"][sl]) and torch.equal(v_out[sl].cpu(), ref["v_out"][sl])
            # planted sinks and needles survive wherever the budget has room for their pooled plateaus
            planted = x.planted[b]
            if kl >= w.pool_kernel * len(planted) and lens[b] > w.avg_budget:
                assert set(planted) <= set(got_idx[sl].tolist()), "planted tokens evicted"
        total = len(ref["counts"]) * w.num_kv_heads
        assert identical >= 0.95 * total, "only %d of %d index lists identical" % (identical, total)


@pytest.mark.parametrize("w,layers", [
    (workloads.LLAMA2_7B, (0, 31)), (workloads.LLAMA3_8B, (0, 31)), (workloads.LLAMA3_70B, (0, 79)),
    (workloads.MISTRAL_RAGGED, (0,)), (workloads.with_budget(workloads.MISTRAL_RAGGED, 2048), (31,)),
], ids=lambda x: getattr(x, "name", str(x)))
def test_full_size_layers_match_oracle(w, layers):
    """The configurations at their full sizes, in the launch shapes bench.py times: every score of the
    layer, every kept list and the gathered rows against the oracle (about a second of CPU per head)."""
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    budgets = pkv.layer_budgets(cfg)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    for layer in layers:
        kl = budgets[layer]
        x = workloads.make_layer(w, layer, device=DEV)
        rows = pkv.total_rows(cfg, kl, lens)
        k_out = torch.empty(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
        v_out = torch.empty_like(k_out)
        idx = torch.empty(rows, dtype=torch.int32, device=DEV)
        scores = torch.full((len(lens), w.num_kv_heads, max(lens)), -1.0, dtype=torch.float32, device=DEV)
        pkv.compress_layer(cfg, layer, x.q_win, x.k, x.v, lens, k_out, v_out, idx, ws, scores=scores)
        pkv.check_status(ws)
        ref = oracle.compress_batch(x.q_win.cpu(), x.k.cpu(), x.v.cpu(), lens, pool_kernel=w.pool_kernel,
                                    avg_budget=w.avg_budget, k_layer=kl)
        got_scores, got_idx = scores.cpu().numpy(), idx.cpu().numpy()
        for b, n in enumerate(lens):
            assert_scores_close(got_scores[b, :, : n - w.window], ref["scores"][b], "%s layer %d seq %d" % (w.name, layer, b))
        identical = 0
        for b, h, sl in packed_rows(ref["counts"], w.num_kv_heads):
            identical += bool(assert_indices_match(got_idx[sl], ref["indices"][sl], ref["scores"][b][h], w.pool_kernel,
                                                   w.window, "%s layer %d b %d h %d" % (w.name, layer, b, h)))
            sel = idx[sl].long()
            assert torch.equal(k_out[sl], x.k[b, h, sel]) and torch.equal(v_out[sl], x.v[b, h, sel])
        assert identical >= 0.95 * len(ref["counts"]) * w.num_kv_heads
        del x, k_out, v_out, scores
        torch.cuda.empty_cache()


def test_layer_calls_can_be_captured_in_a_cuda_graph():
    """Nothing in the per-layer call synchronises or allocates, so a step can be captured once and replayed."""
    w = workloads.scaled(workloads.LLAMA3_8B, num_layers=3, seq_len=3000, name="l3_graph")
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    budgets = pkv.layer_budgets(cfg)
    layers = [workloads.make_layer(w, l, device=DEV) for l in range(w.num_layers)]
    ws = pkv.new_workspace(cfg, 1, max(lens), DEV)
    rows = [pkv.total_rows(cfg, kl, lens) for kl in budgets]
    outs = [(torch.zeros(r, w.head_dim, dtype=torch.bfloat16, device=DEV), torch.zeros(r, w.head_dim, dtype=torch.bfloat16, device=DEV),
             torch.zeros(r, dtype=torch.int32, device=DEV)) for r in rows]

    def step():
        for l, x in enumerate(layers):
            pkv.compress_layer(cfg, l, x.q_win, x.k, x.v, lens, outs[l][0], outs[l][1], outs[l][2], ws)

    step()                                                          # eager: also runs every first-use set-up
    torch.cuda.synchronize()
    want = [tuple(t.clone() for t in o) for o in outs]
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    for o in outs:
        for t in o:
            t.zero_()
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    pkv.check_status(ws)
    for o, wnt in zip(outs, want):
        for a_, b_ in zip(o, wnt):
            assert torch.equal(a_, b_)


@pytest.mark.parametrize("w", [SCALED[0], SCALED[2], SCALED[4]], ids=lambda w: w.name)
def test_decode_attention_and_recall_over_the_compact_cache(w):
    """After compression a new token attends to the kept rows only; recall says how much attention they hold."""
    cfg = pkv.config_of(w)
    lens = small_lens(w)
    layer = 0
    kl = pkv.layer_budgets(cfg)[layer]
    x = workloads.make_layer(w, layer, device=DEV, seq_lens=lens)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    rows = pkv.total_rows(cfg, kl, lens)
    k_out = torch.empty(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
    v_out = torch.empty_like(k_out)
    idx = torch.empty(rows, dtype=torch.int32, device=DEV)
    scores = torch.zeros(len(lens), w.num_kv_heads, max(lens), dtype=torch.float32, device=DEV)
    pkv.compress_layer(cfg, layer, x.q_win, x.k, x.v, lens, k_out, v_out, idx, ws, scores=scores)
    g = torch.Generator(device="cpu").manual_seed(77)
    q_new = torch.randn(len(lens), w.num_q_heads, w.head_dim, generator=g).to(x.k.dtype)
    out = torch.zeros(len(lens), w.num_q_heads, w.head_dim, dtype=torch.float32, device=DEV)
    pkv.decode_attention(cfg, q_new.to(DEV), k_out, v_out, lens, kl, out)
    recall = torch.zeros(len(lens), w.num_kv_heads, dtype=torch.float32, device=DEV)
    pkv.attention_recall(cfg, scores, idx, lens, kl, recall)
    pkv.check_status(ws)
    out_h, rec_h = out.cpu().numpy(), recall.cpu().numpy()
    kc, vc, ic, sc = k_out.cpu(), v_out.cpu(), idx.cpu().numpy(), scores.cpu().numpy()
    counts = [pkv.kept_count(cfg, kl, n) for n in lens]
    for b, h, sl in packed_rows(counts, w.num_kv_heads):
        for gq in range(w.group):
            hq = h * w.group + gq
            want = oracle.decode_attention(q_new[b, hq], kc[sl], vc[sl])
            np.testing.assert_allclose(out_h[b, hq], want, rtol=2e-3, atol=2e-4)
        want_r = oracle.attention_recall(sc[b, h, : lens[b] - w.window], w.window, ic[sl])
        assert abs(rec_h[b, h] - want_r) < 1e-4
        assert 0.0 < rec_h[b, h] <= 1.0 + 1e-5


def test_three_calls_equal_the_fused_call():
    w = workloads.scaled(workloads.LLAMA3_8B, num_layers=2, seq_len=3000, name="l3_3k")
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    kl = pkv.layer_budgets(cfg)[1]
    x = workloads.make_layer(w, 1, device=DEV)
    ws = pkv.new_workspace(cfg, 1, max(lens), DEV)
    rows = pkv.total_rows(cfg, kl, lens)
    outs = []
    for fused in (True, False):
        k_out = torch.empty(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
        v_out = torch.empty_like(k_out)
        idx = torch.empty(rows, dtype=torch.int32, device=DEV)
        scores = torch.zeros(1, w.num_kv_heads, max(lens), dtype=torch.float32, device=DEV)
        if fused:
            pkv.compress_layer(cfg, 1, x.q_win, x.k, x.v, lens, k_out, v_out, idx, ws, scores=scores)
        else:
            pkv.score_window(cfg, x.q_win, x.k, lens, scores, ws)
            pkv.select_topk(cfg, scores, lens, kl, idx, ws)
            pkv.gather_compact(cfg, x.k, x.v, idx, lens, kl, k_out, v_out)
        pkv.check_status(ws)
        outs.append((k_out, v_out, idx, scores))
    for a, b in zip(*outs):
        assert torch.equal(a, b)


@pytest.mark.parametrize("n,B,alpha,G", [(9, 16, 8, 2), (9, 8, 8, 1), (40, 64, 8, 2), (64, 64, 8, 4), (65, 64, 8, 4),
                                         (130, 16, 16, 1), (257, 40, 1, 3), (513, 100, 48, 2)])
def test_edge_cases(n, B, alpha, G):
    """Shortest contexts, contexts that fit the budget, window-only budgets, odd group sizes."""
    hkv, d, w_pool, m = 2, 64, 5, 3
    cfg = pkv.make_config(num_layers=m, num_q_heads=hkv * G, num_kv_heads=hkv, head_dim=d, window=alpha,
                          pool_kernel=w_pool, dtype="fp32", avg_budget=B, beta=20.0)
    g = torch.Generator(device="cpu").manual_seed(n * 3 + B)
    q = torch.randn(1, hkv * G, alpha, d, generator=g)
    k = torch.randn(1, hkv, n, d, generator=g)
    v = torch.randn(1, hkv, n, d, generator=g)
    ws = pkv.new_workspace(cfg, 1, n, DEV)
    budgets = pkv.layer_budgets(cfg)
    for layer, kl in enumerate(budgets):
        c = pkv.kept_count(cfg, kl, n)
        k_out = torch.empty(hkv * c, d, device=DEV)
        v_out = torch.empty_like(k_out)
        idx = torch.empty(hkv * c, dtype=torch.int32, device=DEV)
        pkv.compress_layer(cfg, layer, q.to(DEV), k.to(DEV), v.to(DEV), [n], k_out, v_out, idx, ws)
        pkv.check_status(ws)
        ref = oracle.compress_layer(q[0], k[0], v[0], pool_kernel=w_pool, avg_budget=B, k_layer=kl)
        assert ref["count"] == c
        got = idx.cpu().numpy().reshape(hkv, c)
        for h in range(hkv):
            assert_indices_match(got[h], ref["kept"][h], ref["scores"][h], w_pool, alpha, "edge layer %d h %d" % (layer, h))
            assert torch.equal(k_out.view(hkv, c, d)[h].cpu(), k[0, h, torch.from_numpy(got[h]).long()])
        if n <= B:
            assert (got == np.arange(n)).all()
            assert torch.equal(k_out.cpu().view(hkv, n, d), k[0]) and torch.equal(v_out.cpu().view(hkv, n, d), v[0])


def test_device_errors_are_reported_not_raised_as_faults():
    """Bad arguments with real device buffers: the Python wrapper refuses a mis-sized tensor before the call,
    and the C side (reached directly here, as a C caller would) answers with a status code."""
    import ctypes
    w = workloads.TINY
    cfg = pkv.config_of(w)
    x = workloads.make_layer(w, 0, device=DEV)
    ws = pkv.new_workspace(cfg, 1, 512, DEV)
    scores = torch.zeros(1, w.num_kv_heads, 100, dtype=torch.float32, device=DEV)      # 100 columns for 504 keys
    with pytest.raises(ValueError):
        pkv.score_window(cfg, x.q_win, x.k, [512], scores, ws)
    with pytest.raises(ValueError):                                                     # K shorter than the length given
        pkv.score_window(cfg, x.q_win, x.k[:, :, :300], [512], torch.zeros(1, 2, 512, device=DEV), ws)
    with pytest.raises(ValueError):                                                     # wrong element type
        pkv.score_window(cfg, x.q_win.half(), x.k.half(), [512], torch.zeros(1, 2, 512, device=DEV), ws)
    lens = (ctypes.c_int32 * 1)(512)
    full = torch.zeros(1, 2, 512, device=DEV)
    rc = binding._lib.pyramidkv_score_window(ctypes.byref(cfg), binding._tensor(x.q_win), binding._tensor(x.k), lens, 1,
                                             full.data_ptr(), 100, ws.data_ptr(), ws.numel(), 0)   # ld too small
    assert rc == binding.PKV_ERR_INVALID_ARG
    with pytest.raises(pkv.PkvError) as e:
        pkv.score_window(cfg, x.q_win, x.k, [512], full, ws[:1024])
    assert e.value.status == binding.PKV_ERR_WORKSPACE
    pkv.check_status(ws)


def test_compressing_a_compact_cache_again_sees_the_finished_rows():
    """The score sweeps start before the kernels ahead of them finish, which is only right for inputs those
    kernels do not write.  Here the second call's K and V ARE the first call's outputs, back to back on one
    stream: the library must notice and order them, so the result equals the one taken after a full stop."""
    w = workloads.scaled(workloads.LLAMA3_8B, num_layers=2, seq_len=9000, name="llama3_8b_9k")
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    kl = pkv.layer_budgets(cfg)[0]
    x = workloads.make_layer(w, 0, device=DEV)
    ws = pkv.new_workspace(cfg, 1, max(lens), DEV)
    c1 = pkv.kept_count(cfg, kl, lens[0])
    k1 = torch.empty(w.num_kv_heads * c1, w.head_dim, dtype=x.k.dtype, device=DEV)
    v1 = torch.empty_like(k1)
    i1 = torch.empty(w.num_kv_heads * c1, dtype=torch.int32, device=DEV)
    # second stage: the compact cache (969 rows per head) compressed to a 128-row budget
    cfg2 = pkv.make_config(num_layers=1, num_q_heads=w.num_q_heads, num_kv_heads=w.num_kv_heads, head_dim=w.head_dim,
                           window=w.window, pool_kernel=w.pool_kernel, dtype="bf16", avg_budget=128, beta=1.0)
    c2 = pkv.kept_count(cfg2, 96, c1)
    ws2 = pkv.new_workspace(cfg2, 1, c1, DEV)
    outs = []
    for settle in (True, False, False, False):
        k1.zero_(); v1.zero_()
        k2 = torch.zeros(w.num_kv_heads * c2, w.head_dim, dtype=x.k.dtype, device=DEV)
        v2 = torch.zeros_like(k2)
        i2 = torch.zeros(w.num_kv_heads * c2, dtype=torch.int32, device=DEV)
        torch.cuda.synchronize()
        pkv.compress_layer(cfg, 0, x.q_win, x.k, x.v, lens, k1, v1, i1, ws)
        if settle:
            torch.cuda.synchronize()
        pkv.compress_layer(cfg2, 0, x.q_win, k1.view(1, w.num_kv_heads, c1, w.head_dim),
                           v1.view(1, w.num_kv_heads, c1, w.head_dim), [c1], k2, v2, i2, ws2)
        torch.cuda.synchronize()
        pkv.check_status(ws)
        pkv.check_status(ws2)
        outs.append((i2.clone(), k2.clone(), v2.clone()))
    for got in outs[1:]:
        assert all(torch.equal(a, b) for a, b in zip(got, outs[0]))
    assert int(outs[0][0].max()) == c1 - 1 and (outs[0][1] != 0).any()


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_token_major_and_fused_layouts_give_the_contiguous_result(dtype):
    """K/V/Q as other frameworks store them: token-major [batch][n][heads][d] and K, V interleaved in one
    buffer.  Only the strides in the tensor descriptors differ; the outputs must not."""
    w = workloads.scaled(workloads.LLAMA3_8B, num_layers=2, seq_len=3001, name="llama3_8b_3k", dtype=dtype)
    cfg = pkv.config_of(w)
    lens = [3001, 1777]
    x = workloads.make_layer(w, 1, device=DEV, seq_lens=lens)
    kl = pkv.layer_budgets(cfg)[1]
    rows = pkv.total_rows(cfg, kl, lens)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)

    def run(q, k, v):
        k_out = torch.empty(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
        v_out = torch.empty_like(k_out)
        idx = torch.empty(rows, dtype=torch.int32, device=DEV)
        scores = torch.zeros(len(lens), w.num_kv_heads, max(lens), dtype=torch.float32, device=DEV)
        pkv.compress_layer(cfg, 1, q, k, v, lens, k_out, v_out, idx, ws, scores=scores)
        pkv.check_status(ws)
        return scores.cpu(), idx.cpu(), k_out.cpu(), v_out.cpu()

    want = run(x.q_win, x.k, x.v)
    # token-major storage, viewed head-major
    k_tm = x.k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    v_tm = x.v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    q_tm = x.q_win.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert not k_tm.is_contiguous() and k_tm.stride(1) == w.head_dim
    got = run(q_tm, k_tm, v_tm)
    assert all(torch.equal(a, b) for a, b in zip(got, want))
    # K and V interleaved per token in one buffer
    kv = torch.stack([x.k, x.v], dim=3).contiguous()                  # [batch][H][n][2][d]
    got = run(x.q_win, kv[:, :, :, 0], kv[:, :, :, 1])
    assert all(torch.equal(a, b) for a, b in zip(got, want))


def test_keys_written_by_a_kernel_that_signals_early_are_read_complete():
    """A producer of K that lets its dependents start at once and then takes its time: the score sweeps that follow
    it on the stream (default flags) must still see the finished K.  Same result as with a full stop in between, and
    as the promised-final path after a full stop."""
    w = workloads.scaled(workloads.LLAMA3_8B, num_layers=2, seq_len=9000, name="llama3_8b_9k_slow_producer")
    lens = w.seq_lens()
    x = workloads.make_layer(w, 0, device=DEV)
    results = []
    for mode in ("back_to_back", "full_stop", "full_stop_inputs_final"):
        cfg = pkv.config_of(w, inputs_final=mode == "full_stop_inputs_final")
        kl = pkv.layer_budgets(cfg)[0]
        rows = pkv.total_rows(cfg, kl, lens)
        ws = pkv.new_workspace(cfg, 1, max(lens), DEV)
        k_live = torch.zeros_like(x.k)                       # filled on the stream, right before the call
        k_out = torch.empty(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
        v_out = torch.empty_like(k_out)
        idx = torch.empty(rows, dtype=torch.int32, device=DEV)
        scores = torch.zeros(1, w.num_kv_heads, max(lens), dtype=torch.float32, device=DEV)
        torch.cuda.synchronize()
        binding.slow_copy(k_live, x.k, steps=64)
        if mode != "back_to_back":
            torch.cuda.synchronize()
        pkv.compress_layer(cfg, 0, x.q_win, k_live, x.v, lens, k_out, v_out, idx, ws, scores=scores)
        pkv.check_status(ws)
        assert torch.equal(k_live, x.k)
        results.append((scores.clone(), idx.clone(), k_out.clone(), v_out.clone()))
    for other in results[1:]:
        for a, b in zip(results[0], other):
            assert torch.equal(a, b)


def test_a_wait_that_runs_out_is_reported_and_the_workspace_stays_usable():
    """Every wait inside the tensor-core kernels is bounded.  Here one K tile of one CTA is never loaded and the bound
    is lowered to about a millisecond: the waits for that tile give up, the kernel winds down by itself (all roles
    leave, accumulator memory released), the status word says so, and the next ordinary call on the same workspace
    gives exactly what a fresh workspace gives."""
    w = workloads.scaled(workloads.LLAMA3_8B, num_layers=2, seq_len=7000 + 5, name="llama3_8b_7k_expired_wait")
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    x = workloads.make_layer(w, 1, device=DEV)
    ws = pkv.new_workspace(cfg, 1, max(lens), DEV)
    scores = torch.zeros(1, w.num_kv_heads, max(lens), dtype=torch.float32, device=DEV)
    try:
        binding.test_hooks(wait_clocks=1 << 21, withhold_tile=True)
        pkv.score_window(cfg, x.q_win, x.k, lens, scores, ws)
        with pytest.raises(pkv.PkvError) as e:
            pkv.check_status(ws)
        assert e.value.status == binding.PKV_ERR_DEVICE_STATUS and "0x2" in str(e.value)
    finally:
        binding.test_hooks(0, False)
    ws[:256].zero_()
    again = torch.zeros_like(scores)
    pkv.score_window(cfg, x.q_win, x.k, lens, again, ws)
    pkv.check_status(ws)
    fresh_ws = pkv.new_workspace(cfg, 1, max(lens), DEV)
    fresh = torch.zeros_like(scores)
    pkv.score_window(cfg, x.q_win, x.k, lens, fresh, fresh_ws)
    pkv.check_status(fresh_ws)
    assert torch.equal(again, fresh)
    want, _ = oracle.window_scores(x.q_win[0].cpu(), x.k[0, :, : lens[0]].cpu())
    assert_scores_close(again[0, :, : lens[0] - w.window].cpu().numpy(), want, "after the expired wait")


@pytest.mark.parametrize("hq,hkv,alpha,d,dtype,lens", [
    (8, 8, 32, 128, "bf16", [4096]),                    # the multi-head 4k shape: two tiles per CTA, clusters of 8 ... 4
    (6, 2, 8, 64, "fp16", [41, 3000, 257]),             # 24 window rows of 3 query heads, ragged: some CTAs hold no tile
    (4, 4, 16, 128, "bf16", [16384, 9000]),             # the longest context the kernel takes: 16 tiles per CTA
    (2, 2, 32, 128, "bf16", [2049 + 32]),               # a ragged last tile
])
def test_single_sweep_kernel_for_short_contexts(hq, hkv, alpha, d, dtype, lens):
    """Up to 32 window rows per KV head and 16384 keys: the logits of a head stay in tensor memory across a
    thread-block cluster and K is swept once.  Against the oracle, and against the two-sweep kernels on the same
    inputs (a test switch keeps the call on them): equal within twice the score tolerance."""
    tdt = {"bf16": torch.bfloat16, "fp16": torch.float16}[dtype]
    cfg = pkv.make_config(num_layers=1, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, window=alpha, pool_kernel=7,
                          dtype=dtype, avg_budget=alpha + 8)
    g = torch.Generator(device="cpu").manual_seed(hq * 1000 + alpha + len(lens))
    n_max = max(lens)
    q = (torch.randn(len(lens), hq, alpha, d, generator=g) * 1.5).to(tdt)
    k = torch.randn(len(lens), hkv, n_max, d, generator=g).to(tdt)
    k[:, :, 0] *= 3.0                                          # a sink
    qd, kd = q.to(DEV), k.to(DEV)
    ws = pkv.new_workspace(cfg, len(lens), n_max, DEV)
    both = []
    for two in (False, True):
        scores = torch.full((len(lens), hkv, n_max), -1.0, dtype=torch.float32, device=DEV)
        try:
            binding.test_hooks(two_sweeps=two)
            pkv.score_window(cfg, qd, kd, lens, scores, ws)
            pkv.check_status(ws)
        finally:
            binding.test_hooks()
        both.append(scores.cpu().numpy())
    for b, n in enumerate(lens):
        want, _ = oracle.window_scores(q[b], k[b, :, :n])
        assert_scores_close(both[0][b, :, : n - alpha], want, "single sweep, seq %d" % b)
        assert_scores_close(both[1][b, :, : n - alpha], want, "two sweeps, seq %d" % b)
        assert (both[0][b, :, n - alpha:] == -1.0).all()       # nothing written beyond the prefix


@pytest.mark.parametrize("case", ["mha_4k_layer0", "mha_4k_top_layer", "ragged_with_short", "ties", "mean_pool",
                                  "wide_pool", "alpha8_gqa3"])
def test_short_context_layer_equals_three_calls(case):
    """Short multi-head contexts go through the single-sweep cluster kernel.  The fused per-layer call against the
    three separate calls on the same inputs: identical scores, lists and rows, bit for bit; and the lists are the
    oracle's selection on those scores (max and mean pool, ties everywhere, a batch with a sequence short enough to
    be kept whole, 24 window rows of a 3:1 group)."""
    base = workloads.scaled(workloads.LLAMA2_7B, num_layers=4, num_q_heads=8, num_kv_heads=8, name="tail_" + case)
    layer, lens, same_keys = 0, None, False
    if case == "mha_4k_layer0":
        w = base
    elif case == "mha_4k_top_layer":
        w, layer = base, 3
    elif case == "ragged_with_short":
        w, lens = workloads.scaled(base, batch=4), [4096, 100, 1333, 16384]      # 100 <= B: kept whole
    elif case == "ties":
        w, lens, same_keys = base, [3000], True
    elif case == "mean_pool":
        w = workloads.scaled(base, pool_kind="avg", seq_len=2500)
    elif case == "wide_pool":
        w = workloads.scaled(base, pool_kernel=13, seq_len=5000)
    else:
        w = workloads.scaled(base, num_q_heads=6, num_kv_heads=2, window=8, avg_budget=40, seq_len=7777)
    cfg = pkv.config_of(w)
    lens = lens or w.seq_lens()
    kl = pkv.layer_budgets(cfg)[layer]
    x = workloads.make_layer(w, layer, device=DEV, seq_lens=lens)
    if same_keys:
        x.k[:, :, : min(lens) - w.window] = x.k[:, :, :1]        # every prefix key the same: the ties decide
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    rows = pkv.total_rows(cfg, kl, lens)
    outs = []
    for fused in (True, False):
        k_out = torch.zeros(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
        v_out = torch.zeros_like(k_out)
        idx = torch.full((rows,), -5, dtype=torch.int32, device=DEV)
        scores = torch.zeros(len(lens), w.num_kv_heads, max(lens), dtype=torch.float32, device=DEV)
        if fused:
            pkv.compress_layer(cfg, layer, x.q_win, x.k, x.v, lens, k_out, v_out, idx, ws, scores=scores)
        else:
            pkv.score_window(cfg, x.q_win, x.k, lens, scores, ws)
            pkv.select_topk(cfg, scores, lens, kl, idx, ws)
            pkv.gather_compact(cfg, x.k, x.v, idx, lens, kl, k_out, v_out)
        pkv.check_status(ws)
        outs.append((scores, idx, k_out, v_out))
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    scores, idx = outs[0][0].cpu().numpy(), outs[0][1].cpu().numpy()
    pool = oracle.pool_avg if w.pool_kind == "avg" else oracle.pool_max
    off = 0
    for b, n in enumerate(lens):
        c = pkv.kept_count(cfg, kl, n)
        for h in range(w.num_kv_heads):
            got = idx[off + h * c: off + (h + 1) * c]
            if c < n:
                want = oracle.select_topk(pool(scores[b, h, : n - w.window], w.pool_kernel), c - w.window)
                assert np.array_equal(got[: c - w.window], want)
                assert np.array_equal(got[c - w.window:], np.arange(n - w.window, n))
            else:
                assert np.array_equal(got, np.arange(n))
        off += w.num_kv_heads * c
