"""GPU parity for the paged placement of the compact cache (per-layer block tables)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2406_02069_b200 as pkv
from paper_2406_02069_b200 import binding, workloads
from helpers import packed_rows

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make_tables(cfg, lens, kl, page_size, num_kv_heads, seed, spare=7):
    """A block table as an allocator would hand out: distinct pages in a shuffled order, some left free."""
    pages = [pkv.pages_needed(cfg, kl, n, page_size) for n in lens]
    total = num_kv_heads * sum(pages)
    g = torch.Generator().manual_seed(seed)
    table = torch.randperm(total + spare, generator=g)[:total].to(torch.int32)
    return pages, table, total + spare


def head_slices(pages, num_kv_heads):
    off = 0
    for b, pg in enumerate(pages):
        for h in range(num_kv_heads):
            yield b, h, slice(off + h * pg, off + (h + 1) * pg)
        off += num_kv_heads * pg


@pytest.mark.parametrize("w,page_size", [
    (workloads.TINY, 4),
    (workloads.scaled(workloads.LLAMA3_8B, num_layers=2, seq_len=5037, name="llama3_8b_5k"), 16),
    (workloads.scaled(workloads.MISTRAL_RAGGED, num_layers=2, batch=3, name="mistral_b3"), 16),
    (workloads.scaled(workloads.LLAMA3_70B, num_layers=3, seq_len=3011, name="llama3_70b_3k"), 128),
], ids=lambda x: getattr(x, "name", "ps%s" % x))
def test_paged_layer_equals_packed_layer_and_oracle_placement(w, page_size):
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    if w.batch > 1:
        lens = [300 + (n % 1777) for n in lens]
    budgets = pkv.layer_budgets(cfg)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    for layer in range(w.num_layers):
        kl = budgets[layer]
        x = workloads.make_layer(w, layer, device=DEV, seq_lens=lens)
        rows = pkv.total_rows(cfg, kl, lens)
        counts = [pkv.kept_count(cfg, kl, n) for n in lens]
        # packed call: the reference for which rows are kept
        k_out = torch.empty(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
        v_out = torch.empty_like(k_out)
        idx = torch.empty(rows, dtype=torch.int32, device=DEV)
        pkv.compress_layer(cfg, layer, x.q_win, x.k, x.v, lens, k_out, v_out, idx, ws)
        # paged call
        pages, table, num_pages = make_tables(cfg, lens, kl, page_size, w.num_kv_heads, seed=layer + 1)
        assert pages == [oracle.pages_needed(w.avg_budget, w.window, kl, n, page_size) for n in lens]
        k_pool = torch.full((num_pages, page_size, w.head_dim), -3.0, dtype=x.k.dtype, device=DEV)
        v_pool = torch.full_like(k_pool, -5.0)
        idx2 = torch.empty(rows, dtype=torch.int32, device=DEV)
        pkv.compress_layer_paged(cfg, layer, x.q_win, x.k, x.v, lens, table.to(DEV), k_pool, v_pool, idx2, ws)
        pkv.check_status(ws)
        assert torch.equal(idx, idx2)
        # oracle placement of the packed rows through the same table: pools must agree bit for bit,
        # untouched slots included
        want_k = torch.full((num_pages, page_size, w.head_dim), -3.0, dtype=x.k.dtype)
        want_v = torch.full_like(want_k, -5.0)
        kc, vc, tab = k_out.cpu(), v_out.cpu(), table.numpy()
        for (b, h, rs), (_, _, ts) in zip(packed_rows(counts, w.num_kv_heads), head_slices(pages, w.num_kv_heads)):
            oracle.scatter_paged(kc[rs], tab[ts], page_size, want_k)
            oracle.scatter_paged(vc[rs], tab[ts], page_size, want_v)
        assert torch.equal(k_pool.cpu(), want_k) and torch.equal(v_pool.cpu(), want_v)
        # the stand-alone gather does the same from the index list
        k_pool2 = torch.full_like(k_pool, -3.0)
        v_pool2 = torch.full_like(v_pool, -5.0)
        pkv.gather_paged(cfg, x.k, x.v, idx, lens, kl, table.to(DEV), k_pool2, v_pool2, ws)
        pkv.check_status(ws)
        assert torch.equal(k_pool2, k_pool) and torch.equal(v_pool2, v_pool)
        # decode through the table: the packed kernel's output, and the oracle's
        g = torch.Generator().manual_seed(9)
        q_new = torch.randn(len(lens), w.num_q_heads, w.head_dim, generator=g).to(x.k.dtype)
        out_packed = torch.empty(len(lens), w.num_q_heads, w.head_dim, dtype=torch.float32, device=DEV)
        out_paged = torch.empty_like(out_packed)
        pkv.decode_attention(cfg, q_new.to(DEV), k_out, v_out, lens, kl, out_packed)
        pkv.decode_attention_paged(cfg, q_new.to(DEV), table.to(DEV), k_pool, v_pool, lens, kl, out_paged, ws)
        pkv.check_status(ws)
        assert torch.equal(out_packed, out_paged)            # same rows in the same order: same arithmetic
        got = out_paged.cpu().numpy()
        pool_k, pool_v = k_pool.cpu(), v_pool.cpu()
        for (b, h, ts), c in zip(head_slices(pages, w.num_kv_heads), [c for c in counts for _ in range(w.num_kv_heads)]):
            k_rows = oracle.read_paged(pool_k, tab[ts], c, page_size)
            v_rows = oracle.read_paged(pool_v, tab[ts], c, page_size)
            hq = h * w.group
            want = oracle.decode_attention(q_new[b, hq], k_rows, v_rows)
            np.testing.assert_allclose(got[b, hq], want, rtol=2e-3, atol=2e-4)


def test_single_sweep_mode_places_the_same_pages():
    w = workloads.scaled(workloads.LLAMA3_8B, num_layers=2, seq_len=3001, name="llama3_8b_3k")
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    layer, page_size = 1, 16
    kl = pkv.layer_budgets(cfg)[layer]
    x = workloads.make_layer(w, layer, device=DEV)
    qc, kc = x.q_win.cpu(), x.k.cpu()
    lse = torch.from_numpy(np.stack([oracle.window_lse(qc[b], kc[b, :, :n]) for b, n in enumerate(lens)])
                           .astype(np.float32)).to(DEV)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    rows = pkv.total_rows(cfg, kl, lens)
    pages, table, num_pages = make_tables(cfg, lens, kl, page_size, w.num_kv_heads, seed=3)
    outs = []
    for use in (None, lse):
        k_pool = torch.zeros(num_pages, page_size, w.head_dim, dtype=x.k.dtype, device=DEV)
        v_pool = torch.zeros_like(k_pool)
        idx = torch.empty(rows, dtype=torch.int32, device=DEV)
        pkv.compress_layer_paged(cfg, layer, x.q_win, x.k, x.v, lens, table.to(DEV), k_pool, v_pool, idx, ws,
                                 window_lse=use)
        pkv.check_status(ws)
        outs.append((idx.cpu(), k_pool.cpu(), v_pool.cpu()))
    same = [torch.equal(outs[0][0][sl], outs[1][0][sl]) for _, _, sl in
            packed_rows([pkv.kept_count(cfg, kl, n) for n in lens], w.num_kv_heads)]
    assert np.mean(same) >= 0.75
    if all(same):
        assert torch.equal(outs[0][1], outs[1][1]) and torch.equal(outs[0][2], outs[1][2])


def test_a_page_outside_the_pool_is_reported_and_never_written():
    w = workloads.TINY
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    kl = pkv.layer_budgets(cfg)[0]
    x = workloads.make_layer(w, 0, device=DEV)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    rows = pkv.total_rows(cfg, kl, lens)
    page_size = 8
    pages, table, num_pages = make_tables(cfg, lens, kl, page_size, w.num_kv_heads, seed=1, spare=0)
    bad = table.clone()
    bad[1] = num_pages                                     # one past the pool
    bad[2] = -1
    k_pool = torch.full((num_pages, page_size, w.head_dim), -3.0, dtype=x.k.dtype, device=DEV)
    v_pool = torch.full_like(k_pool, -5.0)
    idx = torch.empty(rows, dtype=torch.int32, device=DEV)
    pkv.compress_layer_paged(cfg, 0, x.q_win, x.k, x.v, lens, bad.to(DEV), k_pool, v_pool, idx, ws)
    with pytest.raises(pkv.PkvError) as e:
        pkv.check_status(ws)
    assert e.value.status == binding.PKV_ERR_DEVICE_STATUS
    # the pages the two bad entries replaced stay untouched; every other page was filled
    for j in (1, 2):
        assert (k_pool[int(table[j])] == -3.0).all() and (v_pool[int(table[j])] == -5.0).all()
    assert not (k_pool[int(table[0])] == -3.0).all()
    ws[:256].zero_()
    out = torch.empty(len(lens), w.num_q_heads, w.head_dim, dtype=torch.float32, device=DEV)
    q_new = torch.randn(len(lens), w.num_q_heads, w.head_dim, device=DEV).to(x.k.dtype)
    pkv.decode_attention_paged(cfg, q_new, bad.to(DEV), k_pool, v_pool, lens, kl, out, ws)
    with pytest.raises(pkv.PkvError):
        pkv.check_status(ws)
    ws[:256].zero_()
    pkv.check_status(ws)
    # host-side refusals
    with pytest.raises(pkv.PkvError):
        pkv.pages_needed(cfg, kl, lens[0], 0)
    with pytest.raises(ValueError):
        pkv.gather_paged(cfg, x.k, x.v, idx, lens, kl, table.to(DEV).long(), k_pool, v_pool, ws)


def test_an_index_outside_its_sequence_is_never_used_as_an_address():
    """Index lists may come from the caller.  An entry below 0 or beyond the sequence is skipped by the gather kernels
    (its output row keeps what it held), the other rows are copied bit for bit, the paged gather records it in the
    status word (bit 3), and the recall diagnostic counts it as not kept."""
    w = workloads.scaled(workloads.LLAMA3_8B, num_layers=2, seq_len=700, avg_budget=64, name="bad_index")
    cfg = pkv.config_of(w)
    lens = w.seq_lens()
    kl = pkv.layer_budgets(cfg)[0]
    x = workloads.make_layer(w, 0, device=DEV)
    ws = pkv.new_workspace(cfg, len(lens), max(lens), DEV)
    rows = pkv.total_rows(cfg, kl, lens)
    good = torch.empty(rows, dtype=torch.int32, device=DEV)
    scores = torch.zeros(1, w.num_kv_heads, max(lens), dtype=torch.float32, device=DEV)
    k_ref = torch.empty(rows, w.head_dim, dtype=x.k.dtype, device=DEV)
    v_ref = torch.empty_like(k_ref)
    pkv.compress_layer(cfg, 0, x.q_win, x.k, x.v, lens, k_ref, v_ref, good, ws, scores=scores)
    pkv.check_status(ws)
    bad = good.clone()
    bad_rows = [3, 17, rows - 1]
    bad[3], bad[17], bad[rows - 1] = -1, lens[0], 2 ** 30      # below, one past the end, far beyond
    ok_rows = torch.ones(rows, dtype=torch.bool, device=DEV)
    ok_rows[bad_rows] = False
    # stand-alone gather: no workspace, so nothing to record; the rows are simply left alone
    k_out = torch.full((rows, w.head_dim), -3.0, dtype=x.k.dtype, device=DEV)
    v_out = torch.full_like(k_out, -5.0)
    pkv.gather_compact(cfg, x.k, x.v, bad, lens, kl, k_out, v_out)
    torch.cuda.synchronize()
    assert torch.equal(k_out[ok_rows], k_ref[ok_rows]) and torch.equal(v_out[ok_rows], v_ref[ok_rows])
    assert (k_out[bad_rows] == -3.0).all() and (v_out[bad_rows] == -5.0).all()
    # paged gather: the same, and the status word says so
    page_size = 16
    pages, table, num_pages = make_tables(cfg, lens, kl, page_size, w.num_kv_heads, seed=3, spare=2)
    k_pool = torch.full((num_pages, page_size, w.head_dim), -3.0, dtype=x.k.dtype, device=DEV)
    v_pool = torch.full_like(k_pool, -5.0)
    pkv.gather_paged(cfg, x.k, x.v, bad, lens, kl, table.to(DEV), k_pool, v_pool, ws)
    with pytest.raises(pkv.PkvError) as e:
        pkv.check_status(ws)
    assert e.value.status == binding.PKV_ERR_DEVICE_STATUS and "0x8" in str(e.value)
    ws[:256].zero_()
    k_pool2 = torch.full_like(k_pool, -3.0)
    v_pool2 = torch.full_like(v_pool, -5.0)
    pkv.gather_paged(cfg, x.k, x.v, good, lens, kl, table.to(DEV), k_pool2, v_pool2, ws)
    pkv.check_status(ws)
    differ = (k_pool != k_pool2).any(dim=2).sum().item()
    assert differ == len(bad_rows)                              # exactly the three skipped slots
    # recall: a bad entry is not a kept position
    rec_good = torch.zeros(1, w.num_kv_heads, dtype=torch.float32, device=DEV)
    rec_bad = torch.zeros_like(rec_good)
    pkv.attention_recall(cfg, scores, good, lens, kl, rec_good)
    pkv.attention_recall(cfg, scores, bad, lens, kl, rec_bad)
    torch.cuda.synchronize()
    assert rec_bad[0, 0] < rec_good[0, 0]                      # rows 3 and 17 belong to head 0: two kept keys fewer
    assert torch.equal(rec_bad[0, 1:], rec_good[0, 1:])        # the last bad entry sits in a window slot: not counted
