"""Pins for the oracle's paged placement of the compact cache (per-layer block tables)."""
import numpy as np
import pytest
import torch

import oracle


@pytest.mark.parametrize("c,ps", [(1, 16), (16, 16), (17, 16), (220, 16), (36, 8), (5, 1), (100, 128)])
def test_scatter_equals_library_indexing_and_read_is_its_inverse(c, ps):
    g = torch.Generator().manual_seed(c * 10 + ps)
    d, num_pages = 64, 40
    rows = torch.randn(c, d, generator=g).to(torch.bfloat16)
    pages = (c + ps - 1) // ps
    table = torch.randperm(num_pages, generator=g)[:pages].numpy().astype(np.int32)     # any free pages, any order
    pool = torch.full((num_pages, ps, d), -3.0, dtype=torch.bfloat16)
    oracle.scatter_paged(rows, table, ps, pool)
    want = torch.full((num_pages, ps, d), -3.0, dtype=torch.bfloat16)
    r = torch.arange(c)
    want[torch.from_numpy(table).long()[r // ps], r % ps] = rows                         # library fancy indexing
    assert torch.equal(pool, want)                     # also: other pages and the tail of the last page untouched
    assert torch.equal(oracle.read_paged(pool, table, c, ps), rows)


def test_pages_needed_is_the_ceiling_of_the_kept_count():
    for n, kl, ps in [(4096, 188, 16), (4096, 4, 16), (100, 188, 16), (5000, 937, 128), (40, 10, 1)]:
        c = oracle.kept_count(128, 32, kl, n)
        assert oracle.pages_needed(128, 32, kl, n, ps) == -(-c // ps)
    with pytest.raises(ValueError):
        oracle.pages_needed(128, 32, 10, 4096, 0)


def test_a_page_outside_the_pool_is_refused():
    rows = torch.zeros(20, 8)
    pool = torch.zeros(4, 16, 8)
    with pytest.raises(ValueError):
        oracle.scatter_paged(rows, np.array([0, 4], dtype=np.int32), 16, pool)
    with pytest.raises(ValueError):
        oracle.read_paged(pool, np.array([-1, 2], dtype=np.int32), 20, 16)
    assert not pool.any()


def test_decode_over_pages_equals_decode_over_the_packed_rows():
    """Attention only needs the rows in list order, so any placement of the pages gives the same output."""
    g = torch.Generator().manual_seed(3)
    c, d, ps = 53, 64, 16
    k_rows, v_rows, q = torch.randn(c, d, generator=g), torch.randn(c, d, generator=g), torch.randn(d, generator=g)
    table = np.array([7, 2, 9, 0], dtype=np.int32)
    kp, vp = torch.zeros(12, ps, d), torch.zeros(12, ps, d)
    oracle.scatter_paged(k_rows, table, ps, kp)
    oracle.scatter_paged(v_rows, table, ps, vp)
    a = oracle.decode_attention(q, oracle.read_paged(kp, table, c, ps), oracle.read_paged(vp, table, c, ps))
    b = oracle.decode_attention(q, k_rows, v_rows)
    assert np.array_equal(a, b)
    want = torch.softmax((k_rows.double() @ q.double()) / 8.0, 0) @ v_rows.double()
    np.testing.assert_allclose(a, want.numpy(), rtol=1e-12, atol=1e-14)
