"""The oracle's widening of 16-bit inputs, pinned against torch's own conversions.

A one-row cache makes decode attention return that row of V unchanged (its softmax weight is exactly 1), so
every finite bit pattern can be pushed through the oracle's element reader and compared with the value the
library conversion gives.
"""
import numpy as np
import pytest
import torch

import oracle


def _all_finite(dtype):
    bits = torch.arange(0, 65536, dtype=torch.int32).to(torch.int16)
    vals = bits.view(dtype)
    return vals[torch.isfinite(vals.float())]


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_every_finite_pattern_widens_exactly(dtype):
    v = _all_finite(dtype).reshape(1, -1).contiguous()
    d = v.shape[1]
    zero = torch.zeros(d, dtype=dtype)
    out = oracle.decode_attention(zero, zero.reshape(1, d), v)
    want = v.double().numpy().reshape(-1)
    assert np.array_equal(out, want)                 # -0 comes back as +0 (it is added to a zero accumulator)
    nz = want != 0
    assert np.array_equal(np.signbit(out[nz]), np.signbit(want[nz]))


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_scores_equal_those_of_the_widened_inputs(dtype):
    g = torch.Generator().manual_seed(11)
    q = torch.randn(4, 8, 64, generator=g).to(dtype)
    k = torch.randn(2, 300, 64, generator=g).to(dtype)
    s16, m16 = oracle.window_scores(q, k)
    s32, m32 = oracle.window_scores(q.float(), k.float())
    assert np.array_equal(s16, s32) and np.array_equal(m16, m32)


def test_fp16_layer_matches_float_layer_bit_for_bit():
    g = torch.Generator().manual_seed(12)
    q = torch.randn(4, 8, 64, generator=g).half()
    k = torch.randn(2, 400, 64, generator=g).half()
    v = torch.randn(2, 400, 64, generator=g).half()
    a = oracle.compress_layer(q, k, v, pool_kernel=5, avg_budget=64, k_layer=40)
    b = oracle.compress_layer(q.float(), k.float(), v.float(), pool_kernel=5, avg_budget=64, k_layer=40)
    assert np.array_equal(a["kept"], b["kept"])
    assert torch.equal(a["k_out"].float(), b["k_out"]) and torch.equal(a["v_out"].float(), b["v_out"])
    assert a["k_out"].dtype == torch.float16
