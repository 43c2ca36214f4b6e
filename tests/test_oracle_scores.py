"""Pins for the oracle's window scores (Section 4.2.2, Eq. 2 and Eq. 3)."""
import math

import numpy as np
import pytest
import torch

import oracle


def draw(hq, hkv, alpha, n, d, seed, dtype=torch.float32):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(hq, alpha, d, generator=g).to(dtype)
    k = torch.randn(hkv, n, d, generator=g).to(dtype)
    return q, k


def library_scores(q, k):
    """Eq. 2-3 through torch's own softmax in float64 (a library routine, not the oracle's loop)."""
    hq, alpha, d = q.shape
    hkv, n, _ = k.shape
    group = hq // hkv
    P = n - alpha
    qd, kd = q.double(), k.double()
    logits = torch.einsum("gjd,gnd->gjn", qd, kd.repeat_interleave(group, dim=0)) / math.sqrt(d)
    pos_q = torch.arange(P, n).view(1, alpha, 1)
    pos_k = torch.arange(n).view(1, 1, n)
    logits = logits.masked_fill(pos_k > pos_q, float("-inf"))
    att = torch.softmax(logits, dim=-1)                      # rows sum to one
    per_q_head = att.sum(dim=1)                              # Eq. 3: sum over the window rows
    per_kv_head = per_q_head.view(hkv, group, n).mean(dim=1)  # mean over the group's query heads
    return per_kv_head[:, :P].numpy(), per_kv_head[:, P:].sum(dim=1).numpy()


@pytest.mark.parametrize("hq,hkv,alpha,n,d,dtype", [
    (4, 2, 8, 97, 64, torch.float32), (4, 4, 5, 40, 16, torch.float32),
    (8, 2, 3, 33, 32, torch.bfloat16), (6, 1, 1, 20, 8, torch.float32),
    (2, 2, 16, 300, 128, torch.bfloat16),
])
def test_matches_library_softmax(hq, hkv, alpha, n, d, dtype):
    q, k = draw(hq, hkv, alpha, n, d, seed=11 + n, dtype=dtype)
    got, mass = oracle.window_scores(q, k)
    want, want_mass = library_scores(q, k)
    np.testing.assert_allclose(got, want, rtol=2e-7, atol=1e-12)   # float rounding of the output
    np.testing.assert_allclose(mass, want_mass, rtol=1e-12)


@pytest.mark.parametrize("hq,hkv,alpha,n,d", [(4, 2, 8, 200, 64), (8, 8, 4, 77, 32), (8, 1, 6, 50, 16)])
def test_attention_mass_sums_to_alpha(hq, hkv, alpha, n, d):
    q, k = draw(hq, hkv, alpha, n, d, seed=5)
    s, mass = oracle.window_scores(q, k)
    total = s.astype(np.float64).sum(axis=1) + mass
    np.testing.assert_allclose(total, np.full(hkv, float(alpha)), rtol=0, atol=1e-5)


def test_zero_queries_give_harmonic_closed_form():
    hq, hkv, alpha, n, d = 4, 2, 6, 64, 16
    _, k = draw(hq, hkv, alpha, n, d, seed=3)
    q = torch.zeros(hq, alpha, d)
    s, mass = oracle.window_scores(q, k)
    P = n - alpha
    want = sum(1.0 / (P + j + 1) for j in range(alpha))     # every visible key gets 1/visible
    np.testing.assert_allclose(s, np.full((hkv, P), want, dtype=np.float32), rtol=2e-7)
    want_mass = sum((j + 1) / (P + j + 1) for j in range(alpha))
    np.testing.assert_allclose(mass, np.full(hkv, want_mass), rtol=1e-12)


def test_single_row_single_head_is_one_softmax_row():
    d, n = 32, 50
    q, k = draw(1, 1, 1, n, d, seed=9)
    s, mass = oracle.window_scores(q, k)
    logits = (k[0].double() @ q[0, 0].double()) / math.sqrt(d)
    row = torch.softmax(logits, dim=0).numpy()
    np.testing.assert_allclose(s[0], row[: n - 1], rtol=2e-7)
    np.testing.assert_allclose(mass[0], row[n - 1], rtol=1e-12)


def test_causal_mask_inside_the_window():
    """Changing window key P+j must not change what earlier window rows contribute."""
    hq, hkv, alpha, n, d = 2, 1, 4, 30, 8
    q, k = draw(hq, hkv, alpha, n, d, seed=21)
    P = n - alpha
    base_first_row = library_scores(q[:, :1], k[:, : P + 1])[0]   # row 0 alone sees keys 0..P
    k2 = k.clone()
    k2[:, P + 1:] = 50.0 * torch.randn(hkv, alpha - 1, d)          # later window keys change
    s1, _ = oracle.window_scores(q[:, :1], k[:, : P + 1])
    np.testing.assert_allclose(s1, base_first_row, rtol=2e-7)
    # with alpha rows: the contribution of row 0 is unchanged, so the difference of full scores
    # between k and k2 must equal the difference computed by the library routine
    a, _ = oracle.window_scores(q, k)
    b, _ = oracle.window_scores(q, k2)
    la, _ = library_scores(q, k)
    lb, _ = library_scores(q, k2)
    np.testing.assert_allclose(a - b, la - lb, atol=1e-6)


def test_logit_shift_leaves_scores_unchanged():
    """An extra feature that adds the same constant to every logit of a row changes nothing."""
    hq, hkv, alpha, n, d = 4, 2, 4, 60, 16
    q, k = draw(hq, hkv, alpha, n, d, seed=8)
    s0, m0 = oracle.window_scores(q, k)
    # large enough that exp() of an unshifted logit overflows: guards the max subtraction
    shift = 4000.0 * (1.0 + torch.rand(hq, alpha, 1))
    scale_fix = math.sqrt((d + 1) / d)                      # keep the 1/sqrt(d) factor of the old part
    q2 = torch.cat([q * scale_fix, shift], dim=2)
    k2 = torch.cat([k, torch.ones(hkv, n, 1)], dim=2)
    s1, m1 = oracle.window_scores(q2, k2)
    np.testing.assert_allclose(s1, s0, rtol=1e-5, atol=1e-9)
    np.testing.assert_allclose(m1, m0, rtol=1e-5)


def test_sink_limit():
    """A prefix key ever more aligned with all queries takes all the prefix attention."""
    hq, hkv, alpha, n, d = 4, 2, 4, 80, 16
    g = torch.Generator().manual_seed(2)
    u = torch.randn(d, generator=g)
    u /= u.norm()
    q = 0.1 * torch.randn(hq, alpha, d, generator=g) + 3.0 * u
    k = torch.randn(hkv, n, d, generator=g)
    prev = None
    for gain in (1.0, 10.0, 100.0):
        k2 = k.clone()
        k2[:, 7] += gain * u
        s, _ = oracle.window_scores(q, k2)
        if prev is not None:
            assert (s[:, 7] > prev).all()
        prev = s[:, 7].copy()
    assert np.all(prev > alpha - 1e-3)
    others = np.delete(s, 7, axis=1)
    assert others.max() < 1e-3


def test_gqa_is_mean_of_per_head_scores():
    hq, hkv, alpha, n, d = 8, 2, 4, 64, 16
    q, k = draw(hq, hkv, alpha, n, d, seed=4)
    s, _ = oracle.window_scores(q, k)
    group = hq // hkv
    for h in range(hkv):
        parts = [oracle.window_scores(q[h * group + g: h * group + g + 1], k[h: h + 1])[0][0].astype(np.float64)
                 for g in range(group)]
        np.testing.assert_allclose(s[h], np.mean(parts, axis=0), rtol=3e-7)


def test_bf16_inputs_are_widened_exactly():
    q, k = draw(2, 1, 4, 40, 16, seed=6, dtype=torch.bfloat16)
    a, _ = oracle.window_scores(q, k)
    b, _ = oracle.window_scores(q.float(), k.float())
    np.testing.assert_array_equal(a, b)


def test_row_lse_matches_library_logsumexp():
    """The log-denominators handed to the single-sweep mode are torch.logsumexp of the masked logits."""
    hq, hkv, alpha, n, d = 6, 2, 5, 70, 16
    q, k = draw(hq, hkv, alpha, n, d, seed=31)
    got = oracle.window_lse(q, k)
    group = hq // hkv
    logits = torch.einsum("gjd,gnd->gjn", q.double(), k.double().repeat_interleave(group, dim=0)) / math.sqrt(d)
    mask = torch.arange(n).view(1, 1, n) > torch.arange(n - alpha, n).view(1, alpha, 1)
    want = torch.logsumexp(logits.masked_fill(mask, float("-inf")), dim=-1).numpy()
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)
    # and scores are exactly exp(logit - lse) summed over rows, averaged over the group
    s, _ = oracle.window_scores(q, k)
    att = torch.exp(logits.masked_fill(mask, float("-inf")) - torch.from_numpy(got).unsqueeze(-1))
    want_s = att.sum(dim=1).view(hkv, group, n).mean(dim=1)[:, : n - alpha].numpy()
    np.testing.assert_allclose(s, want_s, rtol=3e-7)
