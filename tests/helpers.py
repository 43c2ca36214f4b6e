"""Comparison protocol shared by the GPU parity tests."""
import numpy as np
import torch

import oracle

RTOL, ATOL = 2e-3, 1e-5     # score tolerance: |gpu - oracle| <= RTOL * |oracle| + ATOL (fp32)
INDEX_SLACK = 1.0           # index sets may differ where the oracle's pooled score is within this many score
                            # tolerances of its k-th pooled value
# Every kept list compared in this session: [lists, identical lists, largest |pooled - kth| / tolerance among the
# lists that differed].  tests/conftest.py prints it at the end of a run.
INDEX_LOG = {"lists": 0, "identical": 0, "worst": 0.0}


def assert_scores_close(got: np.ndarray, want: np.ndarray, what=""):
    err = np.abs(got.astype(np.float64) - want.astype(np.float64))
    bound = RTOL * np.abs(want.astype(np.float64)) + ATOL
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError("%s scores differ at %s: got %r want %r (%d of %d outside tolerance)"
                             % (what, i, got[i], want[i], int(bad.sum()), bad.size))


def assert_indices_match(got_row: np.ndarray, want_row: np.ndarray, oracle_scores_row: np.ndarray, w: int,
                         alpha: int, what="", pool_kind="max"):
    """Kept lists of one (sequence, head): identical, or differing only where the oracle's pooled
    score is within tolerance of the oracle's k-th pooled value (the threshold)."""
    assert len(got_row) == len(want_row), what
    # window block and ordering are exact requirements
    assert np.array_equal(got_row[len(got_row) - alpha:], want_row[len(want_row) - alpha:]), what + " window block"
    assert np.all(np.diff(got_row) > 0), what + " not strictly ascending"
    INDEX_LOG["lists"] += 1
    if np.array_equal(got_row, want_row):
        INDEX_LOG["identical"] += 1
        return True
    P = oracle_scores_row.shape[0]
    pool = oracle.pool_avg if pool_kind == "avg" else oracle.pool_max
    pooled = pool(oracle_scores_row, w).astype(np.float64)
    k = len(want_row) - alpha
    kth = np.sort(pooled)[::-1][k - 1]
    diff = np.setxor1d(got_row[:k], want_row[:k])
    assert diff.size > 0 and diff.max() < P
    slack = RTOL * abs(kth) + ATOL
    worst = np.max(np.abs(pooled[diff] - kth))
    INDEX_LOG["worst"] = max(INDEX_LOG["worst"], float(worst / slack))
    assert worst <= INDEX_SLACK * slack, "%s: index sets differ away from the threshold (|pooled - kth| = %g, " \
                                         "tolerance %g)" % (what, worst, slack)
    return False


def packed_rows(counts, num_kv_heads):
    """Yield (b, h, slice) over the packed ragged layout."""
    off = 0
    for b, c in enumerate(counts):
        for h in range(num_kv_heads):
            yield b, h, slice(off + h * c, off + (h + 1) * c)
        off += num_kv_heads * c
