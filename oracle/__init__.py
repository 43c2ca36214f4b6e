"""CPU oracle for the PyramidKV prefill KV-cache compression step.

TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  This package wraps the plain C++
restatement in ``pyramidkv_oracle.cpp`` (built with g++ into
``libpyramidkv_oracle.so`` next to it).  It imports nothing from the CUDA
package and the CUDA package imports nothing from here.  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may call it.

All tensors are CPU torch tensors (float32, bfloat16 or float16); shapes are per sequence:
``q_win [H_q][alpha][d]``, ``k, v [H_kv][n][d]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pyramidkv_oracle.cpp")
_LIB = os.path.join(_HERE, "libpyramidkv_oracle.so")
_lib: Optional[ctypes.CDLL] = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA involved).  Returns the library path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        # PKV_ORACLE_LIB names another build of this file's source: the mutation test points it at copies with
        # one planted mistake each, to show that the pins notice.
        other = os.environ.get("PKV_ORACLE_LIB")
        if not other:
            build()
        lib = ctypes.CDLL(other or _LIB)
        lib.orc_layer_budgets.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_double,
                                          ctypes.c_void_p]
        lib.orc_layer_budgets.restype = ctypes.c_int
        lib.orc_layer_budgets_geometric.argtypes = lib.orc_layer_budgets.argtypes
        lib.orc_layer_budgets_geometric.restype = ctypes.c_int
        lib.orc_kept_count.argtypes = [ctypes.c_int] * 4
        lib.orc_kept_count.restype = ctypes.c_int
        lib.orc_window_scores.argtypes = [ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int] * 6 + \
                                         [ctypes.c_void_p, ctypes.c_void_p]
        lib.orc_window_scores.restype = None
        lib.orc_window_scores_lse.argtypes = [ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int] * 6 + \
                                             [ctypes.c_void_p] * 3
        lib.orc_window_scores_lse.restype = None
        lib.orc_pool_max.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
        lib.orc_pool_max.restype = ctypes.c_int
        lib.orc_pool_avg.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
        lib.orc_pool_avg.restype = ctypes.c_int
        lib.orc_select_topk.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
        lib.orc_select_topk.restype = ctypes.c_int
        lib.orc_compress_layer.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int] * 10 + \
                                          [ctypes.c_void_p] * 4
        lib.orc_compress_layer.restype = ctypes.c_int
        lib.orc_window_attention.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int] * 5 + \
                                            [ctypes.c_void_p]
        lib.orc_window_attention.restype = None
        lib.orc_decode_attention.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int] * 3 + [ctypes.c_void_p]
        lib.orc_decode_attention.restype = None
        lib.orc_attention_recall.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_int]
        lib.orc_attention_recall.restype = ctypes.c_double
        lib.orc_pages_needed.argtypes = [ctypes.c_int] * 5
        lib.orc_pages_needed.restype = ctypes.c_int
        lib.orc_scatter_paged.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                          ctypes.c_int, ctypes.c_void_p]
        lib.orc_scatter_paged.restype = ctypes.c_int
        lib.orc_read_paged.argtypes = lib.orc_scatter_paged.argtypes
        lib.orc_read_paged.restype = ctypes.c_int
        lib.orc_num_threads.argtypes = []
        lib.orc_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return 0
    if t.dtype == torch.bfloat16:
        return 1
    if t.dtype == torch.float16:
        return 2
    raise TypeError("oracle takes float32, bfloat16 or float16 tensors, got %s" % t.dtype)


def _host(t: torch.Tensor) -> torch.Tensor:
    if t.device.type != "cpu":
        raise ValueError("oracle inputs must live on the CPU")
    return t.contiguous()


def num_threads() -> int:
    return int(_load().orc_num_threads())


def layer_budgets(num_layers: int, avg_budget: int, alpha: int, beta: float = 20.0,
                  schedule: str = "linear") -> List[int]:
    """Per-layer budgets k^l (prefix rows; the alpha window rows come on top): Eq. 1 ("linear"), or the
    appendix's geometric decay between the same end constraints ("geometric")."""
    out = np.zeros(num_layers, dtype=np.int32)
    fn = {"linear": _load().orc_layer_budgets, "geometric": _load().orc_layer_budgets_geometric}[schedule]
    rc = fn(num_layers, avg_budget, alpha, float(beta), out.ctypes.data)
    if rc != 0:
        raise ValueError("budget schedule undefined for these arguments")
    return [int(x) for x in out]


def kept_count(avg_budget: int, alpha: int, k_layer: int, n: int) -> int:
    return int(_load().orc_kept_count(avg_budget, alpha, k_layer, n))


def window_scores(q_win: torch.Tensor, k: torch.Tensor):
    """Eq. 2-3 for one sequence.  Returns (scores float32 [H_kv][P], window_mass float64 [H_kv])."""
    q_win, k = _host(q_win), _host(k)
    hq, alpha, d = q_win.shape
    hkv, n, d2 = k.shape
    assert d == d2 and hq % hkv == 0 and n > alpha and q_win.dtype == k.dtype
    scores = np.zeros((hkv, n - alpha), dtype=np.float32)
    mass = np.zeros(hkv, dtype=np.float64)
    _load().orc_window_scores(q_win.data_ptr(), k.data_ptr(), _dtype_code(k), hq, hkv, d, alpha, n,
                              scores.ctypes.data, mass.ctypes.data)
    return scores, mass


def window_lse(q_win: torch.Tensor, k: torch.Tensor) -> np.ndarray:
    """Natural-log softmax denominators of the window rows, float64 [H_q][alpha] (Eq. 2, causal rows)."""
    q_win, k = _host(q_win), _host(k)
    hq, alpha, d = q_win.shape
    hkv, n, _ = k.shape
    scores = np.zeros((hkv, n - alpha), dtype=np.float32)
    lse = np.zeros((hq, alpha), dtype=np.float64)
    _load().orc_window_scores_lse(q_win.data_ptr(), k.data_ptr(), _dtype_code(k), hq, hkv, d, alpha, n,
                                  scores.ctypes.data, None, lse.ctypes.data)
    return lse


def pool_max(x: np.ndarray, w: int) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    assert x.ndim == 1
    out = np.empty_like(x)
    if _load().orc_pool_max(x.ctypes.data, x.shape[0], w, out.ctypes.data) != 0:
        raise ValueError("pool width must be odd and >= 1")
    return out


def pool_avg(x: np.ndarray, w: int) -> np.ndarray:
    """Mean-pool variant: zeros outside the prefix, always divided by w, float arithmetic left to right."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    assert x.ndim == 1
    out = np.empty_like(x)
    if _load().orc_pool_avg(x.ctypes.data, x.shape[0], w, out.ctypes.data) != 0:
        raise ValueError("pool width must be odd and >= 1")
    return out


def select_topk(pooled: np.ndarray, k: int) -> np.ndarray:
    pooled = np.ascontiguousarray(pooled, dtype=np.float32)
    assert pooled.ndim == 1
    out = np.empty(max(0, min(k, pooled.shape[0])), dtype=np.int32)
    cnt = _load().orc_select_topk(pooled.ctypes.data, pooled.shape[0], k, out.ctypes.data)
    assert cnt == out.shape[0]
    return out


def compress_layer(q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor, *, pool_kernel: int,
                   avg_budget: int, k_layer: int, want_scores: bool = True,
                   pool_kind: str = "max") -> Dict[str, object]:
    """One layer, one sequence.  Returns kept [H_kv][c] int32, k_out/v_out [H_kv][c][d], scores."""
    q_win, k, v = _host(q_win), _host(k), _host(v)
    hq, alpha, d = q_win.shape
    hkv, n, _ = k.shape
    assert v.shape == k.shape and v.dtype == k.dtype == q_win.dtype
    c = kept_count(avg_budget, alpha, k_layer, n)
    kept = np.zeros((hkv, c), dtype=np.int32)
    k_out = torch.empty((hkv, c, d), dtype=k.dtype)
    v_out = torch.empty((hkv, c, d), dtype=v.dtype)
    scores = np.zeros((hkv, n - alpha), dtype=np.float32) if want_scores else None
    got = _load().orc_compress_layer(q_win.data_ptr(), k.data_ptr(), v.data_ptr(), _dtype_code(k),
                                     hq, hkv, d, alpha, pool_kernel, {"max": 0, "avg": 1}[pool_kind], avg_budget,
                                     k_layer, n,
                                     kept.ctypes.data, k_out.data_ptr(), v_out.data_ptr(),
                                     scores.ctypes.data if want_scores else None)
    assert got == c
    return {"kept": kept, "k_out": k_out, "v_out": v_out, "scores": scores, "count": c}


def compress_batch(q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor, seq_lens: Sequence[int], *,
                   pool_kernel: int, avg_budget: int, k_layer: int, pool_kind: str = "max") -> Dict[str, object]:
    """One layer of a ragged batch (tensors padded to the longest sequence).

    Packed output: sequences in batch order; inside a sequence head after head,
    each head holding that sequence's c_b rows in ascending position.
    """
    rows_k, rows_v, rows_i, scores, counts = [], [], [], [], []
    for b, n in enumerate(seq_lens):
        r = compress_layer(q_win[b], k[b, :, :n], v[b, :, :n], pool_kernel=pool_kernel,
                           avg_budget=avg_budget, k_layer=k_layer, pool_kind=pool_kind)
        d = k.shape[-1]
        rows_k.append(r["k_out"].reshape(-1, d))
        rows_v.append(r["v_out"].reshape(-1, d))
        rows_i.append(r["kept"].reshape(-1))
        scores.append(r["scores"])
        counts.append(r["count"])
    return {"k_out": torch.cat(rows_k), "v_out": torch.cat(rows_v),
            "indices": np.concatenate(rows_i), "scores": scores, "counts": counts}


def window_attention(q_head: torch.Tensor, k_rows: torch.Tensor, v_rows: torch.Tensor,
                     positions: np.ndarray, n: int) -> np.ndarray:
    """Causal softmax attention of one query head's window rows over cached rows.  float64 [alpha][d]."""
    q_head, k_rows, v_rows = _host(q_head), _host(k_rows), _host(v_rows)
    alpha, d = q_head.shape
    c = k_rows.shape[0]
    pos = np.ascontiguousarray(positions, dtype=np.int32)
    out = np.zeros((alpha, d), dtype=np.float64)
    _load().orc_window_attention(q_head.data_ptr(), k_rows.data_ptr(), v_rows.data_ptr(),
                                 pos.ctypes.data, _dtype_code(k_rows), d, alpha, n, c, out.ctypes.data)
    return out


def decode_attention(q_row: torch.Tensor, k_rows: torch.Tensor, v_rows: torch.Tensor) -> np.ndarray:
    """softmax(q K_s^T / sqrt(d)) V_s for one query vector over cached rows.  float64 [d]."""
    q_row, k_rows, v_rows = _host(q_row), _host(k_rows), _host(v_rows)
    c, d = k_rows.shape
    out = np.zeros(d, dtype=np.float64)
    _load().orc_decode_attention(q_row.data_ptr(), k_rows.data_ptr(), v_rows.data_ptr(), _dtype_code(k_rows), d, c,
                                 out.ctypes.data)
    return out


def attention_recall(scores_row: np.ndarray, alpha: int, kept: np.ndarray) -> float:
    """Share of the window's attention on kept keys for one KV head (scores_row: its Eq. 3 scores)."""
    s = np.ascontiguousarray(scores_row, dtype=np.float32)
    kp = np.ascontiguousarray(kept, dtype=np.int32)
    return float(_load().orc_attention_recall(s.ctypes.data, s.shape[0], int(alpha), kp.ctypes.data, kp.shape[0]))


def pages_needed(avg_budget: int, alpha: int, k_layer: int, n: int, page_size: int) -> int:
    """Pages one KV head of an n-token sequence needs in a layer with budget k_layer."""
    got = int(_load().orc_pages_needed(avg_budget, alpha, k_layer, n, page_size))
    if got < 0:
        raise ValueError("page_size must be >= 1")
    return got


def scatter_paged(rows: torch.Tensor, table: np.ndarray, page_size: int, pool: torch.Tensor) -> None:
    """Place rows [c][d] of one head into pool [num_pages][page_size][d] through its block table (in place)."""
    rows = _host(rows)
    assert pool.is_contiguous() and pool.dtype == rows.dtype and pool.shape[1:] == (page_size, rows.shape[1])
    tab = np.ascontiguousarray(table, dtype=np.int32)
    c, d = rows.shape
    assert tab.shape[0] >= (c + page_size - 1) // page_size
    if _load().orc_scatter_paged(rows.data_ptr(), c, d * rows.element_size(), page_size, tab.ctypes.data,
                                 pool.shape[0], pool.data_ptr()) != 0:
        raise ValueError("block table names a page outside the pool")


def read_paged(pool: torch.Tensor, table: np.ndarray, count: int, page_size: int) -> torch.Tensor:
    """The `count` rows of one head, in list order, read back through its block table."""
    assert pool.is_contiguous() and pool.shape[1] == page_size
    tab = np.ascontiguousarray(table, dtype=np.int32)
    rows = torch.empty((count, pool.shape[2]), dtype=pool.dtype)
    if _load().orc_read_paged(pool.data_ptr(), count, pool.shape[2] * pool.element_size(), page_size,
                              tab.ctypes.data, pool.shape[0], rows.data_ptr()) != 0:
        raise ValueError("block table names a page outside the pool")
    return rows
