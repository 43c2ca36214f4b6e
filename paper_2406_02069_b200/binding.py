"""ctypes binding of libpyramidkv.so: same names as the C boundary, argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  torch supplies device
memory and the stream, nothing else.  There is no CPU fallback: if the library
cannot be loaded the import of this module fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import torch

from . import build as _build

PKV_OK = 0
PKV_ERR_INVALID_ARG = 1
PKV_ERR_UNSUPPORTED = 2
PKV_ERR_WORKSPACE = 3
PKV_ERR_CUDA = 4
PKV_ERR_DEVICE_STATUS = 5
PKV_ERR_STATIC_SCRATCH = 6
PKV_MAX_BATCH = 64
PKV_STATIC_SCRATCH_BYTES = 8 << 20

EXPORTS = ("pyramidkv_strerror", "pyramidkv_layer_budgets", "pyramidkv_kept_count",
           "pyramidkv_workspace_bytes", "pyramidkv_score_window", "pyramidkv_select_topk",
           "pyramidkv_gather_compact", "pyramidkv_compress_layer", "pyramidkv_profile_layer",
           "pyramidkv_check_status", "pyramidkv_score_window_static", "pyramidkv_score_window_lse",
           "pyramidkv_compress_layer_lse", "pyramidkv_profile_layer_lse", "pyramidkv_decode_attention",
           "pyramidkv_attention_recall", "pyramidkv_pages_needed", "pyramidkv_gather_paged",
           "pyramidkv_compress_layer_paged", "pyramidkv_decode_attention_paged", "pyramidkv_shard_window_lse",
           "pyramidkv_merge_lse", "pyramidkv_shard_scores", "pyramidkv_shard_gather", "pyramidkv_memory_kind",
           "pyramidkv_lanes_create", "pyramidkv_lanes_destroy", "pyramidkv_lanes_info",
           "pyramidkv_compress_model_lanes")
PKV_MAX_STAGES = 8


class PkvConfig(ctypes.Structure):
    _fields_ = [("num_layers", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
                ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("window", ctypes.c_int32), ("pool_kernel", ctypes.c_int32),
                ("pool_kind", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("avg_budget", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("beta", ctypes.c_double)]


class PkvTensor(ctypes.Structure):
    _fields_ = [("ptr", ctypes.c_void_p), ("stride_batch", ctypes.c_int64),
                ("stride_head", ctypes.c_int64), ("stride_token", ctypes.c_int64)]


class PkvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, strerror(status), status))


def _load() -> ctypes.CDLL:
    path = _build.LIB
    if not os.path.exists(path):
        _build.build_library()
    lib = ctypes.CDLL(path)
    P, I32, I64, SZ = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    CFG = ctypes.POINTER(PkvConfig)
    lib.pyramidkv_strerror.argtypes = [ctypes.c_int]
    lib.pyramidkv_strerror.restype = ctypes.c_char_p
    lib.pyramidkv_layer_budgets.argtypes = [CFG, P]
    lib.pyramidkv_kept_count.argtypes = [CFG, I32, I32]
    lib.pyramidkv_workspace_bytes.argtypes = [CFG, I32, I32]
    lib.pyramidkv_workspace_bytes.restype = SZ
    lib.pyramidkv_score_window.argtypes = [CFG, PkvTensor, PkvTensor, P, I32, P, I64, P, SZ, P]
    lib.pyramidkv_score_window_static.argtypes = [CFG, PkvTensor, PkvTensor, P, I32, P, I64, P]
    lib.pyramidkv_select_topk.argtypes = [CFG, P, I64, P, I32, I32, P, P, SZ, P]
    lib.pyramidkv_gather_compact.argtypes = [CFG, PkvTensor, PkvTensor, P, P, I32, I32, P, P, P]
    lib.pyramidkv_compress_layer.argtypes = [CFG, I32, PkvTensor, PkvTensor, PkvTensor, P, I32, P, P, P, P, I64,
                                             P, SZ, P]
    lib.pyramidkv_profile_layer.argtypes = lib.pyramidkv_compress_layer.argtypes + [P, P, P]
    lib.pyramidkv_score_window_lse.argtypes = [CFG, PkvTensor, PkvTensor, P, P, I32, P, I64, P, SZ, P]
    lib.pyramidkv_compress_layer_lse.argtypes = [CFG, I32, PkvTensor, PkvTensor, PkvTensor, P, P, I32, P, P, P, P,
                                                 I64, P, SZ, P]
    lib.pyramidkv_profile_layer_lse.argtypes = lib.pyramidkv_compress_layer_lse.argtypes + [P, P, P]
    lib.pyramidkv_decode_attention.argtypes = [CFG, P, P, P, P, I32, I32, P, P]
    lib.pyramidkv_attention_recall.argtypes = [CFG, P, I64, P, P, I32, I32, P, P]
    lib.pyramidkv_pages_needed.argtypes = [CFG, I32, I32, I32]
    lib.pyramidkv_gather_paged.argtypes = [CFG, PkvTensor, PkvTensor, P, P, I32, I32, P, I32, I32, P, P, P, SZ, P]
    lib.pyramidkv_compress_layer_paged.argtypes = [CFG, I32, PkvTensor, PkvTensor, PkvTensor, P, P, I32, P, I32, I32,
                                                   P, P, P, P, I64, P, SZ, P]
    lib.pyramidkv_decode_attention_paged.argtypes = [CFG, P, P, P, P, I32, I32, P, I32, I32, P, P, SZ, P]
    lib.pyramidkv_shard_window_lse.argtypes = [CFG, PkvTensor, PkvTensor, P, P, I32, P, P, SZ, P]
    lib.pyramidkv_merge_lse.argtypes = [P, I32, I64, P, P]
    lib.pyramidkv_shard_scores.argtypes = [CFG, PkvTensor, PkvTensor, P, P, P, I32, P, I64, P, SZ, P]
    lib.pyramidkv_shard_gather.argtypes = [CFG, PkvTensor, PkvTensor, P, P, I32, I32, P, P, P, P, P]
    lib.pyramidkv_memory_kind.argtypes = [P]
    lib.pyramidkv_lanes_create.argtypes = [I32, ctypes.POINTER(P)]
    lib.pyramidkv_lanes_destroy.argtypes = [P]
    lib.pyramidkv_lanes_info.argtypes = [P, ctypes.POINTER(I32), ctypes.POINTER(I32)]
    lib.pyramidkv_compress_model_lanes.argtypes = [CFG, P, I32, I32, P, P, P, P, P, I32, P, P, P, P, SZ, P]
    lib.pyramidkv_check_status.argtypes = [P, P, P]
    for name in EXPORTS:
        if name not in ("pyramidkv_strerror", "pyramidkv_workspace_bytes"):
            getattr(lib, name).restype = ctypes.c_int
    return lib


_lib = _load()


def library_path() -> str:
    return _build.LIB


MEM_PAGEABLE_HOST, MEM_PINNED_HOST, MEM_DEVICE, MEM_MANAGED = 0, 1, 2, 3


def memory_kind(t: torch.Tensor) -> int:
    """Where the tensor's storage lives as the CUDA runtime sees it (MEM_*)."""
    kind = _lib.pyramidkv_memory_kind(t.data_ptr())
    if kind < 0:
        raise PkvError(-kind, "pyramidkv_memory_kind")
    return int(kind)


def strerror(status: int) -> str:
    return _lib.pyramidkv_strerror(int(status)).decode()


def make_config(*, num_layers: int, num_q_heads: int, num_kv_heads: int, head_dim: int, window: int,
                pool_kernel: int, dtype: str, avg_budget: int, beta: float = 20.0, pool_kind: int = 0) -> PkvConfig:
    code = {"fp32": 0, "bf16": 1, "fp16": 2, torch.float32: 0, torch.bfloat16: 1, torch.float16: 2}[dtype]
    return PkvConfig(num_layers, num_q_heads, num_kv_heads, head_dim, window, pool_kernel, pool_kind, code,
                     avg_budget, 0, float(beta))


def config_of(w) -> PkvConfig:
    """Config of a workloads.Workload."""
    return make_config(num_layers=w.num_layers, num_q_heads=w.num_q_heads, num_kv_heads=w.num_kv_heads,
                       head_dim=w.head_dim, window=w.window, pool_kernel=w.pool_kernel, dtype=w.dtype,
                       avg_budget=w.avg_budget, beta=w.beta, pool_kind={"max": 0, "avg": 1}[w.pool_kind])


def _tensor(t: Optional[torch.Tensor]) -> PkvTensor:
    """[batch][head][token][d] view -> pkv_tensor (no copy; the last dimension must be contiguous)."""
    if t is None:
        return PkvTensor(None, 0, 0, 0)
    if t.dim() != 4 or t.stride(3) != 1:
        raise ValueError("expected a [batch][head][token][d] tensor with a contiguous last dimension")
    return PkvTensor(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2))


def _lens(seq_lens: Sequence[int]):
    arr = (ctypes.c_int32 * len(seq_lens))(*[int(x) for x in seq_lens])
    return arr, len(seq_lens)


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def _check(status: int, where: str) -> None:
    if status != PKV_OK:
        raise PkvError(status, where)


def layer_budgets(cfg: PkvConfig) -> List[int]:
    out = (ctypes.c_int32 * max(1, cfg.num_layers))()
    _check(_lib.pyramidkv_layer_budgets(ctypes.byref(cfg), out), "pyramidkv_layer_budgets")
    return [int(x) for x in out[: cfg.num_layers]]


def kept_count(cfg: PkvConfig, k_layer: int, seq_len: int) -> int:
    c = _lib.pyramidkv_kept_count(ctypes.byref(cfg), int(k_layer), int(seq_len))
    if c < 0:
        raise PkvError(-c, "pyramidkv_kept_count")
    return int(c)


def pages_needed(cfg: PkvConfig, k_layer: int, seq_len: int, page_size: int) -> int:
    """Pages one KV head of a seq_len-token sequence needs in a layer with budget k_layer."""
    c = _lib.pyramidkv_pages_needed(ctypes.byref(cfg), int(k_layer), int(seq_len), int(page_size))
    if c < 0:
        raise PkvError(-c, "pyramidkv_pages_needed")
    return int(c)


def workspace_bytes(cfg: PkvConfig, batch: int, max_seq_len: int) -> int:
    return int(_lib.pyramidkv_workspace_bytes(ctypes.byref(cfg), int(batch), int(max_seq_len)))


def new_workspace(cfg: PkvConfig, batch: int, max_seq_len: int, device="cuda") -> torch.Tensor:
    """Allocates (with torch) and prepares a workspace: the status bytes are zeroed once."""
    nbytes = workspace_bytes(cfg, batch, max_seq_len)
    if nbytes == 0:
        raise PkvError(PKV_ERR_INVALID_ARG, "pyramidkv_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    ws[:256].zero_()
    return ws


def total_rows(cfg: PkvConfig, k_layer: int, seq_lens: Sequence[int]) -> int:
    return sum(cfg.num_kv_heads * kept_count(cfg, k_layer, n) for n in seq_lens)


def _lse_ptr(window_lse: torch.Tensor) -> int:
    if window_lse.dtype != torch.float32 or not window_lse.is_contiguous():
        raise ValueError("window_lse must be a contiguous float32 [batch][H_q][alpha] tensor")
    return window_lse.data_ptr()


def score_window(cfg: PkvConfig, q_win: torch.Tensor, k: torch.Tensor, seq_lens: Sequence[int],
                 scores: torch.Tensor, workspace: torch.Tensor, stream=None,
                 window_lse: Optional[torch.Tensor] = None) -> None:
    """window_lse given: the prefill's natural-log row normalisers are used and one K sweep is skipped."""
    lens, batch = _lens(seq_lens)
    if window_lse is not None:
        _check(_lib.pyramidkv_score_window_lse(ctypes.byref(cfg), _tensor(q_win), _tensor(k), _lse_ptr(window_lse),
                                               lens, batch, scores.data_ptr(), scores.stride(1),
                                               workspace.data_ptr(), workspace.numel(), _stream(stream)),
               "pyramidkv_score_window_lse")
        return
    _check(_lib.pyramidkv_score_window(ctypes.byref(cfg), _tensor(q_win), _tensor(k), lens, batch,
                                       scores.data_ptr(), scores.stride(1), workspace.data_ptr(),
                                       workspace.numel(), _stream(stream)), "pyramidkv_score_window")


def score_window_static(cfg: PkvConfig, q_win: torch.Tensor, k: torch.Tensor, seq_lens: Sequence[int],
                        scores: torch.Tensor, stream=None) -> None:
    """score_window without a workspace: scratch is the library's built-in 8 MiB array.

    For callers that may not allocate device memory.  Problems that need more
    scratch raise PkvError(PKV_ERR_STATIC_SCRATCH).  Calls on one device share the
    array, so keep them ordered on a stream.
    """
    lens, batch = _lens(seq_lens)
    _check(_lib.pyramidkv_score_window_static(ctypes.byref(cfg), _tensor(q_win), _tensor(k), lens, batch,
                                              scores.data_ptr(), scores.stride(1), _stream(stream)),
           "pyramidkv_score_window_static")


def select_topk(cfg: PkvConfig, scores: torch.Tensor, seq_lens: Sequence[int], k_layer: int,
                indices: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    lens, batch = _lens(seq_lens)
    _check(_lib.pyramidkv_select_topk(ctypes.byref(cfg), scores.data_ptr(), scores.stride(1), lens, batch,
                                      int(k_layer), indices.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                      _stream(stream)), "pyramidkv_select_topk")


def gather_compact(cfg: PkvConfig, k: torch.Tensor, v: Optional[torch.Tensor], indices: torch.Tensor,
                   seq_lens: Sequence[int], k_layer: int, k_out: torch.Tensor, v_out: Optional[torch.Tensor],
                   stream=None) -> None:
    lens, batch = _lens(seq_lens)
    _check(_lib.pyramidkv_gather_compact(ctypes.byref(cfg), _tensor(k), _tensor(v), indices.data_ptr(), lens, batch,
                                         int(k_layer), k_out.data_ptr(),
                                         v_out.data_ptr() if v_out is not None else None, _stream(stream)),
           "pyramidkv_gather_compact")


def compress_layer(cfg: PkvConfig, layer: int, q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                   seq_lens: Sequence[int], k_out: torch.Tensor, v_out: torch.Tensor, indices: torch.Tensor,
                   workspace: torch.Tensor, scores: Optional[torch.Tensor] = None, stream=None,
                   window_lse: Optional[torch.Tensor] = None) -> None:
    lens, batch = _lens(seq_lens)
    if window_lse is not None:
        _check(_lib.pyramidkv_compress_layer_lse(
            ctypes.byref(cfg), int(layer), _tensor(q_win), _tensor(k), _tensor(v), _lse_ptr(window_lse), lens, batch,
            k_out.data_ptr(), v_out.data_ptr(), indices.data_ptr(),
            scores.data_ptr() if scores is not None else None, scores.stride(1) if scores is not None else 0,
            workspace.data_ptr(), workspace.numel(), _stream(stream)), "pyramidkv_compress_layer_lse")
        return
    _check(_lib.pyramidkv_compress_layer(ctypes.byref(cfg), int(layer), _tensor(q_win), _tensor(k), _tensor(v), lens,
                                         batch, k_out.data_ptr(), v_out.data_ptr(), indices.data_ptr(),
                                         scores.data_ptr() if scores is not None else None,
                                         scores.stride(1) if scores is not None else 0,
                                         workspace.data_ptr(), workspace.numel(), _stream(stream)),
           "pyramidkv_compress_layer")


def profile_layer(cfg: PkvConfig, layer: int, q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                  seq_lens: Sequence[int], k_out: torch.Tensor, v_out: torch.Tensor, indices: torch.Tensor,
                  workspace: torch.Tensor, stream=None, window_lse: Optional[torch.Tensor] = None):
    """compress_layer with per-kernel device times: returns [(kernel name, milliseconds), ...]."""
    lens, batch = _lens(seq_lens)
    ms = (ctypes.c_float * PKV_MAX_STAGES)()
    names = ((ctypes.c_char * 32) * PKV_MAX_STAGES)()
    n = ctypes.c_int32(0)
    if window_lse is not None:
        _check(_lib.pyramidkv_profile_layer_lse(
            ctypes.byref(cfg), int(layer), _tensor(q_win), _tensor(k), _tensor(v), _lse_ptr(window_lse), lens, batch,
            k_out.data_ptr(), v_out.data_ptr(), indices.data_ptr(), None, 0, workspace.data_ptr(), workspace.numel(),
            _stream(stream), ms, names, ctypes.byref(n)), "pyramidkv_profile_layer_lse")
        return [(names[i].value.decode(), float(ms[i])) for i in range(n.value)]
    _check(_lib.pyramidkv_profile_layer(ctypes.byref(cfg), int(layer), _tensor(q_win), _tensor(k), _tensor(v), lens,
                                        batch, k_out.data_ptr(), v_out.data_ptr(), indices.data_ptr(), None, 0,
                                        workspace.data_ptr(), workspace.numel(), _stream(stream), ms, names,
                                        ctypes.byref(n)), "pyramidkv_profile_layer")
    return [(names[i].value.decode(), float(ms[i])) for i in range(n.value)]


def decode_attention(cfg: PkvConfig, q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor,
                     seq_lens: Sequence[int], k_layer: int, out: torch.Tensor, stream=None) -> None:
    """One new token per sequence attends to the compact cache of a layer: q [batch][H_q][d] -> out fp32."""
    lens, batch = _lens(seq_lens)
    if not (q.is_contiguous() and k_cache.is_contiguous() and v_cache.is_contiguous() and out.is_contiguous()):
        raise ValueError("decode_attention takes contiguous tensors")
    _check(_lib.pyramidkv_decode_attention(ctypes.byref(cfg), q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(),
                                           lens, batch, int(k_layer), out.data_ptr(), _stream(stream)),
           "pyramidkv_decode_attention")


def attention_recall(cfg: PkvConfig, scores: torch.Tensor, indices: torch.Tensor, seq_lens: Sequence[int],
                     k_layer: int, recall: torch.Tensor, stream=None) -> None:
    """Share of the window's attention that falls on kept keys, per (sequence, KV head)."""
    lens, batch = _lens(seq_lens)
    _check(_lib.pyramidkv_attention_recall(ctypes.byref(cfg), scores.data_ptr(), scores.stride(1),
                                           indices.data_ptr(), lens, batch, int(k_layer), recall.data_ptr(),
                                           _stream(stream)), "pyramidkv_attention_recall")


def check_status(workspace: torch.Tensor, stream=None) -> int:
    """Synchronises the stream; raises PkvError if a kernel flagged a failure."""
    detail = ctypes.c_uint32(0)
    st = _lib.pyramidkv_check_status(workspace.data_ptr(), _stream(stream), ctypes.byref(detail))
    if st != PKV_OK:
        raise PkvError(st, "pyramidkv_check_status (word 0x%x)" % detail.value)
    return 0


def _paged(block_table: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor):
    """(table pointer, page_size, num_pages, k pointer, v pointer) of pools [num_pages][page_size][d]."""
    if block_table.dtype != torch.int32 or not block_table.is_contiguous():
        raise ValueError("block_table must be a contiguous int32 tensor")
    if k_pool.dim() != 3 or k_pool.shape != v_pool.shape or not (k_pool.is_contiguous() and v_pool.is_contiguous()):
        raise ValueError("k_pool and v_pool must be contiguous [num_pages][page_size][d] tensors of one shape")
    return block_table.data_ptr(), int(k_pool.shape[1]), int(k_pool.shape[0]), k_pool.data_ptr(), v_pool.data_ptr()


def gather_paged(cfg: PkvConfig, k: torch.Tensor, v: torch.Tensor, indices: torch.Tensor, seq_lens: Sequence[int],
                 k_layer: int, block_table: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor,
                 workspace: torch.Tensor, stream=None) -> None:
    lens, batch = _lens(seq_lens)
    tab, page_size, num_pages, kp, vp = _paged(block_table, k_pool, v_pool)
    _check(_lib.pyramidkv_gather_paged(ctypes.byref(cfg), _tensor(k), _tensor(v), indices.data_ptr(), lens, batch,
                                       int(k_layer), tab, page_size, num_pages, kp, vp, workspace.data_ptr(),
                                       workspace.numel(), _stream(stream)), "pyramidkv_gather_paged")


def compress_layer_paged(cfg: PkvConfig, layer: int, q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                         seq_lens: Sequence[int], block_table: torch.Tensor, k_pool: torch.Tensor,
                         v_pool: torch.Tensor, indices: torch.Tensor, workspace: torch.Tensor,
                         scores: Optional[torch.Tensor] = None, stream=None,
                         window_lse: Optional[torch.Tensor] = None) -> None:
    lens, batch = _lens(seq_lens)
    tab, page_size, num_pages, kp, vp = _paged(block_table, k_pool, v_pool)
    _check(_lib.pyramidkv_compress_layer_paged(
        ctypes.byref(cfg), int(layer), _tensor(q_win), _tensor(k), _tensor(v),
        _lse_ptr(window_lse) if window_lse is not None else None, lens, batch, tab, page_size, num_pages, kp, vp,
        indices.data_ptr(), scores.data_ptr() if scores is not None else None,
        scores.stride(1) if scores is not None else 0, workspace.data_ptr(), workspace.numel(), _stream(stream)),
        "pyramidkv_compress_layer_paged")


def decode_attention_paged(cfg: PkvConfig, q: torch.Tensor, block_table: torch.Tensor, k_pool: torch.Tensor,
                           v_pool: torch.Tensor, seq_lens: Sequence[int], k_layer: int, out: torch.Tensor,
                           workspace: torch.Tensor, stream=None) -> None:
    lens, batch = _lens(seq_lens)
    if not (q.is_contiguous() and out.is_contiguous()):
        raise ValueError("decode_attention_paged takes contiguous q and out")
    tab, page_size, num_pages, kp, vp = _paged(block_table, k_pool, v_pool)
    _check(_lib.pyramidkv_decode_attention_paged(ctypes.byref(cfg), q.data_ptr(), kp, vp, tab, page_size, num_pages,
                                                 lens, batch, int(k_layer), out.data_ptr(), workspace.data_ptr(),
                                                 workspace.numel(), _stream(stream)),
           "pyramidkv_decode_attention_paged")


# ----------------------------------------------------------------------------- sequence-sharded steps
def shard_window_lse(cfg: PkvConfig, q_win: torch.Tensor, k_shard: torch.Tensor, shard_keys: Sequence[int],
                     window_keys: Sequence[int], lse_out: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    """Partial normalisers (natural log) of the window rows over this shard's keys -> lse_out [batch][H_q][alpha]."""
    keys, batch = _lens(shard_keys)
    wkeys, _ = _lens(window_keys)
    _check(_lib.pyramidkv_shard_window_lse(ctypes.byref(cfg), _tensor(q_win), _tensor(k_shard), keys, wkeys, batch,
                                           _lse_ptr(lse_out), workspace.data_ptr(), workspace.numel(),
                                           _stream(stream)), "pyramidkv_shard_window_lse")


def merge_lse(parts: torch.Tensor, out: torch.Tensor, stream=None) -> None:
    """parts [num_shards][...] float32 -> out [...] = log(sum over shards of exp(part))."""
    if parts.dtype != torch.float32 or out.dtype != torch.float32 or not (parts.is_contiguous() and out.is_contiguous()):
        raise ValueError("merge_lse takes contiguous float32 tensors")
    if parts.numel() != parts.shape[0] * out.numel():
        raise ValueError("parts must be [num_shards] + out.shape")
    _check(_lib.pyramidkv_merge_lse(parts.data_ptr(), int(parts.shape[0]), out.numel(), out.data_ptr(),
                                    _stream(stream)), "pyramidkv_merge_lse")


def shard_scores(cfg: PkvConfig, q_win: torch.Tensor, k_shard: torch.Tensor, window_lse: torch.Tensor,
                 shard_keys: Sequence[int], window_keys: Sequence[int], scores: torch.Tensor,
                 workspace: torch.Tensor, stream=None) -> None:
    keys, batch = _lens(shard_keys)
    wkeys, _ = _lens(window_keys)
    _check(_lib.pyramidkv_shard_scores(ctypes.byref(cfg), _tensor(q_win), _tensor(k_shard), _lse_ptr(window_lse), keys,
                                       wkeys, batch, scores.data_ptr(), scores.stride(1), workspace.data_ptr(),
                                       workspace.numel(), _stream(stream)), "pyramidkv_shard_scores")


def shard_gather(cfg: PkvConfig, k_shard: torch.Tensor, v_shard: torch.Tensor, indices: torch.Tensor,
                 seq_lens: Sequence[int], k_layer: int, shard_begin: Sequence[int], shard_keys: Sequence[int],
                 k_out: torch.Tensor, v_out: torch.Tensor, stream=None) -> None:
    lens, batch = _lens(seq_lens)
    begin, _ = _lens(shard_begin)
    keys, _ = _lens(shard_keys)
    _check(_lib.pyramidkv_shard_gather(ctypes.byref(cfg), _tensor(k_shard), _tensor(v_shard), indices.data_ptr(), lens,
                                       batch, int(k_layer), begin, keys, k_out.data_ptr(), v_out.data_ptr(),
                                       _stream(stream)), "pyramidkv_shard_gather")


# ----------------------------------------------------------------------------- two lanes
class Lanes:
    """The device's SMs split into a group for the score sweeps and a small one for selection and gather."""

    def __init__(self, select_sms: int = 8):
        handle = ctypes.c_void_p()
        _check(_lib.pyramidkv_lanes_create(int(select_sms), ctypes.byref(handle)), "pyramidkv_lanes_create")
        self._handle = handle
        a, b = ctypes.c_int32(), ctypes.c_int32()
        _check(_lib.pyramidkv_lanes_info(handle, ctypes.byref(a), ctypes.byref(b)), "pyramidkv_lanes_info")
        self.score_sms, self.select_sms = a.value, b.value

    def close(self) -> None:
        if self._handle is not None:
            _lib.pyramidkv_lanes_destroy(self._handle)
            self._handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def compress_model_lanes(cfg: PkvConfig, lanes: Lanes, layers, seq_lens: Sequence[int], k_out, v_out, indices,
                         workspaces, first_layer: int = 0, stream=None) -> None:
    """layers: objects with .q_win/.k/.v (and optionally .window_lse, on all or none of them); k_out, v_out,
    indices: per-layer output tensors; workspaces: two workspace tensors of one size."""
    lens, batch = _lens(seq_lens)
    m = len(layers)
    if not (len(k_out) == len(v_out) == len(indices) == m) or len(workspaces) != 2:
        raise ValueError("one output per layer and exactly two workspaces are needed")
    if workspaces[0].numel() != workspaces[1].numel():
        raise ValueError("the two workspaces must have one size")
    tensors = lambda name: (PkvTensor * m)(*[_tensor(getattr(x, name)) for x in layers])
    pointers = lambda ts: (ctypes.c_void_p * m)(*[t.data_ptr() for t in ts])
    with_lse = [getattr(x, "window_lse", None) is not None for x in layers]
    if any(with_lse) and not all(with_lse):
        raise ValueError("window_lse must be given for every layer or for none")
    lse = (ctypes.c_void_p * m)(*[_lse_ptr(x.window_lse) for x in layers]) if all(with_lse) and m else None
    _check(_lib.pyramidkv_compress_model_lanes(
        ctypes.byref(cfg), lanes._handle, int(first_layer), m, tensors("q_win"), tensors("k"), tensors("v"), lse, lens,
        batch, pointers(k_out), pointers(v_out), pointers(indices),
        (ctypes.c_void_p * 2)(workspaces[0].data_ptr(), workspaces[1].data_ptr()), workspaces[0].numel(),
        _stream(stream)), "pyramidkv_compress_model_lanes")
