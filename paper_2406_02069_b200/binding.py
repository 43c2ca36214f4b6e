"""ctypes binding of libpyramidkv.so: same names as the C boundary, argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  torch supplies device
memory and the stream, nothing else.  There is no CPU fallback: the library is
loaded (and built first when it is missing or older than its sources) by the first
call that needs it, and that call raises if it cannot be.

The wrappers check what the C side cannot see: that the tensors are as large as the
configuration and the sequence lengths say, of the configured type, and on a device.
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
           "pyramidkv_check_status", "pyramidkv_score_window_static", "pyramidkv_check_status_static",
           "pyramidkv_score_window_lse",
           "pyramidkv_compress_layer_lse", "pyramidkv_profile_layer_lse", "pyramidkv_decode_attention",
           "pyramidkv_attention_recall", "pyramidkv_pages_needed", "pyramidkv_gather_paged",
           "pyramidkv_compress_layer_paged", "pyramidkv_decode_attention_paged", "pyramidkv_shard_window_lse",
           "pyramidkv_merge_lse", "pyramidkv_shard_scores", "pyramidkv_shard_gather", "pyramidkv_memory_kind",
           "pyramidkv_lanes_create", "pyramidkv_lanes_destroy", "pyramidkv_lanes_info",
           "pyramidkv_compress_model_lanes", "pyramidkv_test_hooks", "pyramidkv_test_slow_copy",
           "pyramidkv_attend_window", "pyramidkv_attend_compress_layer",
           "pyramidkv_profile_attend_compress_layer")
PKV_MAX_STAGES = 8


class PkvConfig(ctypes.Structure):
    _fields_ = [("num_layers", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
                ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("window", ctypes.c_int32), ("pool_kernel", ctypes.c_int32),
                ("pool_kind", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("avg_budget", ctypes.c_int32), ("schedule", ctypes.c_int32),
                ("beta", ctypes.c_double), ("flags", ctypes.c_uint32), ("sweep_ctas", ctypes.c_uint32)]


class PkvTensor(ctypes.Structure):
    _fields_ = [("ptr", ctypes.c_void_p), ("stride_batch", ctypes.c_int64),
                ("stride_head", ctypes.c_int64), ("stride_token", ctypes.c_int64)]


class PkvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, strerror(status), status))


def _load() -> ctypes.CDLL:
    path = _build.build_library()          # compiles only when the library is missing or its sources changed
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
    lib.pyramidkv_attend_window.argtypes = [CFG, PkvTensor, PkvTensor, PkvTensor, P, I32, P, P, I64, P, SZ, P]
    lib.pyramidkv_attend_compress_layer.argtypes = [CFG, I32, PkvTensor, PkvTensor, PkvTensor, P, I32, P, P, P, P, P,
                                                    I64, P, SZ, P]
    lib.pyramidkv_profile_attend_compress_layer.argtypes = lib.pyramidkv_attend_compress_layer.argtypes + [P, P, P]
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
    lib.pyramidkv_test_hooks.argtypes = [I64, I32]
    lib.pyramidkv_test_slow_copy.argtypes = [P, P, SZ, I32, P]
    lib.pyramidkv_check_status_static.argtypes = [P, P]
    for name in EXPORTS:
        if name not in ("pyramidkv_strerror", "pyramidkv_workspace_bytes"):
            getattr(lib, name).restype = ctypes.c_int
    return lib


class _LazyLibrary:
    """Loads libpyramidkv.so on first use, so that importing the package (for its input generators, say) maps
    no native code."""
    _real = None

    def __getattr__(self, name):
        if _LazyLibrary._real is None:
            _LazyLibrary._real = _load()
        return getattr(_LazyLibrary._real, name)


_lib = _LazyLibrary()


def library_path() -> str:
    """Path of libpyramidkv.so, built first if it is missing or older than its sources."""
    return _build.build_library()


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
                pool_kernel: int, dtype: str, avg_budget: int, beta: float = 20.0, pool_kind: int = 0,
                schedule: str = "linear", inputs_final: bool = False, sweep_ctas: int = 0) -> PkvConfig:
    """inputs_final sets PKV_FLAG_INPUTS_FINAL: nothing still running on the stream writes q_win or k when a call is
    enqueued, so the score kernels may read them before the kernels ahead of them have finished.  sweep_ctas > 0
    caps the CTAs of the persistent score sweeps (a share of the SMs for callers that run layers on several streams)."""
    code = {"fp32": 0, "bf16": 1, "fp16": 2, torch.float32: 0, torch.bfloat16: 1, torch.float16: 2}[dtype]
    return PkvConfig(num_layers, num_q_heads, num_kv_heads, head_dim, window, pool_kernel, pool_kind, code,
                     avg_budget, {"linear": 0, "geometric": 1}[schedule], float(beta), 1 if inputs_final else 0, int(sweep_ctas))


def config_of(w, inputs_final: bool = False, sweep_ctas: int = 0) -> PkvConfig:
    """Config of a workloads.Workload."""
    return make_config(num_layers=w.num_layers, num_q_heads=w.num_q_heads, num_kv_heads=w.num_kv_heads,
                       head_dim=w.head_dim, window=w.window, pool_kernel=w.pool_kernel, dtype=w.dtype,
                       avg_budget=w.avg_budget, beta=w.beta, pool_kind={"max": 0, "avg": 1}[w.pool_kind],
                       schedule=getattr(w, "schedule", "linear"), inputs_final=inputs_final, sweep_ctas=sweep_ctas)


def _tensor(t: Optional[torch.Tensor]) -> PkvTensor:
    """[batch][head][token][d] view -> pkv_tensor (no copy; the last dimension must be contiguous)."""
    if t is None:
        return PkvTensor(None, 0, 0, 0)
    if t.dim() != 4 or t.stride(3) != 1:
        raise ValueError("expected a [batch][head][token][d] tensor with a contiguous last dimension")
    return PkvTensor(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2))


_TORCH_DTYPE = {0: torch.float32, 1: torch.bfloat16, 2: torch.float16}


def _on_device(t: torch.Tensor) -> bool:
    return t.is_cuda or t.is_pinned()      # pinned host memory is mapped on the device (see memory_kind)


def _want(ok: bool, what: str) -> None:
    if not ok:
        raise ValueError(what)


def _check_kv(cfg: PkvConfig, t: torch.Tensor, name: str, batch: int, tokens: int) -> None:
    """A K or V tensor as large as the call will read: [>= batch][H_kv][>= tokens][d], configured type."""
    _want(t.dim() == 4 and t.stride(3) == 1, "%s must be [batch][H_kv][token][d] with a contiguous last dimension" % name)
    _want(t.dtype == _TORCH_DTYPE[cfg.dtype], "%s has type %s, the configuration says %s" % (name, t.dtype, _TORCH_DTYPE[cfg.dtype]))
    _want(_on_device(t), "%s must live in device memory (or pinned host memory)" % name)
    _want(t.shape[0] >= batch and t.shape[1] == cfg.num_kv_heads and t.shape[3] == cfg.head_dim,
          "%s has shape %s, expected [>=%d][%d][token][%d]" % (name, tuple(t.shape), batch, cfg.num_kv_heads, cfg.head_dim))
    _want(t.shape[2] >= tokens, "%s holds %d tokens per sequence, the lengths given need %d" % (name, t.shape[2], tokens))
    _want((batch == 1 or t.stride(0) > 0) and (cfg.num_kv_heads == 1 or t.stride(1) > 0) and t.stride(2) >= cfg.head_dim,
          "%s: batch, head and token strides must be positive (no broadcast views)" % name)


def _check_q(cfg: PkvConfig, q_win: torch.Tensor, batch: int) -> None:
    _want(q_win.dim() == 4 and q_win.stride(3) == 1, "q_win must be [batch][H_q][alpha][d] with a contiguous last dimension")
    _want(q_win.dtype == _TORCH_DTYPE[cfg.dtype], "q_win has type %s, the configuration says %s" % (q_win.dtype, _TORCH_DTYPE[cfg.dtype]))
    _want(_on_device(q_win), "q_win must live in device memory")
    _want(q_win.shape[0] >= batch and tuple(q_win.shape[1:]) == (cfg.num_q_heads, cfg.window, cfg.head_dim),
          "q_win has shape %s, expected [>=%d][%d][%d][%d]" % (tuple(q_win.shape), batch, cfg.num_q_heads, cfg.window, cfg.head_dim))


def _check_scores(cfg: PkvConfig, scores: torch.Tensor, batch: int, columns: int) -> None:
    """scores [>= batch][H_kv][ld] float32 with ld >= columns; rows of one sequence one after another."""
    _want(scores.dim() == 3 and scores.dtype == torch.float32 and scores.is_cuda, "scores must be a float32 [batch][H_kv][ld] device tensor")
    _want(scores.shape[0] >= batch and scores.shape[1] == cfg.num_kv_heads and scores.shape[2] >= columns,
          "scores has shape %s, expected [>=%d][%d][>=%d]" % (tuple(scores.shape), batch, cfg.num_kv_heads, columns))
    _want(scores.stride(2) == 1 and scores.stride(1) >= columns and
          (batch == 1 or scores.stride(0) == cfg.num_kv_heads * scores.stride(1)),
          "scores: rows must be contiguous and a sequence's heads evenly spaced (stride(0) = H_kv * stride(1))")


def _check_rows(cfg: PkvConfig, rows: int, k_out: Optional[torch.Tensor], v_out: Optional[torch.Tensor],
                indices: Optional[torch.Tensor]) -> None:
    """Packed outputs with room for `rows` rows."""
    for name, t in (("k_out", k_out), ("v_out", v_out)):
        if t is None:
            continue
        _want(t.is_cuda and t.is_contiguous() and t.dtype == _TORCH_DTYPE[cfg.dtype], "%s must be a contiguous device tensor of the configured type" % name)
        _want(t.numel() >= rows * cfg.head_dim, "%s holds %d elements, %d rows need %d" % (name, t.numel(), rows, rows * cfg.head_dim))
    if indices is not None:
        _want(indices.is_cuda and indices.is_contiguous() and indices.dtype == torch.int32, "indices must be a contiguous int32 device tensor")
        _want(indices.numel() >= rows, "indices holds %d entries, %d are needed" % (indices.numel(), rows))


def _check_workspace(ws: torch.Tensor) -> None:
    _want(ws.is_cuda and ws.dtype == torch.uint8 and ws.is_contiguous(), "the workspace must be a contiguous uint8 device tensor")


def _check_layer_call(cfg: PkvConfig, layer: int, q_win, k, v, seq_lens, k_out, v_out, indices, workspace, scores) -> None:
    batch = len(seq_lens)
    _check_q(cfg, q_win, batch)
    _check_kv(cfg, k, "k", batch, max(seq_lens))
    _check_kv(cfg, v, "v", batch, max(seq_lens))
    _check_rows(cfg, _layer_rows(cfg, layer, seq_lens), k_out, v_out, indices)
    _check_workspace(workspace)
    if scores is not None:
        _check_scores(cfg, scores, batch, max(seq_lens) - cfg.window)


_budget_cache = {}


def _layer_rows(cfg: PkvConfig, layer: int, seq_lens: Sequence[int]) -> int:
    """Packed output rows of a layer (host arithmetic, remembered per configuration and lengths: the per-layer call
    is on the hot path of short configurations)."""
    _want(0 <= int(layer) < cfg.num_layers, "layer %d outside [0, %d)" % (layer, cfg.num_layers))
    key = (cfg.num_layers, cfg.num_kv_heads, cfg.window, cfg.avg_budget, cfg.schedule, cfg.beta, tuple(seq_lens))
    rows = _budget_cache.get(key)
    if rows is None:
        rows = [total_rows(cfg, kl, seq_lens) for kl in layer_budgets(cfg)]
        if len(_budget_cache) > 64:
            _budget_cache.clear()
        _budget_cache[key] = rows
    return rows[int(layer)]


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
    _check_q(cfg, q_win, batch)
    _check_kv(cfg, k, "k", batch, max(seq_lens))
    _check_scores(cfg, scores, batch, max(seq_lens) - cfg.window)
    _check_workspace(workspace)
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
    _check_q(cfg, q_win, batch)
    _check_kv(cfg, k, "k", batch, max(seq_lens))
    _check_scores(cfg, scores, batch, max(seq_lens) - cfg.window)
    _check(_lib.pyramidkv_score_window_static(ctypes.byref(cfg), _tensor(q_win), _tensor(k), lens, batch,
                                              scores.data_ptr(), scores.stride(1), _stream(stream)),
           "pyramidkv_score_window_static")


def test_hooks(wait_clocks: int = 0, withhold_tile: bool = False, two_sweeps: bool = False,
               withhold_attend_tile: bool = False) -> None:
    """Test aid: bound of the waits inside the tensor-core kernels (0 = default), the withheld K tile (of the row
    statistics sweep, or of the window-attention kernel), and short contexts kept on the two-sweep kernels."""
    _check(_lib.pyramidkv_test_hooks(int(wait_clocks), (1 if withhold_tile else 0) | (2 if two_sweeps else 0) |
                                     (4 if withhold_attend_tile else 0)),
           "pyramidkv_test_hooks")


test_hooks.__test__ = False      # not a test case, whatever its name says to a collector


def slow_copy(dst: torch.Tensor, src: torch.Tensor, steps: int = 64, stream=None) -> None:
    """Test aid: dst <- src by a deliberately slow kernel that lets the kernels behind it on the stream start early."""
    if dst.numel() * dst.element_size() != src.numel() * src.element_size() or not (dst.is_contiguous() and src.is_contiguous()):
        raise ValueError("slow_copy takes two contiguous tensors of one size")
    _check(_lib.pyramidkv_test_slow_copy(dst.data_ptr(), src.data_ptr(), dst.numel() * dst.element_size(), int(steps),
                                         _stream(stream)), "pyramidkv_test_slow_copy")


def check_status_static(stream=None) -> int:
    """check_status for score_window_static: synchronises the stream and reads the status word of the built-in
    scratch; raises PkvError if a kernel flagged a failure."""
    detail = ctypes.c_uint32(0)
    st = _lib.pyramidkv_check_status_static(_stream(stream), ctypes.byref(detail))
    if st != PKV_OK:
        raise PkvError(st, "pyramidkv_check_status_static (word 0x%x)" % detail.value)
    return 0


def select_topk(cfg: PkvConfig, scores: torch.Tensor, seq_lens: Sequence[int], k_layer: int,
                indices: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    lens, batch = _lens(seq_lens)
    _check_scores(cfg, scores, batch, max(seq_lens) - cfg.window)
    _check_rows(cfg, total_rows(cfg, k_layer, seq_lens), None, None, indices)
    _check_workspace(workspace)
    _check(_lib.pyramidkv_select_topk(ctypes.byref(cfg), scores.data_ptr(), scores.stride(1), lens, batch,
                                      int(k_layer), indices.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                      _stream(stream)), "pyramidkv_select_topk")


def gather_compact(cfg: PkvConfig, k: torch.Tensor, v: Optional[torch.Tensor], indices: torch.Tensor,
                   seq_lens: Sequence[int], k_layer: int, k_out: torch.Tensor, v_out: Optional[torch.Tensor],
                   stream=None) -> None:
    lens, batch = _lens(seq_lens)
    _check_kv(cfg, k, "k", batch, max(seq_lens))
    if v is not None:
        _check_kv(cfg, v, "v", batch, max(seq_lens))
    _check_rows(cfg, total_rows(cfg, k_layer, seq_lens), k_out, v_out, indices)
    _check(_lib.pyramidkv_gather_compact(ctypes.byref(cfg), _tensor(k), _tensor(v), indices.data_ptr(), lens, batch,
                                         int(k_layer), k_out.data_ptr(),
                                         v_out.data_ptr() if v_out is not None else None, _stream(stream)),
           "pyramidkv_gather_compact")


def compress_layer(cfg: PkvConfig, layer: int, q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                   seq_lens: Sequence[int], k_out: torch.Tensor, v_out: torch.Tensor, indices: torch.Tensor,
                   workspace: torch.Tensor, scores: Optional[torch.Tensor] = None, stream=None,
                   window_lse: Optional[torch.Tensor] = None) -> None:
    lens, batch = _lens(seq_lens)
    _check_layer_call(cfg, layer, q_win, k, v, seq_lens, k_out, v_out, indices, workspace, scores)
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


def _check_attn_out(cfg: PkvConfig, attn_out: torch.Tensor, batch: int) -> None:
    _want(attn_out.is_cuda and attn_out.dtype == torch.float32 and attn_out.is_contiguous() and
          tuple(attn_out.shape) == (batch, cfg.num_q_heads, cfg.window, cfg.head_dim),
          "attn_out must be a contiguous float32 device tensor [batch][H_q][window][d]")


def attend_window(cfg: PkvConfig, q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor, seq_lens: Sequence[int],
                  attn_out: torch.Tensor, scores: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    """The window rows' attention output and the window scores from one fused pass."""
    lens, batch = _lens(seq_lens)
    _check_q(cfg, q_win, batch)
    _check_kv(cfg, k, "k", batch, max(seq_lens))
    _check_kv(cfg, v, "v", batch, max(seq_lens))
    _check_attn_out(cfg, attn_out, batch)
    _check_scores(cfg, scores, batch, max(seq_lens) - cfg.window)
    _check_workspace(workspace)
    _check(_lib.pyramidkv_attend_window(ctypes.byref(cfg), _tensor(q_win), _tensor(k), _tensor(v), lens, batch,
                                        attn_out.data_ptr(), scores.data_ptr(), scores.stride(1),
                                        workspace.data_ptr(), workspace.numel(), _stream(stream)),
           "pyramidkv_attend_window")


def attend_compress_layer(cfg: PkvConfig, layer: int, q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                          seq_lens: Sequence[int], attn_out: torch.Tensor, k_out: torch.Tensor, v_out: torch.Tensor,
                          indices: torch.Tensor, workspace: torch.Tensor, scores: Optional[torch.Tensor] = None,
                          stream=None) -> None:
    """compress_layer that also returns the window rows' attention output."""
    lens, batch = _lens(seq_lens)
    _check_layer_call(cfg, layer, q_win, k, v, seq_lens, k_out, v_out, indices, workspace, scores)
    _check_attn_out(cfg, attn_out, batch)
    _check(_lib.pyramidkv_attend_compress_layer(
        ctypes.byref(cfg), int(layer), _tensor(q_win), _tensor(k), _tensor(v), lens, batch, attn_out.data_ptr(),
        k_out.data_ptr(), v_out.data_ptr(), indices.data_ptr(),
        scores.data_ptr() if scores is not None else None, scores.stride(1) if scores is not None else 0,
        workspace.data_ptr(), workspace.numel(), _stream(stream)), "pyramidkv_attend_compress_layer")


def profile_layer(cfg: PkvConfig, layer: int, q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                  seq_lens: Sequence[int], k_out: torch.Tensor, v_out: torch.Tensor, indices: torch.Tensor,
                  workspace: torch.Tensor, stream=None, window_lse: Optional[torch.Tensor] = None,
                  attn_out: Optional[torch.Tensor] = None):
    """compress_layer (attend_compress_layer when attn_out is given) with per-kernel device times: returns
    [(kernel name, milliseconds), ...]."""
    lens, batch = _lens(seq_lens)
    _check_layer_call(cfg, layer, q_win, k, v, seq_lens, k_out, v_out, indices, workspace, None)
    ms = (ctypes.c_float * PKV_MAX_STAGES)()
    names = ((ctypes.c_char * 32) * PKV_MAX_STAGES)()
    n = ctypes.c_int32(0)
    if attn_out is not None:
        _check_attn_out(cfg, attn_out, batch)
        _check(_lib.pyramidkv_profile_attend_compress_layer(
            ctypes.byref(cfg), int(layer), _tensor(q_win), _tensor(k), _tensor(v), lens, batch, attn_out.data_ptr(),
            k_out.data_ptr(), v_out.data_ptr(), indices.data_ptr(), None, 0, workspace.data_ptr(), workspace.numel(),
            _stream(stream), ms, names, ctypes.byref(n)), "pyramidkv_profile_attend_compress_layer")
        return [(names[i].value.decode(), float(ms[i])) for i in range(n.value)]
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
