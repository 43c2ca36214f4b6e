"""Whole-model drivers over the per-layer C-ABI call.

`compress_model` runs every layer of a model whose K/V already live on the device.
`compress_model_from_host` is the end-to-end form for callers whose prefill K/V
sit in (pinned) host memory, e.g. an offloaded cache: each layer is copied to the
device on a copy stream while the previous layer is being compressed, and the
compact cache and its index list are copied back.  V can stay where it is: only
its kept rows are ever read, and the kernels can read pinned host memory.  Both only marshal arguments
and order streams; all arithmetic is in the library's kernels.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as pkv


class LayerOutputs:
    """Preallocated packed outputs of every layer of a model (device)."""

    def __init__(self, cfg: pkv.PkvConfig, seq_lens: Sequence[int], dtype: torch.dtype, device="cuda"):
        self.budgets = pkv.layer_budgets(cfg)
        self.rows = [pkv.total_rows(cfg, kl, seq_lens) for kl in self.budgets]
        self.k = [torch.empty(r, cfg.head_dim, dtype=dtype, device=device) for r in self.rows]
        self.v = [torch.empty(r, cfg.head_dim, dtype=dtype, device=device) for r in self.rows]
        self.idx = [torch.empty(r, dtype=torch.int32, device=device) for r in self.rows]


class LayerStreams:
    """A few CUDA streams with a workspace each.  The layers of a model are independent of one another, so
    `compress_model` can enqueue them round robin on these streams: the short kernels of one layer (selection and
    gather, the tails of the sweeps) then run beside the sweeps of the next layers instead of leaving SMs idle."""

    def __init__(self, cfg: pkv.PkvConfig, seq_lens: Sequence[int], count: int, device="cuda"):
        if count < 1:
            raise ValueError("at least one stream")
        self.streams = [torch.cuda.Stream(device=device) for _ in range(count)]
        self.workspaces = [pkv.new_workspace(cfg, len(seq_lens), max(seq_lens), device) for _ in range(count)]
        self.fork = torch.cuda.Event()
        self.joins = [torch.cuda.Event() for _ in range(count)]

    def check_status(self) -> None:
        for ws in self.workspaces:
            pkv.check_status(ws)


def compress_model(cfg: pkv.PkvConfig, layers, seq_lens: Sequence[int], out: LayerOutputs,
                   workspace, stream: Optional[torch.cuda.Stream] = None, lanes=None,
                   layer_streams: Optional[LayerStreams] = None) -> None:
    """layers: sequence of objects with .q_win, .k, .v device tensors, one per layer; a layer that also
    has .window_lse (the prefill's log-sum-exp of the window rows) is scored in a single K sweep; one that has
    .attn_out ([batch][H_q][window][d] float32) also gets the window rows' attention output written there.
    With `lanes` (binding.Lanes) and `workspace` a pair of workspaces, the score sweeps of a layer run beside
    the selection and gather of the layer before it, each on its own group of SMs.
    With `layer_streams` (`workspace` is then not used) layer l runs on stream l mod count with that stream's
    workspace; the streams start after the work already enqueued on `stream` (the current stream if None) and
    `stream` continues after all of them: to the caller the call is ordered like the single-stream one, and its
    results are the same bit for bit."""
    if lanes is not None:
        pkv.compress_model_lanes(cfg, lanes, layers, seq_lens, out.k, out.v, out.idx, workspace, stream=stream)
        return
    if layer_streams is not None:
        cur = stream if stream is not None else torch.cuda.current_stream()
        layer_streams.fork.record(cur)
        for s in layer_streams.streams:
            s.wait_event(layer_streams.fork)
        count = len(layer_streams.streams)
        for l, x in enumerate(layers):
            _compress_one(cfg, l, x, seq_lens, out, layer_streams.workspaces[l % count], layer_streams.streams[l % count])
        for s, e in zip(layer_streams.streams, layer_streams.joins):
            e.record(s)
            cur.wait_event(e)
        return
    for l, x in enumerate(layers):
        _compress_one(cfg, l, x, seq_lens, out, workspace, stream)


def _compress_one(cfg, l, x, seq_lens, out, workspace, stream) -> None:
    if getattr(x, "attn_out", None) is not None:           # the window rows' attention output is wanted too
        pkv.attend_compress_layer(cfg, l, x.q_win, x.k, x.v, seq_lens, x.attn_out, out.k[l], out.v[l], out.idx[l],
                                  workspace, stream=stream)
        return
    pkv.compress_layer(cfg, l, x.q_win, x.k, x.v, seq_lens, out.k[l], out.v[l], out.idx[l], workspace,
                       stream=stream, window_lse=getattr(x, "window_lse", None))


class HostPipeline:
    """Double-buffered host -> device -> host pipeline for one model shape."""

    def __init__(self, cfg: pkv.PkvConfig, seq_lens: Sequence[int], q_shape, kv_shape, dtype: torch.dtype,
                 device="cuda", zero_copy_v: bool = True):
        """zero_copy_v: leave V in the caller's pinned host memory and let the gather read the kept rows over
        the bus (only they are ever needed); V is then not copied to the device at all."""
        self.cfg, self.seq_lens = cfg, list(seq_lens)
        self.zero_copy_v = zero_copy_v
        self.budgets = pkv.layer_budgets(cfg)
        self.rows = [pkv.total_rows(cfg, kl, seq_lens) for kl in self.budgets]
        max_rows = max(self.rows)
        self.dev = [dict(q=torch.empty(q_shape, dtype=dtype, device=device),
                         k=torch.empty(kv_shape, dtype=dtype, device=device),
                         v=torch.empty(kv_shape, dtype=dtype, device=device),
                         ko=torch.empty(max_rows, cfg.head_dim, dtype=dtype, device=device),
                         vo=torch.empty(max_rows, cfg.head_dim, dtype=dtype, device=device),
                         io=torch.empty(max_rows, dtype=torch.int32, device=device),
                         lse=torch.empty(q_shape[:3], dtype=torch.float32, device=device)) for _ in range(2)]
        self.workspace = pkv.new_workspace(cfg, len(self.seq_lens), max(self.seq_lens), device)
        self.copy_in = torch.cuda.Stream(device=device)
        self.compute = torch.cuda.Stream(device=device)
        self.copy_out = torch.cuda.Stream(device=device)
        self.h2d_bytes = 0
        self.d2h_bytes = 0

    def run(self, host_layers, host_out) -> None:
        """host_layers[l] has pinned .q_win/.k/.v; host_out[l] has pinned .k/.v/.idx sized rows[l]."""
        m = self.cfg.num_layers
        loaded = [torch.cuda.Event() for _ in range(m)]
        computed = [torch.cuda.Event() for _ in range(m)]
        drained = [torch.cuda.Event() for _ in range(m)]
        self.h2d_bytes = self.d2h_bytes = 0
        for l in range(m):
            buf, src, dst, r = self.dev[l & 1], host_layers[l], host_out[l], self.rows[l]
            with torch.cuda.stream(self.copy_in):
                if l >= 2:
                    self.copy_in.wait_event(computed[l - 2])      # buffer free once its layer was compressed
                direct_v = self.zero_copy_v and pkv.memory_kind(src.v) == pkv.MEM_PINNED_HOST
                buf["q"].copy_(src.q_win, non_blocking=True)
                buf["k"].copy_(src.k, non_blocking=True)
                if not direct_v:
                    buf["v"].copy_(src.v, non_blocking=True)
                lse = getattr(src, "window_lse", None)
                if lse is not None:
                    buf["lse"].copy_(lse, non_blocking=True)
                loaded[l].record(self.copy_in)
            moved = [src.q_win, src.k] + ([] if direct_v else [src.v]) + ([lse] if lse is not None else [])
            self.h2d_bytes += sum(t.numel() * t.element_size() for t in moved)
            if direct_v:                                          # the kept rows of V cross the bus inside the kernel
                self.h2d_bytes += r * self.cfg.head_dim * src.v.element_size()
            with torch.cuda.stream(self.compute):
                self.compute.wait_event(loaded[l])
                if l >= 2:
                    self.compute.wait_event(drained[l - 2])       # outputs of this buffer were copied out
                pkv.compress_layer(self.cfg, l, buf["q"], buf["k"], src.v if direct_v else buf["v"], self.seq_lens,
                                   buf["ko"], buf["vo"],
                                   buf["io"], self.workspace, stream=self.compute,
                                   window_lse=buf["lse"] if lse is not None else None)
                computed[l].record(self.compute)
            with torch.cuda.stream(self.copy_out):
                self.copy_out.wait_event(computed[l])
                dst.k.copy_(buf["ko"][:r], non_blocking=True)
                dst.v.copy_(buf["vo"][:r], non_blocking=True)
                dst.idx.copy_(buf["io"][:r], non_blocking=True)
                drained[l].record(self.copy_out)
            self.d2h_bytes += sum(t.numel() * t.element_size() for t in (dst.k, dst.v, dst.idx))
        cur = torch.cuda.current_stream()
        cur.wait_stream(self.copy_out)
        cur.wait_stream(self.compute)
