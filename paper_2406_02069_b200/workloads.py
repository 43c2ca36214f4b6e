"""Seeded synthetic inputs for the prefill KV-cache compression step.

This module only draws tensors. It holds none of the method's arithmetic (no
budgets, no scores, no selection), so the CUDA path and the CPU oracle can both
be fed from it without sharing any of the code under test.

The tensors stand in for the paper's long-context workloads (LongBench,
Needle-in-a-Haystack, the 128k setting), whose items and model weights are not
used here.  What is kept from the paper is the structure it describes in its
observation section: broad, near-uniform attention in low layers, attention
concentrating on a few tokens in high layers, a few attention-sink tokens at the
start of the sequence, and a needle planted at some depth.

Recipe, per layer l of m and per KV head h:
  * every element of window-Q, K and V is i.i.d. N(0,1), rounded to the dtype;
  * a unit vector u[l,h] is drawn; all window queries of the head's GQA group
    get  + gamma_l * u  with gamma_l rising linearly from gamma_lo (layer 0) to
    gamma_hi (layer m-1), so attention sharpens with depth;
  * sink keys (positions 0..n_sink-1) get  + sink_gain * sqrt(d) * u;
  * needle keys get  + needle_gain * sqrt(d) * u  at seeded positions, either
    `needles` single positions or one block of `needle_block` consecutive ones;
  * V is left as drawn: the path only moves it.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Tuple

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    num_layers: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    batch: int
    seq_len_lo: int          # per-sequence length is uniform in [lo, hi]
    seq_len_hi: int
    dtype: str               # "fp32" | "bf16" | "fp16"
    window: int              # alpha
    pool_kernel: int         # w
    avg_budget: int          # B, window rows included
    beta: float = 20.0
    n_sink: int = 4
    needles: int = 0         # number of single planted keys per sequence
    needle_block: int = 0    # length of one planted block (0 = none)
    gamma_lo: float = 2.0
    gamma_hi: float = 6.0
    sink_gain: float = 2.0
    needle_gain: float = 1.5
    seed: int = 0
    pool_kind: str = "max"   # "max" | "avg" (the mean-pool variant)
    needle_depth: float = -1.0   # in [0, 1]: where the planted block starts in the prefix; < 0: drawn from the seed
    schedule: str = "linear"     # "linear" | "geometric": shape of the per-layer budgets (a configuration label only)

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    def torch_dtype(self) -> torch.dtype:
        return {"fp32": torch.float32, "bf16": torch.bfloat16, "fp16": torch.float16}[self.dtype]

    def seq_lens(self) -> List[int]:
        """Per-sequence context lengths, drawn once from the workload seed."""
        if self.seq_len_lo == self.seq_len_hi:
            return [self.seq_len_lo] * self.batch
        g = torch.Generator(device="cpu")
        g.manual_seed(7919 * (self.seed + 1))
        r = torch.randint(self.seq_len_lo, self.seq_len_hi + 1, (self.batch,), generator=g)
        return [int(x) for x in r]

    def gamma(self, layer: int) -> float:
        if self.num_layers == 1:
            return self.gamma_lo
        return self.gamma_lo + (self.gamma_hi - self.gamma_lo) * layer / (self.num_layers - 1)


# The five named workloads.  "configs[i]" below refers to their order here.
TINY = Workload("tiny_fp32", 2, 4, 2, 64, 1, 512, 512, "fp32", 8, 5, 64,
                n_sink=1, gamma_lo=4.0, gamma_hi=4.0, seed=1)
LLAMA2_7B = Workload("llama2_7b_4k", 32, 32, 32, 128, 1, 4096, 4096, "bf16", 32, 7, 128,
                     needles=16, seed=2)
LLAMA3_8B = Workload("llama3_8b_32k", 32, 32, 8, 128, 1, 32768, 32768, "bf16", 32, 7, 512,
                     needles=32, seed=3)
LLAMA3_70B = Workload("llama3_70b_128k", 80, 64, 8, 128, 1, 131072, 131072, "bf16", 32, 7, 128,
                      needle_block=64, seed=4)
MISTRAL_RAGGED = Workload("mistral_7b_ragged", 32, 32, 8, 128, 8, 4096, 16384, "bf16", 32, 7, 512,
                          needles=8, seed=5)
MISTRAL_BUDGETS = (64, 128, 256, 512, 2048)

# Retrieval-shaped sweep (appendix on fact retrieval across context lengths): Mistral-7B heads, contexts up to
# 32k, one planted block at a chosen depth, cache sizes 64 / 96 / 128.
MISTRAL_NEEDLE_32K = Workload("mistral_7b_32k_needle", 32, 32, 8, 128, 1, 32768, 32768, "bf16", 8, 7, 128,
                              needle_block=16, needle_depth=0.5, seed=6)
NEEDLE_BUDGETS = (64, 96, 128)

WORKLOADS = {w.name: w for w in (TINY, LLAMA2_7B, LLAMA3_8B, LLAMA3_70B, MISTRAL_RAGGED, MISTRAL_NEEDLE_32K)}


def needle_case(seq_len: int, depth: float, avg_budget: int, num_layers: int = 32) -> Workload:
    """One cell of the retrieval sweep: context length, needle depth in [0, 1], cache size."""
    return dataclasses.replace(MISTRAL_NEEDLE_32K, name="needle_n%d_d%02d_b%d" % (seq_len, round(depth * 100), avg_budget),
                               seq_len_lo=seq_len, seq_len_hi=seq_len, needle_depth=depth, avg_budget=avg_budget,
                               num_layers=num_layers)


def with_budget(w: Workload, avg_budget: int) -> Workload:
    return dataclasses.replace(w, avg_budget=avg_budget)


def scaled(w: Workload, *, num_layers: Optional[int] = None, seq_len: Optional[int] = None,
           batch: Optional[int] = None, name: Optional[str] = None, **fields) -> Workload:
    """A smaller case of the same shape family (for tests the oracle finishes in seconds); further keyword
    arguments replace fields by name (dtype, pool_kind, window, beta ...)."""
    kw = dict(fields)
    if num_layers is not None:
        kw["num_layers"] = num_layers
    if seq_len is not None:
        kw["seq_len_lo"] = seq_len
        kw["seq_len_hi"] = seq_len
    if batch is not None:
        kw["batch"] = batch
    kw["name"] = name or (w.name + "_scaled")
    return dataclasses.replace(w, **kw)


@dataclasses.dataclass
class LayerInputs:
    """One layer's tensors.  K and V are padded to the longest sequence."""
    q_win: torch.Tensor      # [batch][H_q][alpha][d]
    k: torch.Tensor          # [batch][H_kv][n_max][d]
    v: torch.Tensor          # [batch][H_kv][n_max][d]
    seq_lens: List[int]
    planted: List[List[int]]  # per sequence: sink + needle positions


def _planted_positions(w: Workload, layer: int, b: int, n: int) -> Tuple[List[int], List[int]]:
    """Sink positions and needle positions of sequence b (same in every layer)."""
    prefix = n - w.window
    sinks = list(range(min(w.n_sink, prefix)))
    g = torch.Generator(device="cpu")
    g.manual_seed(104729 * (w.seed + 1) + 31 * b)
    needles: List[int] = []
    lo = len(sinks)
    if w.needle_block > 0 and prefix - lo > w.needle_block:
        start = int(torch.randint(lo, prefix - w.needle_block, (1,), generator=g))
        if w.needle_depth >= 0.0:
            start = lo + int(round(min(w.needle_depth, 1.0) * (prefix - w.needle_block - lo - 1)))
        needles = list(range(start, start + w.needle_block))
    elif w.needles > 0 and prefix - lo > w.needles:
        perm = torch.randperm(prefix - lo, generator=g)[: w.needles] + lo
        needles = sorted(int(x) for x in perm)
    return sinks, needles


def make_layer(w: Workload, layer: int, device: str = "cpu",
               seq_lens: Optional[List[int]] = None) -> LayerInputs:
    """Draw layer `layer` of workload `w` on `device` (seed = 1000*w.seed + layer)."""
    lens = list(seq_lens) if seq_lens is not None else w.seq_lens()
    n_max = max(lens)
    d = w.head_dim
    dt = w.torch_dtype()
    g = torch.Generator(device=device)
    g.manual_seed(1000 * w.seed + layer)

    def randn(*shape):
        return torch.randn(*shape, generator=g, device=device, dtype=torch.float32)

    u = randn(len(lens), w.num_kv_heads, d)
    u = u / u.norm(dim=-1, keepdim=True)
    gam = w.gamma(layer)
    root_d = math.sqrt(d)

    q = randn(len(lens), w.num_q_heads, w.window, d)
    q += gam * u.repeat_interleave(w.group, dim=1).unsqueeze(2)
    q = q.to(dt)

    k = randn(len(lens), w.num_kv_heads, n_max, d)
    planted: List[List[int]] = []
    for b, n in enumerate(lens):
        sinks, needles = _planted_positions(w, layer, b, n)
        if sinks:
            k[b, :, sinks, :] += (w.sink_gain * root_d) * u[b].unsqueeze(1)
        if needles:
            k[b, :, needles, :] += (w.needle_gain * root_d) * u[b].unsqueeze(1)
        planted.append(sinks + needles)
    k = k.to(dt)
    v = randn(len(lens), w.num_kv_heads, n_max, d).to(dt)
    return LayerInputs(q, k, v, lens, planted)


def checksum(t: torch.Tensor) -> int:
    """Order-independent 64-bit checksum of a tensor's bytes (for logging what was drawn)."""
    if t.element_size() == 2:
        raw = t.contiguous().view(torch.int16).to(torch.int64) & 0xFFFF
    else:
        raw = t.contiguous().view(torch.int32).to(torch.int64) & 0xFFFFFFFF
    return int(raw.sum().item()) & 0xFFFFFFFFFFFFFFFF
