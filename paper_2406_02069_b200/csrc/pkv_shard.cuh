// Sequence-sharded compression: the keys of one long context are split into contiguous ranges, one per GPU
// (the window queries are small and every GPU holds them).  Eq. 2's softmax then needs one exchange: each
// shard's partial row normalisers are merged into the row's full normaliser, after which every shard scores
// its own keys (Eq. 3) exactly as in the single-sweep mode.  The kernels here are the small pieces around
// the score kernels: exporting and merging normalisers, and gathering the kept rows a shard owns.
#pragma once

#include "pkv_common.cuh"

namespace pkv {

constexpr int kShardThreads = 256;

// lse2 holds log2(sum of 2^x) + log2(G) per window row; the exchange format is the natural logarithm of the
// plain sum of exponentials, the same quantity the single-sweep mode takes.
__global__ void __launch_bounds__(kShardThreads) export_lse_kernel(const float* lse2, float log2_group, float* out,
                                                                    int64_t count) {
  pdl_trigger();
  pdl_wait();
  const int64_t i = static_cast<int64_t>(blockIdx.x) * kShardThreads + threadIdx.x;
  if (i < count) out[i] = (lse2[i] - log2_group) * 0.6931471805599453f;
}

// out[i] = log(sum over shards s of exp(parts[s][i])), evaluated around the largest part.
__global__ void __launch_bounds__(kShardThreads) merge_lse_kernel(const float* parts, int shards, int64_t count,
                                                                   float* out) {
  pdl_trigger();
  pdl_wait();
  const int64_t i = static_cast<int64_t>(blockIdx.x) * kShardThreads + threadIdx.x;
  if (i >= count) return;
  float m = -INFINITY;
  for (int s = 0; s < shards; ++s) m = fmaxf(m, parts[s * count + i]);
  float z = 0.f;
  for (int s = 0; s < shards; ++s) z += expf(parts[s * count + i] - m);
  out[i] = m + logf(z);
}

struct GatherShardParams {
  TensorView k, v;          // this shard's keys: token t of the view is position begin[b] + t of the sequence
  const int32_t* indices;   // packed rows of the whole layer: original positions
  void* k_out;              // packed rows of the whole layer; only rows this shard owns are written
  void* v_out;
  SeqTable seq;             // counts and row offsets of the whole sequences
  int32_t begin[PKV_MAX_BATCH];
  int32_t keys[PKV_MAX_BATCH];
  int32_t num_kv_heads;
  int32_t elem_bytes;
  int32_t pieces;
  int64_t total_rows;
};

__global__ void __launch_bounds__(kShardThreads) gather_shard_kernel(const GatherShardParams p) {
  pdl_trigger();
  pdl_wait();
  const int64_t gid = static_cast<int64_t>(blockIdx.x) * kShardThreads + threadIdx.x;
  const int64_t row = gid / p.pieces;
  const int piece = static_cast<int>(gid % p.pieces);
  if (row >= p.total_rows) return;
  int b = 0;
  while (b + 1 < p.seq.batch && row >= p.seq.row_off[b + 1]) ++b;
  const int h = static_cast<int>((row - p.seq.row_off[b]) / p.seq.count[b]);
  const int local = p.indices[row] - p.begin[b];
  if (local < 0 || local >= p.keys[b]) return;                  // another shard owns this row
  const int64_t dst = row * p.pieces + piece;
  const char* ksrc = static_cast<const char*>(p.k.ptr) +
                     (b * p.k.sb + h * p.k.sh + static_cast<int64_t>(local) * p.k.st) * p.elem_bytes;
  static_cast<uint4*>(p.k_out)[dst] = reinterpret_cast<const uint4*>(ksrc)[piece];
  const char* vsrc = static_cast<const char*>(p.v.ptr) +
                     (b * p.v.sb + h * p.v.sh + static_cast<int64_t>(local) * p.v.st) * p.elem_bytes;
  static_cast<uint4*>(p.v_out)[dst] = reinterpret_cast<const uint4*>(vsrc)[piece];
}

}  // namespace pkv
