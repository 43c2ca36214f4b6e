// Eviction by gather: copy the kept rows of K and V into the packed compact cache
// (appendix on torch.gather; Section 4.1: K_s, V_s are sub-matrices of K, V).
//
// Pure data movement.  Each thread moves one 16-byte piece of a row of K and the
// same piece of V, so a 256-byte bf16 row is one coalesced access of 16 threads.
// The index list is the caller's: an entry outside [0, n_b) is never used as an
// address, its output row is left untouched.
#pragma once

#include "pkv_common.cuh"

namespace pkv {

constexpr int kGatherThreads = 256;

struct GatherParams {
  TensorView k, v;
  const int32_t* indices;   // packed rows: original position of each output row
  void* k_out;
  void* v_out;              // may be null together with v.ptr
  SeqTable seq;
  int32_t num_kv_heads;
  int32_t elem_bytes;       // 4 or 2
  int32_t pieces;           // 16-byte pieces per row = d * elem_bytes / 16
  int64_t total_rows;
};

__global__ void __launch_bounds__(kGatherThreads) gather_rows_kernel(const GatherParams p) {
  pdl_trigger();
  pdl_wait();
  const int64_t gid = static_cast<int64_t>(blockIdx.x) * kGatherThreads + threadIdx.x;
  const int64_t row = gid / p.pieces;
  const int piece = static_cast<int>(gid % p.pieces);
  if (row >= p.total_rows) return;
  int b = 0;
  while (b + 1 < p.seq.batch && row >= p.seq.row_off[b + 1]) ++b;
  const int h = static_cast<int>((row - p.seq.row_off[b]) / p.seq.count[b]);
  const int pos = p.indices[row];
  if (pos < 0 || pos >= p.seq.n[b]) return;                 // not a position of this sequence: nothing is read
  const int64_t dst = row * p.pieces + piece;
  {
    const char* src = static_cast<const char*>(p.k.ptr) +
                      (b * p.k.sb + h * p.k.sh + static_cast<int64_t>(pos) * p.k.st) * p.elem_bytes;
    static_cast<uint4*>(p.k_out)[dst] = reinterpret_cast<const uint4*>(src)[piece];
  }
  if (p.v_out) {
    const char* src = static_cast<const char*>(p.v.ptr) +
                      (b * p.v.sb + h * p.v.sh + static_cast<int64_t>(pos) * p.v.st) * p.elem_bytes;
    static_cast<uint4*>(p.v_out)[dst] = reinterpret_cast<const uint4*>(src)[piece];
  }
}

}  // namespace pkv
