// Shared definitions of the PyramidKV compression kernels (device + host side of the library).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "pyramidkv.h"

namespace pkv {

// Per-call table of the sequences of a batch, passed to kernels by value.
struct SeqTable {
  int32_t batch;
  int32_t alpha;
  int32_t n[PKV_MAX_BATCH];              // keys of sequence b held by the K tensor of this call
  int32_t prefix[PKV_MAX_BATCH];         // how many of them are scored prefix keys: n - alpha for a whole
                                         // sequence; all of them on a shard that does not hold the window
  int32_t count[PKV_MAX_BATCH];          // rows each KV head of sequence b keeps in this layer
  int64_t row_off[PKV_MAX_BATCH];        // first packed output row of sequence b
  int32_t stat_off[PKV_MAX_BATCH + 1];   // running sum of key chunks per sequence (row statistics sweep)
  int32_t score_off[PKV_MAX_BATCH + 1];  // running sum of prefix key tiles per sequence (score sweep)
};

// Strided view of a [batch][head][token][d] tensor.
struct TensorView {
  const void* ptr;
  int64_t sb, sh, st;
};

// Status word values (first word of the workspace); kernels only ever OR bits in.
enum : uint32_t {
  kStatusSelectMismatch = 1u << 0,   // selection emitted a count other than k
  kStatusWaitExpired = 1u << 1,      // a bounded wait ran out
  kStatusBadPage = 1u << 2,          // a block-table entry named a page outside the pool (row skipped)
  kStatusBadIndex = 1u << 3,         // a caller-supplied index list named a position outside its sequence (row skipped)
};

// Programmatic dependent launch: every kernel of the library is launched so that it may start while
// the kernel before it in the stream is still draining.  A kernel first lets its own successor be
// scheduled (pdl_trigger), does whatever set-up touches no global memory, and then waits for the
// preceding kernel to have completed and flushed its writes (pdl_wait) before it reads or writes
// global memory.  Without a preceding kernel both are no-ops.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ float to_float(__half x) { return __half2float(x); }

// Which sequence owns global tile `t` (off is ascending, off[batch] = total).
__device__ __forceinline__ int find_sequence(const int32_t* off, int batch, int t) {
  int b = 0;
  while (b + 1 < batch && t >= off[b + 1]) ++b;
  return b;
}

}  // namespace pkv
