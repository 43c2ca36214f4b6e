// Paged placement of the compact cache (appendix on paged attention: block tables per layer, so that a layer
// with a small budget holds few pages and a paged allocator can free the rest).
//
// A pool holds pages of page_size rows of one KV head.  One layer's block table lists, sequence after
// sequence and inside a sequence head after head, the pages of that head's kept list: row r of the list
// sits in page table[r / page_size] at slot r % page_size.  The caller's allocator fills the table; the
// kernels only follow it.  A table entry outside [0, num_pages) is never dereferenced: the kernel records
// kStatusBadPage in the status word and skips that row.  The same goes for an entry of the index list
// outside [0, n_b): kStatusBadIndex, row skipped.
#pragma once

#include "pkv_common.cuh"

namespace pkv {

struct PageTable {
  const int32_t* table;                  // device, packed as described above
  int64_t tab_off[PKV_MAX_BATCH];        // first table entry of sequence b
  int32_t pages[PKV_MAX_BATCH];          // pages per KV head of sequence b = ceil(count[b] / page_size)
  int32_t page_size;
  int32_t num_pages;
};

// Row (in units of rows) of the pool that holds row r of head h of sequence b, or -1 for a bad table entry.
__device__ __forceinline__ int64_t paged_row(const PageTable& t, int b, int h, int r) {
  const int page = __ldg(t.table + t.tab_off[b] + static_cast<int64_t>(h) * t.pages[b] + r / t.page_size);
  if (page < 0 || page >= t.num_pages) return -1;
  return static_cast<int64_t>(page) * t.page_size + r % t.page_size;
}

constexpr int kPagedThreads = 256;

struct GatherPagedParams {
  TensorView k, v;
  const int32_t* indices;   // packed rows: original position of each kept row
  void* k_pool;             // [num_pages][page_size][d]
  void* v_pool;
  SeqTable seq;
  PageTable pt;
  int32_t num_kv_heads;
  int32_t elem_bytes;       // 4 or 2
  int32_t pieces;           // 16-byte pieces per row
  int64_t total_rows;
  uint32_t* status;
};

// One thread moves one 16-byte piece of a kept row of K and the same piece of V into its page slot.
__global__ void __launch_bounds__(kPagedThreads) gather_paged_kernel(const GatherPagedParams p) {
  pdl_trigger();
  pdl_wait();
  const int64_t gid = static_cast<int64_t>(blockIdx.x) * kPagedThreads + threadIdx.x;
  const int64_t row = gid / p.pieces;
  const int piece = static_cast<int>(gid % p.pieces);
  if (row >= p.total_rows) return;
  int b = 0;
  while (b + 1 < p.seq.batch && row >= p.seq.row_off[b + 1]) ++b;
  const int64_t local = row - p.seq.row_off[b];
  const int h = static_cast<int>(local / p.seq.count[b]);
  const int r = static_cast<int>(local - static_cast<int64_t>(h) * p.seq.count[b]);
  const int64_t slot = paged_row(p.pt, b, h, r);
  if (slot < 0) {
    if (piece == 0) atomicOr(p.status, kStatusBadPage);
    return;
  }
  const int pos = p.indices[row];
  if (pos < 0 || pos >= p.seq.n[b]) {
    if (piece == 0) atomicOr(p.status, kStatusBadIndex);
    return;
  }
  const int64_t dst = slot * p.pieces + piece;
  const char* ksrc = static_cast<const char*>(p.k.ptr) +
                     (b * p.k.sb + h * p.k.sh + static_cast<int64_t>(pos) * p.k.st) * p.elem_bytes;
  static_cast<uint4*>(p.k_pool)[dst] = reinterpret_cast<const uint4*>(ksrc)[piece];
  const char* vsrc = static_cast<const char*>(p.v.ptr) +
                     (b * p.v.sb + h * p.v.sh + static_cast<int64_t>(pos) * p.v.st) * p.elem_bytes;
  static_cast<uint4*>(p.v_pool)[dst] = reinterpret_cast<const uint4*>(vsrc)[piece];
}

}  // namespace pkv
