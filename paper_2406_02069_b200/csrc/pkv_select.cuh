// Fused max-pool + per-head top-k + window retention (Section 4.2.2).
//
// One thread-block cluster per (sequence, KV head).  The prefix positions are
// split into contiguous slices, one per CTA of the cluster; each CTA pools its
// slice (reading a halo of (w-1)/2 scores on both sides) and keeps the pooled
// values in shared memory as order-preserving 32-bit keys.  The k-th largest key
// is found by a most-significant-digit radix search (4 passes of 8 bits): every
// CTA histograms its slice, the histograms are summed across the cluster through
// distributed shared memory, and every CTA walks the summed histogram to the same
// digit.  Ties at the threshold go to the smaller position, and kept positions
// are written in ascending order, so the result is one canonical list:
//   kept = { i : key_i > T }  plus the leftmost (k - |{key > T}|) positions with key_i == T.
// The alpha window positions are appended after them.
//
// Only cluster barriers are used for synchronisation (no flag spinning).
#pragma once

#include <cooperative_groups.h>

#include "pkv_common.cuh"

namespace pkv {

namespace cg = cooperative_groups;

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelMaxCluster = 8;
constexpr int kSelSliceCap = 48 * 1024;   // keys a CTA can hold in shared memory (192 KB)

struct SelectParams {
  const float* scores;      // [batch][H_kv][ld]
  int64_t ld_scores;
  int32_t* indices;         // packed rows
  SeqTable seq;
  int32_t num_kv_heads;
  int32_t pool_radius;      // (w - 1) / 2
  int32_t slice_cap;        // keys of shared memory each CTA has (0: keys are recomputed from global)
  uint32_t* status;
};

// Monotone map float -> uint32 (larger float, larger key).  -0 is folded into +0 first.
__device__ __forceinline__ uint32_t ordered_key(float x) {
  const uint32_t u = __float_as_uint(x + 0.0f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ uint32_t pooled_key(const float* s, int i, int P, int radius) {
  const int lo = max(0, i - radius), hi = min(P - 1, i + radius);
  float best = s[lo];
  for (int t = lo + 1; t <= hi; ++t) best = fmaxf(best, s[t]);
  return ordered_key(best);
}

// grid (cluster * H_kv, batch), cluster (cluster, 1, 1), block kSelThreads,
// dynamic shared memory slice_cap * 4 bytes.
__global__ void __launch_bounds__(kSelThreads) pool_select_kernel(const SelectParams p) {
  extern __shared__ __align__(16) uint32_t keys[];          // this CTA's pooled keys (if cached)
  __shared__ uint32_t hist[2][256];                         // per-pass digit histogram (double buffered)
  __shared__ uint32_t total[256];                           // histogram summed over the cluster
  __shared__ uint32_t warp_gt[kSelWarps], warp_eq[kSelWarps];
  __shared__ uint32_t cta_cnt[2];                           // (greater, equal) counts of this CTA
  __shared__ uint32_t sel_digit, sel_above;

  cg::cluster_group cluster = cg::this_cluster();
  const int C = cluster.dim_blocks().x;
  const int rank = cluster.block_rank();
  const int h = blockIdx.x / C, b = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  const int n = p.seq.n[b], alpha = p.seq.alpha, P = n - alpha;
  const int count = p.seq.count[b];
  const int k = count - alpha;                              // prefix rows to keep, 0 <= k <= P
  int32_t* out = p.indices + p.seq.row_off[b] + static_cast<int64_t>(h) * count;

  // The window positions close the list (Section 4.2.1: always retained).
  if (rank == 0)
    for (int j = tid; j < alpha; j += kSelThreads) out[k + j] = P + j;
  if (k >= P) {                                             // nothing to evict: identity list
    for (int i = rank * kSelThreads + tid; i < P; i += C * kSelThreads) out[i] = i;
    return;                                                 // uniform over the cluster
  }
  if (k == 0) return;

  const float* s = p.scores + (static_cast<int64_t>(b) * p.num_kv_heads + h) * p.ld_scores;
  const int slice = ((P + C - 1) / C + 31) & ~31;           // multiple of 32 positions per CTA
  const int lo = min(P, rank * slice), hi = min(P, lo + slice);
  const bool cached = p.slice_cap >= slice;

  if (cached)
    for (int i = lo + tid; i < hi; i += kSelThreads) keys[i - lo] = pooled_key(s, i, P, p.pool_radius);
  auto key_at = [&](int i) -> uint32_t {
    return cached ? keys[i - lo] : pooled_key(s, i, P, p.pool_radius);
  };
  for (int i = tid; i < 512; i += kSelThreads) (&hist[0][0])[i] = 0;
  __syncthreads();

  // ---- radix search for the k-th largest key
  uint32_t prefix = 0, mask = 0, remaining = k;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    uint32_t* hcur = hist[pass & 1];
    for (int base = lo + warp * 32; base < hi; base += kSelThreads) {
      const int i = base + lane;
      uint32_t digit = 256;                                 // 256 = does not take part
      if (i < hi) {
        const uint32_t key = key_at(i);
        if ((key & mask) == prefix) digit = (key >> shift) & 255u;
      }
      const uint32_t peers = __match_any_sync(0xffffffffu, digit);
      if (digit < 256 && lane == __ffs(peers) - 1) atomicAdd(&hcur[digit], __popc(peers));
    }
    cluster.sync();                                         // all histograms of this pass complete
    if (tid < 256) {
      uint32_t t = 0;
      for (int c = 0; c < C; ++c) t += cluster.map_shared_rank(hcur, c)[tid];
      total[tid] = t;
      hist[(pass + 1) & 1][tid] = 0;                        // next pass's buffer: last read two syncs ago
    }
    __syncthreads();
    if (warp == 0) {
      // lane L owns digits 8L .. 8L+7; find the digit where the count from the top reaches `remaining`
      uint32_t mine = 0;
      for (int t = 0; t < 8; ++t) mine += total[lane * 8 + t];
      uint32_t above = mine;                                // inclusive suffix sum over lanes
      for (int off = 1; off < 32; off <<= 1) {
        const uint32_t v = __shfl_down_sync(0xffffffffu, above, off);
        if (lane + off < 32) above += v;
      }
      const uint32_t higher = above - mine;                 // keys in digits owned by higher lanes
      if (higher < remaining && remaining <= above) {
        uint32_t acc = higher;
        for (int t = 7; t >= 0; --t) {
          const uint32_t c = total[lane * 8 + t];
          if (acc + c >= remaining) { sel_digit = lane * 8 + t; sel_above = acc; break; }
          acc += c;
        }
      }
    }
    __syncthreads();
    prefix |= sel_digit << shift;
    mask |= 255u << shift;
    remaining -= sel_above;
  }
  const uint32_t T = prefix;                                // the k-th largest key
  const uint32_t need_eq = remaining;                       // ties at T to take, from the left

  // ---- count keys above / at the threshold: warp w owns a contiguous run of the slice
  const int run = ((slice / kSelWarps) + 31) & ~31;
  const int wlo = min(hi, lo + warp * run), whi = min(hi, wlo + run);
  uint32_t ngt = 0, neq = 0;
  for (int base = wlo; base < whi; base += 32) {
    const int i = base + lane;
    const uint32_t key = i < whi ? key_at(i) : 0u;
    ngt += __popc(__ballot_sync(0xffffffffu, i < whi && key > T));
    neq += __popc(__ballot_sync(0xffffffffu, i < whi && key == T));
  }
  if (lane == 0) { warp_gt[warp] = ngt; warp_eq[warp] = neq; }
  __syncthreads();
  if (warp == 0) {
    uint32_t g = warp_gt[lane], e = warp_eq[lane];
    const uint32_t g0 = g, e0 = e;
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t vg = __shfl_up_sync(0xffffffffu, g, off), ve = __shfl_up_sync(0xffffffffu, e, off);
      if (lane >= off) { g += vg; e += ve; }
    }
    warp_gt[lane] = g - g0;                                 // exclusive prefix inside the CTA
    warp_eq[lane] = e - e0;
    if (lane == 31) { cta_cnt[0] = g; cta_cnt[1] = e; }
  }
  cluster.sync();                                           // counts of every CTA visible
  uint32_t gt_before = warp_gt[warp], eq_before = warp_eq[warp];
  uint32_t all_gt = 0;
  for (int c = 0; c < C; ++c) {
    const uint32_t* rc = cluster.map_shared_rank(cta_cnt, c);
    const uint32_t g = rc[0], e = rc[1];
    if (c < rank) { gt_before += g; eq_before += e; }
    all_gt += g;
  }
  if (rank == 0 && tid == 0 && all_gt + need_eq != static_cast<uint32_t>(k))
    atomicOr(p.status, kStatusSelectMismatch);

  // ---- emit in ascending position: rank of i among the kept = (#greater before i) + min(#equal before i, need_eq)
  for (int base = wlo; base < whi; base += 32) {
    const int i = base + lane;
    const uint32_t key = i < whi ? key_at(i) : 0u;
    const bool is_gt = i < whi && key > T, is_eq = i < whi && key == T;
    const uint32_t bg = __ballot_sync(0xffffffffu, is_gt), be = __ballot_sync(0xffffffffu, is_eq);
    const uint32_t lt = (1u << lane) - 1u;
    const uint32_t g = gt_before + __popc(bg & lt), e = eq_before + __popc(be & lt);
    if (is_gt || (is_eq && e < need_eq)) out[g + min(e, need_eq)] = i;
    gt_before += __popc(bg);
    eq_before += __popc(be);
  }
  cluster.sync();                                           // nobody leaves while its shared memory may be read
}

}  // namespace pkv
