// Fused max-pool + per-head top-k + window retention (+ optional eviction by gather), Section 4.2.2.
//
// One thread-block cluster per (sequence, KV head).  The prefix positions are
// split into contiguous slices, one per CTA of the cluster, and inside a CTA into
// contiguous runs, one per warp, so that position order is (CTA rank, warp, order
// inside the warp's run).
//
//  1. Every CTA stages its slice of raw scores in shared memory (coalesced), pools
//     them (halo of (w-1)/2 scores on both sides, clipped to the prefix) into
//     order-preserving 32-bit keys held in registers.
//  2. Candidate filter.  Every thread remembers the largest key it produced.  The
//     k-th largest of those per-thread maxima is a lower bound of the k-th largest
//     key (k distinct keys >= it exist); its top 22 bits are found with two CTA-local
//     11-bit histogram passes.  The CTA writes the (key, position) pairs of its slice
//     that reach the bound, in position order, to its region of a scratch buffer in
//     global memory.  Typically a few times k pairs survive in the whole cluster; in
//     the worst case (all keys equal, or k larger than the thread count) all do.
//  3. After one cluster barrier CTA 0 alone finishes: it concatenates the regions
//     (they are already in position order), finds the k-th largest key T by a
//     most-significant-digit radix search in three passes (11, 11, 10 bits) over the
//     candidates, and emits
//       kept = { i : key_i > T } plus the leftmost (k - |{key > T}|) positions with key_i == T
//     in ascending position; the alpha window positions follow.
//  4. After a second cluster barrier all CTAs of the cluster copy the kept rows of K
//     and V (when asked to).
//
// Ties therefore go to the smaller position and the list is canonical.  Only
// block and cluster barriers are used for synchronisation (no flag spinning).
#pragma once

#include <cooperative_groups.h>

#include "pkv_common.cuh"

namespace pkv {

namespace cg = cooperative_groups;

constexpr int kSelThreads = 1024;
constexpr int kSelThreadsSmall = 512;      // the instance for short slices (it can take up to 8192 positions)
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelMaxCluster = 8;
constexpr int kSelBins = 2048;
constexpr int kSelSliceCap = 16384;        // positions a CTA can hold in shared memory (6 bytes each)
constexpr int kSelRunMax = kSelSliceCap / kSelWarps;   // positions per warp in that case
constexpr int kSelPerLane = kSelRunMax / 32;           // ... and per lane
constexpr int kSelHalo = 16;               // largest pool radius the shared-memory path stages

struct SelectParams {
  const float* scores;      // [batch][H_kv][ld]
  int64_t ld_scores;
  int32_t* indices;         // packed rows
  SeqTable seq;
  int32_t num_kv_heads;
  int32_t pool_radius;      // (w - 1) / 2
  int32_t cached;           // 1: the pool radius fits kSelHalo, slices are staged in shared memory round by round
  int32_t smem_pairs;       // (key, position) pairs CTA 0 can hold in its dynamic shared memory
  uint2* cand;              // scratch: [batch * H_kv][cand_stride] candidate pairs, one region per CTA rank
  int64_t cand_stride;      // >= cluster * slice
  uint32_t* cand_cnt;       // scratch: [batch * H_kv][kSelMaxCluster] pairs written per region
  uint32_t* status;
  // Optional fused eviction by gather (k_out == nullptr: indices only).  Once a head's list is complete
  // the cluster that produced it copies the listed rows of K and V into the packed cache.
  TensorView k, v;
  void* k_out;
  void* v_out;
  int32_t elem_bytes;       // 4 or 2
  int32_t pieces;           // 16-byte pieces per row = d * elem_bytes / 16
};

// Monotone map float -> uint32 (larger float, larger key).  -0 is folded into +0 first.
__device__ __forceinline__ uint32_t ordered_key(float x) {
  const uint32_t u = __float_as_uint(x + 0.0f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// The mean pool decides a top-k, so its rounding is fixed: float additions from the left-most position of the
// window to the right-most, then one float division by the width.
__device__ __forceinline__ uint32_t pooled_key(const float* s, int i, int P, int radius, int avg) {
  const int lo = max(0, i - radius), hi = min(P - 1, i + radius);
  float best = s[lo];
  if (avg) {
    for (int t = lo + 1; t <= hi; ++t) best = __fadd_rn(best, s[t]);
    best = __fdiv_rn(best, static_cast<float>(2 * radius + 1));
  } else {
    for (int t = lo + 1; t <= hi; ++t) best = fmaxf(best, s[t]);
  }
  return ordered_key(best);
}

// Copies the rows named by one head's finished list into the packed cache: 16 bytes of K and of V per thread
// and piece.  `first` / `stride` spread the pieces over the threads of the cluster.  Kept out of line so that
// its registers are allocated apart from the selection's.  Long lists (large budgets move hundreds of
// megabytes here) take four pieces per step with the index loads, the row loads and the stores issued as
// batches; a one-piece loop would be bound by its latency chain.
__device__ __noinline__ void gather_listed_rows(const int32_t* out, const char* kb, const char* vb, int64_t k_step,
                                                int64_t v_step, uint4* k_dst, uint4* v_dst, int64_t row0, int total,
                                                int pieces, int first, int stride) {
  constexpr int kUnroll = 4;
  int g0 = first;
  {
    for (; g0 + (kUnroll - 1) * stride < total; g0 += kUnroll * stride) {
      int piece[kUnroll], pos[kUnroll];
      int64_t dst[kUnroll];
      uint4 val[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int g = g0 + u * stride;
        const int row = g / pieces;
        piece[u] = g - row * pieces;
        pos[u] = __ldcg(out + row);                           // written by other CTAs of the cluster: skip L1
        dst[u] = (row0 + row) * pieces + piece[u];
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u)
        val[u] = reinterpret_cast<const uint4*>(kb + pos[u] * k_step)[piece[u]];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) k_dst[dst[u]] = val[u];
      if (v_dst) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
          val[u] = reinterpret_cast<const uint4*>(vb + pos[u] * v_step)[piece[u]];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) v_dst[dst[u]] = val[u];
      }
    }
  }
  for (; g0 < total; g0 += stride) {
    const int row = g0 / pieces, piece = g0 - row * pieces;
    const int pos = __ldcg(out + row);
    const int64_t dst = (row0 + row) * pieces + piece;
    k_dst[dst] =
        reinterpret_cast<const uint4*>(kb + pos * k_step)[piece];
    if (v_dst)
      v_dst[dst] =
          reinterpret_cast<const uint4*>(vb + pos * v_step)[piece];
  }
}

// grid (cluster * H_kv, batch), cluster (cluster, 1, 1), block kSelThreads,
// dynamic shared memory (6 bytes per slice position + 8 * kSelHalo) when cached, else none.
// MULTI: some CTA's slice is longer than kSelSliceCap and is taken in several rounds.
// GROUPS: maxima each thread keeps for the lower bound of step 2 (1 for small budgets, 8 when k nears or
// passes the thread count, so that the bound stays tight).
template <bool AVG, bool MULTI, int GROUPS, int THREADS = kSelThreads>
__global__ void __launch_bounds__(THREADS, THREADS == kSelThreads ? 1 : 2) pool_select_kernel(const SelectParams p) {
  // THREADS = 512 is the instance for short slices (at most 8192 positions): half the registers of an SM, so that
  // two such CTAs, or one and a CTA of another layer's score kernel, share an SM
  constexpr int WARPS = THREADS / 32;
  constexpr int CAP = kSelSliceCap / (kSelThreads / THREADS);   // positions a CTA holds per round
  constexpr int PER_LANE = kSelPerLane;
  constexpr int BPT = kSelBins / THREADS;                        // histogram bins every thread scans: 2 or 4
  static_assert(BPT == 2 || BPT == 4, "thread count of the selection kernel");
  extern __shared__ __align__(16) uint32_t sel_smem[];      // [halo | slice | halo] raw scores; later CTA 0's pairs
  __shared__ uint32_t hist[2][kSelBins];                    // per-pass digit histogram (double buffered)
  __shared__ uint32_t warp_sum[WARPS];
  __shared__ uint32_t warp_gt[WARPS], warp_eq[WARPS];
  __shared__ uint32_t sel_digit, sel_above, bound_digit;

  pdl_trigger();
  pdl_wait();
  cg::cluster_group cluster = cg::this_cluster();
  const int C = cluster.dim_blocks().x;
  const int rank = cluster.block_rank();
  const int h = blockIdx.x / C, b = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lt = (1u << lane) - 1u;

  const int n = p.seq.n[b], alpha = p.seq.alpha, P = n - alpha;
  const int count = p.seq.count[b];
  const int k = count - alpha;                              // prefix rows to keep, 0 <= k <= P
  int32_t* out = p.indices + p.seq.row_off[b] + static_cast<int64_t>(h) * count;
  const bool selecting = k > 0 && k < P;                    // uniform over the cluster

  // The window positions close the list (Section 4.2.1: always retained).
  if (rank == 0)
    for (int j = tid; j < alpha; j += THREADS) out[k + j] = P + j;
  if (k >= P) {                                             // nothing to evict: identity list
    for (int i = rank * THREADS + tid; i < P; i += C * THREADS) out[i] = i;
  }

  const int64_t head = static_cast<int64_t>(b) * p.num_kv_heads + h;
  const int slice = ((P + C - 1) / C + 31) & ~31;           // multiple of 32 positions per CTA
  uint2* regions = p.cand + head * p.cand_stride;           // region of CTA c starts at c * slice
  uint32_t* counts = p.cand_cnt + head * kSelMaxCluster;
  for (int i = tid; i < 2 * kSelBins; i += THREADS) (&hist[0][0])[i] = 0;
  // A cluster of one keeps its candidates in shared memory when they fit: no trip through global memory.
  bool local_pairs = false;
  int local_count = 0;

  if (selecting) {
    const float* s = p.scores + head * p.ld_scores;
    const int lo = min(P, rank * slice), hi = min(P, lo + slice);
    const int radius = p.pool_radius;
    uint2* region = regions + static_cast<int64_t>(rank) * slice;
    if (p.cached) {                                         // the pool's reach fits the staged halo
      // The slice is taken in rounds of at most CAP positions (one round up to 131072 keys per head
      // with a cluster of 8).  Round: stage raw scores with a halo (outside the prefix: -inf for the max, 0
      // for the mean), pool them into one key per lane and step.
      float* raw = reinterpret_cast<float*>(sel_smem + kSelHalo);
      const float outside = AVG ? 0.0f : -INFINITY;
      const float width = static_cast<float>(2 * radius + 1);
      const int rounds = MULTI ? (hi - lo + CAP - 1) / CAP : 1;
      const int run = ((min(slice, CAP) / WARPS) + 31) & ~31;   // positions per warp and round
      uint32_t pk[PER_LANE];
      int wlo = hi, whi = hi;
      auto pool_round = [&](int r) {
        const int rlo = lo + r * CAP, rhi = min(hi, rlo + CAP);
        if (MULTI) __syncthreads();                         // the previous round's readers are done
        for (int i = rlo - kSelHalo + tid; i < rhi + kSelHalo; i += THREADS)
          raw[i - rlo] = (i >= 0 && i < P) ? s[i] : outside;
        __syncthreads();
        wlo = min(rhi, rlo + warp * run);
        whi = min(rhi, wlo + run);
#pragma unroll
        for (int it = 0; it < PER_LANE; ++it) {
          const int i = wlo + it * 32 + lane;
          pk[it] = 0;
          if (i < whi) {
            float best;
            if (AVG) {                                      // left to right; adding the zeros outside changes nothing
              best = raw[i - rlo - radius];
              for (int t = 1 - radius; t <= radius; ++t) best = __fadd_rn(best, raw[i - rlo + t]);
              best = __fdiv_rn(best, width);
            } else {
              best = raw[i - rlo];
              for (int t = 1; t <= radius; ++t) best = fmaxf(best, fmaxf(raw[i - rlo - t], raw[i - rlo + t]));
            }
            pk[it] = ordered_key(best);
          }
        }
      };
      // ---- 1. every thread's largest pooled keys over the whole slice: one per group of its positions
      //         (position step `it` belongs to group it mod GROUPS)
      uint32_t tmax[GROUPS];
#pragma unroll
      for (int g = 0; g < GROUPS; ++g) tmax[g] = 0;
#pragma unroll
      for (int it = 0; it < PER_LANE; ++it) pk[it] = 0;
      for (int r = 0; r < rounds; ++r) {
        pool_round(r);
#pragma unroll
        for (int it = 0; it < PER_LANE; ++it) tmax[it % GROUPS] = max(tmax[it % GROUPS], pk[it]);
      }
      // ---- 2. lower bound of the k-th largest key: the k-th largest of these maxima (maxima of disjoint
      //         groups of positions, so at least k keys are no smaller), resolved to its top 22 bits by two
      //         CTA-local histogram passes
      uint32_t bprefix = 0, bmask = 0, brem = static_cast<uint32_t>(k);
      for (int bp = 0; bp < 2; ++bp) {
        const int shift = bp == 0 ? 21 : 10;
        // maxima that left the searched prefix do not take part in the second pass
#pragma unroll
        for (int g = 0; g < GROUPS; ++g) {
          const uint32_t digit = ((tmax[g] & bmask) == bprefix) ? ((tmax[g] >> shift) & 2047u) : kSelBins;
          const uint32_t peers = __match_any_sync(0xffffffffu, digit);
          if (digit < kSelBins && lane == __ffs(peers) - 1) atomicAdd(&hist[1][digit], __popc(peers));
        }
        __syncthreads();
        uint32_t bins[BPT];                                 // every thread owns BPT adjacent digits
#pragma unroll
        for (int j = 0; j < BPT; ++j) bins[j] = hist[1][BPT * tid + j];
        uint32_t mine = 0;
#pragma unroll
        for (int j = 0; j < BPT; ++j) mine += bins[j];
        uint32_t incl = mine;
        for (int off = 1; off < 32; off <<= 1) {
          const uint32_t u = __shfl_down_sync(0xffffffffu, incl, off);
          if (lane + off < 32) incl += u;
        }
        if (lane == 0) warp_sum[warp] = incl;
        if (tid == 0) { bound_digit = kSelBins; sel_above = 0; }   // kSelBins: fewer than brem maxima in play
        __syncthreads();
        uint32_t higher = incl - mine;
        for (int w2 = warp + 1; w2 < WARPS; ++w2) higher += warp_sum[w2];
        if (higher < brem && brem <= higher + mine) {
          uint32_t above = higher;                          // from the thread's highest digit down
#pragma unroll
          for (int j = BPT - 1; j >= 0; --j) {
            if (above < brem && brem <= above + bins[j]) { bound_digit = BPT * tid + j; sel_above = above; }
            above += bins[j];
          }
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < BPT; ++j) hist[1][BPT * tid + j] = 0;
        const uint32_t bd = bound_digit;
        if (bd == kSelBins) {                               // cannot bound (k exceeds the number of maxima): keep all
          if (bp == 0) { bprefix = 0; bmask = 0; }
          __syncthreads();
          break;
        }
        bprefix |= bd << shift;
        bmask |= 2047u << shift;
        brem -= sel_above;
        __syncthreads();                                    // histogram zeroed, bound_digit consumed
      }
      const uint32_t bound = bprefix;                       // lower edge of the resolved digits
      // ---- 2b. candidates (keys >= bound) of every round, in position order, to this CTA's region
      uint32_t filled = 0;
      for (int r = 0; r < rounds; ++r) {
        if (MULTI) pool_round(r);                           // a single round still holds its keys in registers
        uint32_t wc = 0;
#pragma unroll
        for (int it = 0; it < PER_LANE; ++it) {
          const int i = wlo + it * 32 + lane;
          wc += __popc(__ballot_sync(0xffffffffu, i < whi && pk[it] >= bound));
        }
        if (lane == 0) warp_gt[warp] = wc;
        __syncthreads();
        uint32_t base = filled, all_cand = 0;
        for (int w2 = 0; w2 < WARPS; ++w2) {
          if (w2 < warp) base += warp_gt[w2];
          all_cand += warp_gt[w2];
        }
        local_pairs = !MULTI && C == 1 && static_cast<int>(all_cand) <= p.smem_pairs;
        uint2* dst = local_pairs ? reinterpret_cast<uint2*>(sel_smem) : region;   // the raw scores are dead by now
#pragma unroll
        for (int it = 0; it < PER_LANE; ++it) {
          const int i = wlo + it * 32 + lane;
          const bool c = i < whi && pk[it] >= bound;
          const uint32_t bal = __ballot_sync(0xffffffffu, c);
          if (c) dst[base + __popc(bal & lt)] = make_uint2(pk[it], static_cast<uint32_t>(i));
          base += __popc(bal);
        }
        filled += all_cand;
      }
      local_count = static_cast<int>(filled);
      if (tid == 0) counts[rank] = filled;
    } else {
      // a very wide pool: every position is a candidate
      for (int i = lo + tid; i < hi; i += THREADS) region[i - lo] = make_uint2(pooled_key(s, i, P, radius, AVG ? 1 : 0), i);
      if (tid == 0) counts[rank] = hi - lo;
    }
  }
  if (C == 1) __syncthreads(); else cluster.sync();         // every region and its count are written

  if (selecting && rank == 0) {
    // ---- 3. CTA 0: concatenate the regions, radix search, emit
    uint32_t pre[kSelMaxCluster + 1];
    pre[0] = 0;
#pragma unroll
    for (int c = 0; c < kSelMaxCluster; ++c) pre[c + 1] = pre[c] + (c < C ? __ldcg(counts + c) : 0u);
    const int N = local_pairs ? local_count : static_cast<int>(pre[kSelMaxCluster]);
    auto fetch = [&](int j) -> uint2 {                      // pair j of the concatenation, from global memory
      int c = 0;
#pragma unroll
      for (int q = 1; q < kSelMaxCluster; ++q) c += static_cast<uint32_t>(j) >= pre[q] ? 1 : 0;
      return __ldcg(regions + static_cast<int64_t>(c) * slice + (j - static_cast<int>(pre[c])));
    };
    uint2* flat = reinterpret_cast<uint2*>(sel_smem);
    const int held = min(N, p.smem_pairs);
    if (!local_pairs) {
      for (int j = tid; j < held; j += THREADS) flat[j] = fetch(j);
      __syncthreads();
    }
    auto item = [&](int j) -> uint2 { return j < held ? flat[j] : fetch(j); };

    uint32_t prefix = 0, mask = 0, remaining = k;
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
      const uint32_t dmask = pass == 2 ? 1023u : 2047u;
      uint32_t* hcur = hist[pass & 1];
      for (int j0 = warp * 32; j0 < N; j0 += THREADS) {
        const int j = j0 + lane;
        uint32_t digit = kSelBins;                          // kSelBins = does not take part
        if (j < N) {
          const uint32_t key = item(j).x;
          if ((key & mask) == prefix) digit = (key >> shift) & dmask;
        }
        const uint32_t peers = __match_any_sync(0xffffffffu, digit);
        if (digit < kSelBins && lane == __ffs(peers) - 1) atomicAdd(&hcur[digit], __popc(peers));
      }
      __syncthreads();
      uint32_t bins[BPT];                                   // every thread owns BPT adjacent digits
      uint32_t mine = 0;
#pragma unroll
      for (int j = 0; j < BPT; ++j) {
        bins[j] = hcur[BPT * tid + j];
        hist[(pass + 1) & 1][BPT * tid + j] = 0;            // next pass's buffer
        mine += bins[j];
      }
      uint32_t incl = mine;                                 // keys in this and the higher threads of the warp
      for (int off = 1; off < 32; off <<= 1) {
        const uint32_t u = __shfl_down_sync(0xffffffffu, incl, off);
        if (lane + off < 32) incl += u;
      }
      if (lane == 0) warp_sum[warp] = incl;
      __syncthreads();
      uint32_t higher = incl - mine;
      for (int w2 = warp + 1; w2 < WARPS; ++w2) higher += warp_sum[w2];
      if (higher < remaining && remaining <= higher + mine) {  // exactly one thread: the k-th key is in its digits
        uint32_t above = higher;                            // from the thread's highest digit down
#pragma unroll
        for (int j = BPT - 1; j >= 0; --j) {
          if (above < remaining && remaining <= above + bins[j]) { sel_digit = BPT * tid + j; sel_above = above; }
          above += bins[j];
        }
      }
      __syncthreads();
      prefix |= sel_digit << shift;
      mask |= dmask << shift;
      remaining -= sel_above;
      __syncthreads();                                      // sel_* are rewritten next pass
    }
    const uint32_t T = prefix;                              // the k-th largest key
    const uint32_t need_eq = remaining;                     // ties at T to take, from the left

    // keys above / at the threshold, warp by warp over contiguous chunks of the concatenation
    const int chunk = (((N + WARPS - 1) / WARPS) + 31) & ~31;
    const int j_lo = min(N, warp * chunk), j_hi = min(N, j_lo + chunk);
    uint32_t ngt = 0, neq = 0;
    for (int j0 = j_lo; j0 < j_hi; j0 += 32) {
      const int j = j0 + lane;
      const uint32_t key = j < j_hi ? item(j).x : 0u;
      ngt += __popc(__ballot_sync(0xffffffffu, j < j_hi && key > T));
      neq += __popc(__ballot_sync(0xffffffffu, j < j_hi && key == T));
    }
    if (lane == 0) { warp_gt[warp] = ngt; warp_eq[warp] = neq; }
    __syncthreads();
    uint32_t gt_before = 0, eq_before = 0;
    for (int w2 = 0; w2 < warp; ++w2) { gt_before += warp_gt[w2]; eq_before += warp_eq[w2]; }
    if (tid == THREADS - 1) {                           // the last thread can see the grand total
      if (gt_before + ngt + min(eq_before + neq, need_eq) != static_cast<uint32_t>(k))
        atomicOr(p.status, kStatusSelectMismatch);
    }
    // rank of a kept position = (#greater before it) + min(#equal before it, need_eq)
    for (int j0 = j_lo; j0 < j_hi; j0 += 32) {
      const int j = j0 + lane;
      const uint2 kv = j < j_hi ? item(j) : make_uint2(0u, 0u);
      const bool is_gt = j < j_hi && kv.x > T, is_eq = j < j_hi && kv.x == T;
      const uint32_t bg = __ballot_sync(0xffffffffu, is_gt), be = __ballot_sync(0xffffffffu, is_eq);
      const uint32_t g = gt_before + __popc(bg & lt), e = eq_before + __popc(be & lt);
      if (is_gt || (is_eq && e < need_eq)) out[g + min(e, need_eq)] = static_cast<int32_t>(kv.y);
      gt_before += __popc(bg);
      eq_before += __popc(be);
    }
  }
  if (C == 1) __syncthreads(); else cluster.sync();         // the list is complete

  // ---- 5. eviction by gather (appendix on torch.gather), spread over the cluster
  if (p.k_out != nullptr) {
    const char* kb = static_cast<const char*>(p.k.ptr) + (b * p.k.sb + h * p.k.sh) * p.elem_bytes;
    const char* vb = static_cast<const char*>(p.v.ptr) + (b * p.v.sb + h * p.v.sh) * p.elem_bytes;
    const int64_t row0 = p.seq.row_off[b] + static_cast<int64_t>(h) * count;
    const int total = count * p.pieces, stride = C * THREADS;
    if (total >= 8 * stride) {                              // a long list: the batched copy
      gather_listed_rows(out, kb, vb, p.k.st * p.elem_bytes, p.v.st * p.elem_bytes, static_cast<uint4*>(p.k_out),
                         static_cast<uint4*>(p.v_out), row0, total, p.pieces, rank * THREADS + tid, stride);
    } else {
      for (int g = rank * THREADS + tid; g < total; g += stride) {
        const int row = g / p.pieces, piece = g - row * p.pieces;
        const int pos = __ldcg(out + row);                  // written by other CTAs of the cluster: skip L1
        const int64_t dst = (row0 + row) * p.pieces + piece;
        static_cast<uint4*>(p.k_out)[dst] =
            reinterpret_cast<const uint4*>(kb + static_cast<int64_t>(pos) * p.k.st * p.elem_bytes)[piece];
        if (p.v_out)
          static_cast<uint4*>(p.v_out)[dst] =
              reinterpret_cast<const uint4*>(vb + static_cast<int64_t>(pos) * p.v.st * p.elem_bytes)[piece];
      }
    }
  }
}

}  // namespace pkv
