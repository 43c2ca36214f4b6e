// Window scores in ONE sweep over K for short contexts (Section 4.2.2, Eq. 2 and Eq. 3), bf16 or fp16 inputs.
//
// The two-sweep kernels of pkv_score_tc.cuh read K twice because the score of a key needs every window row's
// normaliser, which is known only after the row's last key.  When the logits of a whole (sequence, KV head) fit
// in the tensor memory of a few SMs there is no need for that: a thread-block cluster takes the head, every CTA
// of it keeps the logits of its share of the keys in TMEM, and the row statistics travel between the CTAs
// through distributed shared memory:
//
//   D[key i][row r] = K Q^T          M = 128 keys per tile, N = 32 window rows, one 32-column TMEM slice per tile,
//                                    up to 16 tiles (2048 keys) per CTA, up to 8 CTAs per head
//   statistics   as the tiles arrive: every thread keeps, per row, a running maximum and the sum of 2^(x - max)
//                over its own keys; afterwards lanes -> warps -> CTAs merge these pairs (one cluster barrier)
//   scores       s_i = sum_r 2^(x_ri - lse2_r) from the logits still in TMEM, written for the prefix keys
//
// K is read once, the contraction runs once, and one launch replaces two.  Taken for R = G * alpha <= 32 window
// rows per KV head (multi-head attention with the usual windows) and contexts of at most 8 x 2048 keys; everything
// else goes to the two-sweep kernels.  Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2..5 = epilogue (one per quarter of the TMEM lanes).  Every wait on an mbarrier is bounded as in the
// two-sweep kernels; a CTA that gave up still walks through the two cluster barriers, so its peers are never
// left waiting, and the status word gets kStatusWaitExpired.
#pragma once

#include <cooperative_groups.h>

#include "pkv_score_tc.cuh"

namespace pkv {

constexpr int kRsThreads = 192;
constexpr int kRsRows = 32;                 // window rows (columns of a tile's accumulator)
constexpr int kRsTileKeys = 128;
constexpr int kRsMaxTiles = 512 / kRsRows;  // tiles a CTA keeps in its 512 TMEM columns
constexpr int kRsMaxCluster = 8;
constexpr int kRsStages = 6;                // K tiles in flight per CTA ...
constexpr int kRsStagesShort = 3;           // ... or 3 when a CTA has at most 8 tiles: half the shared memory and (with 256 TMEM
                                            // columns) room for two CTAs per SM, so that two layers' kernels can share the device

template <int D, int STAGES>
struct RsSmem {
  static constexpr int kStageBytes = kRsTileKeys * D * 2;
  static constexpr int kQBytes = kRsRows * D * 2;
  static constexpr int kQOff = 0;
  static constexpr int kKOff = 8192;                          // Q takes at most 8 KB
  static constexpr int kMiscOff = kKOff + STAGES * kStageBytes;
  static constexpr int kMiscBytes = 4096;
  static constexpr int kTotal = kMiscOff + kMiscBytes + 1024;  // + slack for manual 1024-byte alignment
};

__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}

// grid (cluster * H_kv, batch), cluster (cluster, 1, 1), block kRsThreads, dynamic shared memory RsSmem<D, STAGES>::kTotal.
// Uses of TcParams: seq (n, prefix, alpha), num_kv_heads, group, rows (<= 32), fp16, early, scale_log2, log2_group,
// scores, ld_scores, status, wait_clocks.
template <int D, int STAGES>
__global__ void __launch_bounds__(kRsThreads, 1)
score_resident_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                      const TcParams p) {
  namespace cg = cooperative_groups;
  using L = RsSmem<D, STAGES>;
  constexpr int kHalves = D / 64;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem + L::kQOff;
  uint8_t* k_s = smem + L::kKOff;
  uint8_t* misc = smem + L::kMiscOff;
  uint64_t* bars = reinterpret_cast<uint64_t*>(misc);          // [0..5] k_full, [6..11] k_empty, [12] q_full, [13..28] t_full
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 260);
  float2* warp_stat = reinterpret_cast<float2*>(misc + 512);   // [4 epilogue warps][32 rows] (maximum, sum)
  float2* cta_stat = reinterpret_cast<float2*>(misc + 1536);   // [32]: read by the other CTAs of the cluster

  cg::cluster_group cluster = cg::this_cluster();
  const int C = cluster.dim_blocks().x;
  const int rank = cluster.block_rank();
  const int h = blockIdx.x / C, b = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar0 = smem_u32(bars);
  auto k_full = [&](int s) { return bar0 + 8u * s; };
  auto k_empty = [&](int s) { return bar0 + 8u * (STAGES + s); };
  const uint32_t q_full = bar0 + 8u * (2 * STAGES);
  auto t_full = [&](int t) { return bar0 + 8u * (2 * STAGES + 1 + t); };

  // this CTA's tiles of the sequence: tiles_per consecutive ones from rank * tiles_per on
  const int n = p.seq.n[b], alpha = p.seq.alpha, P = p.seq.prefix[b];
  const int ntiles = (n + kRsTileKeys - 1) / kRsTileKeys;
  const int tiles_per = (ntiles + C - 1) / C;                  // <= kRsMaxTiles (the host checks)
  const int tile0 = min(ntiles, rank * tiles_per), tile1 = min(ntiles, tile0 + tiles_per);
  const int T = tile1 - tile0;
  // TMEM columns: 32 per tile, a power of two; CTAs that need 256 or fewer leave room for a second CTA on the SM
  uint32_t tmem_cols = 32;
  while (tmem_cols < static_cast<uint32_t>(tiles_per * kRsRows)) tmem_cols <<= 1;

  // ---- set-up (shared memory and TMEM only: it may overlap the tail of the preceding kernel)
  pdl_trigger();
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(k_full(s), 1); mbar_init(k_empty(s), 1); }
    mbar_init(q_full, 1);
    for (int t = 0; t < kRsMaxTiles; ++t) mbar_init(t_full(t), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // rows of the Q tile beyond R stay zero (TMA only ever writes R rows)
  for (int i = threadIdx.x; i < L::kQBytes / 16; i += kRsThreads) reinterpret_cast<uint4*>(q_s)[i] = make_uint4(0, 0, 0, 0);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (!p.early) pdl_wait();

  if (warp == 0) {
    // =========================================================== TMA producer
    if (lane == 0 && T > 0) {
      mbar_expect_tx(q_full, static_cast<uint32_t>(p.rows) * D * 2);
      for (int half = 0; half < kHalves; ++half)
        tma_load_4d(smem_u32(q_s) + half * kRsRows * 128, &q_map, q_full, half * 64, 0, h * p.group, b);
      bool ok = true;
      int issued = 0;
      for (int t = 0; t < T && ok; ++t) {
        const int s = t % STAGES;
        ok = mbar_wait(k_empty(s), ((t / STAGES) & 1) ^ 1, abort_flag, p.wait_clocks);
        if (!ok) break;
        mbar_expect_tx(k_full(s), L::kStageBytes);
        for (int half = 0; half < kHalves; ++half)
          tma_load_4d(smem_u32(k_s) + s * L::kStageBytes + half * kRsTileKeys * 128, &k_map, k_full(s), half * 64,
                      (tile0 + t) * kRsTileKeys, h, b);
        issued = t + 1;
      }
      if (!ok) {
        // drain: wait (bounded) for the copies still in flight before shared memory is given up
        for (int j = max(0, issued - STAGES); j < issued; ++j)
          for (uint32_t spin = 0; spin < (1u << 16) && !mbar_test(k_full(j % STAGES), (j / STAGES) & 1); ++spin)
            __nanosleep(64);
        for (uint32_t spin = 0; spin < (1u << 16) && !mbar_test(q_full, 0); ++spin) __nanosleep(64);
      }
    }
  } else if (warp == 1) {
    // =========================================================== MMA issuer
    if (lane == 0 && T > 0) {
      const uint32_t idesc = instr_desc_16bit(kRsTileKeys, kRsRows, p.fp16);
      bool ok = mbar_wait(q_full, 0, abort_flag, p.wait_clocks);
      for (int t = 0; t < T && ok; ++t) {
        const int s = t % STAGES;
        ok = mbar_wait(k_full(s), (t / STAGES) & 1, abort_flag, p.wait_clocks);
        if (!ok) break;
        tc_fence_after();
        const uint32_t k_addr = smem_u32(k_s) + s * L::kStageBytes, q_addr = smem_u32(q_s);
        const uint32_t d_addr = tmem_base + t * kRsRows;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t ka = k_addr + (kk / 4) * kRsTileKeys * 128 + (kk % 4) * 32;
          const uint32_t qa = q_addr + (kk / 4) * kRsRows * 128 + (kk % 4) * 32;
          tc_mma_f16kind(d_addr, smem_desc_sw128(ka), smem_desc_sw128(qa), idesc, kk > 0);
        }
        tc_commit(k_empty(s));
        tc_commit(t_full(t));                                 // arrives when this tile's logits are in TMEM
      }
    }
  }

  // =========================================================== epilogue (warps 2..5), in step with the cluster
  const bool epi = warp >= 2;
  const int quarter = warp & 3;                               // TMEM lanes 32 * quarter .. + 31 are this warp's
  const int lane_row = quarter * 32 + lane;
  const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
  const float c2 = p.scale_log2;
  bool ok = true;
  // a tile that ends inside the prefix is seen whole by every row: no mask to evaluate (all but the last one or two)
  auto whole = [&](int t) -> bool { return (tile0 + t + 1) * kRsTileKeys <= P; };
  // (maximum, sum) pairs merge like this; -inf marks "nothing yet"
  auto merge = [](float& m, float& z, float m2, float z2) {
    const float mn = fmaxf(m, m2);
    z = (m > -INFINITY ? z * ex2(m - mn) : 0.f) + (m2 > -INFINITY ? z2 * ex2(m2 - mn) : 0.f);
    m = mn;
  };

  // ---- statistics, tile by tile as the MMAs complete: per thread and row a running maximum and the sum of
  //      2^(x - maximum) over the thread's own keys (x = logit in log2 units; a row (g, jj) sees keys 0 .. P + jj)
  float lse2 = 0.f;                                            // of row `lane`, after the cluster barrier
  if (epi) {
    float m[kRsRows], z[kRsRows];
#pragma unroll
    for (int j = 0; j < kRsRows; ++j) { m[j] = -INFINITY; z[j] = 0.f; }
    for (int t = 0; t < T && ok; ++t) {
      ok = mbar_wait(t_full(t), 0, abort_flag, p.wait_clocks);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t v[32];
      tc_ld32(lane_addr + t * kRsRows, v);
      tc_wait_ld();
      if (whole(t)) {
#pragma unroll
        for (int j = 0; j < kRsRows; ++j) {
          const float x = __uint_as_float(v[j]) * c2, mn = fmaxf(m[j], x);
          z[j] = z[j] * ex2(m[j] - mn) + ex2(x - mn);          // m = -inf the first time: 0 * 0 + 1
          m[j] = mn;
        }
      } else {
        const int i = (tile0 + t) * kRsTileKeys + lane_row;
#pragma unroll
        for (int j = 0; j < kRsRows; ++j)
          if (i <= min(P + (j % alpha), n - 1)) {
            const float x = __uint_as_float(v[j]) * c2, mn = fmaxf(m[j], x);
            z[j] = z[j] * ex2(m[j] - mn) + ex2(x - mn);
            m[j] = mn;
          }
      }
    }
    // lanes, then the four warps, then (behind the cluster barrier) the CTAs
#pragma unroll
    for (int j = 0; j < kRsRows; ++j)
      for (int o = 16; o > 0; o >>= 1)
        merge(m[j], z[j], __shfl_xor_sync(0xffffffffu, m[j], o), __shfl_xor_sync(0xffffffffu, z[j], o));
    float2 mine = make_float2(-INFINITY, 0.f);
#pragma unroll
    for (int j = 0; j < kRsRows; ++j)
      if (lane == j) mine = make_float2(m[j], z[j]);
    warp_stat[(warp - 2) * kRsRows + lane] = mine;
    asm volatile("bar.sync 1, 128;" ::: "memory");             // the four epilogue warps
    if (warp == 2) {
      float2 r = warp_stat[lane];
#pragma unroll
      for (int w2 = 1; w2 < 4; ++w2) merge(r.x, r.y, warp_stat[w2 * kRsRows + lane].x, warp_stat[w2 * kRsRows + lane].y);
      cta_stat[lane] = r;
    }
  }
  cluster.sync();                                              // barrier 1: every CTA's row statistics are in place
  if (epi) {
    float rm = -INFINITY, rz = 0.f;
    for (int c = 0; c < C; ++c) {                              // the same order in every CTA
      const float2 o = cluster.map_shared_rank(cta_stat, c)[lane];
      merge(rm, rz, o.x, o.y);
    }
    lse2 = rm + __log2f(rz) + p.log2_group;
  }

  // ---- scores of the prefix keys, from the logits still in TMEM (loads double buffered)
  if (epi) {
    pdl_wait();                                                // the score buffer may still be read by the call before
    float nl[kRsRows];
#pragma unroll
    for (int j = 0; j < kRsRows; ++j) {
      const float l = __shfl_sync(0xffffffffu, lse2, j);
      nl[j] = j < p.rows ? -l : -INFINITY;
    }
    float* srow = p.scores + (static_cast<int64_t>(b) * p.num_kv_heads + h) * p.ld_scores;
    auto score_tile = [&](int t, const uint32_t (&v)[32]) {
      float s0 = 0.f, s1 = 0.f;
#pragma unroll
      for (int j = 0; j < kRsRows; j += 2) {                   // a prefix key is seen by every row: no mask
        s0 += ex2(fmaf(__uint_as_float(v[j]), c2, nl[j]));
        s1 += ex2(fmaf(__uint_as_float(v[j + 1]), c2, nl[j + 1]));
      }
      const int i = (tile0 + t) * kRsTileKeys + lane_row;
      if (i < P) srow[i] = s0 + s1;
    };
    if (ok && T > 0) {
      uint32_t va[32], vb[32];
      tc_ld32(lane_addr, va);
      for (int t = 0; t < T; t += 2) {
        tc_wait_ld();
        if (t + 1 < T) tc_ld32(lane_addr + (t + 1) * kRsRows, vb);
        score_tile(t, va);
        if (t + 1 < T) {
          tc_wait_ld();
          if (t + 2 < T) tc_ld32(lane_addr + (t + 2) * kRsRows, va);
          score_tile(t + 1, vb);
        }
      }
    }
  }
  cluster.sync();                                              // barrier 2: nobody reads this CTA's shared memory any more

  // ---- teardown
  pdl_wait();                                                  // never finish before the kernels ahead in the stream
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, kStatusWaitExpired);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

}  // namespace pkv
