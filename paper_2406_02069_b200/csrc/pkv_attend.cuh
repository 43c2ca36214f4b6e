// The window rows' attention and the window scores from one pass over K and V (Section 4.1 and
// Section 4.2.2, Eq. 2 and Eq. 3): the scores of Eq. 3 are column sums of the very attention matrix
// whose rows, multiplied by V, are what the prefill attention returns for the last alpha queries.
// This kernel is that attention for those rows (all query heads of a KV head at once) and emits the
// scores from inside it:
//
//   S[key i][row r]   = K Q^T                       tcgen05.mma, TMEM lane = key   (as the score sweep)
//   e_ri              = 2^(x_ri - lse2_r + 15)      x = S * log2(e) / sqrt(d); lse2 = the row's final
//                                                   normaliser (from the row-statistics sweep) + log2 G
//   score_i           = 2^-15 * sum_r e_ri          Eq. 3 (mean over the group's query heads)
//   O^T[c][row r]    += sum_i V[i][c] * e_ri        tcgen05.mma, A = V tile (d-major), B = e rounded to the
//                                                   inputs' 16-bit type in shared memory (row-major per key)
//   out[r][c]         = G * 2^-15 * O^T[c][r]       summed over the CTAs that share a head (reduce kernel)
//
// The normalisers are final before the pass starts, so the accumulators are never rescaled.  The factor
// 2^15 keeps binary16 probabilities of long contexts out of the subnormal range; it is exact.
//
// Warp roles: 0 = TMA producer of Q and K, 1 = MMA issuer and TMEM owner, 2 = TMA producer of V,
// 4..19 = epilogue in four groups of four warps (TMEM lane quarter = warp % 4), all on the same K tile.
// Per tile the issuer queues ONE product K Q^T over all window rows (N up to 256: an MMA costs the issuing
// thread about 100 clocks whatever its width, so few wide ones) into the single 256-column S stage; the
// epilogue takes the rows in halves of (up to) 128: it loads a half's logits into registers, and once the last
// half is loaded gives the S stage back, so the next tile's K Q^T runs beside the exponentials; each half's e
// values go to their own P buffer and V^T P of a half is queued when the buffer is full, behind the next tile's
// K Q^T.
// TMEM: columns 0..255 the S stage, 256..511 O^T (lane = channel c, column = window row).
// Shared memory: Q 64 KB, one K tile, two V tiles, two P buffers of 32 KB each (128 keys x 128 rows).
//
// Every wait on an mbarrier is bounded, as in the score sweeps: a wait that runs out sets the abort
// flag, all roles leave their loops, copies in flight are drained, TMEM is released.
#pragma once

#include "pkv_score_tc.cuh"

namespace pkv {

constexpr int kAtThreads = 640;
constexpr int kAtEpiWarp0 = 4;
constexpr int kAtEpiWarps = 16;
constexpr int kAtTileKeys = 128;
constexpr int kAtD = 128;                // head dimension this kernel is built for
constexpr int kAtVStages = 2;            // V tiles in shared memory (one K tile: it is free again as soon as K Q^T ran)
constexpr int kAtShift = 15;             // e values carry a factor 2^15
constexpr int kAtTileBytes = kAtTileKeys * kAtD * 2;        // a K or V tile, or one P buffer (128 keys x 128 rows)
constexpr int kAtQOff = 0;
constexpr int kAtQBytes = kTcMaxRows * kAtD * 2;
constexpr int kAtKOff = kAtQOff + kAtQBytes;
constexpr int kAtVOff = kAtKOff + kAtTileBytes;
constexpr int kAtPOff = kAtVOff + kAtVStages * kAtTileBytes;
constexpr int kAtMiscOff = kAtPOff + 2 * kAtTileBytes;
constexpr int kAtMiscBytes = 3072;       // barriers 0.., TMEM slot 256, abort flag 260, exchange 512.., -lse2 2048..
constexpr int kAtSmemBytes = kAtMiscOff + kAtMiscBytes;     // 227 KB: all a CTA can have
static_assert(kAtSmemBytes <= 232448, "shared memory of the window-attention kernel");

struct AtParams {
  SeqTable seq;                 // score_off counts this kernel's work items: chunks of chunk_tiles tiles over ALL n keys
  int32_t num_kv_heads, group, rows, rows_pad, fp16;
  int32_t chunk_tiles;
  int32_t withhold;             // test aid: CTA 0 never loads its last K tile (its waits then run out)
  long long wait_clocks;
  float scale_log2;             // log2(e) / sqrt(d)
  const float* lse2;            // [batch][H_kv][R]: log2 of the row's sum of 2^x, plus log2 G
  float* scores;                // [batch][H_kv][ld]: the prefix positions are written
  int64_t ld_scores;
  float* o_partial;             // [segment][R][d]: a segment is one CTA's run over one (sequence, head)
  float* out;                   // reduce kernel: [batch][H_q][alpha][d]
  int32_t grid;                 // CTAs the attention kernel runs with (the reduce kernel finds a head's segments from it)
  uint32_t* status;
};

// The MMA issuer is one thread and this kernel issues 24 MMAs per K tile, so the descriptors are split into their
// 32-bit halves: the high half (strides, version, swizzle) is a constant, the low half (start address and leading
// offset) is formed once per product and advanced by a compile-time constant per MMA.  (Measured: an MMA still takes
// the issuer about 100 clocks at N = 128 and 90 at N = 256, whatever it costs in instructions; hence few, wide MMAs.)
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // stride 1024 B, version 1, 128-byte swizzle
__device__ __forceinline__ uint32_t desc_lo_k_major(uint32_t addr) { return ((addr & 0x3FFFFu) >> 4) | (1u << 16); }
__device__ __forceinline__ uint32_t desc_lo_mn_major(uint32_t addr, uint32_t block_bytes) {
  return ((addr & 0x3FFFFu) >> 4) | ((block_bytes >> 4) << 16);
}
template <bool ACC>
__device__ __forceinline__ void tc_mma_halves(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(kDescHi), "r"(idesc), "n"(ACC ? 1 : 0)
      : "memory");
}

__device__ __forceinline__ uint32_t pack_16bit(float lo, float hi, int fp16) {
  if (fp16) {
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
  }
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// 16 window rows of one key, all visible: e = 2^(v * c2 + nl), summed into acc (a packed pair of partial sums)
// and rounded to 16 bits into two 16-byte chunks (c0, c0 + 1, swizzled by sw) of the key's line of the P buffer.
template <bool FP16>
__device__ __forceinline__ void at_chunk(const uint32_t (&v)[16], unsigned long long cc, const float* nl, uint8_t* blk,
                                         int c0, int sw, unsigned long long& acc) {
  uint32_t pk[8];
#pragma unroll
  for (int j = 0; j < 8; j += 2) {
    const ulonglong2 l = *reinterpret_cast<const ulonglong2*>(nl + 2 * j);   // four floats as two packed pairs
    float x0, x1, x2, x3;
    unpack2(fma2(pack2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])), cc, l.x), x0, x1);
    unpack2(fma2(pack2(__uint_as_float(v[2 * j + 2]), __uint_as_float(v[2 * j + 3])), cc, l.y), x2, x3);
    const float e0 = ex2(x0), e1 = ex2(x1), e2 = ex2(x2), e3 = ex2(x3);
    acc = add2(acc, add2(pack2(e0, e1), pack2(e2, e3)));
    pk[j] = pack_16bit(e0, e1, FP16 ? 1 : 0);
    pk[j + 1] = pack_16bit(e2, e3, FP16 ? 1 : 0);
  }
  *reinterpret_cast<uint4*>(blk + ((c0 ^ sw) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
  *reinterpret_cast<uint4*>(blk + (((c0 + 1) ^ sw) << 4)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
}

__global__ void __launch_bounds__(kAtThreads, 1)
window_attend_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                     const __grid_constant__ CUtensorMap v_map, const AtParams p) {
  extern __shared__ __align__(1024) uint8_t at_smem[];
  uint8_t* smem = at_smem;
  pdl_trigger();
  if (smem_u32(smem) & 1023u) {                                // the carve-up below needs this; never seen otherwise
    if (threadIdx.x == 0) atomicOr(p.status, kStatusWaitExpired);
    return;
  }
  uint8_t* q_s = smem + kAtQOff;
  uint8_t* k_s = smem + kAtKOff;
  uint8_t* v_s = smem + kAtVOff;
  uint8_t* p_s = smem + kAtPOff;
  uint8_t* misc = smem + kAtMiscOff;
  uint64_t* bars = reinterpret_cast<uint64_t*>(misc);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 260);
  float* xch = reinterpret_cast<float*>(misc + 512);           // [3][128] partial score sums handed between groups
  float* lse_all = reinterpret_cast<float*>(misc + 2048);      // [256] shifted -lse2 of the current head

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar0 = smem_u32(bars);
  const uint32_t k_full = bar0, k_empty = bar0 + 8u;
  auto v_full = [&](int s) { return bar0 + 8u * (2 + s); };
  auto v_empty = [&](int s) { return bar0 + 8u * (4 + s); };
  const uint32_t s_full = bar0 + 8u * 6, s_empty = bar0 + 8u * 7;
  auto p_full = [&](int s) { return bar0 + 8u * (8 + s); };
  auto p_empty = [&](int s) { return bar0 + 8u * (10 + s); };
  const uint32_t q_full = bar0 + 8u * 12, q_empty = bar0 + 8u * 13;
  const uint32_t o_full = bar0 + 8u * 14, o_empty = bar0 + 8u * 15;
  const uint32_t x_full = bar0 + 8u * 16, x_empty = bar0 + 8u * 17;
  const uint32_t lse_full = bar0 + 8u * 18;

  const int halves = p.rows_pad > 128 ? 2 : 1;                 // row halves the epilogue takes a tile in
  const int n_half = halves == 2 ? 128 : p.rows_pad;           // window rows (columns) of one half
  const int n_pv = n_half < 64 ? 64 : n_half;                  // ... and of its P x V product (whole 64-row blocks)

  if (threadIdx.x == 0) {
    mbar_init(k_full, 1); mbar_init(k_empty, 1);
    mbar_init(s_full, 1); mbar_init(s_empty, kAtEpiWarps);
    for (int s = 0; s < 2; ++s) {
      mbar_init(v_full(s), 1); mbar_init(v_empty(s), 1);
      mbar_init(p_full(s), kAtEpiWarps); mbar_init(p_empty(s), 1);
    }
    mbar_init(q_full, 1); mbar_init(q_empty, 1);
    mbar_init(o_full, 1); mbar_init(o_empty, kAtEpiWarps);
    mbar_init(x_full, 12); mbar_init(x_empty, 4);
    mbar_init(lse_full, kAtEpiWarps);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Q rows beyond R and P rows beyond a half's width stay zero for the whole kernel
  for (int i = threadIdx.x; i < kAtQBytes / 16; i += kAtThreads) reinterpret_cast<uint4*>(q_s)[i] = make_uint4(0, 0, 0, 0);
  for (int i = threadIdx.x; i < 2 * kAtTileBytes / 16; i += kAtThreads) reinterpret_cast<uint4*>(p_s)[i] = make_uint4(0, 0, 0, 0);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                                                  // the normalisers come from the kernels before

  const int32_t* off = p.seq.score_off;
  const int total = p.num_kv_heads * off[p.seq.batch];
  const int per = total / gridDim.x, rem = total % gridDim.x;
  const int item0 = blockIdx.x * per + min(static_cast<int>(blockIdx.x), rem);
  const int item1 = item0 + per + (static_cast<int>(blockIdx.x) < rem ? 1 : 0);
  auto tiles_of = [&](const TcItem& w, int& tile0, int& tile1) {
    tile0 = w.c * p.chunk_tiles;
    tile1 = min(tile0 + p.chunk_tiles, (p.seq.n[w.b] + kAtTileKeys - 1) / kAtTileKeys);
  };

  if (warp == 0) {
    // =========================================================== TMA producer: Q per head, K per tile
    if (lane == 0) {
      uint32_t it = 0, heads_loaded = 0;
      int cur_b = -1, cur_h = -1;
      bool ok = true;
      for (int id = item0; id < item1 && ok; ++id) {
        const TcItem w = tc_item(off, p.seq.batch, p.num_kv_heads, id);
        if (w.b != cur_b || w.h != cur_h) {
          if (heads_loaded > 0) ok = mbar_wait(q_empty, (heads_loaded - 1) & 1, abort_flag, p.wait_clocks);
          if (!ok) break;
          mbar_expect_tx(q_full, static_cast<uint32_t>(p.rows) * kAtD * 2);
          for (int half = 0; half < 2; ++half)
            tma_load_4d(smem_u32(q_s) + half * kTcMaxRows * 128, &q_map, q_full, half * 64, 0, w.h * p.group, w.b);
          ++heads_loaded;
          cur_b = w.b; cur_h = w.h;
        }
        int tile0, tile1;
        tiles_of(w, tile0, tile1);
        for (int t = tile0; t < tile1 && ok; ++t, ++it) {
          ok = mbar_wait(k_empty, (it & 1) ^ 1, abort_flag, p.wait_clocks);
          if (!ok) break;
          if (p.withhold && blockIdx.x == 0 && id + 1 == item1 && t + 1 == tile1) continue;   // test aid: never arrives
          mbar_expect_tx(k_full, kAtTileBytes);
          for (int half = 0; half < 2; ++half)
            tma_load_4d(smem_u32(k_s) + half * kAtTileKeys * 128, &k_map, k_full, half * 64, t * kAtTileKeys, w.h, w.b);
        }
      }
      if (!ok) {
        if (it > 0)
          for (uint32_t spin = 0; spin < (1u << 16) && !mbar_test(k_full, (it - 1) & 1); ++spin) __nanosleep(64);
        if (heads_loaded > 0)
          for (uint32_t spin = 0; spin < (1u << 16) && !mbar_test(q_full, (heads_loaded - 1) & 1); ++spin) __nanosleep(64);
      }
    }
  } else if (warp == 2) {
    // =========================================================== TMA producer: V per tile
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int id = item0; id < item1 && ok; ++id) {
        const TcItem w = tc_item(off, p.seq.batch, p.num_kv_heads, id);
        int tile0, tile1;
        tiles_of(w, tile0, tile1);
        for (int t = tile0; t < tile1 && ok; ++t, ++it) {
          const int s = it & 1;
          ok = mbar_wait(v_empty(s), ((it >> 1) & 1) ^ 1, abort_flag, p.wait_clocks);
          if (!ok) break;
          mbar_expect_tx(v_full(s), kAtTileBytes);
          for (int half = 0; half < 2; ++half)
            tma_load_4d(smem_u32(v_s) + s * kAtTileBytes + half * kAtTileKeys * 128, &v_map, v_full(s), half * 64,
                        t * kAtTileKeys, w.h, w.b);
        }
      }
      if (!ok) {
        const uint32_t first = it > 2 ? it - 2 : 0;
        for (uint32_t j = first; j < it; ++j)
          for (uint32_t spin = 0; spin < (1u << 16) && !mbar_test(v_full(j & 1), (j >> 1) & 1); ++spin) __nanosleep(64);
      }
    }
  } else if (warp == 1) {
    // =========================================================== MMA issuer
    if (lane == 0) {
      // all window rows at once; with two halves always 256 columns, so that the second half holds zeros (Q rows
      // beyond R are zero) rather than what the stage held before
      const uint32_t idesc_s = instr_desc_16bit(kAtTileKeys, halves == 2 ? 256 : p.rows_pad, p.fp16);
      const uint32_t idesc_pv = instr_desc_16bit(kAtD, n_pv, p.fp16) | (1u << 15) | (1u << 16);   // A and B M/N-major
      uint32_t it = 0, heads_seen = 0, runs = 0;
      int cur_b = -1, cur_h = -1;
      bool ok = true, fresh = true, wait_o = false, pend = false;   // pend: the products V^T P of tile it - 1 are still to be queued
      // V^T P of both row halves of tile j, each as soon as its P buffer is full
      auto issue_pv = [&](uint32_t j) -> bool {
        const int vs = j & 1;
        if (!mbar_wait(v_full(vs), (j >> 1) & 1, abort_flag, p.wait_clocks)) return false;
        if (wait_o) {                                          // the epilogue has read the accumulators of the run before
          if (!mbar_wait(o_empty, (runs - 1) & 1, abort_flag, p.wait_clocks)) return false;
          wait_o = false;
        }
        const uint32_t v_lo = desc_lo_mn_major(smem_u32(v_s) + vs * kAtTileBytes, kAtTileKeys * 128);
        for (int hf = 0; hf < halves; ++hf) {
          if (!mbar_wait(p_full(hf), j & 1, abort_flag, p.wait_clocks)) return false;
          tc_fence_after();
          const uint32_t d_addr = tmem_base + 256 + hf * 128;
          const uint32_t p_lo = desc_lo_mn_major(smem_u32(p_s) + hf * kAtTileBytes, kAtTileKeys * 128);
          if (fresh) tc_mma_halves<false>(d_addr, v_lo, p_lo, idesc_pv);
          else tc_mma_halves<true>(d_addr, v_lo, p_lo, idesc_pv);
#pragma unroll
          for (int kk = 1; kk < kAtTileKeys / 16; ++kk)        // 16 keys further: 2048 bytes in both operands
            tc_mma_halves<true>(d_addr, v_lo + kk * (2048 >> 4), p_lo + kk * (2048 >> 4), idesc_pv);
          tc_commit(p_empty(hf));
        }
        fresh = false;
        tc_commit(v_empty(vs));
        return true;
      };
      auto end_run = [&]() -> bool {
        if (pend && !issue_pv(it - 1)) return false;
        pend = false;
        tc_commit(o_full);
        ++runs;
        wait_o = true;
        fresh = true;
        return true;
      };
      for (int id = item0; id < item1 && ok; ++id) {
        const TcItem w = tc_item(off, p.seq.batch, p.num_kv_heads, id);
        if (w.b != cur_b || w.h != cur_h) {
          if (cur_b >= 0) ok = end_run();
          if (!ok) break;
          ok = mbar_wait(q_full, heads_seen & 1, abort_flag, p.wait_clocks);
          if (!ok) break;
          ++heads_seen;
          cur_b = w.b; cur_h = w.h;
        }
        bool last_of_head = id + 1 >= item1;
        if (!last_of_head) {
          const TcItem nx = tc_item(off, p.seq.batch, p.num_kv_heads, id + 1);
          last_of_head = nx.b != w.b || nx.h != w.h;
        }
        int tile0, tile1;
        tiles_of(w, tile0, tile1);
        for (int t = tile0; t < tile1 && ok; ++t, ++it) {
          ok = mbar_wait(k_full, it & 1, abort_flag, p.wait_clocks);
          if (!ok) break;
          ok = mbar_wait(s_empty, (it & 1) ^ 1, abort_flag, p.wait_clocks);   // the tile before is in registers
          if (!ok) break;
          tc_fence_after();
          const uint32_t k_lo = desc_lo_k_major(smem_u32(k_s)), q_lo = desc_lo_k_major(smem_u32(q_s));
          tc_mma_halves<false>(tmem_base, k_lo, q_lo, idesc_s);
#pragma unroll
          for (int kk = 1; kk < kAtD / 16; ++kk) {             // 16 channels further: 32 bytes, the next 64-channel block
            constexpr int kBlock = kAtTileKeys * 128 >> 4, kQBlock = kTcMaxRows * 128 >> 4;        // after four steps
            tc_mma_halves<true>(tmem_base, k_lo + (kk / 4) * kBlock + (kk % 4) * 2, q_lo + (kk / 4) * kQBlock + (kk % 4) * 2,
                                idesc_s);
          }
          tc_commit(s_full);
          tc_commit(k_empty);
          // the products of the tile before come behind this tile's logits in the queue: the logits are what the
          // epilogue waits for next
          if (pend) ok = issue_pv(it - 1);
          pend = true;
        }
        if (ok && last_of_head) tc_commit(q_empty);
      }
      if (ok && cur_b >= 0) end_run();
    }
  } else if (warp >= kAtEpiWarp0) {
    // =========================================================== epilogue
    // Sixteen warps, all on the same tile.  A half's 16-column pieces are dealt round to the four groups (a group
    // = the four warps that cover the 128 TMEM lanes).  A thread carries its key's partial score sum through the
    // halves; group 0 then collects the other groups' sums and writes the score.
    const int e = warp - kAtEpiWarp0;
    const int quarter = warp & 3, g4 = e >> 2;
    const int lane_row = quarter * 32 + lane;                  // TMEM lane: key of a tile in S, channel in O^T
    const uint32_t lanes = static_cast<uint32_t>(quarter * 32) << 16;
    const float c2 = p.scale_log2;
    const float unshift = 1.0f / static_cast<float>(1 << kAtShift);
    const int cg_a = g4 * 16, cg_b = cg_a + 64;                // this group's pieces of a half
    const bool has_a = cg_a < n_half, has_b = cg_b < n_half;
    uint32_t it = 0, lse_rounds = 0, runs = 0;
    int cur_b = -1, cur_h = -1;
    bool ok = true;
    // Hands the accumulators of the run that ends to global memory (raw: the reduce kernel scales).
    auto flush_o = [&]() -> bool {
      bool good = mbar_wait(o_full, runs & 1, abort_flag, p.wait_clocks);
      good = __all_sync(0xffffffffu, good);
      if (!good) return false;
      tc_fence_after();
      const int ncols = halves == 2 ? 256 : n_pv;
      const int64_t seg = static_cast<int64_t>(blockIdx.x) + cur_b * p.num_kv_heads + cur_h;
      float* dst = p.o_partial + seg * p.rows * kAtD + lane_row;
      for (int cg = g4 * 16; cg < ncols; cg += 64) {           // 16-column pieces dealt round to the four groups
        uint32_t v[16];
        tc_ld16(tmem_base + lanes + 256 + cg, v);
        tc_wait_ld();
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (cg + j < p.rows) dst[static_cast<int64_t>(cg + j) * kAtD] = __uint_as_float(v[j]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(o_empty);
      ++runs;
      return true;
    };
    // One meeting of the sixteen warps.
    auto meet = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(lse_full);
      bool good = mbar_wait(lse_full, lse_rounds & 1u, abort_flag, p.wait_clocks);
      ++lse_rounds;
      return __all_sync(0xffffffffu, good);
    };
    for (int id = item0; id < item1 && ok; ++id) {
      const TcItem w = tc_item(off, p.seq.batch, p.num_kv_heads, id);
      const int n = p.seq.n[w.b], alpha = p.seq.alpha, P = p.seq.prefix[w.b];
      if (w.b != cur_b || w.h != cur_h) {
        if (cur_b >= 0) ok = flush_o();
        if (!ok) break;
        // the head's normalisers, negated and shifted: written once everybody is done with the old ones, read
        // once everybody has written
        ok = meet();
        if (!ok) break;
        const int r = e * 32 + lane;
        if (r < kTcMaxRows) {
          const float* src = p.lse2 + (static_cast<int64_t>(w.b) * p.num_kv_heads + w.h) * p.rows;
          lse_all[r] = r < p.rows ? static_cast<float>(kAtShift) - src[r] : -INFINITY;
        }
        ok = meet();
        if (!ok) break;
        cur_b = w.b; cur_h = w.h;
      }
      float* srow = p.scores + (static_cast<int64_t>(w.b) * p.num_kv_heads + w.h) * p.ld_scores;
      int tile0, tile1;
      tiles_of(w, tile0, tile1);
      for (int t = tile0; t < tile1 && ok; ++t, ++it) {
        const int i = t * kAtTileKeys + lane_row;
        const bool in_seq = i < n;
        const int jp = i - P;                                  // window key P + jp is seen by rows j >= jp
        const bool plain = __all_sync(0xffffffffu, in_seq && jp <= 0);   // no mask anywhere in this warp's keys
        ok = mbar_wait(s_full, it & 1, abort_flag, p.wait_clocks);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        float sum = 0.f;
        for (int hf = 0; hf < halves && ok; ++hf) {
          const uint32_t taddr = tmem_base + lanes + hf * 128;
          uint32_t va[16], vb[16];
          if (has_a) tc_ld16(taddr + cg_a, va);
          if (has_b) tc_ld16(taddr + cg_b, vb);
          tc_wait_ld();
          if (hf == halves - 1) {                              // this tile's logits are in registers: the stage is free
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(s_empty);
          }
          ok = mbar_wait(p_empty(hf), (it & 1) ^ 1, abort_flag, p.wait_clocks);   // V^T P of the tile before has read the buffer
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          uint8_t* prow = p_s + hf * kAtTileBytes + lane_row * 128;
          const float* nlr = lse_all + hf * 128;
          if (plain) {
            unsigned long long acc = pack2(0.f, 0.f);
            const unsigned long long cc = pack2(c2, c2);
            const int sw = lane_row & 7;
            if (has_a) {
              if (p.fp16) at_chunk<true>(va, cc, nlr + cg_a, prow, cg_a >> 3, sw, acc);
              else at_chunk<false>(va, cc, nlr + cg_a, prow, cg_a >> 3, sw, acc);
            }
            if (has_b) {
              if (p.fp16) at_chunk<true>(vb, cc, nlr + cg_b, prow + kAtTileKeys * 128, (cg_b & 63) >> 3, sw, acc);
              else at_chunk<false>(vb, cc, nlr + cg_b, prow + kAtTileKeys * 128, (cg_b & 63) >> 3, sw, acc);
            }
            float lo, hi;
            unpack2(acc, lo, hi);
            sum += lo + hi;
          } else {
#pragma unroll
            for (int piece = 0; piece < 2; ++piece) {
              if (piece == 0 ? !has_a : !has_b) continue;
              const int cg = piece == 0 ? cg_a : cg_b;
              const uint32_t (&v)[16] = piece == 0 ? va : vb;
              float ev[16];
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                const float x = ex2(fmaf(__uint_as_float(v[j]), c2, nlr[cg + j]));
                const bool vis = in_seq && (jp <= 0 || (hf * 128 + cg + j) % alpha >= jp);
                ev[j] = vis ? x : 0.f;
              }
              uint32_t pk[8];
#pragma unroll
              for (int j = 0; j < 16; j += 2) {
                sum += ev[j] + ev[j + 1];
                pk[j >> 1] = pack_16bit(ev[j], ev[j + 1], p.fp16);
              }
              const int nb = cg >> 6, c0 = (cg & 63) >> 3;     // 64-row block and first 16-byte chunk inside it
              uint8_t* blk = prow + nb * (kAtTileKeys * 128);
              *reinterpret_cast<uint4*>(blk + ((c0 ^ (lane_row & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
              *reinterpret_cast<uint4*>(blk + (((c0 + 1) ^ (lane_row & 7)) << 4)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
            }
          }
          if (hf == 0 && g4 == 0 && (t + 1) * kAtTileKeys > n) {
            // last tile of a sequence: what lies behind the sequence in V may be anything, and 0 x NaN is NaN
            ok = mbar_wait(v_full(it & 1), (it >> 1) & 1, abort_flag, p.wait_clocks);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (!in_seq)
              for (int half = 0; half < 2; ++half)
#pragma unroll
                for (int c = 0; c < 8; ++c)
                  reinterpret_cast<uint4*>(v_s + (it & 1) * kAtTileBytes + half * kAtTileKeys * 128 + lane_row * 128)[c] =
                      make_uint4(0, 0, 0, 0);
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(p_full(hf));
        }
        if (!ok) break;
        // the key's score: the other groups' partial sums, added in a fixed order
        if (g4 == 0) {
          ok = mbar_wait(x_full, it & 1, abort_flag, p.wait_clocks);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          sum += xch[lane_row] + xch[128 + lane_row] + xch[256 + lane_row];
          __syncwarp();
          if (lane == 0) mbar_arrive(x_empty);
          if (i < P) srow[i] = sum * unshift;
        } else {
          ok = mbar_wait(x_empty, (it & 1) ^ 1, abort_flag, p.wait_clocks);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          xch[(g4 - 1) * 128 + lane_row] = sum;
          __syncwarp();
          if (lane == 0) mbar_arrive(x_full);
        }
      }
    }
    if (ok && cur_b >= 0) flush_o();
  }

  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, kStatusWaitExpired);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

// out[b][h * G + g][j][c] = G * 2^-15 * sum over the head's segments of o_partial[segment][g * alpha + j][c].
// grid (R, H_kv, batch), block d.
__global__ void __launch_bounds__(kAtD) window_attend_reduce_kernel(const AtParams p) {
  pdl_trigger();
  pdl_wait();
  const int r = blockIdx.x, h = blockIdx.y, b = blockIdx.z, c = threadIdx.x;
  const int nc = p.seq.score_off[b + 1] - p.seq.score_off[b];
  const int total = p.num_kv_heads * p.seq.score_off[p.seq.batch];
  const int per = total / p.grid, rem = total % p.grid, edge = rem * (per + 1);
  const int i0 = p.num_kv_heads * p.seq.score_off[b] + h * nc, i1 = i0 + nc - 1;
  const int c0 = i0 < edge ? i0 / (per + 1) : rem + (i0 - edge) / per;
  const int c1 = i1 < edge ? i1 / (per + 1) : rem + (i1 - edge) / per;
  const int hg = b * p.num_kv_heads + h;
  float acc = 0.f;
  for (int s = c0 + hg; s <= c1 + hg; ++s) acc += __ldcg(p.o_partial + (static_cast<int64_t>(s) * p.rows + r) * kAtD + c);
  const int alpha = p.seq.alpha, g = r / alpha, j = r % alpha;
  const int64_t hq = static_cast<int64_t>(b) * p.num_kv_heads * p.group + h * p.group + g;
  p.out[(hq * alpha + j) * kAtD + c] = acc * static_cast<float>(p.group) / static_cast<float>(1 << kAtShift);
}

}  // namespace pkv
