// Window-score kernels on the sm_100a tensor cores (Section 4.2.2, Eq. 2 and Eq. 3), bf16 or fp16 inputs.
//
// Two sweeps over K, because the score of a key sums softmax rows that each have
// their own normaliser (known only after a whole row has been seen):
//
//   sweep A  D[row r][key i] = Q K^T   (A operand = 128 window rows, B operand = 256-key tile)
//            TMEM lane = window row, so each epilogue thread owns one row and keeps its
//            reference exponent and sum of 2^x privately: no cross-thread reduction at all.
//   sweep B  D[key i][row r] = K Q^T   (A operand = 128-key tile, B operand = all window rows)
//            TMEM lane = key, so each epilogue thread owns one key and sums
//            2^(x_ri - lse2_r) over the rows r, reading lse2 from shared memory.
//
// x = (q . k) * log2(e) / sqrt(d).  Operands arrive by plain per-CTA TMA loads into
// 128-byte-swizzled shared memory; tcgen05.mma accumulates in TMEM (two to four
// accumulator stages of up to 256 columns); epilogue warps read TMEM with tcgen05.ld.
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 4..19 =
// epilogue.  The exponentials bound both sweeps (16 per clock per SM); four epilogue
// warps per scheduler are what it takes to keep that unit busy.  The 16 epilogue
// warps form four groups (TMEM lane quarter = warp % 4, group = (warp - 4) / 4).
// Accumulator stage u % 2 is read by the two groups g with g % 2 == u % 2, each taking
// half of its columns, so while one pair of groups works on a stage the MMAs of the
// next stage run.  CTAs are persistent: each takes a contiguous range of (sequence,
// KV head, key chunk) work items.
//
// Every wait on an mbarrier is bounded.  A wait that runs out sets an abort flag in
// shared memory and a status bit in the workspace; all roles then leave their loops,
// the producer drains the copies it still has in flight, TMEM is released and the
// kernel returns.
#pragma once

#include <cuda.h>

#include "pkv_common.cuh"

namespace pkv {

constexpr int kTcThreads = 640;         // 20 warps: producer, MMA issuer, 2 idle, 16 epilogue
constexpr int kTcEpiWarp0 = 4;          // first epilogue warp
constexpr int kTcEpiWarps = 16;         // four per scheduler, which is what keeps the exp unit fed
constexpr int kTcTileKeysA = 256;       // keys per K tile in sweep A (the N of its MMAs)
constexpr int kTcTileKeysB = 128;       // keys per K tile in sweep B (the M of its MMAs)
constexpr int kTcKBytes = 128 * 1024;   // shared memory given to K stages (2 x 64 KB or 4 x 32 KB at d = 128)
constexpr int kTcMaxGrid = 256;         // CTAs of a sweep at most (the workspace holds a partial segment per CTA)
constexpr int kTcMaxRows = 256;         // window rows (G * alpha) the tensor-core path takes
constexpr long long kTcWaitCycles = 1ll << 31;   // bound of any one wait, in SM clocks
constexpr int kTcStatSlots = 4;         // partial (reference, sum) slots per run segment and row in sweep A, at most
// ... and how many of them a sweep with `row_blocks` blocks of 128 window rows writes (one per epilogue warp
// group that works on a row)
__host__ __device__ constexpr int tc_stat_slots(int row_blocks) { return row_blocks == 2 ? 2 : 4; }

struct TcParams {
  SeqTable seq;                 // stat_off / score_off count CHUNKS of chunk_tiles tiles
  int32_t num_kv_heads, group, rows;      // rows = group * alpha (R)
  int32_t rows_pad;             // R rounded up to 32
  int32_t fp16;                 // 1: Q and K hold binary16, 0: bfloat16 (both operands always share the type)
  int32_t early;                // 1: the caller vouches for Q and K (PKV_FLAG_INPUTS_FINAL) and they are not outputs
                                // of a library kernel that may still run: start reading them at once
  int32_t withhold;             // test aid: CTA 0 of sweep A never loads its last K tile (its waits then run out)
  long long wait_clocks;        // bound of any one wait, in SM clocks
  int32_t row_blocks;           // ceil(R / 128): M-blocks of sweep A
  int32_t chunk_tiles_a;        // 256-key tiles per work item of sweep A
  int32_t chunk_tiles_b;        // 128-key tiles per work item of sweep B
  float scale_log2;             // log2(e) / sqrt(d)
  float2* partial;              // sweep A out: [segment][slots][R] (reference exponent, sum); a segment is one
                                // CTA's run over one (sequence, head); slots = 2 with two row blocks, 4 with
                                // one: every epilogue warp group writes its own slot
  const float* lse2;            // sweep B in:  [batch][H_kv][R] row normalisers (log of the row's sum of exps)
  float lse_scale, lse_add;     // lse2_r = lse2[r] * lse_scale + lse_add: (1, 0) for the library's own sweep A,
                                // (log2 e, log2 G) for natural-log normalisers handed in by the caller
  int32_t merge;                // sweep B: 1 = lse2 is not read; every CTA merges the partials of sweep A for the
                                // heads it works on (no merge kernel between the sweeps)
  int32_t stat_grid;            // CTAs sweep A ran with (which segments belong to a head follows from it)
  float log2_group;             // log2 G, added to the merged normalisers
  float* scores;                // sweep B out: [batch][H_kv][ld]
  int64_t ld_scores;
  uint32_t* status;
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Non-blocking test of a barrier phase.
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Hardware-suspended wait for a barrier phase: the thread sleeps until the phase completes or the time hint (in
// nanoseconds) has passed, whichever comes first; returns false in the second case.  The hint matters: with the
// default (short) limit the waiting warps of this kernel spent a fifth of all issued instructions on re-trying.
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(20000u)
      : "memory");
  return ok != 0;
}
// Bounded wait.  The thread is suspended by the hardware between checks (no sleeping in software, which
// would add its wake-up latency to every hand-off of the pipeline).  Gives up after `limit` SM
// clocks (kTcWaitCycles, of the order of a second, unless a test lowers it) or when another thread gave up (abort flag); returns false then.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long limit) {
  if (mbar_try(bar, parity)) return true;
  const long long start = clock64();
  for (;;) {
    if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - start > limit) break;
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_f16kind(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// The special-function unit evaluates 16 exponentials per clock per SM, which is what bounds both
// sweeps when every 2^x goes through it.  A fixed share of the exponentials is therefore evaluated on
// the FMA pipe instead, two at a time with the packed fp32 instructions.  Of every eight consecutive
// pairs of values (16 accumulator columns), kTcPolyPairs go this way, spread evenly over the eight.
#ifndef PKV_POLY_PAIRS
#define PKV_POLY_PAIRS 2
#endif
constexpr int kTcPolyPairs = PKV_POLY_PAIRS;    // 0 = every exponential on the special-function unit
__host__ __device__ constexpr bool tc_pair_is_poly(int pair) {
  return ((pair % 8 + 1) * kTcPolyPairs) / 8 != ((pair % 8) * kTcPolyPairs) / 8;
}

// Packed pairs of fp32 (one instruction for two multiply-adds or two adds): the scale-and-shift in front
// of each exponential, the polynomial and the accumulation behind it go through these, which halves
// their issue slots.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(unsigned long long r, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(r));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float fma_sat(float a, float b, float c) {   // a * b + c clamped to [0, 1]
  float d;
  asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// acc + (2^x0, 2^x1), evaluated on the FMA pipe.
//   y = sat((x + 126) / 253)            one instruction rescales x and clamps it to [-126, 127], so that the
//                                       exponent arithmetic below cannot wrap (-inf and NaN give y = 0)
//   t = 253 y + (1.5 * 2^23 + 1)        rounds to an integer: the low mantissa bits of t hold n + 127, n = round(x)
//   f = 253 y + (1.5 * 2^23 + 1 - t)    = x - n in [-0.5, 0.5]
//   2^f by a cubic minimax polynomial (largest relative error 7.5e-5, far inside the 2e-3 the scores are held to);
//   2^n is the float whose exponent field is n + 127, i.e. t << 23;  result = acc + 2^f * 2^n.
__device__ __forceinline__ unsigned long long ex2_poly_add(float x0, float x1, unsigned long long acc) {
  const float kMagic1 = 12582913.0f;
  const float y0 = fma_sat(x0, 1.0f / 253.0f, 126.0f / 253.0f), y1 = fma_sat(x1, 1.0f / 253.0f, 126.0f / 253.0f);
  const unsigned long long y = pack2(y0, y1), k253 = pack2(253.0f, 253.0f), km = pack2(kMagic1, kMagic1);
  const unsigned long long t = fma2(y, k253, km);
  const unsigned long long g = fma2(t, pack2(-1.0f, -1.0f), km);
  const unsigned long long f = fma2(y, k253, g);
  unsigned long long q = fma2(f, pack2(0.0551716685295105f, 0.0551716685295105f),
                              pack2(0.2426111251115799f, 0.2426111251115799f));
  q = fma2(q, f, pack2(0.6932609677314758f, 0.6932609677314758f));
  q = fma2(q, f, pack2(0.9999280571937561f, 0.9999280571937561f));
  float t0, t1;
  unpack2(t, t0, t1);
  const unsigned long long scale = pack2(__int_as_float(__float_as_int(t0) << 23), __int_as_float(__float_as_int(t1) << 23));
  return fma2(q, scale, acc);
}

// acc[j % 4] += (2^x0, 2^x1) for the eight packed pairs xs[j] of one 16-column chunk, each pair by the unit its
// position selects.
__device__ __forceinline__ void ex2_accumulate8(const unsigned long long (&xs)[8], unsigned long long (&acc)[4]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    float x0, x1;
    unpack2(xs[j], x0, x1);
    if (tc_pair_is_poly(j)) acc[j & 3] = ex2_poly_add(x0, x1, acc[j & 3]);
    else acc[j & 3] = add2(acc[j & 3], pack2(ex2(x0), ex2(x1)));
  }
}

// Sweep A, 16 logits of one window row, fast path: acc += 2^(v_j * c2 - m) in four packed pairs of partial sums.
// m is a reference exponent, not necessarily the running maximum; the caller adds the partial sums up once per
// unit and falls back to rowstats_rescue when the total is not a moderate finite number.
__device__ __forceinline__ void rowstats_accumulate(const uint32_t (&v)[16], unsigned long long cc,
                                                    unsigned long long mm, unsigned long long (&acc)[4]) {
  unsigned long long xs[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) xs[j] = fma2(pack2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])), cc, mm);
  ex2_accumulate8(xs, acc);
}
__device__ __forceinline__ float sum_pairs(const unsigned long long (&acc)[4]) {
  float a[8];
#pragma unroll
  for (int q = 0; q < 4; ++q) unpack2(acc[q], a[2 * q], a[2 * q + 1]);
  return ((a[0] + a[1]) + (a[2] + a[3])) + ((a[4] + a[5]) + (a[6] + a[7]));
}
// Sweep A, slow path for the same 16 logits: moves the reference exponent up to a whole number at or above the
// running maximum first (the row's first chunk, where m = -inf, or a logit some 60 binades above the reference).
// `live` is false for threads that only keep the warp's loads aligned.
__device__ __forceinline__ void rowstats_rescue(const uint32_t (&v)[16], float c2, bool live, float& m, float& z) {
  if (!live) return;
  float gm = __uint_as_float(v[0]);
#pragma unroll
  for (int j = 1; j < 16; ++j) gm = fmaxf(gm, __uint_as_float(v[j]));
  const float mn = fmaxf(m, ceilf(gm * c2));
  z *= ex2(m - mn);
  m = mn;
  float g = 0.f;
#pragma unroll
  for (int j = 0; j < 16; ++j) g += ex2(fmaf(__uint_as_float(v[j]), c2, -m));
  z += g;
}

// Sweep B, 16 window rows of one key: acc += 2^(v_j * c2 + nlse_j); nlse = -lse2 sits in shared memory
// (negated when it was loaded), acc holds four packed pairs of partial sums.
__device__ __forceinline__ void score_group(const uint32_t (&v)[16], unsigned long long cc, const float* nlse,
                                            unsigned long long (&acc)[4]) {
  unsigned long long xs[8];
#pragma unroll
  for (int j = 0; j < 8; j += 2) {
    const ulonglong2 l = *reinterpret_cast<const ulonglong2*>(nlse + 2 * j);   // four floats as two packed pairs
    xs[j] = fma2(pack2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])), cc, l.x);
    xs[j + 1] = fma2(pack2(__uint_as_float(v[2 * j + 2]), __uint_as_float(v[2 * j + 3])), cc, l.y);
  }
  ex2_accumulate8(xs, acc);
}

// Shared-memory matrix descriptor of a K-major bf16 operand whose rows are 128 bytes wide and
// stored with the 128-byte swizzle: 8-row groups are 1024 bytes apart.  `addr` is the byte address
// of the first row, plus 32 bytes per 16-element step along the contraction dimension.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr & 0x3FFFFu) >> 4);          // start address
  d |= static_cast<uint64_t>(1) << 16;                         // leading byte offset (unused with swizzle), 16 B
  d |= static_cast<uint64_t>(1024 >> 4) << 32;                 // stride byte offset: 1024 B between 8-row groups
  d |= static_cast<uint64_t>(1) << 46;                         // descriptor version of this architecture
  d |= static_cast<uint64_t>(2) << 61;                         // 128-byte swizzle
  return d;
}
// Instruction descriptor: 16-bit x 16-bit -> fp32, both operands K-major and of one type (format code 1 =
// bf16, 0 = fp16, for A at bit 7 and B at bit 10), M x N tile.
__device__ __forceinline__ uint32_t instr_desc_16bit(int M, int N, int fp16) {
  const uint32_t fmt = fp16 ? 0u : 1u;
  return (1u << 4) | (fmt << 7) | (fmt << 10) | (static_cast<uint32_t>(N >> 3) << 17) |
         (static_cast<uint32_t>(M >> 4) << 24);
}

// Work item -> (sequence, head, chunk).  Items are ordered sequence, head, chunk.
struct TcItem { int b, h, c, nchunks; };
__device__ __forceinline__ TcItem tc_item(const int32_t* off, int batch, int heads, int id) {
  int b = 0;
  while (b + 1 < batch && id >= heads * off[b + 1]) ++b;
  const int local = id - heads * off[b];
  const int nc = off[b + 1] - off[b];
  return TcItem{b, local / nc, local % nc, nc};
}

// Dynamic shared memory carve-up (bytes), all regions 1024-aligned.
template <int D>
struct TcSmem {
  static constexpr int kHalves = D / 64;                       // 64-element (128-byte) column blocks
  static constexpr int kQBytes = kTcMaxRows * D * 2;
  static constexpr int kQOff = 0;
  static constexpr int kKOff = kQBytes;
  static constexpr int kMiscOff = kKOff + kTcKBytes;
  static constexpr int kMiscBytes = 20 * 1024;                 // barriers, exchange buffers, per-warp lse2 copies
  static constexpr int kTotal = kMiscOff + kMiscBytes + 1024;  // + slack for manual 1024-byte alignment
};

// SWEEP 0 = row statistics (A), 1 = scores (B).
template <int D, int SWEEP>
__global__ void __launch_bounds__(kTcThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                const TcParams p) {
  using L = TcSmem<D>;
  constexpr int kTileKeys = SWEEP == 0 ? kTcTileKeysA : kTcTileKeysB;
  // Sweep B walks each CTA's items and tiles from the last to the first: sweep A has just read the same keys in
  // ascending order, so the end of every range is what the L2 still holds.
  constexpr bool kReverse = SWEEP == 1;
  constexpr int kStageBytes = kTileKeys * D * 2;               // one K tile in shared memory
  constexpr int kKStages = kTcKBytes / kStageBytes >= 4 ? 4 : kTcKBytes / kStageBytes;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem + L::kQOff;
  uint8_t* k_s = smem + L::kKOff;
  uint8_t* misc = smem + L::kMiscOff;
  uint64_t* bars = reinterpret_cast<uint64_t*>(misc);          // [0..3] k_full, [4..7] k_empty, [8..11] t_full,
                                                               // [12..15] t_empty, [16] q_full, [17] q_empty,
                                                               // [18..19] x_full, [20..21] x_empty, [22] lse_full
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 260);
  float* xch = reinterpret_cast<float*>(misc + 1024);          // sweep B: [2][128] partial sums handed between groups
  float* lse_all = reinterpret_cast<float*>(misc + 4096);      // sweep B: [2][256] -lse2 of the current / next head

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar0 = smem_u32(bars);
  auto k_full = [&](int s) { return bar0 + 8u * s; };
  auto k_empty = [&](int s) { return bar0 + 8u * (4 + s); };
  auto t_full = [&](int s) { return bar0 + 8u * (8 + s); };
  auto t_empty = [&](int s) { return bar0 + 8u * (12 + s); };
  const uint32_t q_full = bar0 + 8u * 16, q_empty = bar0 + 8u * 17;
  auto x_full = [&](int s) { return bar0 + 8u * (18 + s); };
  auto x_empty = [&](int s) { return bar0 + 8u * (20 + s); };
  const uint32_t lse_full = bar0 + 8u * 22;

  // Accumulator stages.  Sweep A: 256 key columns per unit (one row block x one K tile): two stages.
  // Sweep B: rows_pad columns per unit (one K tile), rounded up to a power of two: two to four stages.
  int stage_cols = 256;
  if (SWEEP == 1) {
    stage_cols = p.rows_pad <= 32 ? 32 : (p.rows_pad <= 64 ? 64 : (p.rows_pad <= 128 ? 128 : 256));
  }
  const int t_stages = SWEEP == 0 ? 2 : min(4, 512 / stage_cols);
  const bool two_blocks = p.row_blocks == 2;                   // sweep A: units per K tile
  const int split_b = ((p.rows_pad / 2) + 31) & ~31;           // sweep B: columns [0, split) and [split, rows_pad)
  const bool second_half = SWEEP == 0 || split_b < p.rows_pad; // do the groups 2, 3 have columns to read?

  // ---- set-up (shared memory and TMEM only: it may overlap the tail of the preceding kernel)
  pdl_trigger();
  if (threadIdx.x == 0) {
    for (int s = 0; s < 4; ++s) { mbar_init(k_full(s), 1); mbar_init(k_empty(s), 1); }
    const uint32_t consumers = second_half ? 8 : 4;            // epilogue warps that read one accumulator stage
    for (int s = 0; s < 4; ++s) { mbar_init(t_full(s), 1); mbar_init(t_empty(s), consumers); }
    mbar_init(q_full, 1);
    mbar_init(q_empty, 1);
    for (int s = 0; s < 2; ++s) { mbar_init(x_full(s), 4); mbar_init(x_empty(s), 4); }
    mbar_init(lse_full, kTcEpiWarps);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // rows of the Q tile beyond R stay zero for the whole kernel (TMA only ever writes R rows)
  for (int i = threadIdx.x; i < L::kQBytes / 16; i += kTcThreads) reinterpret_cast<uint4*>(q_s)[i] = make_uint4(0, 0, 0, 0);
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
  // Neither sweep waits here for the kernels ahead of it in the stream: copies and MMAs touch only the caller's Q
  // and K, so they start at once, beside the tail of those kernels.  Sweep A waits just before its first write
  // (its partials), sweep B's epilogue just before it reads the row normalisers; both wait again before they end.
  // (When Q or K may be the output of a library kernel still in flight, e.g. a compact cache that is compressed
  // again, the host clears `early` and the kernel waits here like any other.)
  if (!p.early) pdl_wait();

  // ---- this CTA's contiguous range of work items
  const int32_t* off = SWEEP == 0 ? p.seq.stat_off : p.seq.score_off;
  const int chunk_tiles = SWEEP == 0 ? p.chunk_tiles_a : p.chunk_tiles_b;
  const int total = p.num_kv_heads * off[p.seq.batch];
  const int per = total / gridDim.x, rem = total % gridDim.x;
  const int item0 = blockIdx.x * per + min(static_cast<int>(blockIdx.x), rem);
  const int item1 = item0 + per + (static_cast<int>(blockIdx.x) < rem ? 1 : 0);
  // keys an item of sequence b spans: sweep A covers all n keys, sweep B the prefix only
  auto span_keys = [&](int b) { return SWEEP == 0 ? p.seq.n[b] : p.seq.prefix[b]; };

  if (warp == 0) {
    // =========================================================== TMA producer
    if (lane == 0) {
      uint32_t it = 0, heads_loaded = 0;                       // it counts K tiles
      int cur_b = -1, cur_h = -1;
      bool ok = true;
      for (int ii = 0; ii < item1 - item0 && ok; ++ii) {
        const int id = kReverse ? item1 - 1 - ii : item0 + ii;
        const TcItem w = tc_item(off, p.seq.batch, p.num_kv_heads, id);
        if (w.b != cur_b || w.h != cur_h) {
          if (heads_loaded > 0) ok = mbar_wait(q_empty, (heads_loaded - 1) & 1, abort_flag, p.wait_clocks);
          if (!ok) break;
          mbar_expect_tx(q_full, static_cast<uint32_t>(p.rows) * D * 2);
          for (int half = 0; half < L::kHalves; ++half)
            tma_load_4d(smem_u32(q_s) + half * kTcMaxRows * 128, &q_map, q_full, half * 64, 0, w.h * p.group, w.b);
          ++heads_loaded;
          cur_b = w.b; cur_h = w.h;
        }
        const int keys = span_keys(w.b);
        const int tile0 = w.c * chunk_tiles;
        const int tile1 = min(tile0 + chunk_tiles, (keys + kTileKeys - 1) / kTileKeys);
        for (int tt = 0; tt < tile1 - tile0 && ok; ++tt, ++it) {
          const int t = kReverse ? tile1 - 1 - tt : tile0 + tt;
          const int s = it % kKStages;
          ok = mbar_wait(k_empty(s), ((it / kKStages) & 1) ^ 1, abort_flag, p.wait_clocks);
          if (!ok) break;
          if (SWEEP == 0 && p.withhold && blockIdx.x == 0 && ii + 1 == item1 - item0 && tt + 1 == tile1 - tile0)
            continue;                                       // test aid: this tile never arrives
          mbar_expect_tx(k_full(s), kStageBytes);
          for (int half = 0; half < L::kHalves; ++half)
            tma_load_4d(smem_u32(k_s) + s * kStageBytes + half * kTileKeys * 128, &k_map, k_full(s), half * 64,
                        t * kTileKeys, w.h, w.b);
        }
      }
      if (!ok) {
        // drain: wait (bounded) for the copies still in flight before shared memory is given up
        const uint32_t first = it > kKStages ? it - kKStages : 0;
        for (uint32_t j = first; j < it; ++j)
          for (uint32_t spin = 0; spin < (1u << 16) && !mbar_test(k_full(j % kKStages), (j / kKStages) & 1); ++spin)
            __nanosleep(64);
        if (heads_loaded > 0)
          for (uint32_t spin = 0; spin < (1u << 16) && !mbar_test(q_full, (heads_loaded - 1) & 1); ++spin) __nanosleep(64);
      }
    }
  } else if (warp == 1) {
    // =========================================================== MMA issuer
    if (lane == 0) {
      uint32_t it = 0, u = 0, heads_seen = 0;                  // it counts K tiles, u accumulator units
      int cur_b = -1, cur_h = -1;
      bool ok = true;
      const uint32_t idesc = SWEEP == 0 ? instr_desc_16bit(128, kTcTileKeysA, p.fp16)
                                        : instr_desc_16bit(kTcTileKeysB, p.rows_pad, p.fp16);
      for (int ii = 0; ii < item1 - item0 && ok; ++ii) {
        const int id = kReverse ? item1 - 1 - ii : item0 + ii;
        const TcItem w = tc_item(off, p.seq.batch, p.num_kv_heads, id);
        if (w.b != cur_b || w.h != cur_h) {
          ok = mbar_wait(q_full, heads_seen & 1, abort_flag, p.wait_clocks);
          if (!ok) break;
          ++heads_seen;
          cur_b = w.b; cur_h = w.h;
        }
        // does the next item belong to another head?  then Q may be overwritten after this item's MMAs
        bool last_of_head = ii + 1 >= item1 - item0;
        if (!last_of_head) {
          const TcItem nx = tc_item(off, p.seq.batch, p.num_kv_heads, kReverse ? id - 1 : id + 1);
          last_of_head = nx.b != w.b || nx.h != w.h;
        }
        const int keys = span_keys(w.b);
        const int tile0 = w.c * chunk_tiles;
        const int tile1 = min(tile0 + chunk_tiles, (keys + kTileKeys - 1) / kTileKeys);
        for (int tt = 0; tt < tile1 - tile0 && ok; ++tt, ++it) {
          const int s = it % kKStages;
          ok = mbar_wait(k_full(s), (it / kKStages) & 1, abort_flag, p.wait_clocks);
          if (!ok) break;
          const uint32_t k_addr = smem_u32(k_s) + s * kStageBytes;
          const uint32_t q_addr = smem_u32(q_s);
          const int units = SWEEP == 0 ? p.row_blocks : 1;
          for (int rb = 0; rb < units && ok; ++rb, ++u) {
            const int ts = u % t_stages;
            ok = mbar_wait(t_empty(ts), ((u / t_stages) & 1) ^ 1, abort_flag, p.wait_clocks);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_addr = tmem_base + ts * stage_cols;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              const uint32_t qa = q_addr + (kk / 4) * kTcMaxRows * 128 + rb * 128 * 128 + (kk % 4) * 32;
              const uint32_t ka = k_addr + (kk / 4) * kTileKeys * 128 + (kk % 4) * 32;
              if (SWEEP == 0) tc_mma_f16kind(d_addr, smem_desc_sw128(qa), smem_desc_sw128(ka), idesc, kk > 0);
              else tc_mma_f16kind(d_addr, smem_desc_sw128(ka), smem_desc_sw128(qa), idesc, kk > 0);
            }
            tc_commit(t_full(ts));
          }
          if (ok) tc_commit(k_empty(s));
        }
        if (ok && last_of_head) tc_commit(q_empty);
      }
    }
  } else if (warp >= kTcEpiWarp0) {
    // =========================================================== epilogue
    const int e = warp - kTcEpiWarp0;
    const int quarter = warp & 3;               // TMEM lanes 32*quarter .. +31 are this warp's
    const int grp = e >> 2;                     // 0..3
    const int par = grp & 1;                    // this group reads the units u with u % 2 == par
    const int ch = grp >> 1;                    // ... and this half of their columns
    const int lane_row = quarter * 32 + lane;   // TMEM lane of this thread
    const float c2 = p.scale_log2;
    uint32_t u = 0, mine = 0;                   // units seen by the CTA / units this group's pair has read
    uint32_t heads_seen = 0;                    // sweep B: (sequence, head) changes so far
    const float* lse_s = lse_all;               // sweep B: the current head's -lse2
    int cur_b = -1, cur_h = -1;
    bool ok = true;
    // Sweep A: a thread's (reference, sum) runs on over consecutive work items of one (sequence, head) and is
    // written once per run, to the segment numbered blockIdx.x + head: along the item order either the CTA
    // or the head advances from one run to the next, so the numbers are distinct, and the merge kernel finds
    // a head's segments from the CTAs its items fall to.
    float m = -INFINITY, z = 0.f;
    int run_b = -1, run_h = -1;
    auto flush_run = [&]() {
      const int r = (two_blocks ? par * 128 : 0) + lane_row;
      if (run_b < 0 || r >= p.rows) return;
      pdl_wait();                                             // the partials of the call before have been merged
      const int slots = tc_stat_slots(p.row_blocks);
      const int slot = two_blocks ? ch : grp;
      const int64_t seg = static_cast<int64_t>(blockIdx.x) + run_b * p.num_kv_heads + run_h;
      p.partial[(seg * slots + slot) * p.rows + r] = make_float2(m, z);
    };
    for (int ii = 0; ii < item1 - item0 && ok; ++ii) {
      const int id = kReverse ? item1 - 1 - ii : item0 + ii;
      const TcItem w = tc_item(off, p.seq.batch, p.num_kv_heads, id);
      const int n = p.seq.n[w.b], alpha = p.seq.alpha, P = p.seq.prefix[w.b];
      const int keys = span_keys(w.b);
      const int tile0 = w.c * chunk_tiles;
      const int tile1 = min(tile0 + chunk_tiles, (keys + kTileKeys - 1) / kTileKeys);
      if (SWEEP == 0) {
        // thread -> window row.  With two row blocks the unit parity is the row block, so a group always
        // works on the same block; with one, the pairs of groups take alternate K tiles.  Either way a
        // thread keeps one (reference, sum) per run of work items and every group writes its own partial slot.
        const int r = (two_blocks ? par * 128 : 0) + lane_row;
        const int last_visible = min(P + (r % alpha), n - 1); // row (g, j) sees keys 0 .. P + j that exist here
        const int units = p.row_blocks;
        // a warp whose 32 TMEM lanes are all padding rows (R < 128) has nothing to evaluate
        const bool warp_has_rows = (two_blocks ? par * 128 : 0) + quarter * 32 < p.rows;
        if (w.b != run_b || w.h != run_h) {
          flush_run();
          m = -INFINITY;
          z = 0.f;
          run_b = w.b;
          run_h = w.h;
        }
        for (int t = tile0; t < tile1 && ok; ++t) {
          for (int rb = 0; rb < units && ok; ++rb, ++u) {
            if (static_cast<int>(u & 1u) != par) continue;    // the other pair's unit
            const int ts = u & 1;
            ok = mbar_wait(t_full(ts), (u >> 1) & 1, abort_flag, p.wait_clocks);
            ok = __all_sync(0xffffffffu, ok);                 // whole warp proceeds together or not at all
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + ts * stage_cols + ch * 128;
            const int key_base = t * kTcTileKeysA + ch * 128;
            if (!warp_has_rows) {
              // only the hand-shake below
            } else if (key_base + 127 <= min(P, n - 1)) {     // every key visible to every row: no mask
              // fast path over the 128 columns; the sums are only looked at once, at the end
              const unsigned long long cc = pack2(c2, c2), mm = pack2(-m, -m);
              unsigned long long acc[4] = {pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f)};
              // 16-column loads, double buffered: the next load is in flight while a chunk is evaluated
              uint32_t va[16], vb[16];
              tc_ld16(taddr, va);
#pragma unroll
              for (int cg = 0; cg < 128; cg += 32) {
                tc_wait_ld();
                tc_ld16(taddr + cg + 16, vb);
                rowstats_accumulate(va, cc, mm, acc);
                tc_wait_ld();
                if (cg + 32 < 128) tc_ld16(taddr + cg + 32, va);
                rowstats_accumulate(vb, cc, mm, acc);
              }
              const float g = sum_pairs(acc);
              const bool good = g < 1.0e18f;                  // false for inf and NaN too
              if (good) z += g;
              if (!__all_sync(0xffffffffu, good)) {           // rare: the warp reads its columns again, slow path
                for (int cg = 0; cg < 128; cg += 16) {
                  tc_ld16(taddr + cg, va);
                  tc_wait_ld();
                  rowstats_rescue(va, c2, !good, m, z);
                }
              }
            } else {
              for (int cg = 0; cg < 128; cg += 16) {
                uint32_t v[16];
                tc_ld16(taddr + cg, v);
                tc_wait_ld();
                float gm = -INFINITY;
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                  const bool vis = key_base + cg + j <= last_visible;
                  const float x = vis ? __uint_as_float(v[j]) * c2 : -INFINITY;
                  v[j] = __float_as_uint(x);
                  gm = fmaxf(gm, x);
                }
                if (gm > -INFINITY) {
                  const float mn = fmaxf(m, ceilf(gm));
                  z *= ex2(m - mn);
                  m = mn;
                  float a0 = 0.f;
#pragma unroll
                  for (int j = 0; j < 16; ++j) a0 += ex2(__uint_as_float(v[j]) - m);
                  z += a0;
                }
              }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(t_empty(ts));
          }
        }
        if (!ok) break;
      } else {
        // thread -> key.  The pairs of groups take alternate K tiles; inside a pair the groups split the
        // window rows (columns) of a key and group ch = 1 hands its partial sum to group ch = 0.
        // The head's normalisers, negated (the epilogue adds them), in one of two buffers that alternate from
        // head to head.  The sixteen warps fill a buffer together (512 threads over the rows, 2 to 16 lanes per
        // row), then meet at a barrier; a buffer is written again only after every warp has passed the barrier of
        // the head in between, i.e. after all of them are done with it.  The values come either from the caller
        // (or the merge kernel), or straight from sweep A's partial (reference, sum) pairs of this head, which
        // every CTA that works on the head merges for itself, always in the same order.
        if (w.b != cur_b || w.h != cur_h) {
          pdl_wait();                                         // normalisers and partials are written by kernels before
          float* dst = lse_all + (heads_seen & 1u) * 256;
          const int rows_p2 = p.rows_pad <= 32 ? 32 : (p.rows_pad <= 64 ? 64 : (p.rows_pad <= 128 ? 128 : 256));
          const int per_row = (kTcEpiWarps * 32) / rows_p2;   // lanes that share a row: 2, 4, 8 or 16
          const int r = (e * 32 + lane) / per_row, part = (e * 32 + lane) % per_row;
          float val = -INFINITY;
          if (p.merge) {
            // sweep A's CTAs took contiguous item ranges (items ordered sequence, head, chunk): the first `rem`
            // CTAs per + 1 items, the others per; this head's items fell to CTAs c0..c1, one segment each
            const int nc = p.seq.stat_off[w.b + 1] - p.seq.stat_off[w.b];
            const int total_a = p.num_kv_heads * p.seq.stat_off[p.seq.batch];
            const int per_a = total_a / p.stat_grid, rem_a = total_a % p.stat_grid, edge = rem_a * (per_a + 1);
            const int i0 = p.num_kv_heads * p.seq.stat_off[w.b] + w.h * nc, i1 = i0 + nc - 1;
            const int c0 = i0 < edge ? i0 / (per_a + 1) : rem_a + (i0 - edge) / per_a;
            const int c1 = i1 < edge ? i1 / (per_a + 1) : rem_a + (i1 - edge) / per_a;
            const int hg = w.b * p.num_kv_heads + w.h, slots = tc_stat_slots(p.row_blocks);
            const int t0 = (c0 + hg) * slots, t1 = (c1 + hg + 1) * slots;
            float m = -INFINITY, z = 0.f;
            if (r < p.rows) {
              const float2* base = p.partial + r;
              for (int t = t0 + part; t < t1; t += 4 * per_row) {
                float2 pz[4];
#pragma unroll
                for (int q = 0; q < 4; ++q)
                  pz[q] = t + q * per_row < t1 ? __ldcg(base + static_cast<int64_t>(t + q * per_row) * p.rows)
                                               : make_float2(-INFINITY, 0.f);
#pragma unroll
                for (int q = 0; q < 4; ++q)
                  if (pz[q].x > -INFINITY) {                  // (-inf, 0) marks a slot that saw no key of this row
                    const float mn = fmaxf(m, pz[q].x);
                    z = z * ex2(m - mn) + pz[q].y * ex2(pz[q].x - mn);
                    m = mn;
                  }
              }
            }
            for (int o = 1; o < per_row; o <<= 1) {           // the lanes of a row meet pairwise; both partners of a
              const float m2 = __shfl_xor_sync(0xffffffffu, m, o), z2 = __shfl_xor_sync(0xffffffffu, z, o);   // pair
              const float mm = fmaxf(m, m2);                                        // compute the same merged value
              z = (m > -INFINITY ? z * ex2(m - mm) : 0.f) + (m2 > -INFINITY ? z2 * ex2(m2 - mm) : 0.f);
              m = mm;
            }
            if (r < p.rows) val = -(m + __log2f(z) + p.log2_group);
          } else if (r < p.rows) {
            const float* src = p.lse2 + (static_cast<int64_t>(w.b) * p.num_kv_heads + w.h) * p.rows;
            val = -fmaf(src[r], p.lse_scale, p.lse_add);
          }
          if (part == 0) dst[r] = val;
          __syncwarp();
          if (lane == 0) mbar_arrive(lse_full);
          ok = mbar_wait(lse_full, heads_seen & 1u, abort_flag, p.wait_clocks);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          lse_s = dst;
          ++heads_seen;
          cur_b = w.b; cur_h = w.h;
        }
        float* srow = p.scores + (static_cast<int64_t>(w.b) * p.num_kv_heads + w.h) * p.ld_scores;
        const int col0 = ch == 0 ? 0 : split_b, col1 = ch == 0 ? split_b : p.rows_pad;
        for (int tt = 0; tt < tile1 - tile0 && ok; ++tt, ++u) {
          const int t = kReverse ? tile1 - 1 - tt : tile0 + tt;
          if (static_cast<int>(u & 1u) != par) continue;      // the other pair's tile
          if (ch == 1 && !second_half) continue;              // nothing for this group to read
          const int ts = u % t_stages;
          ok = mbar_wait(t_full(ts), (u / t_stages) & 1, abort_flag, p.wait_clocks);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + ts * stage_cols;
          unsigned long long acc[4] = {pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f)};
          const unsigned long long cc = pack2(c2, c2);
          {
            uint32_t va[16], vb[16];
            tc_ld16(taddr + col0, va);
            for (int cg = col0; cg < col1; cg += 32) {
              tc_wait_ld();
              tc_ld16(taddr + cg + 16, vb);
              score_group(va, cc, lse_s + cg, acc);
              tc_wait_ld();
              if (cg + 32 < col1) tc_ld16(taddr + cg + 32, va);
              score_group(vb, cc, lse_s + cg + 16, acc);
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(t_empty(ts));
          float sum = sum_pairs(acc);
          if (second_half) {
            if (ch == 1) {
              ok = mbar_wait(x_empty(par), (mine & 1) ^ 1, abort_flag, p.wait_clocks);
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) break;
              xch[par * 128 + lane_row] = sum;
              __syncwarp();
              if (lane == 0) mbar_arrive(x_full(par));
            } else {
              ok = mbar_wait(x_full(par), mine & 1, abort_flag, p.wait_clocks);
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) break;
              sum += xch[par * 128 + lane_row];
              __syncwarp();
              if (lane == 0) mbar_arrive(x_empty(par));
            }
          }
          ++mine;
          const int i = t * kTcTileKeysB + lane_row;
          if (ch == 0 && i < P) srow[i] = sum;
        }
        if (!ok) break;
      }
    }
    if (SWEEP == 0 && ok) flush_run();                        // the CTA's last run
  }

  // ---- teardown
  pdl_wait();                                                  // never finish before the kernels ahead in the stream
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, kStatusWaitExpired);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

}  // namespace pkv
