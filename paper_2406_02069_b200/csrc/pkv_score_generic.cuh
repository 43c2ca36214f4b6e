// Window-score kernels on the plain fp32 pipes (Section 4.2.2, Eq. 2 and Eq. 3).
//
// These cover every dtype / shape the boundary admits (fp32 inputs, any window,
// any group size) and are the path of small fp32 problems.  The tensor-core
// kernels in pkv_score_tc.cuh take over for bf16 inputs when their shape rules hold.
//
// The score of a key mixes softmax rows that each have their own normaliser, so
// the normalisers must be known before any score can be formed.  Three launches:
//   rowstats    one thread per window row r = (query head g, window row j): running
//               max and sum of exp over one chunk of keys     -> partial (max, sum)
//   combine     merges the chunks of a (sequence, KV head)     -> lse2[r] = log2 sum_i 2^(x_ri)
//   scores      one thread per key: s_i = sum_r 2^(x_ri - lse2[r] - log2 G)
// with x_ri = q_r . k_i * log2(e) / sqrt(d); both sweeps form x with the same
// sequence of operations, so the two agree bit for bit.
#pragma once

#include "pkv_common.cuh"

namespace pkv {

constexpr int kGenChunk = 128;       // keys per rowstats CTA (= the chunk the workspace is sized for)
constexpr int kGenKeyTile = 16;      // keys staged in shared memory at a time
constexpr int kGenRowBlock = 256;    // window rows per rowstats CTA pass (= its thread count)
constexpr int kGenScoreKeys = 128;   // keys (= threads) per scores CTA
constexpr int kGenQRows = 32;        // window rows staged per pass in the scores kernel

struct ScoreParams {
  TensorView q, k;
  SeqTable seq;
  int32_t num_kv_heads, group, rows;     // rows = group * alpha
  float scale_log2;                      // log2(e) / sqrt(d)
  float2* partial;                       // [sum_b chunks_b][slots_per_chunk][H_kv][rows] (max, sum)
  int32_t slots_per_chunk;               // partial slots each chunk writes (1 here, 2 for the tensor-core sweep)
  float* lse2;                           // [batch][H_kv][rows]
  const float* lse_in;                   // normalisers the score sweep reads: lse2, or the caller's
  float lse_scale, lse_add;              // applied on load: (1, 0), or (log2 e, log2 G) for natural-log input
  float* scores;                         // [batch][H_kv][ld]
  int64_t ld_scores;
  int32_t stats_only;                    // host side: stop after the row normalisers (no score sweep)
  int32_t stat_grid;                     // 0: partial is [chunk][slot][H_kv][rows] (fp32-pipe sweep).  > 0: CTAs of
                                         // the tensor-core sweep, which writes [segment][slot][rows] with segment =
                                         // CTA + head for every run of a CTA over one head's chunks
};

// grid (total chunks, H_kv), block kGenRowBlock.
template <typename T, int D>
__global__ void __launch_bounds__(kGenRowBlock) rowstats_generic_kernel(const ScoreParams p) {
  __shared__ __align__(16) float ktile[kGenKeyTile][D];
  pdl_trigger();
  pdl_wait();
  const int tile = blockIdx.x, h = blockIdx.y;
  const int b = find_sequence(p.seq.stat_off, p.seq.batch, tile);
  const int n = p.seq.n[b], alpha = p.seq.alpha, P = p.seq.prefix[b];
  const int key0 = (tile - p.seq.stat_off[b]) * kGenChunk;
  const int key1 = min(n, key0 + kGenChunk);
  const T* kbase = static_cast<const T*>(p.k.ptr) + b * p.k.sb + h * p.k.sh;

  for (int r0 = 0; r0 < p.rows; r0 += kGenRowBlock) {
    const int r = r0 + threadIdx.x;
    const bool live = r < p.rows;
    const int g = live ? r / alpha : 0, j = live ? r % alpha : 0;
    const int last_visible = P + j;                  // row j sees keys 0 .. P + j
    float qreg[D];
    {
      const T* qrow = static_cast<const T*>(p.q.ptr) + b * p.q.sb +
                      static_cast<int64_t>(h * p.group + g) * p.q.sh + j * p.q.st;
#pragma unroll
      for (int c = 0; c < D; ++c) qreg[c] = live ? to_float(qrow[c]) : 0.f;
    }
    float m = -INFINITY, z = 0.f;
    for (int t0 = key0; t0 < key1; t0 += kGenKeyTile) {
      __syncthreads();
      for (int e = threadIdx.x; e < kGenKeyTile * D; e += blockDim.x) {
        const int kk = e / D, c = e % D;
        const int i = t0 + kk;
        ktile[kk][c] = i < key1 ? to_float(kbase[static_cast<int64_t>(i) * p.k.st + c]) : 0.f;
      }
      __syncthreads();
      float x[kGenKeyTile];
      float tmax = -INFINITY;
#pragma unroll
      for (int kk = 0; kk < kGenKeyTile; ++kk) {
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < D; c += 4) {
          const float4 kv = *reinterpret_cast<const float4*>(&ktile[kk][c]);
          dot = fmaf(qreg[c], kv.x, dot);
          dot = fmaf(qreg[c + 1], kv.y, dot);
          dot = fmaf(qreg[c + 2], kv.z, dot);
          dot = fmaf(qreg[c + 3], kv.w, dot);
        }
        const int i = t0 + kk;
        x[kk] = (i < key1 && i <= last_visible) ? dot * p.scale_log2 : -INFINITY;
        tmax = fmaxf(tmax, x[kk]);
      }
      if (tmax > -INFINITY) {
        const float mn = fmaxf(m, tmax);
        float acc = 0.f;
#pragma unroll
        for (int kk = 0; kk < kGenKeyTile; ++kk) acc += exp2f(x[kk] - mn);
        z = z * exp2f(m - mn) + acc;                 // exp2f(-inf) = 0 on the first tile
        m = mn;
      }
    }
    if (live) p.partial[(static_cast<int64_t>(tile) * p.num_kv_heads + h) * p.rows + r] = make_float2(m, z);
  }
}

// grid (ceil(rows / 32), H_kv, batch), block 1024: merge the chunk partials of each window row.
// Thread (rl, sg) = (tid % 32, tid / 32) takes row r0 + rl and every 32nd partial slot starting at sg, so
// a warp reads 32 consecutive rows of one slot (256 contiguous bytes); loads are issued four at a time
// before they are used.  The 32 slot groups of a row are merged through shared memory.
// extra_log2 = log2(G) folds the mean over the group's query heads into the normaliser.
constexpr int kCombineThreads = 1024;
__global__ void __launch_bounds__(kCombineThreads) combine_stats_kernel(const ScoreParams p, float extra_log2) {
  __shared__ float sm[32][33], sz[32][33];
  pdl_trigger();
  pdl_wait();
  const int h = blockIdx.y, b = blockIdx.z;
  const int rl = threadIdx.x & 31, sg = threadIdx.x >> 5;
  const int r = blockIdx.x * 32 + rl;
  int t0 = p.seq.stat_off[b] * p.slots_per_chunk, t1 = p.seq.stat_off[b + 1] * p.slots_per_chunk;
  int64_t slot_stride = static_cast<int64_t>(p.num_kv_heads) * p.rows;
  int64_t first = static_cast<int64_t>(h) * p.rows;
  if (p.stat_grid > 0) {
    // The sweep's CTAs take contiguous item ranges (items ordered sequence, head, chunk): the first `rem`
    // CTAs per + 1 items, the others per.  This head's items fall to CTAs c0..c1, one segment each.
    const int nc = p.seq.stat_off[b + 1] - p.seq.stat_off[b];
    const int total = p.num_kv_heads * p.seq.stat_off[p.seq.batch];
    const int per = total / p.stat_grid, rem = total % p.stat_grid;
    const int edge = rem * (per + 1);
    const int i0 = p.num_kv_heads * p.seq.stat_off[b] + h * nc, i1 = i0 + nc - 1;
    const int c0 = i0 < edge ? i0 / (per + 1) : rem + (i0 - edge) / per;
    const int c1 = i1 < edge ? i1 / (per + 1) : rem + (i1 - edge) / per;
    const int hg = b * p.num_kv_heads + h;
    t0 = (c0 + hg) * p.slots_per_chunk;
    t1 = (c1 + hg + 1) * p.slots_per_chunk;
    slot_stride = p.rows;
    first = 0;
  }
  float m = -INFINITY, z = 0.f;
  if (r < p.rows) {
    const float2* base = p.partial + first + r;
    for (int t = t0 + sg; t < t1; t += 4 * 32) {
      float2 pz[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        pz[u] = t + 32 * u < t1 ? base[(t + 32 * u) * slot_stride] : make_float2(-INFINITY, 0.f);
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (pz[u].x > -INFINITY) {                 // (-inf, 0) marks a slot that saw no key of this row
          const float mn = fmaxf(m, pz[u].x);
          z = z * exp2f(m - mn) + pz[u].y * exp2f(pz[u].x - mn);
          m = mn;
        }
    }
  }
  sm[sg][rl] = m;
  sz[sg][rl] = z;
  __syncthreads();
  if (sg == 0 && r < p.rows) {
    float mm = -INFINITY;
    for (int g = 0; g < 32; ++g) mm = fmaxf(mm, sm[g][rl]);
    float zz = 0.f;
    for (int g = 0; g < 32; ++g)
      if (sm[g][rl] > -INFINITY) zz += sz[g][rl] * exp2f(sm[g][rl] - mm);
    p.lse2[(static_cast<int64_t>(b) * p.num_kv_heads + h) * p.rows + r] = mm + log2f(zz) + extra_log2;
  }
}

// grid (total prefix tiles, H_kv), block kGenScoreKeys: one thread per prefix key.
template <typename T, int D>
__global__ void __launch_bounds__(kGenScoreKeys) scores_generic_kernel(const ScoreParams p) {
  __shared__ __align__(16) float qs[kGenQRows][D];
  __shared__ float lse_s[kGenQRows];
  pdl_trigger();
  pdl_wait();
  const int tile = blockIdx.x, h = blockIdx.y;
  const int b = find_sequence(p.seq.score_off, p.seq.batch, tile);
  const int alpha = p.seq.alpha, P = p.seq.prefix[b];
  const int i = (tile - p.seq.score_off[b]) * kGenScoreKeys + threadIdx.x;
  const bool live = i < P;
  float kreg[D];
  {
    const T* krow = static_cast<const T*>(p.k.ptr) + b * p.k.sb + h * p.k.sh +
                    static_cast<int64_t>(live ? i : 0) * p.k.st;
#pragma unroll
    for (int c = 0; c < D; ++c) kreg[c] = to_float(krow[c]);
  }
  float s = 0.f;
  for (int r0 = 0; r0 < p.rows; r0 += kGenQRows) {
    __syncthreads();
    for (int e = threadIdx.x; e < kGenQRows * D; e += blockDim.x) {
      const int rr = e / D, c = e % D, r = r0 + rr;
      float v = 0.f;
      if (r < p.rows) {
        const int g = r / alpha, j = r % alpha;
        v = to_float(static_cast<const T*>(p.q.ptr)[b * p.q.sb + static_cast<int64_t>(h * p.group + g) * p.q.sh +
                                                     j * p.q.st + c]);
      }
      qs[rr][c] = v;
    }
    if (threadIdx.x < kGenQRows) {
      const int r = r0 + threadIdx.x;
      lse_s[threadIdx.x] =
          r < p.rows ? fmaf(p.lse_in[(static_cast<int64_t>(b) * p.num_kv_heads + h) * p.rows + r], p.lse_scale, p.lse_add)
                     : INFINITY;
    }
    __syncthreads();
    const int rn = min(kGenQRows, p.rows - r0);
    for (int rr = 0; rr < rn; ++rr) {
      float dot = 0.f;
#pragma unroll
      for (int c = 0; c < D; c += 4) {
        const float4 qv = *reinterpret_cast<const float4*>(&qs[rr][c]);
        dot = fmaf(qv.x, kreg[c], dot);
        dot = fmaf(qv.y, kreg[c + 1], dot);
        dot = fmaf(qv.z, kreg[c + 2], dot);
        dot = fmaf(qv.w, kreg[c + 3], dot);
      }
      s += exp2f(dot * p.scale_log2 - lse_s[rr]);
    }
  }
  if (live) p.scores[(static_cast<int64_t>(b) * p.num_kv_heads + h) * p.ld_scores + i] = s;
}

}  // namespace pkv
