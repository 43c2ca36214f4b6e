// Consumers of the compact cache: decode attention over the kept rows (Section 4.1: after compression
// only K_s, V_s are used for inference) and the attention-recall diagnostic (appendix on attention recall).
#pragma once

#include "pkv_common.cuh"
#include "pkv_paged.cuh"

namespace pkv {

constexpr int kDecThreads = 128;

struct DecodeParams {
  const void* q;            // [batch][H_q][d], config dtype, contiguous
  const void* k_cache;      // packed rows [sum_b H_kv * c_b][d]; with PAGED the pool [num_pages][page_size][d]
  const void* v_cache;
  PageTable pt;             // PAGED only
  uint32_t* status;         // PAGED only: where a bad table entry is recorded
  float* out;               // [batch][H_q][d] fp32
  SeqTable seq;
  int32_t num_kv_heads, group;
  float scale_log2;         // log2(e) / sqrt(d)
};

// grid (H_q, batch), block kDecThreads.  One new token's query of one head attends to every kept row of
// its KV head: out = softmax(q K_s^T / sqrt(d)) V_s.  Each 16-lane half-warp takes one cached row at a
// time (16 bytes per lane); running (max, sum, weighted V) are kept per half-warp and merged at the end.
// PAGED: the rows are found through the layer's block table instead of at fixed offsets.
template <typename T, int D, bool PAGED = false>
__global__ void __launch_bounds__(kDecThreads) decode_attention_kernel(const DecodeParams p) {
  constexpr int kPer = D / 16;                  // elements per lane
  __shared__ float s_m[kDecThreads / 16], s_z[kDecThreads / 16];
  __shared__ float s_acc[kDecThreads / 16][D];
  pdl_trigger();
  pdl_wait();
  const int hq = blockIdx.x, b = blockIdx.y;
  const int h = hq / p.group;
  const int count = p.seq.count[b];
  const int64_t row0 = p.seq.row_off[b] + static_cast<int64_t>(h) * count;
  const int sub = threadIdx.x & 15, team = threadIdx.x >> 4, teams = kDecThreads / 16;
  const uint32_t half_mask = 0xffffu << (threadIdx.x & 16);   // the two half-warps leave the row loop separately

  float qv[kPer], acc[kPer];
  const T* qrow = static_cast<const T*>(p.q) + (static_cast<int64_t>(b) * gridDim.x + hq) * D + sub * kPer;
#pragma unroll
  for (int c = 0; c < kPer; ++c) { qv[c] = to_float(qrow[c]); acc[c] = 0.f; }
  float m = -INFINITY, z = 0.f;
  for (int r = team; r < count; r += teams) {
    int64_t at = row0 + r;
    if (PAGED) {
      at = paged_row(p.pt, b, h, r);
      if (at < 0) {                                           // uniform over the half-warp
        if (sub == 0) atomicOr(p.status, kStatusBadPage);
        continue;
      }
    }
    const T* kr = static_cast<const T*>(p.k_cache) + at * D + sub * kPer;
    const T* vr = static_cast<const T*>(p.v_cache) + at * D + sub * kPer;
    float dot = 0.f;
#pragma unroll
    for (int c = 0; c < kPer; ++c) dot = fmaf(qv[c], to_float(kr[c]), dot);
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) dot += __shfl_xor_sync(half_mask, dot, o, 16);
    const float x = dot * p.scale_log2;
    const float mn = fmaxf(m, x);
    const float corr = exp2f(m - mn), w = exp2f(x - mn);
    z = z * corr + w;
#pragma unroll
    for (int c = 0; c < kPer; ++c) acc[c] = fmaf(acc[c], corr, w * to_float(vr[c]));
    m = mn;
  }
  if (sub == 0) { s_m[team] = m; s_z[team] = z; }
#pragma unroll
  for (int c = 0; c < kPer; ++c) s_acc[team][sub * kPer + c] = acc[c];
  __syncthreads();
  for (int c = threadIdx.x; c < D; c += kDecThreads) {
    float mm = -INFINITY;
    for (int t = 0; t < teams; ++t) mm = fmaxf(mm, s_m[t]);
    float zz = 0.f, a = 0.f;
    for (int t = 0; t < teams; ++t) {
      if (s_m[t] == -INFINITY) continue;         // team saw no row
      const float f = exp2f(s_m[t] - mm);
      zz += s_z[t] * f;
      a += s_acc[t][c] * f;
    }
    p.out[(static_cast<int64_t>(b) * gridDim.x + hq) * D + c] = a / zz;
  }
}

struct RecallParams {
  const float* scores;      // [batch][H_kv][ld]
  int64_t ld_scores;
  const int32_t* indices;   // packed rows
  float* recall;            // [batch][H_kv]
  SeqTable seq;
  int32_t num_kv_heads;
};

// grid (H_kv, batch), block 256.  Share of the window's attention that falls on kept keys:
//   recall = 1 - (sum of the scores of the evicted prefix keys) / alpha,
// because every window row's attention sums to one over the prefix and window keys, and window keys are kept.
__global__ void __launch_bounds__(256) attention_recall_kernel(const RecallParams p) {
  __shared__ float part[2][8];
  pdl_trigger();
  pdl_wait();
  const int h = blockIdx.x, b = blockIdx.y;
  const int alpha = p.seq.alpha, P = p.seq.n[b] - alpha, count = p.seq.count[b], k = count - alpha;
  const float* s = p.scores + (static_cast<int64_t>(b) * p.num_kv_heads + h) * p.ld_scores;
  const int32_t* idx = p.indices + p.seq.row_off[b] + static_cast<int64_t>(h) * count;
  float all = 0.f, kept = 0.f;
  for (int i = threadIdx.x; i < P; i += 256) all += s[i];
  for (int j = threadIdx.x; j < k; j += 256) {
    const int i = idx[j];
    if (i >= 0 && i < P) kept += s[i];                      // an entry that is no prefix position counts as not kept
  }
  for (int o = 16; o > 0; o >>= 1) {
    all += __shfl_xor_sync(0xffffffffu, all, o);
    kept += __shfl_xor_sync(0xffffffffu, kept, o);
  }
  if ((threadIdx.x & 31) == 0) { part[0][threadIdx.x >> 5] = all; part[1][threadIdx.x >> 5] = kept; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float a = 0.f, kk = 0.f;
    for (int w = 0; w < 8; ++w) { a += part[0][w]; kk += part[1][w]; }
    p.recall[b * p.num_kv_heads + h] = 1.0f - (a - kk) / static_cast<float>(alpha);
  }
}

}  // namespace pkv
