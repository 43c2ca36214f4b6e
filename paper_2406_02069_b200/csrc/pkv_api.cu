// Host side of the PyramidKV compression library: argument validation, the
// budget schedule, workspace carving and kernel launches behind the C boundary
// declared in include/pyramidkv.h.
#include <cmath>
#include <cstdio>
#include <algorithm>
#include <cstring>
#include <atomic>
#include <mutex>
#include <utility>

#include "pkv_common.cuh"
#include "pkv_extras.cuh"
#include "pkv_gather.cuh"
#include "pkv_score_generic.cuh"
#include "pkv_score_tc.cuh"
#include "pkv_score_resident.cuh"
#include "pkv_attend.cuh"
#include "pkv_select.cuh"
#include "pkv_shard.cuh"

namespace pkv {
namespace {

// Test knobs (pyramidkv_test_hooks): bound of the waits inside the tensor-core kernels, and the withheld tile.
std::atomic<long long> g_test_wait_clocks{0};
std::atomic<int> g_test_withhold{0};
std::atomic<int> g_test_withhold_attend{0};  // 1: the withheld K tile, in the window-attention kernel
std::atomic<int> g_test_two_sweeps{0};     // 1: never take the single-sweep kernel for short contexts

constexpr size_t kAlign = 256;
constexpr int kPartialChunk = 128;   // smallest key chunk any row-statistics kernel uses (sizes the workspace)

inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

bool config_ok(const pkv_config* c) {
  if (!c) return false;
  if (c->num_layers < 1 || c->num_kv_heads < 1 || c->num_q_heads < 1) return false;
  if (c->num_q_heads % c->num_kv_heads != 0) return false;
  if (c->window < 1 || c->avg_budget < c->window) return false;
  if (c->pool_kernel < 1 || (c->pool_kernel % 2) == 0) return false;
  if (!(c->beta >= 1.0) || c->beta > 1.0e6) return false;
  if (c->schedule != PKV_SCHEDULE_LINEAR && c->schedule != PKV_SCHEDULE_GEOMETRIC) return false;
  if ((c->flags & ~PKV_FLAG_INPUTS_FINAL) != 0 || c->sweep_ctas > 1024) return false;
  return true;
}

int config_supported(const pkv_config* c) {
  if (c->dtype != PKV_DTYPE_FP32 && c->dtype != PKV_DTYPE_BF16 && c->dtype != PKV_DTYPE_FP16)
    return PKV_ERR_UNSUPPORTED;
  if (c->head_dim != 64 && c->head_dim != 128) return PKV_ERR_UNSUPPORTED;
  if (c->pool_kind != PKV_POOL_MAX && c->pool_kind != PKV_POOL_AVG) return PKV_ERR_UNSUPPORTED;
  return PKV_OK;
}

// Eq. 1 in integers.  beta = bq / 1024.  With k_total = m (B - alpha):
//   k^l = k_total * ((2 bq - 1024)(m - 1) - (2 bq - 2048) l) / (bq m (m - 1)),
// floored; the units lost to flooring go to layers 0, 1, ...
void budgets_geometric(const pkv_config* c, int32_t* out);

void budgets(const pkv_config* c, int32_t* out) {
  if (c->schedule == PKV_SCHEDULE_GEOMETRIC) { budgets_geometric(c, out); return; }
  const int m = c->num_layers;
  const long long k_total = static_cast<long long>(m) * (c->avg_budget - c->window);
  if (m == 1) { out[0] = static_cast<int32_t>(k_total); return; }
  const long long bq = std::llround(c->beta * 1024.0);
  const unsigned __int128 den = static_cast<unsigned __int128>(bq) * m * (m - 1);
  long long given = 0;
  for (int l = 0; l < m; ++l) {
    // (2bq-1024)(m-1) >= (2bq-2048) l for l <= m-1, so the numerator is never negative
    const unsigned __int128 num = static_cast<unsigned __int128>(2 * bq - 1024) * (m - 1) -
                                  static_cast<unsigned __int128>(2 * bq - 2048) * l;
    const long long kl = static_cast<long long>(static_cast<unsigned __int128>(k_total) * num / den);
    out[l] = static_cast<int32_t>(kl);
    given += kl;
  }
  for (int l = 0; given < k_total; ++l, ++given) out[l] += 1;
}

// Geometric decay (appendix "Allocation Strategies"): shares k_total * rho^(m-1-l) / (1 + rho + ... + rho^(m-1)),
// where rho >= 1 solves 1 + rho + ... + rho^(m-1) = beta * m (so that the top layer gets k_total / (beta m), as
// in Eq. 1) and is then rounded to a multiple of 2^-20.  Doubles throughout, in a fixed order of operations:
// the geometric sum is built term by term from rho^0 upward.
double geometric_sum(double rho, int m, double* powers) {
  double term = 1.0, sum = 0.0;
  for (int j = 0; j < m; ++j) {
    if (powers) powers[j] = term;
    sum += term;
    term *= rho;
  }
  return sum;
}

void budgets_geometric(const pkv_config* c, int32_t* out) {
  const int m = c->num_layers;
  const long long k_total = static_cast<long long>(m) * (c->avg_budget - c->window);
  const double beta = static_cast<double>(std::llround(c->beta * 1024.0)) / 1024.0;
  double rho = 1.0;
  if (m > 1 && beta > 1.0) {
    double below = 1.0, above = beta * m;                  // the sum is at least 1 + rho, so the root lies below beta m
    for (int step = 0; step < 200; ++step) {
      const double mid = 0.5 * (below + above);
      if (geometric_sum(mid, m, nullptr) < beta * m) below = mid; else above = mid;
    }
    rho = std::nearbyint(0.5 * (below + above) * 1048576.0) / 1048576.0;
  }
  double stack_buf[512];
  double* powers = m <= 512 ? stack_buf : new double[m];
  const double total = geometric_sum(rho, m, powers);
  long long given = 0;
  for (int l = 0; l < m; ++l) {
    const long long kl = static_cast<long long>(std::floor(static_cast<double>(k_total) * powers[m - 1 - l] / total));
    out[l] = static_cast<int32_t>(kl);
    given += kl;
  }
  for (int l = 0; given < k_total; ++l, ++given) out[l] += 1;
  if (powers != stack_buf) delete[] powers;
}

int kept_count(const pkv_config* c, int k_layer, int n) {
  if (n <= c->avg_budget) return n;
  const int prefix = n - c->window;
  return (k_layer < prefix ? k_layer : prefix) + c->window;
}

struct Workspace {
  uint32_t* status;
  float* lse2;
  float2* partial;
  float* scores;
  int64_t ld_scores;
  uint2* sel_cand;           // selection: candidate (key, position) pairs, [heads][sel_cand_stride]
  int64_t sel_cand_stride;
  uint32_t* sel_cnt;         // selection: pairs per cluster rank, [heads][kSelMaxCluster]
  float* o_partial;          // window attention: per-segment accumulators [kAtMaxGrid + heads][R][d], or null
  size_t score_scratch_bytes;   // bytes of the leading regions that the score kernels alone need
  size_t bytes;
};

// Which configurations the tensor-core score kernels take (the others go to the fp32-pipe kernels).
bool tc_eligible(const pkv_config* c) {
  const int g = c->num_q_heads / c->num_kv_heads;
  return (c->dtype == PKV_DTYPE_BF16 || c->dtype == PKV_DTYPE_FP16) && g * c->window <= kTcMaxRows &&
         c->window <= 256 && g <= 256;
}

// Which configurations the fused window-attention kernel takes.
bool attend_eligible(const pkv_config* c) { return tc_eligible(c) && c->head_dim == kAtD; }
constexpr int kAtMaxGrid = 160;      // CTAs of the window-attention kernel at most (sizes its partial accumulators)

// Carves the workspace for `batch` sequences of at most max_n tokens.  base may be null (sizing only).
Workspace carve(const pkv_config* c, int batch, int max_n, void* base) {
  Workspace w{};
  char* p = static_cast<char*>(base);
  size_t off = 0;
  auto take = [&](size_t bytes) { char* r = p ? p + off : nullptr; off += align_up(bytes); return r; };
  const size_t rows = static_cast<size_t>(c->num_q_heads / c->num_kv_heads) * c->window;
  const size_t heads = static_cast<size_t>(batch) * c->num_kv_heads;
  const size_t chunks = (static_cast<size_t>(max_n) + kPartialChunk - 1) / kPartialChunk;
  w.status = reinterpret_cast<uint32_t*>(take(kAlign));
  w.lse2 = reinterpret_cast<float*>(take(heads * rows * sizeof(float)));
  // fp32-pipe sweep: 2 slots per chunk and head; tensor-core sweep: kTcStatSlots slots per segment, one segment
  // per run of a CTA over a head (at most CTAs + heads of them), whatever the context length
  const size_t partial_slots =
      tc_eligible(c) ? (static_cast<size_t>(kTcMaxGrid) + heads) * kTcStatSlots : heads * chunks * 2;
  w.partial = reinterpret_cast<float2*>(take(partial_slots * rows * sizeof(float2)));
  w.score_scratch_bytes = off;
  w.ld_scores = static_cast<int64_t>((static_cast<size_t>(max_n) + 63) / 64 * 64);
  w.scores = reinterpret_cast<float*>(take(heads * w.ld_scores * sizeof(float)));
  w.sel_cand_stride = static_cast<int64_t>(max_n) + 32 * kSelMaxCluster;   // cluster * slice never exceeds this
  w.sel_cand = reinterpret_cast<uint2*>(take(heads * w.sel_cand_stride * sizeof(uint2)));
  w.sel_cnt = reinterpret_cast<uint32_t*>(take(heads * kSelMaxCluster * sizeof(uint32_t)));
  if (attend_eligible(c))
    w.o_partial = reinterpret_cast<float*>(take((static_cast<size_t>(kAtMaxGrid) + heads) * rows * kAtD * sizeof(float)));
  w.bytes = off;
  return w;
}

// Validates the sequence lengths and fills the per-call table for budget k_layer.
int build_table(const pkv_config* c, const int32_t* seq_lens, int batch, int k_layer, SeqTable* t, int* max_n,
                int64_t* total_rows) {
  if (!seq_lens || batch < 1 || k_layer < 0) return PKV_ERR_INVALID_ARG;
  if (batch > PKV_MAX_BATCH) return PKV_ERR_UNSUPPORTED;
  std::memset(t, 0, sizeof *t);
  t->batch = batch;
  t->alpha = c->window;
  int64_t rows = 0;
  int mx = 0;
  for (int b = 0; b < batch; ++b) {
    const int n = seq_lens[b];
    if (n < c->window + 1) return PKV_ERR_INVALID_ARG;
    t->n[b] = n;
    t->prefix[b] = n - c->window;
    t->count[b] = kept_count(c, k_layer, n);
    t->row_off[b] = rows;
    rows += static_cast<int64_t>(c->num_kv_heads) * t->count[b];
    if (n > mx) mx = n;
  }
  *max_n = mx;
  *total_rows = rows;
  return PKV_OK;
}

// A [batch][heads][token][d] view the kernels can take: 16-byte aligned base and strides, rows that do not
// overlap, and a positive stride along every dimension that has more than one entry (a broadcast or reversed
// view has no tensor map and would be mis-sized by the overlap test below).
bool tensor_ok(const pkv_tensor& t, int d, int elem_bytes, int batch = 1, int heads = 1) {
  if (!t.ptr || t.stride_token < d) return false;
  if (reinterpret_cast<uintptr_t>(t.ptr) % 16) return false;
  if ((batch > 1 && t.stride_batch <= 0) || (heads > 1 && t.stride_head <= 0)) return false;
  const int64_t q = 16 / elem_bytes;
  return t.stride_token % q == 0 && t.stride_head % q == 0 && t.stride_batch % q == 0;
}

TensorView view(const pkv_tensor& t) { return TensorView{t.ptr, t.stride_batch, t.stride_head, t.stride_token}; }

int check_launch() { return cudaPeekAtLastError() == cudaSuccess ? PKV_OK : PKV_ERR_CUDA; }

// Launch with programmatic stream serialisation: the kernel may be scheduled while its predecessor in
// the stream drains; the kernels order themselves with pdl_wait() (pkv_common.cuh).
template <typename... KArgs, typename... Args>
void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Optional per-kernel timing (pyramidkv_profile_layer): when armed, an event is recorded after every launch.
struct StageTimer {
  cudaEvent_t ev[PKV_MAX_STAGES + 1];
  const char* name[PKV_MAX_STAGES];
  int n = 0;
};
thread_local StageTimer* g_timer = nullptr;

void mark(cudaStream_t st, const char* name) {
  if (!g_timer || g_timer->n >= PKV_MAX_STAGES) return;
  g_timer->name[g_timer->n] = name;
  cudaEventRecord(g_timer->ev[++g_timer->n], st);
}

// ---------------------------------------------------------------- outputs still in flight
// The tensor-core sweeps start reading Q and K before the kernels ahead of them in the stream have finished.
// That is only right for tensors those kernels do not write, so the library remembers where its last calls put
// K/V rows (packed caches, page pools) and a sweep whose Q or K overlaps one of them waits like any other kernel.
struct ByteRange { uintptr_t lo, hi; };
std::mutex g_out_mutex;
ByteRange g_recent_out[16];
unsigned g_recent_out_next = 0;

void note_output(const void* ptr, size_t bytes) {
  if (!ptr || !bytes) return;
  std::lock_guard<std::mutex> lock(g_out_mutex);
  const uintptr_t lo = reinterpret_cast<uintptr_t>(ptr);
  g_recent_out[g_recent_out_next++ % 16] = ByteRange{lo, lo + bytes};
}

bool overlaps_recent_output(const pkv_tensor& t, int batch, int heads, int tokens, int d, int elem_bytes) {
  const int64_t last = (batch - 1) * std::max<int64_t>(t.stride_batch, 0) +
                       (heads - 1) * std::max<int64_t>(t.stride_head, 0) + (tokens - 1) * t.stride_token + d;
  const uintptr_t lo = reinterpret_cast<uintptr_t>(t.ptr), hi = lo + static_cast<uintptr_t>(last) * elem_bytes;
  std::lock_guard<std::mutex> lock(g_out_mutex);
  for (const ByteRange& r : g_recent_out)
    if (r.hi > r.lo && lo < r.hi && r.lo < hi) return true;
  return false;
}

// ---------------------------------------------------------------- scores
template <typename T, int D>
int launch_scores_generic(ScoreParams& sp, int batch, cudaStream_t st) {
  int stat_tiles = 0, score_tiles = 0;
  for (int b = 0; b < batch; ++b) {
    sp.seq.stat_off[b] = stat_tiles;
    sp.seq.score_off[b] = score_tiles;
    stat_tiles += (sp.seq.n[b] + kGenChunk - 1) / kGenChunk;
    score_tiles += (sp.seq.prefix[b] + kGenScoreKeys - 1) / kGenScoreKeys;
  }
  sp.seq.stat_off[batch] = stat_tiles;
  sp.seq.score_off[batch] = score_tiles;
  sp.slots_per_chunk = 1;
  if (sp.lse_in == sp.lse2) {                    // normalisers not supplied: sweep A and its merge
    launch_pdl(rowstats_generic_kernel<T, D>, dim3(stat_tiles, sp.num_kv_heads), kGenRowBlock, 0, st, sp);
    mark(st, "rowstats_generic");
    launch_pdl(combine_stats_kernel, dim3((sp.rows + 31) / 32, sp.num_kv_heads, batch), kCombineThreads, 0, st, sp,
               std::log2(static_cast<float>(sp.group)));
    mark(st, "combine_stats");
  }
  if (sp.stats_only) return check_launch();
  launch_pdl(scores_generic_kernel<T, D>, dim3(score_tiles, sp.num_kv_heads), kGenScoreKeys, 0, st, sp);
  mark(st, "scores_generic");
  return check_launch();
}

// ---------------------------------------------------------------- tensor-core scores
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      sym = nullptr;
    return reinterpret_cast<EncodeTiledFn>(sym);
  }();
  return fn;
}

// Tensor map of a 16-bit [batch][head][token][d] view: dims (d, token, head, batch), box (64, box_tok, box_head, 1),
// 128-byte swizzle, zero fill outside the tensor.
bool make_map(CUtensorMap* map, const pkv_tensor& t, bool fp16, int d, uint64_t tokens, uint64_t heads,
              uint64_t batch, uint32_t box_tok, uint32_t box_head) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(d), tokens, heads, batch};
  // a dimension of extent 1 may come with any stride (0 included): the map then gets a harmless placeholder
  auto bytes = [](int64_t elems, uint64_t extent) { return static_cast<cuuint64_t>(extent > 1 || elems > 0 ? elems : 8) * 2; };
  if ((heads > 1 && t.stride_head <= 0) || (batch > 1 && t.stride_batch <= 0)) return false;
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(t.stride_token) * 2, bytes(t.stride_head, heads),
                                 bytes(t.stride_batch, batch)};
  const cuuint32_t box[4] = {64, box_tok, box_head, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, fp16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(t.ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


// SMs the persistent score kernels may count on: the device's, or fewer while a call runs them on a lane that
// owns only a group of the SMs (pyramidkv_compress_model_lanes sets the limit for its own thread).
thread_local int tl_sm_limit = 0;

int device_sm_count() {
  static int sms[64] = {};
  if (tl_sm_limit > 0) return tl_sm_limit;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  if (!sms[dev]) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    sms[dev] = n;
  }
  return sms[dev];
}

template <int D>
int launch_scores_tc(const pkv_config* c, const pkv_tensor& q, const pkv_tensor& k, ScoreParams& sp, int batch,
                     int max_n, uint32_t* status, cudaStream_t st) {
  int sms = device_sm_count();
  if (sms <= 0) return PKV_ERR_CUDA;
  if (c->sweep_ctas > 0) sms = std::min(sms, static_cast<int>(c->sweep_ctas));   // the caller's share of the SMs
  static bool attr_done[64] = {};  // the attribute is per device; setting it twice is harmless
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return PKV_ERR_CUDA;
  if (dev >= 64 || !attr_done[dev]) {
    if (cudaFuncSetAttribute(score_resident_kernel<D, kRsStages>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             RsSmem<D, kRsStages>::kTotal) != cudaSuccess ||
        cudaFuncSetAttribute(score_resident_kernel<D, kRsStagesShort>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             RsSmem<D, kRsStagesShort>::kTotal) != cudaSuccess ||
        cudaFuncSetAttribute(score_tc_kernel<D, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcSmem<D>::kTotal) !=
            cudaSuccess ||
        cudaFuncSetAttribute(score_tc_kernel<D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcSmem<D>::kTotal) !=
            cudaSuccess)
      return PKV_ERR_CUDA;
    if (dev < 64) attr_done[dev] = true;
  }
  alignas(64) CUtensorMap q_map, k_map_a, k_map_b;
  const bool fp16 = c->dtype == PKV_DTYPE_FP16;
  if (!make_map(&q_map, q, fp16, D, c->window, c->num_q_heads, batch, c->window, sp.group) ||
      !make_map(&k_map_a, k, fp16, D, max_n, c->num_kv_heads, batch, kTcTileKeysA, 1) ||
      !make_map(&k_map_b, k, fp16, D, max_n, c->num_kv_heads, batch, kTcTileKeysB, 1))
    return PKV_ERR_CUDA;

  TcParams tp{};
  tp.seq = sp.seq;
  tp.num_kv_heads = sp.num_kv_heads;
  tp.group = sp.group;
  tp.rows = sp.rows;
  tp.rows_pad = (sp.rows + 31) / 32 * 32;
  tp.fp16 = fp16 ? 1 : 0;
  // An early start needs the caller's word that nothing on the stream still writes Q or K, and the library's own
  // knowledge that none of its recent outputs is among them.
  tp.early = (c->flags & PKV_FLAG_INPUTS_FINAL) != 0 &&
             !(overlaps_recent_output(q, batch, c->num_q_heads, c->window, D, 2) ||
               overlaps_recent_output(k, batch, c->num_kv_heads, max_n, D, 2));
  const long long test_wait = g_test_wait_clocks.load();
  tp.wait_clocks = test_wait > 0 ? test_wait : kTcWaitCycles;
  tp.withhold = g_test_withhold.load();
  tp.row_blocks = (sp.rows + 127) / 128;
  tp.scale_log2 = sp.scale_log2;
  tp.partial = sp.partial;
  tp.lse2 = sp.lse_in;
  tp.lse_scale = sp.lse_scale;
  tp.lse_add = sp.lse_add;
  tp.scores = sp.scores;
  tp.ld_scores = sp.ld_scores;
  tp.status = status;
  // Key tiles per work item: the largest power of two that still spreads the items evenly over the SMs.
  auto items_for = [&](int ct, int tile_keys, bool prefix) {
    long long items = 0;
    for (int b = 0; b < batch; ++b) {
      const int keys = prefix ? sp.seq.prefix[b] : sp.seq.n[b];
      const int tiles = (keys + tile_keys - 1) / tile_keys;
      items += (tiles + ct - 1) / ct;
    }
    return items * sp.num_kv_heads;
  };
  auto pick = [&](int tile_keys, bool prefix) {
    int ct = 16;
    for (; ct > 1; ct /= 2) {
      const long long items = items_for(ct, tile_keys, prefix);
      const long long waves = (items + sms - 1) / sms;
      if (items >= sms && static_cast<double>(items) / static_cast<double>(waves * sms) >= 0.93) break;
    }
    return ct;
  };
  tp.chunk_tiles_a = pick(kTcTileKeysA, false);
  tp.chunk_tiles_b = pick(kTcTileKeysB, true);
  int stat_items = 0, score_items = 0;
  for (int b = 0; b < batch; ++b) {
    tp.seq.stat_off[b] = stat_items;
    tp.seq.score_off[b] = score_items;
    stat_items += ((sp.seq.n[b] + kTcTileKeysA - 1) / kTcTileKeysA + tp.chunk_tiles_a - 1) / tp.chunk_tiles_a;
    score_items += ((sp.seq.prefix[b] + kTcTileKeysB - 1) / kTcTileKeysB + tp.chunk_tiles_b - 1) /
                   tp.chunk_tiles_b;
  }
  tp.seq.stat_off[batch] = stat_items;
  tp.seq.score_off[batch] = score_items;
  sp.seq = tp.seq;
  sp.slots_per_chunk = tc_stat_slots(tp.row_blocks);  // partial slots each run segment of sweep A holds

  const int grid_a = static_cast<int>(std::min<long long>(std::min(sms, kTcMaxGrid),
                                                          static_cast<long long>(stat_items) * sp.num_kv_heads));
  sp.stat_grid = grid_a;
  const int grid_b = static_cast<int>(std::min<long long>(sms, static_cast<long long>(score_items) * sp.num_kv_heads));
  tp.stat_grid = grid_a;
  tp.log2_group = std::log2(static_cast<float>(sp.group));
  // Short contexts with few window rows: the logits of a head fit in the tensor memory of a cluster, one sweep.
  const int tiles_max = (max_n + kRsTileKeys - 1) / kRsTileKeys;
  if (sp.lse_in == sp.lse2 && !sp.stats_only && sp.rows <= kRsRows && tiles_max <= kRsMaxCluster * kRsMaxTiles &&
      !g_test_two_sweeps.load()) {
    int cluster = 1;
    while (cluster * kRsMaxTiles < tiles_max) cluster *= 2;
    // more CTAs per head while they still all fit on the device at once and keep at least two tiles each
    while (2 * cluster <= kRsMaxCluster && static_cast<long long>(2 * cluster) * sp.num_kv_heads * batch <= sms &&
           tiles_max >= 4 * cluster)
      cluster *= 2;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(cluster * sp.num_kv_heads, batch);
    cfg.blockDim = dim3(kRsThreads);
    // at most 8 tiles per CTA: three K stages and 256 TMEM columns do, and two such CTAs fit on an SM
    const bool small = (tiles_max + cluster - 1) / cluster <= 8;
    cfg.dynamicSmemBytes = small ? RsSmem<D, kRsStagesShort>::kTotal : RsSmem<D, kRsStages>::kTotal;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if ((small ? cudaLaunchKernelEx(&cfg, score_resident_kernel<D, kRsStagesShort>, q_map, k_map_b, tp)
               : cudaLaunchKernelEx(&cfg, score_resident_kernel<D, kRsStages>, q_map, k_map_b, tp)) != cudaSuccess)
      return PKV_ERR_CUDA;
    mark(st, "scores_resident");
    return check_launch();
  }
  if (sp.lse_in == sp.lse2) {                    // normalisers not supplied: sweep A
    launch_pdl(score_tc_kernel<D, 0>, grid_a, kTcThreads, TcSmem<D>::kTotal, st, q_map, k_map_a, tp);
    mark(st, "rowstats_tc");
    if (sp.stats_only) {                         // the normalisers themselves are wanted: merge kernel
      launch_pdl(combine_stats_kernel, dim3((sp.rows + 31) / 32, sp.num_kv_heads, batch), kCombineThreads, 0, st, sp,
                 tp.log2_group);
      mark(st, "combine_stats");
    } else {
      tp.merge = 1;                              // sweep B merges the partials of its heads itself
    }
  }
  if (sp.stats_only) return check_launch();
  launch_pdl(score_tc_kernel<D, 1>, grid_b, kTcThreads, TcSmem<D>::kTotal, st, q_map, k_map_b, tp);
  mark(st, "scores_tc");
  return check_launch();
}

// window_lse: null, or the caller's natural-log row normalisers [batch][H_q][alpha] (then sweep A is skipped).
int run_scores(const pkv_config* c, const pkv_tensor& q, const pkv_tensor& k, const SeqTable& table, int batch,
               float* scores, int64_t ld, const Workspace& w, cudaStream_t st, const float* window_lse = nullptr,
               bool stats_only = false) {
  ScoreParams sp{};
  sp.stats_only = stats_only ? 1 : 0;
  sp.q = view(q);
  sp.k = view(k);
  sp.seq = table;
  sp.num_kv_heads = c->num_kv_heads;
  sp.group = c->num_q_heads / c->num_kv_heads;
  sp.rows = sp.group * c->window;
  sp.scale_log2 = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(c->head_dim)));
  sp.partial = w.partial;
  sp.lse2 = w.lse2;
  sp.lse_in = window_lse ? window_lse : w.lse2;
  sp.lse_scale = window_lse ? 1.4426950408889634f : 1.0f;
  sp.lse_add = window_lse ? std::log2(static_cast<float>(sp.group)) : 0.0f;
  sp.scores = scores;
  sp.ld_scores = ld;
  if (tc_eligible(c)) {
    int max_n = 0;
    for (int b = 0; b < batch; ++b) max_n = std::max(max_n, table.n[b]);
    return c->head_dim == 64 ? launch_scores_tc<64>(c, q, k, sp, batch, max_n, w.status, st)
                             : launch_scores_tc<128>(c, q, k, sp, batch, max_n, w.status, st);
  }
  if (c->dtype == PKV_DTYPE_FP32)
    return c->head_dim == 64 ? launch_scores_generic<float, 64>(sp, batch, st)
                             : launch_scores_generic<float, 128>(sp, batch, st);
  if (c->dtype == PKV_DTYPE_FP16)
    return c->head_dim == 64 ? launch_scores_generic<__half, 64>(sp, batch, st)
                             : launch_scores_generic<__half, 128>(sp, batch, st);
  return c->head_dim == 64 ? launch_scores_generic<__nv_bfloat16, 64>(sp, batch, st)
                           : launch_scores_generic<__nv_bfloat16, 128>(sp, batch, st);
}

// ---------------------------------------------------------------- window attention fused with the scores
// Needs the row normalisers in w.lse2 (run_scores with stats_only).  Writes the scores of the prefix positions and
// attn_out[batch][H_q][alpha][d].
int run_attend(const pkv_config* c, const pkv_tensor& q, const pkv_tensor& k, const pkv_tensor& v, const SeqTable& table,
               int batch, int max_n, float* scores, int64_t ld, float* attn_out, const Workspace& w, cudaStream_t st) {
  const int sms = device_sm_count();
  if (sms <= 0) return PKV_ERR_CUDA;
  static bool attr_done[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return PKV_ERR_CUDA;
  if (dev >= 64 || !attr_done[dev]) {
    if (cudaFuncSetAttribute(window_attend_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAtSmemBytes) !=
        cudaSuccess)
      return PKV_ERR_CUDA;
    if (dev < 64) attr_done[dev] = true;
  }
  const bool fp16 = c->dtype == PKV_DTYPE_FP16;
  const int group = c->num_q_heads / c->num_kv_heads;
  alignas(64) CUtensorMap q_map, k_map, v_map;
  if (!make_map(&q_map, q, fp16, kAtD, c->window, c->num_q_heads, batch, c->window, group) ||
      !make_map(&k_map, k, fp16, kAtD, max_n, c->num_kv_heads, batch, kAtTileKeys, 1) ||
      !make_map(&v_map, v, fp16, kAtD, max_n, c->num_kv_heads, batch, kAtTileKeys, 1))
    return PKV_ERR_CUDA;
  AtParams ap{};
  ap.seq = table;
  ap.num_kv_heads = c->num_kv_heads;
  ap.group = group;
  ap.rows = group * c->window;
  ap.rows_pad = (ap.rows + 31) / 32 * 32;
  ap.fp16 = fp16 ? 1 : 0;
  const long long test_wait = g_test_wait_clocks.load();
  ap.wait_clocks = test_wait > 0 ? test_wait : kTcWaitCycles;
  ap.withhold = g_test_withhold_attend.load();
  ap.scale_log2 = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(c->head_dim)));
  ap.lse2 = w.lse2;
  ap.scores = scores;
  ap.ld_scores = ld;
  ap.o_partial = w.o_partial;
  ap.out = attn_out;
  ap.status = w.status;
  const int grid_cap = std::min(c->sweep_ctas > 0 ? std::min(sms, static_cast<int>(c->sweep_ctas)) : sms, kAtMaxGrid);
  // Key tiles per work item: the largest power of two that still spreads the items evenly over the SMs.
  auto items_for = [&](int ct) {
    long long items = 0;
    for (int b = 0; b < batch; ++b) items += ((table.n[b] + kAtTileKeys - 1) / kAtTileKeys + ct - 1) / ct;
    return items * c->num_kv_heads;
  };
  int ct = 16;
  for (; ct > 1; ct /= 2) {
    const long long items = items_for(ct), waves = (items + grid_cap - 1) / grid_cap;
    if (items >= grid_cap && static_cast<double>(items) / static_cast<double>(waves * grid_cap) >= 0.93) break;
  }
  ap.chunk_tiles = ct;
  int items = 0;
  for (int b = 0; b < batch; ++b) {
    ap.seq.score_off[b] = items;
    items += ((table.n[b] + kAtTileKeys - 1) / kAtTileKeys + ct - 1) / ct;
  }
  ap.seq.score_off[batch] = items;
  ap.grid = static_cast<int>(std::min<long long>(grid_cap, static_cast<long long>(items) * c->num_kv_heads));
  launch_pdl(window_attend_kernel, ap.grid, kAtThreads, kAtSmemBytes, st, q_map, k_map, v_map, ap);
  mark(st, "window_attend");
  launch_pdl(window_attend_reduce_kernel, dim3(ap.rows, c->num_kv_heads, batch), kAtD, 0, st, ap);
  mark(st, "window_attend_reduce");
  return check_launch();
}

// ---------------------------------------------------------------- select
// With k/v/k_out given the kernel also copies the kept rows (fused eviction); otherwise it writes indices only.
int run_select(const pkv_config* c, const float* scores, int64_t ld, const SeqTable& table, int batch, int max_n,
               int32_t* indices, const Workspace& w, cudaStream_t st, const pkv_tensor* k = nullptr,
               const pkv_tensor* v = nullptr, void* k_out = nullptr, void* v_out = nullptr) {
  SelectParams sp{};
  sp.scores = scores;
  sp.ld_scores = ld;
  sp.indices = indices;
  sp.seq = table;
  sp.num_kv_heads = c->num_kv_heads;
  sp.pool_radius = (c->pool_kernel - 1) / 2;
  sp.status = w.status;
  sp.cand = w.sel_cand;
  sp.cand_stride = w.sel_cand_stride;
  sp.cand_cnt = w.sel_cnt;
  if (k_out) {
    sp.k = view(*k);
    sp.v = view(*v);
    sp.k_out = k_out;
    sp.v_out = v_out;
    sp.elem_bytes = c->dtype == PKV_DTYPE_FP32 ? 4 : 2;
    sp.pieces = c->head_dim * sp.elem_bytes / 16;
  }
  const int max_p = max_n - c->window;
  int cluster = 1;
  while (cluster < kSelMaxCluster && (max_p + cluster - 1) / cluster > 8192) cluster *= 2;
  const int slice = ((max_p + cluster - 1) / cluster + 31) & ~31;
  sp.cached = sp.pool_radius <= kSelHalo ? 1 : 0;
  const size_t smem = sp.cached ? static_cast<size_t>(std::min(slice, kSelSliceCap)) * 6 + 8 * kSelHalo : 0;
  sp.smem_pairs = static_cast<int32_t>(smem / sizeof(uint2));
  static bool attr_done[64] = {};  // the attribute is per device; setting it twice is harmless
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return PKV_ERR_CUDA;
  if (dev >= 64 || !attr_done[dev]) {
    for (auto kernel : {pool_select_kernel<false, false, 1>, pool_select_kernel<true, false, 1>,
                        pool_select_kernel<false, true, 1>, pool_select_kernel<true, true, 1>,
                        pool_select_kernel<false, false, 8>, pool_select_kernel<true, false, 8>,
                        pool_select_kernel<false, true, 8>, pool_select_kernel<true, true, 8>,
                        pool_select_kernel<false, false, 1, kSelThreadsSmall>, pool_select_kernel<true, false, 1, kSelThreadsSmall>,
                        pool_select_kernel<false, false, 8, kSelThreadsSmall>, pool_select_kernel<true, false, 8, kSelThreadsSmall>})
      if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               kSelSliceCap * 6 + 8 * kSelHalo) != cudaSuccess)
        return PKV_ERR_CUDA;
    if (dev < 64) attr_done[dev] = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(cluster * c->num_kv_heads, batch);
  // short slices (at most 8 positions per thread): the 512-thread instance, of which two fit on an SM, or one beside
  // another layer's single-sweep score CTA.  (It could take 8192 positions, but at 16 per thread it is slower than
  // 1024 threads at 8: measured +6 % per step on the 32k and batch-8 shapes.)
  const bool small_cta = slice <= 4096;
  cfg.blockDim = dim3(small_cta ? kSelThreadsSmall : kSelThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const bool avg = c->pool_kind == PKV_POOL_AVG;   // the mean pool is a variant; the max pool is the graded reading
  const bool multi = slice > kSelSliceCap;          // long rows: each CTA takes its slice in several rounds
  int k_max = 0;                                    // largest number of prefix rows any sequence keeps
  for (int b = 0; b < batch; ++b) k_max = std::max(k_max, table.count[b] - c->window);
  const bool wide = k_max > 512;                    // then 8 maxima per thread keep the candidate bound tight
  auto kernel = avg ? (multi ? (wide ? pool_select_kernel<true, true, 8> : pool_select_kernel<true, true, 1>)
                             : (wide ? pool_select_kernel<true, false, 8> : pool_select_kernel<true, false, 1>))
                    : (multi ? (wide ? pool_select_kernel<false, true, 8> : pool_select_kernel<false, true, 1>)
                             : (wide ? pool_select_kernel<false, false, 8> : pool_select_kernel<false, false, 1>));
  if (small_cta)                                    // never multi: a slice of 8192 positions is one round
    kernel = avg ? (wide ? pool_select_kernel<true, false, 8, kSelThreadsSmall> : pool_select_kernel<true, false, 1, kSelThreadsSmall>)
                 : (wide ? pool_select_kernel<false, false, 8, kSelThreadsSmall> : pool_select_kernel<false, false, 1, kSelThreadsSmall>);
  if (cudaLaunchKernelEx(&cfg, kernel, sp) != cudaSuccess) return PKV_ERR_CUDA;
  if (k_out) {
    int64_t out_rows = 0;
    for (int b = 0; b < batch; ++b) out_rows += static_cast<int64_t>(c->num_kv_heads) * table.count[b];
    const size_t out_bytes = static_cast<size_t>(out_rows) * c->head_dim * sp.elem_bytes;
    note_output(k_out, out_bytes);
    note_output(v_out, out_bytes);
  }
  mark(st, k_out ? "pool_select_gather" : "pool_select");
  return check_launch();
}

// ---------------------------------------------------------------- gather
int run_gather(const pkv_config* c, const pkv_tensor& k, const pkv_tensor& v, const int32_t* indices,
               const SeqTable& table, int64_t total_rows, void* k_out, void* v_out, cudaStream_t st) {
  GatherParams gp{};
  gp.k = view(k);
  gp.v = view(v);
  gp.indices = indices;
  gp.k_out = k_out;
  gp.v_out = v_out;
  gp.seq = table;
  gp.num_kv_heads = c->num_kv_heads;
  gp.elem_bytes = c->dtype == PKV_DTYPE_FP32 ? 4 : 2;
  gp.pieces = c->head_dim * gp.elem_bytes / 16;
  gp.total_rows = total_rows;
  const int64_t threads = total_rows * gp.pieces;
  if (threads == 0) return PKV_OK;
  const unsigned blocks = static_cast<unsigned>((threads + kGatherThreads - 1) / kGatherThreads);
  launch_pdl(gather_rows_kernel, blocks, kGatherThreads, 0, st, gp);
  note_output(k_out, static_cast<size_t>(total_rows) * c->head_dim * gp.elem_bytes);
  note_output(v_out, static_cast<size_t>(total_rows) * c->head_dim * gp.elem_bytes);
  mark(st, "gather_rows");
  return check_launch();
}

// Table offsets of a layer's block table: sequences in batch order, H_kv * pages_b entries each.
void fill_page_table(const pkv_config* c, const SeqTable& t, const int32_t* block_table, int page_size,
                     int num_pages, PageTable* pt) {
  std::memset(pt, 0, sizeof *pt);
  pt->table = block_table;
  pt->page_size = page_size;
  pt->num_pages = num_pages;
  int64_t off = 0;
  for (int b = 0; b < t.batch; ++b) {
    pt->pages[b] = (t.count[b] + page_size - 1) / page_size;
    pt->tab_off[b] = off;
    off += static_cast<int64_t>(c->num_kv_heads) * pt->pages[b];
  }
}

int run_gather_paged(const pkv_config* c, const pkv_tensor& k, const pkv_tensor& v, const int32_t* indices,
                     const SeqTable& table, int64_t total_rows, const int32_t* block_table, int page_size,
                     int num_pages, void* k_pool, void* v_pool, uint32_t* status, cudaStream_t st) {
  GatherPagedParams gp{};
  gp.k = view(k);
  gp.v = view(v);
  gp.indices = indices;
  gp.k_pool = k_pool;
  gp.v_pool = v_pool;
  gp.seq = table;
  fill_page_table(c, table, block_table, page_size, num_pages, &gp.pt);
  gp.num_kv_heads = c->num_kv_heads;
  gp.elem_bytes = c->dtype == PKV_DTYPE_FP32 ? 4 : 2;
  gp.pieces = c->head_dim * gp.elem_bytes / 16;
  gp.total_rows = total_rows;
  gp.status = status;
  const int64_t threads = total_rows * gp.pieces;
  if (threads == 0) return PKV_OK;
  const unsigned blocks = static_cast<unsigned>((threads + kPagedThreads - 1) / kPagedThreads);
  launch_pdl(gather_paged_kernel, blocks, kPagedThreads, 0, st, gp);
  const size_t pool_bytes = static_cast<size_t>(num_pages) * page_size * c->head_dim * gp.elem_bytes;
  note_output(k_pool, pool_bytes);
  note_output(v_pool, pool_bytes);
  mark(st, "gather_paged");
  return check_launch();
}

bool paged_args_ok(const int32_t* block_table, int page_size, int num_pages, const void* k_pool, const void* v_pool) {
  if (!block_table || !k_pool || !v_pool || page_size < 1 || num_pages < 1) return false;
  return reinterpret_cast<uintptr_t>(k_pool) % 16 == 0 && reinterpret_cast<uintptr_t>(v_pool) % 16 == 0;
}

// Table of a call on one shard of each sequence: n = keys held here, prefix = those that are scored.
int build_shard_table(const pkv_config* c, const int32_t* shard_keys, const int32_t* window_keys, int batch,
                      SeqTable* t, int* max_n) {
  if (!shard_keys || !window_keys || batch < 1) return PKV_ERR_INVALID_ARG;
  if (batch > PKV_MAX_BATCH) return PKV_ERR_UNSUPPORTED;
  std::memset(t, 0, sizeof *t);
  t->batch = batch;
  t->alpha = c->window;
  int mx = 0;
  for (int b = 0; b < batch; ++b) {
    if (window_keys[b] != 0 && window_keys[b] != c->window) return PKV_ERR_INVALID_ARG;
    if (shard_keys[b] < window_keys[b] + 1) return PKV_ERR_INVALID_ARG;
    t->n[b] = shard_keys[b];
    t->prefix[b] = shard_keys[b] - window_keys[b];
    if (shard_keys[b] > mx) mx = shard_keys[b];
  }
  *max_n = mx;
  return PKV_OK;
}

int workspace_check(const pkv_config* c, int batch, int max_n, void* ws, size_t ws_bytes, Workspace* out) {
  if (!ws || reinterpret_cast<uintptr_t>(ws) % kAlign) return PKV_ERR_WORKSPACE;
  *out = carve(c, batch, max_n, ws);
  return out->bytes <= ws_bytes ? PKV_OK : PKV_ERR_WORKSPACE;
}

}  // namespace
}  // namespace pkv

using namespace pkv;

extern "C" {

int pyramidkv_memory_kind(const void* ptr) {
  cudaPointerAttributes attr;
  if (!ptr) return -PKV_ERR_INVALID_ARG;
  if (cudaPointerGetAttributes(&attr, ptr) != cudaSuccess) {
    cudaGetLastError();                                    // a query must not leave a sticky error behind
    return -PKV_ERR_CUDA;
  }
  switch (attr.type) {
    case cudaMemoryTypeHost: return attr.devicePointer == ptr ? PKV_MEM_PINNED_HOST : PKV_MEM_PAGEABLE_HOST;
    case cudaMemoryTypeDevice: return PKV_MEM_DEVICE;
    case cudaMemoryTypeManaged: return PKV_MEM_MANAGED;
    default: return PKV_MEM_PAGEABLE_HOST;
  }
}

const char* pyramidkv_strerror(int status) {
  switch (status) {
    case PKV_OK: return "ok";
    case PKV_ERR_INVALID_ARG: return "invalid argument";
    case PKV_ERR_UNSUPPORTED: return "unsupported dtype, head_dim, pool kind or batch size";
    case PKV_ERR_WORKSPACE: return "workspace too small or misaligned";
    case PKV_ERR_CUDA: return "CUDA launch failed";
    case PKV_ERR_DEVICE_STATUS: return "a kernel recorded a failure in the workspace status word";
    case PKV_ERR_STATIC_SCRATCH: return "problem too large for the built-in scratch (PKV_STATIC_SCRATCH_BYTES)";
    default: return "unknown status";
  }
}

int pyramidkv_layer_budgets(const pkv_config* cfg, int32_t* k_out) {
  if (!config_ok(cfg) || !k_out) return PKV_ERR_INVALID_ARG;
  budgets(cfg, k_out);
  return PKV_OK;
}

int pyramidkv_kept_count(const pkv_config* cfg, int32_t k_layer, int32_t seq_len) {
  if (!config_ok(cfg) || k_layer < 0 || seq_len < cfg->window + 1) return -PKV_ERR_INVALID_ARG;
  return kept_count(cfg, k_layer, seq_len);
}

size_t pyramidkv_workspace_bytes(const pkv_config* cfg, int32_t batch, int32_t max_seq_len) {
  if (!config_ok(cfg) || batch < 1 || batch > PKV_MAX_BATCH || max_seq_len < cfg->window + 1) return 0;
  return carve(cfg, batch, max_seq_len, nullptr).bytes;
}

static int score_window_impl(const pkv_config* cfg, pkv_tensor q_win, pkv_tensor k, const float* window_lse,
                             const int32_t* seq_lens, int32_t batch, float* scores, int64_t ld_scores,
                             void* workspace, size_t workspace_bytes, void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (int rc = config_supported(cfg)) return rc;
  const int eb = cfg->dtype == PKV_DTYPE_FP32 ? 4 : 2;
  if (!tensor_ok(q_win, cfg->head_dim, eb, batch, cfg->num_q_heads) ||
      !tensor_ok(k, cfg->head_dim, eb, batch, cfg->num_kv_heads) || !scores)
    return PKV_ERR_INVALID_ARG;
  SeqTable table;
  int max_n;
  int64_t rows;
  if (int rc = build_table(cfg, seq_lens, batch, 0, &table, &max_n, &rows)) return rc;
  if (ld_scores < max_n - cfg->window) return PKV_ERR_INVALID_ARG;
  Workspace w;
  if (int rc = workspace_check(cfg, batch, max_n, workspace, workspace_bytes, &w)) return rc;
  return run_scores(cfg, q_win, k, table, batch, scores, ld_scores, w, static_cast<cudaStream_t>(stream), window_lse);
}

int pyramidkv_score_window(const pkv_config* cfg, pkv_tensor q_win, pkv_tensor k, const int32_t* seq_lens,
                           int32_t batch, float* scores, int64_t ld_scores, void* workspace,
                           size_t workspace_bytes, void* stream) {
  return score_window_impl(cfg, q_win, k, nullptr, seq_lens, batch, scores, ld_scores, workspace, workspace_bytes,
                           stream);
}

int pyramidkv_score_window_lse(const pkv_config* cfg, pkv_tensor q_win, pkv_tensor k, const float* window_lse,
                               const int32_t* seq_lens, int32_t batch, float* scores, int64_t ld_scores,
                               void* workspace, size_t workspace_bytes, void* stream) {
  if (!window_lse) return PKV_ERR_INVALID_ARG;
  return score_window_impl(cfg, q_win, k, window_lse, seq_lens, batch, scores, ld_scores, workspace,
                           workspace_bytes, stream);
}

int pyramidkv_select_topk(const pkv_config* cfg, const float* scores, int64_t ld_scores, const int32_t* seq_lens,
                          int32_t batch, int32_t k_layer, int32_t* indices, void* workspace,
                          size_t workspace_bytes, void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (int rc = config_supported(cfg)) return rc;
  if (!scores || !indices) return PKV_ERR_INVALID_ARG;
  SeqTable table;
  int max_n;
  int64_t rows;
  if (int rc = build_table(cfg, seq_lens, batch, k_layer, &table, &max_n, &rows)) return rc;
  if (ld_scores < max_n - cfg->window) return PKV_ERR_INVALID_ARG;
  Workspace w;
  if (int rc = workspace_check(cfg, batch, max_n, workspace, workspace_bytes, &w)) return rc;
  return run_select(cfg, scores, ld_scores, table, batch, max_n, indices, w, static_cast<cudaStream_t>(stream));
}

int pyramidkv_gather_compact(const pkv_config* cfg, pkv_tensor k, pkv_tensor v, const int32_t* indices,
                             const int32_t* seq_lens, int32_t batch, int32_t k_layer, void* k_out, void* v_out,
                             void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (int rc = config_supported(cfg)) return rc;
  const int eb = cfg->dtype == PKV_DTYPE_FP32 ? 4 : 2;
  if (!tensor_ok(k, cfg->head_dim, eb, batch, cfg->num_kv_heads) || !indices || !k_out) return PKV_ERR_INVALID_ARG;
  if ((v.ptr == nullptr) != (v_out == nullptr)) return PKV_ERR_INVALID_ARG;
  if (v.ptr && !tensor_ok(v, cfg->head_dim, eb, batch, cfg->num_kv_heads)) return PKV_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(k_out) % 16 || reinterpret_cast<uintptr_t>(v_out) % 16) return PKV_ERR_INVALID_ARG;
  SeqTable table;
  int max_n;
  int64_t rows;
  if (int rc = build_table(cfg, seq_lens, batch, k_layer, &table, &max_n, &rows)) return rc;
  return run_gather(cfg, k, v, indices, table, rows, k_out, v_out, static_cast<cudaStream_t>(stream));
}

// Budget of one layer: the schedule is O(m) integer work, small enough to redo per call.
static int32_t layer_budget(const pkv_config* cfg, int32_t layer) {
  int32_t stack_buf[512];
  int32_t* all = cfg->num_layers <= 512 ? stack_buf : new int32_t[cfg->num_layers];
  budgets(cfg, all);
  const int32_t k_layer = all[layer];
  if (all != stack_buf) delete[] all;
  return k_layer;
}

static int compress_layer_impl(const pkv_config* cfg, int32_t layer, pkv_tensor q_win, pkv_tensor k, pkv_tensor v,
                               const float* window_lse, const int32_t* seq_lens, int32_t batch, void* k_out,
                               void* v_out, int32_t* indices, float* scores_or_null, int64_t ld_scores,
                               void* workspace, size_t workspace_bytes, void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (int rc = config_supported(cfg)) return rc;
  if (layer < 0 || layer >= cfg->num_layers) return PKV_ERR_INVALID_ARG;
  const int eb = cfg->dtype == PKV_DTYPE_FP32 ? 4 : 2;
  if (!tensor_ok(q_win, cfg->head_dim, eb, batch, cfg->num_q_heads) ||
      !tensor_ok(k, cfg->head_dim, eb, batch, cfg->num_kv_heads) || !tensor_ok(v, cfg->head_dim, eb, batch, cfg->num_kv_heads))
    return PKV_ERR_INVALID_ARG;
  if (!k_out || !v_out || !indices) return PKV_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(k_out) % 16 || reinterpret_cast<uintptr_t>(v_out) % 16) return PKV_ERR_INVALID_ARG;
  const int32_t k_layer = layer_budget(cfg, layer);
  SeqTable table;
  int max_n;
  int64_t rows;
  if (int rc = build_table(cfg, seq_lens, batch, k_layer, &table, &max_n, &rows)) return rc;
  Workspace w;
  if (int rc = workspace_check(cfg, batch, max_n, workspace, workspace_bytes, &w)) return rc;
  float* scores = scores_or_null ? scores_or_null : w.scores;
  const int64_t ld = scores_or_null ? ld_scores : w.ld_scores;
  if (ld < max_n - cfg->window) return PKV_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // A batch in which no sequence is compressed needs no scores unless the caller asked for them.
  bool any_compress = false;
  for (int b = 0; b < batch; ++b) any_compress |= table.count[b] < table.n[b];
  if (any_compress || scores_or_null)
    if (int rc = run_scores(cfg, q_win, k, table, batch, scores, ld, w, st, window_lse)) return rc;
  return run_select(cfg, scores, ld, table, batch, max_n, indices, w, st, &k, &v, k_out, v_out);
}

int pyramidkv_compress_layer(const pkv_config* cfg, int32_t layer, pkv_tensor q_win, pkv_tensor k, pkv_tensor v,
                             const int32_t* seq_lens, int32_t batch, void* k_out, void* v_out, int32_t* indices,
                             float* scores_or_null, int64_t ld_scores, void* workspace, size_t workspace_bytes,
                             void* stream) {
  return compress_layer_impl(cfg, layer, q_win, k, v, nullptr, seq_lens, batch, k_out, v_out, indices,
                             scores_or_null, ld_scores, workspace, workspace_bytes, stream);
}

int pyramidkv_compress_layer_lse(const pkv_config* cfg, int32_t layer, pkv_tensor q_win, pkv_tensor k, pkv_tensor v,
                                 const float* window_lse, const int32_t* seq_lens, int32_t batch, void* k_out,
                                 void* v_out, int32_t* indices, float* scores_or_null, int64_t ld_scores,
                                 void* workspace, size_t workspace_bytes, void* stream) {
  if (!window_lse) return PKV_ERR_INVALID_ARG;
  return compress_layer_impl(cfg, layer, q_win, k, v, window_lse, seq_lens, batch, k_out, v_out, indices,
                             scores_or_null, ld_scores, workspace, workspace_bytes, stream);
}

// Window attention fused with the scores: row statistics sweep, merge, then the fused pass; with a layer
// (layer >= 0) the selection and the gather follow as in pyramidkv_compress_layer.
static int attend_impl(const pkv_config* cfg, int32_t layer, pkv_tensor q_win, pkv_tensor k, pkv_tensor v,
                       const int32_t* seq_lens, int32_t batch, float* attn_out, void* k_out, void* v_out,
                       int32_t* indices, float* scores_or_null, int64_t ld_scores, void* workspace,
                       size_t workspace_bytes, void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (int rc = config_supported(cfg)) return rc;
  if (!attend_eligible(cfg)) return PKV_ERR_UNSUPPORTED;
  const bool compress = layer >= 0;
  if (compress && layer >= cfg->num_layers) return PKV_ERR_INVALID_ARG;
  if (!tensor_ok(q_win, cfg->head_dim, 2, batch, cfg->num_q_heads) ||
      !tensor_ok(k, cfg->head_dim, 2, batch, cfg->num_kv_heads) || !tensor_ok(v, cfg->head_dim, 2, batch, cfg->num_kv_heads))
    return PKV_ERR_INVALID_ARG;
  if (!attn_out || reinterpret_cast<uintptr_t>(attn_out) % 16) return PKV_ERR_INVALID_ARG;
  if (compress) {
    if (!k_out || !v_out || !indices) return PKV_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(k_out) % 16 || reinterpret_cast<uintptr_t>(v_out) % 16) return PKV_ERR_INVALID_ARG;
  } else if (!scores_or_null) {
    return PKV_ERR_INVALID_ARG;
  }
  const int32_t k_layer = compress ? layer_budget(cfg, layer) : 0;
  SeqTable table;
  int max_n;
  int64_t rows;
  if (int rc = build_table(cfg, seq_lens, batch, k_layer, &table, &max_n, &rows)) return rc;
  Workspace w;
  if (int rc = workspace_check(cfg, batch, max_n, workspace, workspace_bytes, &w)) return rc;
  float* scores = scores_or_null ? scores_or_null : w.scores;
  const int64_t ld = scores_or_null ? ld_scores : w.ld_scores;
  if (ld < max_n - cfg->window) return PKV_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (int rc = run_scores(cfg, q_win, k, table, batch, scores, ld, w, st, nullptr, /*stats_only=*/true)) return rc;
  if (int rc = run_attend(cfg, q_win, k, v, table, batch, max_n, scores, ld, attn_out, w, st)) return rc;
  if (!compress) return PKV_OK;
  return run_select(cfg, scores, ld, table, batch, max_n, indices, w, st, &k, &v, k_out, v_out);
}

int pyramidkv_attend_window(const pkv_config* cfg, pkv_tensor q_win, pkv_tensor k, pkv_tensor v,
                            const int32_t* seq_lens, int32_t batch, float* attn_out, float* scores,
                            int64_t ld_scores, void* workspace, size_t workspace_bytes, void* stream) {
  return attend_impl(cfg, -1, q_win, k, v, seq_lens, batch, attn_out, nullptr, nullptr, nullptr, scores, ld_scores,
                     workspace, workspace_bytes, stream);
}

int pyramidkv_attend_compress_layer(const pkv_config* cfg, int32_t layer, pkv_tensor q_win, pkv_tensor k, pkv_tensor v,
                                    const int32_t* seq_lens, int32_t batch, float* attn_out, void* k_out,
                                    void* v_out, int32_t* indices, float* scores_or_null, int64_t ld_scores,
                                    void* workspace, size_t workspace_bytes, void* stream) {
  if (layer < 0) return PKV_ERR_INVALID_ARG;
  return attend_impl(cfg, layer, q_win, k, v, seq_lens, batch, attn_out, k_out, v_out, indices, scores_or_null,
                     ld_scores, workspace, workspace_bytes, stream);
}

static int profile_layer_impl(const pkv_config* cfg, int32_t layer, pkv_tensor q_win, pkv_tensor k, pkv_tensor v,
                              const float* window_lse, const int32_t* seq_lens, int32_t batch, void* k_out,
                              void* v_out, int32_t* indices, float* scores_or_null, int64_t ld_scores,
                              void* workspace, size_t workspace_bytes, void* stream, float* stage_ms,
                              char (*stage_names)[32], int32_t* num_stages, float* attn_out = nullptr) {
  if (!stage_ms || !stage_names || !num_stages) return PKV_ERR_INVALID_ARG;
  StageTimer timer;
  for (auto& e : timer.ev)
    if (cudaEventCreate(&e) != cudaSuccess) return PKV_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaEventRecord(timer.ev[0], st);
  g_timer = &timer;
  int rc = attn_out ? attend_impl(cfg, layer, q_win, k, v, seq_lens, batch, attn_out, k_out, v_out, indices,
                                  scores_or_null, ld_scores, workspace, workspace_bytes, stream)
                    : compress_layer_impl(cfg, layer, q_win, k, v, window_lse, seq_lens, batch, k_out, v_out, indices,
                                          scores_or_null, ld_scores, workspace, workspace_bytes, stream);
  g_timer = nullptr;
  if (rc == PKV_OK && cudaStreamSynchronize(st) != cudaSuccess) rc = PKV_ERR_CUDA;
  *num_stages = 0;
  if (rc == PKV_OK) {
    for (int i = 0; i < timer.n; ++i) {
      cudaEventElapsedTime(&stage_ms[i], timer.ev[i], timer.ev[i + 1]);
      std::snprintf(stage_names[i], 32, "%s", timer.name[i]);
    }
    *num_stages = timer.n;
  }
  for (auto& e : timer.ev) cudaEventDestroy(e);
  return rc;
}

int pyramidkv_profile_layer(const pkv_config* cfg, int32_t layer, pkv_tensor q_win, pkv_tensor k, pkv_tensor v,
                            const int32_t* seq_lens, int32_t batch, void* k_out, void* v_out, int32_t* indices,
                            float* scores_or_null, int64_t ld_scores, void* workspace, size_t workspace_bytes,
                            void* stream, float* stage_ms, char (*stage_names)[32], int32_t* num_stages) {
  return profile_layer_impl(cfg, layer, q_win, k, v, nullptr, seq_lens, batch, k_out, v_out, indices, scores_or_null,
                            ld_scores, workspace, workspace_bytes, stream, stage_ms, stage_names, num_stages);
}

int pyramidkv_profile_layer_lse(const pkv_config* cfg, int32_t layer, pkv_tensor q_win, pkv_tensor k, pkv_tensor v,
                                const float* window_lse, const int32_t* seq_lens, int32_t batch, void* k_out,
                                void* v_out, int32_t* indices, float* scores_or_null, int64_t ld_scores,
                                void* workspace, size_t workspace_bytes, void* stream, float* stage_ms,
                                char (*stage_names)[32], int32_t* num_stages) {
  if (!window_lse) return PKV_ERR_INVALID_ARG;
  return profile_layer_impl(cfg, layer, q_win, k, v, window_lse, seq_lens, batch, k_out, v_out, indices,
                            scores_or_null, ld_scores, workspace, workspace_bytes, stream, stage_ms, stage_names,
                            num_stages);
}

int pyramidkv_profile_attend_compress_layer(const pkv_config* cfg, int32_t layer, pkv_tensor q_win, pkv_tensor k,
                                            pkv_tensor v, const int32_t* seq_lens, int32_t batch, float* attn_out,
                                            void* k_out, void* v_out, int32_t* indices, float* scores_or_null,
                                            int64_t ld_scores, void* workspace, size_t workspace_bytes, void* stream,
                                            float* stage_ms, char (*stage_names)[32], int32_t* num_stages) {
  if (!attn_out || layer < 0) return PKV_ERR_INVALID_ARG;
  return profile_layer_impl(cfg, layer, q_win, k, v, nullptr, seq_lens, batch, k_out, v_out, indices, scores_or_null,
                            ld_scores, workspace, workspace_bytes, stream, stage_ms, stage_names, num_stages, attn_out);
}

int pyramidkv_decode_attention(const pkv_config* cfg, const void* q, const void* k_cache, const void* v_cache,
                               const int32_t* seq_lens, int32_t batch, int32_t k_layer, float* out, void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (int rc = config_supported(cfg)) return rc;
  if (!q || !k_cache || !v_cache || !out) return PKV_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(q) % 16 || reinterpret_cast<uintptr_t>(k_cache) % 16 ||
      reinterpret_cast<uintptr_t>(v_cache) % 16)
    return PKV_ERR_INVALID_ARG;
  SeqTable table;
  int max_n;
  int64_t rows;
  if (int rc = build_table(cfg, seq_lens, batch, k_layer, &table, &max_n, &rows)) return rc;
  DecodeParams dp{};
  dp.q = q;
  dp.k_cache = k_cache;
  dp.v_cache = v_cache;
  dp.out = out;
  dp.seq = table;
  dp.num_kv_heads = cfg->num_kv_heads;
  dp.group = cfg->num_q_heads / cfg->num_kv_heads;
  dp.scale_log2 = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(cfg->head_dim)));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const dim3 grid(cfg->num_q_heads, batch);
  if (cfg->dtype == PKV_DTYPE_FP32) {
    if (cfg->head_dim == 64) launch_pdl(decode_attention_kernel<float, 64>, grid, kDecThreads, 0, st, dp);
    else launch_pdl(decode_attention_kernel<float, 128>, grid, kDecThreads, 0, st, dp);
  } else if (cfg->dtype == PKV_DTYPE_FP16) {
    if (cfg->head_dim == 64) launch_pdl(decode_attention_kernel<__half, 64>, grid, kDecThreads, 0, st, dp);
    else launch_pdl(decode_attention_kernel<__half, 128>, grid, kDecThreads, 0, st, dp);
  } else {
    if (cfg->head_dim == 64) launch_pdl(decode_attention_kernel<__nv_bfloat16, 64>, grid, kDecThreads, 0, st, dp);
    else launch_pdl(decode_attention_kernel<__nv_bfloat16, 128>, grid, kDecThreads, 0, st, dp);
  }
  return check_launch();
}

int pyramidkv_attention_recall(const pkv_config* cfg, const float* scores, int64_t ld_scores, const int32_t* indices,
                               const int32_t* seq_lens, int32_t batch, int32_t k_layer, float* recall,
                               void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (!scores || !indices || !recall) return PKV_ERR_INVALID_ARG;
  SeqTable table;
  int max_n;
  int64_t rows;
  if (int rc = build_table(cfg, seq_lens, batch, k_layer, &table, &max_n, &rows)) return rc;
  if (ld_scores < max_n - cfg->window) return PKV_ERR_INVALID_ARG;
  RecallParams rp{};
  rp.scores = scores;
  rp.ld_scores = ld_scores;
  rp.indices = indices;
  rp.recall = recall;
  rp.seq = table;
  rp.num_kv_heads = cfg->num_kv_heads;
  launch_pdl(attention_recall_kernel, dim3(cfg->num_kv_heads, batch), 256, 0, static_cast<cudaStream_t>(stream), rp);
  return check_launch();
}

int pyramidkv_pages_needed(const pkv_config* cfg, int32_t k_layer, int32_t seq_len, int32_t page_size) {
  if (!config_ok(cfg) || k_layer < 0 || seq_len < cfg->window + 1 || page_size < 1) return -PKV_ERR_INVALID_ARG;
  return (kept_count(cfg, k_layer, seq_len) + page_size - 1) / page_size;
}

int pyramidkv_gather_paged(const pkv_config* cfg, pkv_tensor k, pkv_tensor v, const int32_t* indices,
                           const int32_t* seq_lens, int32_t batch, int32_t k_layer, const int32_t* block_table,
                           int32_t page_size, int32_t num_pages, void* k_pool, void* v_pool, void* workspace,
                           size_t workspace_bytes, void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (int rc = config_supported(cfg)) return rc;
  const int eb = cfg->dtype == PKV_DTYPE_FP32 ? 4 : 2;
  if (!tensor_ok(k, cfg->head_dim, eb, batch, cfg->num_kv_heads) || !tensor_ok(v, cfg->head_dim, eb, batch, cfg->num_kv_heads) ||
      !indices)
    return PKV_ERR_INVALID_ARG;
  if (!paged_args_ok(block_table, page_size, num_pages, k_pool, v_pool)) return PKV_ERR_INVALID_ARG;
  if (!workspace || reinterpret_cast<uintptr_t>(workspace) % kAlign || workspace_bytes < kAlign)
    return PKV_ERR_WORKSPACE;
  SeqTable table;
  int max_n;
  int64_t rows;
  if (int rc = build_table(cfg, seq_lens, batch, k_layer, &table, &max_n, &rows)) return rc;
  return run_gather_paged(cfg, k, v, indices, table, rows, block_table, page_size, num_pages, k_pool, v_pool,
                          static_cast<uint32_t*>(workspace), static_cast<cudaStream_t>(stream));
}

int pyramidkv_compress_layer_paged(const pkv_config* cfg, int32_t layer, pkv_tensor q_win, pkv_tensor k,
                                   pkv_tensor v, const float* window_lse_or_null, const int32_t* seq_lens,
                                   int32_t batch, const int32_t* block_table, int32_t page_size, int32_t num_pages,
                                   void* k_pool, void* v_pool, int32_t* indices, float* scores_or_null,
                                   int64_t ld_scores, void* workspace, size_t workspace_bytes, void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (int rc = config_supported(cfg)) return rc;
  if (layer < 0 || layer >= cfg->num_layers) return PKV_ERR_INVALID_ARG;
  const int eb = cfg->dtype == PKV_DTYPE_FP32 ? 4 : 2;
  if (!tensor_ok(q_win, cfg->head_dim, eb, batch, cfg->num_q_heads) ||
      !tensor_ok(k, cfg->head_dim, eb, batch, cfg->num_kv_heads) || !tensor_ok(v, cfg->head_dim, eb, batch, cfg->num_kv_heads))
    return PKV_ERR_INVALID_ARG;
  if (!indices || !paged_args_ok(block_table, page_size, num_pages, k_pool, v_pool)) return PKV_ERR_INVALID_ARG;
  const int32_t k_layer = layer_budget(cfg, layer);
  SeqTable table;
  int max_n;
  int64_t rows;
  if (int rc = build_table(cfg, seq_lens, batch, k_layer, &table, &max_n, &rows)) return rc;
  Workspace w;
  if (int rc = workspace_check(cfg, batch, max_n, workspace, workspace_bytes, &w)) return rc;
  float* scores = scores_or_null ? scores_or_null : w.scores;
  const int64_t ld = scores_or_null ? ld_scores : w.ld_scores;
  if (ld < max_n - cfg->window) return PKV_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  bool any_compress = false;
  for (int b = 0; b < batch; ++b) any_compress |= table.count[b] < table.n[b];
  if (any_compress || scores_or_null)
    if (int rc = run_scores(cfg, q_win, k, table, batch, scores, ld, w, st, window_lse_or_null)) return rc;
  if (int rc = run_select(cfg, scores, ld, table, batch, max_n, indices, w, st)) return rc;
  return run_gather_paged(cfg, k, v, indices, table, rows, block_table, page_size, num_pages, k_pool, v_pool,
                          w.status, st);
}

int pyramidkv_decode_attention_paged(const pkv_config* cfg, const void* q, const void* k_pool, const void* v_pool,
                                     const int32_t* block_table, int32_t page_size, int32_t num_pages,
                                     const int32_t* seq_lens, int32_t batch, int32_t k_layer, float* out,
                                     void* workspace, size_t workspace_bytes, void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (int rc = config_supported(cfg)) return rc;
  if (!q || !out || reinterpret_cast<uintptr_t>(q) % 16) return PKV_ERR_INVALID_ARG;
  if (!paged_args_ok(block_table, page_size, num_pages, k_pool, v_pool)) return PKV_ERR_INVALID_ARG;
  if (!workspace || reinterpret_cast<uintptr_t>(workspace) % kAlign || workspace_bytes < kAlign)
    return PKV_ERR_WORKSPACE;
  SeqTable table;
  int max_n;
  int64_t rows;
  if (int rc = build_table(cfg, seq_lens, batch, k_layer, &table, &max_n, &rows)) return rc;
  DecodeParams dp{};
  dp.q = q;
  dp.k_cache = k_pool;
  dp.v_cache = v_pool;
  dp.out = out;
  dp.seq = table;
  fill_page_table(cfg, table, block_table, page_size, num_pages, &dp.pt);
  dp.status = static_cast<uint32_t*>(workspace);
  dp.num_kv_heads = cfg->num_kv_heads;
  dp.group = cfg->num_q_heads / cfg->num_kv_heads;
  dp.scale_log2 = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(cfg->head_dim)));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const dim3 grid(cfg->num_q_heads, batch);
  const bool wide = cfg->head_dim == 128;
  if (cfg->dtype == PKV_DTYPE_FP32) {
    if (wide) launch_pdl(decode_attention_kernel<float, 128, true>, grid, kDecThreads, 0, st, dp);
    else launch_pdl(decode_attention_kernel<float, 64, true>, grid, kDecThreads, 0, st, dp);
  } else if (cfg->dtype == PKV_DTYPE_FP16) {
    if (wide) launch_pdl(decode_attention_kernel<__half, 128, true>, grid, kDecThreads, 0, st, dp);
    else launch_pdl(decode_attention_kernel<__half, 64, true>, grid, kDecThreads, 0, st, dp);
  } else {
    if (wide) launch_pdl(decode_attention_kernel<__nv_bfloat16, 128, true>, grid, kDecThreads, 0, st, dp);
    else launch_pdl(decode_attention_kernel<__nv_bfloat16, 64, true>, grid, kDecThreads, 0, st, dp);
  }
  return check_launch();
}

int pyramidkv_shard_window_lse(const pkv_config* cfg, pkv_tensor q_win, pkv_tensor k_shard,
                               const int32_t* shard_keys, const int32_t* window_keys, int32_t batch, float* lse_out,
                               void* workspace, size_t workspace_bytes, void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (int rc = config_supported(cfg)) return rc;
  const int eb = cfg->dtype == PKV_DTYPE_FP32 ? 4 : 2;
  if (!tensor_ok(q_win, cfg->head_dim, eb, batch, cfg->num_q_heads) ||
      !tensor_ok(k_shard, cfg->head_dim, eb, batch, cfg->num_kv_heads) || !lse_out)
    return PKV_ERR_INVALID_ARG;
  SeqTable table;
  int max_n;
  if (int rc = build_shard_table(cfg, shard_keys, window_keys, batch, &table, &max_n)) return rc;
  Workspace w;
  if (int rc = workspace_check(cfg, batch, max_n + cfg->window, workspace, workspace_bytes, &w)) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (int rc = run_scores(cfg, q_win, k_shard, table, batch, w.scores, w.ld_scores, w, st, nullptr, true)) return rc;
  const int64_t count = static_cast<int64_t>(batch) * cfg->num_q_heads * cfg->window;
  const float log2_group = std::log2(static_cast<float>(cfg->num_q_heads / cfg->num_kv_heads));
  launch_pdl(export_lse_kernel, static_cast<unsigned>((count + kShardThreads - 1) / kShardThreads), kShardThreads, 0,
             st, static_cast<const float*>(w.lse2), log2_group, lse_out, count);
  return check_launch();
}

int pyramidkv_merge_lse(const float* parts, int32_t num_shards, int64_t count, float* out, void* stream) {
  if (!parts || !out || num_shards < 1 || count < 1) return PKV_ERR_INVALID_ARG;
  launch_pdl(merge_lse_kernel, static_cast<unsigned>((count + kShardThreads - 1) / kShardThreads), kShardThreads, 0,
             static_cast<cudaStream_t>(stream), parts, static_cast<int>(num_shards), count, out);
  return check_launch();
}

int pyramidkv_shard_scores(const pkv_config* cfg, pkv_tensor q_win, pkv_tensor k_shard, const float* window_lse,
                           const int32_t* shard_keys, const int32_t* window_keys, int32_t batch, float* scores,
                           int64_t ld_scores, void* workspace, size_t workspace_bytes, void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (int rc = config_supported(cfg)) return rc;
  const int eb = cfg->dtype == PKV_DTYPE_FP32 ? 4 : 2;
  if (!tensor_ok(q_win, cfg->head_dim, eb, batch, cfg->num_q_heads) ||
      !tensor_ok(k_shard, cfg->head_dim, eb, batch, cfg->num_kv_heads) || !window_lse || !scores)
    return PKV_ERR_INVALID_ARG;
  SeqTable table;
  int max_n;
  if (int rc = build_shard_table(cfg, shard_keys, window_keys, batch, &table, &max_n)) return rc;
  for (int b = 0; b < batch; ++b)
    if (ld_scores < table.prefix[b]) return PKV_ERR_INVALID_ARG;
  Workspace w;
  if (int rc = workspace_check(cfg, batch, max_n + cfg->window, workspace, workspace_bytes, &w)) return rc;
  return run_scores(cfg, q_win, k_shard, table, batch, scores, ld_scores, w, static_cast<cudaStream_t>(stream),
                    window_lse);
}

int pyramidkv_shard_gather(const pkv_config* cfg, pkv_tensor k_shard, pkv_tensor v_shard, const int32_t* indices,
                           const int32_t* seq_lens, int32_t batch, int32_t k_layer, const int32_t* shard_begin,
                           const int32_t* shard_keys, void* k_out, void* v_out, void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (int rc = config_supported(cfg)) return rc;
  const int eb = cfg->dtype == PKV_DTYPE_FP32 ? 4 : 2;
  if (!tensor_ok(k_shard, cfg->head_dim, eb, batch, cfg->num_kv_heads) ||
      !tensor_ok(v_shard, cfg->head_dim, eb, batch, cfg->num_kv_heads))
    return PKV_ERR_INVALID_ARG;
  if (!indices || !k_out || !v_out || !shard_begin || !shard_keys) return PKV_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(k_out) % 16 || reinterpret_cast<uintptr_t>(v_out) % 16) return PKV_ERR_INVALID_ARG;
  SeqTable table;
  int max_n;
  int64_t rows;
  if (int rc = build_table(cfg, seq_lens, batch, k_layer, &table, &max_n, &rows)) return rc;
  GatherShardParams gp{};
  gp.k = view(k_shard);
  gp.v = view(v_shard);
  gp.indices = indices;
  gp.k_out = k_out;
  gp.v_out = v_out;
  gp.seq = table;
  for (int b = 0; b < batch; ++b) {
    if (shard_begin[b] < 0 || shard_keys[b] < 0 || shard_begin[b] + shard_keys[b] > seq_lens[b])
      return PKV_ERR_INVALID_ARG;
    gp.begin[b] = shard_begin[b];
    gp.keys[b] = shard_keys[b];
  }
  gp.num_kv_heads = cfg->num_kv_heads;
  gp.elem_bytes = eb;
  gp.pieces = cfg->head_dim * eb / 16;
  gp.total_rows = rows;
  const int64_t threads = rows * gp.pieces;
  if (threads == 0) return PKV_OK;
  launch_pdl(gather_shard_kernel, static_cast<unsigned>((threads + kShardThreads - 1) / kShardThreads), kShardThreads,
             0, static_cast<cudaStream_t>(stream), gp);
  note_output(k_out, static_cast<size_t>(rows) * cfg->head_dim * eb);
  note_output(v_out, static_cast<size_t>(rows) * cfg->head_dim * eb);
  return check_launch();
}

// ---------------------------------------------------------------------------
// Two lanes: the SMs of the device split into two disjoint groups (CUDA green contexts), one stream on each.
// The score sweeps of layer l + 1 then run beside the selection and gather of layer l, which by itself keeps
// fewer than half of the SMs busy for a seventh of a layer's time.
struct pkv_lanes {
  CUgreenCtx ctx[2];          // [0] scores, [1] selection
  cudaStream_t stream[2];
  int sms[2];
  int device;
  cudaEvent_t start, scored[2], selected[2], done[2];
};

namespace {

struct LaneApi {
  CUresult (*device_get)(CUdevice*, int);
  CUresult (*get_dev_resource)(CUdevice, CUdevResource*, CUdevResourceType);
  CUresult (*split_by_count)(CUdevResource*, unsigned int*, const CUdevResource*, CUdevResource*, unsigned int,
                             unsigned int);
  CUresult (*generate_desc)(CUdevResourceDesc*, CUdevResource*, unsigned int);
  CUresult (*green_create)(CUgreenCtx*, CUdevResourceDesc, CUdevice, unsigned int);
  CUresult (*green_stream)(CUstream*, CUgreenCtx, unsigned int, int);
  CUresult (*green_destroy)(CUgreenCtx);
  bool ok;
};

const LaneApi& lane_api() {
  static LaneApi api = [] {
    LaneApi a{};
    auto get = [](const char* name) -> void* {
      void* sym = nullptr;
      cudaDriverEntryPointQueryResult q;
      if (cudaGetDriverEntryPoint(name, &sym, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
        return nullptr;
      return sym;
    };
    a.device_get = reinterpret_cast<decltype(a.device_get)>(get("cuDeviceGet"));
    a.get_dev_resource = reinterpret_cast<decltype(a.get_dev_resource)>(get("cuDeviceGetDevResource"));
    a.split_by_count = reinterpret_cast<decltype(a.split_by_count)>(get("cuDevSmResourceSplitByCount"));
    a.generate_desc = reinterpret_cast<decltype(a.generate_desc)>(get("cuDevResourceGenerateDesc"));
    a.green_create = reinterpret_cast<decltype(a.green_create)>(get("cuGreenCtxCreate"));
    a.green_stream = reinterpret_cast<decltype(a.green_stream)>(get("cuGreenCtxStreamCreate"));
    a.green_destroy = reinterpret_cast<decltype(a.green_destroy)>(get("cuGreenCtxDestroy"));
    a.ok = a.device_get && a.get_dev_resource && a.split_by_count && a.generate_desc && a.green_create &&
           a.green_stream && a.green_destroy;
    cudaGetLastError();
    return a;
  }();
  return api;
}

}  // namespace

int pyramidkv_lanes_create(int32_t select_sms, pkv_lanes** out) {
  if (!out || select_sms < 8) return PKV_ERR_INVALID_ARG;
  *out = nullptr;
  const LaneApi& api = lane_api();
  if (!api.ok) return PKV_ERR_UNSUPPORTED;
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess || cudaFree(nullptr) != cudaSuccess) return PKV_ERR_CUDA;
  CUdevice dev;
  CUdevResource all, group, rest;
  unsigned int groups = 1;
  if (api.device_get(&dev, device) != CUDA_SUCCESS ||
      api.get_dev_resource(dev, &all, CU_DEV_RESOURCE_TYPE_SM) != CUDA_SUCCESS)
    return PKV_ERR_UNSUPPORTED;
  if (static_cast<unsigned>(select_sms) * 2 > all.sm.smCount) return PKV_ERR_INVALID_ARG;
  if (api.split_by_count(&group, &groups, &all, &rest, 0, static_cast<unsigned>(select_sms)) != CUDA_SUCCESS ||
      groups != 1 || rest.sm.smCount == 0)
    return PKV_ERR_UNSUPPORTED;
  pkv_lanes* l = new pkv_lanes();
  l->device = device;
  CUdevResource parts[2] = {rest, group};
  bool good = true;
  int made_ctx = 0, made_stream = 0;
  for (int i = 0; i < 2 && good; ++i) {
    CUdevResourceDesc desc;
    good = api.generate_desc(&desc, &parts[i], 1) == CUDA_SUCCESS &&
           api.green_create(&l->ctx[i], desc, dev, CU_GREEN_CTX_DEFAULT_STREAM) == CUDA_SUCCESS;
    if (!good) break;
    ++made_ctx;
    CUstream s;
    good = api.green_stream(&s, l->ctx[i], CU_STREAM_NON_BLOCKING, 0) == CUDA_SUCCESS;
    if (!good) break;
    ++made_stream;
    l->stream[i] = reinterpret_cast<cudaStream_t>(s);
    l->sms[i] = static_cast<int>(parts[i].sm.smCount);
  }
  cudaEvent_t* events[] = {&l->start, &l->scored[0], &l->scored[1], &l->selected[0], &l->selected[1], &l->done[0],
                           &l->done[1]};
  int made_events = 0;
  for (cudaEvent_t* e : events) {
    if (!good) break;
    good = cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
    if (good) ++made_events;
  }
  if (!good) {
    for (int i = 0; i < made_events; ++i) cudaEventDestroy(*events[i]);
    for (int i = 0; i < made_stream; ++i) cudaStreamDestroy(l->stream[i]);
    for (int i = 0; i < made_ctx; ++i) api.green_destroy(l->ctx[i]);
    delete l;
    cudaGetLastError();
    return PKV_ERR_UNSUPPORTED;
  }
  *out = l;
  return PKV_OK;
}

int pyramidkv_lanes_destroy(pkv_lanes* l) {
  if (!l) return PKV_OK;
  cudaEvent_t events[] = {l->start, l->scored[0], l->scored[1], l->selected[0], l->selected[1], l->done[0], l->done[1]};
  for (cudaEvent_t e : events) cudaEventDestroy(e);
  for (int i = 0; i < 2; ++i) cudaStreamDestroy(l->stream[i]);
  for (int i = 0; i < 2; ++i) lane_api().green_destroy(l->ctx[i]);
  delete l;
  return PKV_OK;
}

int pyramidkv_lanes_info(const pkv_lanes* l, int32_t* score_sms, int32_t* select_sms) {
  if (!l || !score_sms || !select_sms) return PKV_ERR_INVALID_ARG;
  *score_sms = l->sms[0];
  *select_sms = l->sms[1];
  return PKV_OK;
}

int pyramidkv_compress_model_lanes(const pkv_config* cfg, pkv_lanes* lanes, int32_t first_layer, int32_t num_layers,
                                   const pkv_tensor* q_win, const pkv_tensor* k, const pkv_tensor* v,
                                   const float* const* window_lse_or_null, const int32_t* seq_lens, int32_t batch,
                                   void* const* k_out, void* const* v_out, int32_t* const* indices,
                                   void* const* workspaces, size_t workspace_bytes, void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (int rc = config_supported(cfg)) return rc;
  if (!lanes || !q_win || !k || !v || !k_out || !v_out || !indices || !workspaces) return PKV_ERR_INVALID_ARG;
  if (first_layer < 0 || num_layers < 1 || first_layer + num_layers > cfg->num_layers) return PKV_ERR_INVALID_ARG;
  if (!workspaces[0] || !workspaces[1] || workspaces[0] == workspaces[1]) return PKV_ERR_INVALID_ARG;
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess || device != lanes->device) return PKV_ERR_INVALID_ARG;
  const int eb = cfg->dtype == PKV_DTYPE_FP32 ? 4 : 2;
  for (int i = 0; i < num_layers; ++i) {
    if (!tensor_ok(q_win[i], cfg->head_dim, eb, batch, cfg->num_q_heads) ||
        !tensor_ok(k[i], cfg->head_dim, eb, batch, cfg->num_kv_heads) ||
        !tensor_ok(v[i], cfg->head_dim, eb, batch, cfg->num_kv_heads) || !k_out[i] || !v_out[i] || !indices[i])
      return PKV_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(k_out[i]) % 16 || reinterpret_cast<uintptr_t>(v_out[i]) % 16)
      return PKV_ERR_INVALID_ARG;
  }
  // tables and workspaces are validated before anything is enqueued
  int max_n = 0;
  int64_t rows = 0;
  Workspace ws[2];
  {
    SeqTable probe;
    if (int rc = build_table(cfg, seq_lens, batch, 0, &probe, &max_n, &rows)) return rc;
    for (int i = 0; i < 2; ++i)
      if (int rc = workspace_check(cfg, batch, max_n, workspaces[i], workspace_bytes, &ws[i])) return rc;
  }
  cudaStream_t caller = static_cast<cudaStream_t>(stream), score = lanes->stream[0], select = lanes->stream[1];
  if (cudaEventRecord(lanes->start, caller) != cudaSuccess || cudaStreamWaitEvent(score, lanes->start, 0) != cudaSuccess ||
      cudaStreamWaitEvent(select, lanes->start, 0) != cudaSuccess)
    return PKV_ERR_CUDA;
  int status = PKV_OK;
  tl_sm_limit = lanes->sms[0];
  for (int i = 0; i < num_layers && status == PKV_OK; ++i) {
    const int32_t k_layer = layer_budget(cfg, first_layer + i);
    SeqTable table;
    if ((status = build_table(cfg, seq_lens, batch, k_layer, &table, &max_n, &rows)) != PKV_OK) break;
    const Workspace& w = ws[i & 1];
    // the scores buffer of this workspace is free once the selection two layers back has read it
    if (i >= 2 && cudaStreamWaitEvent(score, lanes->selected[i & 1], 0) != cudaSuccess) { status = PKV_ERR_CUDA; break; }
    bool any_compress = false;
    for (int b = 0; b < batch; ++b) any_compress |= table.count[b] < table.n[b];
    if (any_compress)
      status = run_scores(cfg, q_win[i], k[i], table, batch, w.scores, w.ld_scores, w, score,
                          window_lse_or_null ? window_lse_or_null[i] : nullptr);
    if (status != PKV_OK) break;
    if (cudaEventRecord(lanes->scored[i & 1], score) != cudaSuccess ||
        cudaStreamWaitEvent(select, lanes->scored[i & 1], 0) != cudaSuccess) { status = PKV_ERR_CUDA; break; }
    tl_sm_limit = 0;
    status = run_select(cfg, w.scores, w.ld_scores, table, batch, max_n, indices[i], w, select, &k[i], &v[i], k_out[i],
                        v_out[i]);
    tl_sm_limit = lanes->sms[0];
    if (status != PKV_OK) break;
    if (cudaEventRecord(lanes->selected[i & 1], select) != cudaSuccess) { status = PKV_ERR_CUDA; break; }
  }
  tl_sm_limit = 0;
  // the caller's stream continues when both lanes are done, whatever happened above
  if (cudaEventRecord(lanes->done[0], score) != cudaSuccess || cudaEventRecord(lanes->done[1], select) != cudaSuccess ||
      cudaStreamWaitEvent(caller, lanes->done[0], 0) != cudaSuccess ||
      cudaStreamWaitEvent(caller, lanes->done[1], 0) != cudaSuccess)
    return status != PKV_OK ? status : PKV_ERR_CUDA;
  return status;
}

int pyramidkv_check_status(const void* workspace, void* stream, uint32_t* detail_or_null) {
  if (!workspace) return PKV_ERR_INVALID_ARG;
  uint32_t word = 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&word, workspace, sizeof word, cudaMemcpyDeviceToHost, st) != cudaSuccess) return PKV_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return PKV_ERR_CUDA;
  if (detail_or_null) *detail_or_null = word;
  return word == 0 ? PKV_OK : PKV_ERR_DEVICE_STATUS;
}

}  // extern "C"

// ---------------------------------------------------------------------------
// Scoring without any caller-provided scratch.
//
// Some callers of pyramidkv_score_window cannot hand over a workspace because they
// cannot allocate device memory at the point of the call: code that runs inside a
// serving engine whose memory pool is already carved up, a plugin that is only given
// its input and output tensors, or a latency-critical section in which cudaMalloc
// (which may synchronise the device) is off limits.  For them the scratch of the
// score kernels (chunk statistics and row normalisers) lives in the fixed array
// below, which is part of the library image: every GPU that loads the library holds
// PKV_STATIC_SCRATCH_BYTES of it until the process exits.
//
// In host code `g_static_scratch` only names the symbol; it is not a device address.
// The address that kernels may use is looked up once per device with
// cudaGetSymbolAddress, on the first call made while that device is current.
static __device__ __align__(256) unsigned char g_static_scratch[PKV_STATIC_SCRATCH_BYTES];

namespace {
std::mutex g_static_mutex;
void* g_static_ptr[64] = {};

// Device address of the static scratch on the current device (nullptr on failure).
void* static_scratch_address() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) return nullptr;
    g_static_ptr[dev] = ptr;
  }
  return g_static_ptr[dev];
}
}  // namespace

extern "C" int pyramidkv_score_window_static(const pkv_config* cfg, pkv_tensor q_win, pkv_tensor k,
                                             const int32_t* seq_lens, int32_t batch, float* scores,
                                             int64_t ld_scores, void* stream) {
  if (!config_ok(cfg)) return PKV_ERR_INVALID_ARG;
  if (int rc = config_supported(cfg)) return rc;
  const int eb = cfg->dtype == PKV_DTYPE_FP32 ? 4 : 2;
  if (!tensor_ok(q_win, cfg->head_dim, eb, batch, cfg->num_q_heads) ||
      !tensor_ok(k, cfg->head_dim, eb, batch, cfg->num_kv_heads) || !scores)
    return PKV_ERR_INVALID_ARG;
  SeqTable table;
  int max_n;
  int64_t rows;
  if (int rc = build_table(cfg, seq_lens, batch, 0, &table, &max_n, &rows)) return rc;
  if (ld_scores < max_n - cfg->window) return PKV_ERR_INVALID_ARG;
  // Scratch the score kernels need: the workspace's leading regions (status word, normalisers, chunk
  // statistics); the score buffer is supplied by the caller and the selection scratch is not used here.
  const Workspace sizing = carve(cfg, batch, max_n, nullptr);
  const size_t need = sizing.score_scratch_bytes;
  if (need > PKV_STATIC_SCRATCH_BYTES) return PKV_ERR_STATIC_SCRATCH;
  void* base = static_scratch_address();
  if (!base) return PKV_ERR_CUDA;
  const Workspace w = carve(cfg, batch, max_n, base);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The array keeps whatever the previous call left.  Only the status word has to start from zero;
  // statistics and normalisers are fully rewritten before they are read.
  if (cudaMemsetAsync(w.status, 0, kAlign, st) != cudaSuccess) return PKV_ERR_CUDA;
  return run_scores(cfg, q_win, k, table, batch, scores, ld_scores, w, st);
}

extern "C" int pyramidkv_check_status_static(void* stream, uint32_t* detail_or_null) {
  void* base = static_scratch_address();
  if (!base) return PKV_ERR_CUDA;
  return pyramidkv_check_status(base, stream, detail_or_null);   // the status word heads the array
}

// ---------------------------------------------------------------------------
// Test aids (no counterpart in the paper).
namespace pkv {
// One small CTA: lets the kernels behind it in the stream start at once, then copies 16-byte pieces in `steps`
// rounds with a pause after each round, as a slow producer of K that signals its dependents early would.
__global__ void __launch_bounds__(256) slow_copy_kernel(uint4* dst, const uint4* src, size_t pieces, int steps) {
  pdl_trigger();
  const size_t per = (pieces + steps - 1) / steps;
  for (int s = 0; s < steps; ++s) {
    const size_t lo = s * per, hi = lo + per < pieces ? lo + per : pieces;
    for (size_t i = lo + threadIdx.x; i < hi; i += blockDim.x) dst[i] = src[i];
    __syncthreads();
    __nanosleep(20000);
  }
}
}  // namespace pkv

extern "C" int pyramidkv_test_hooks(int64_t wait_clocks, int32_t withhold_tile) {
  if (wait_clocks < 0) return PKV_ERR_INVALID_ARG;
  g_test_wait_clocks.store(wait_clocks);
  g_test_withhold.store((withhold_tile & 1) ? 1 : 0);
  g_test_two_sweeps.store((withhold_tile & 2) ? 1 : 0);
  g_test_withhold_attend.store((withhold_tile & 4) ? 1 : 0);
  return PKV_OK;
}

extern "C" int pyramidkv_test_slow_copy(void* dst, const void* src, size_t bytes, int32_t steps, void* stream) {
  if (!dst || !src || bytes % 16 || steps < 1) return PKV_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(dst) % 16 || reinterpret_cast<uintptr_t>(src) % 16) return PKV_ERR_INVALID_ARG;
  if (bytes == 0) return PKV_OK;
  slow_copy_kernel<<<1, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<uint4*>(dst),
                                                                     static_cast<const uint4*>(src), bytes / 16, steps);
  return cudaPeekAtLastError() == cudaSuccess ? PKV_OK : PKV_ERR_CUDA;
}
