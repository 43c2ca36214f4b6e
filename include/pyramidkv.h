/*
 * pyramidkv.h: C boundary of the B200 (sm_100a) PyramidKV prefill KV-cache
 * compression library.
 *
 * The library implements one step of the paper (arXiv 2406.02069, Section 4.2):
 * at the end of prefill, for each transformer layer, score every cached key by
 * the attention it receives from the last alpha ("instruction") tokens, smooth
 * the scores with a 1-D max pool, keep the k^l best positions per KV head under
 * the pyramidal per-layer budget, always keep the alpha window tokens, and copy
 * the survivors into a compact ragged K/V cache with a list of their original
 * positions.
 *
 * Conventions that hold for every call
 *   - C linkage; every function returns an int status (PKV_OK = 0) unless noted.
 *   - "host" pointers are dereferenced on the CPU before the call returns;
 *     "device" pointers are only touched by kernels enqueued on `stream`.
 *   - The caller owns every buffer.  The library never allocates or frees
 *     device memory, never synchronises the stream (except
 *     pyramidkv_check_status), and enqueues all device work on `stream`
 *     (a cudaStream_t passed as void*; NULL is the default stream).
 *   - Arguments are validated before anything is enqueued; on an error status
 *     other than PKV_ERR_CUDA no device work has been submitted by that call.
 *   - Output sizes are pure functions of host-known values (the config, the
 *     sequence lengths and the layer budget): nothing is read back from the
 *     device to size a buffer.
 *   - Sequences of a batch are independent; each has its own length n_b.
 *     P_b = n_b - alpha is its prefix length.
 *   - Kernels of consecutive calls on one stream overlap at their edges (programmatic dependent
 *     launch): a kernel of the library does its set-up while its predecessor drains, and waits for the
 *     predecessor's completion before it touches global memory.  The one exception is opt-in: with
 *     PKV_FLAG_INPUTS_FINAL in cfg->flags the score kernels read q_win and k without that wait (see the
 *     flag).  Even then the library orders them itself when q_win or k lies inside a cache or page pool
 *     that one of its own recent calls writes.
 *   - Calls on different streams may run at the same time as long as each has a workspace of its own (a
 *     call keeps its intermediate results there); the layers of a model are independent of one another, so a
 *     caller may spread them over a few streams to keep the device busy during the short kernels of a layer.
 *     Ordering between streams (a call that reads what a call on another stream writes) is the caller's, by events.
 *
 * Tensor layout
 *   K, V     [batch][H_kv][n_max][d]   element strides given per tensor
 *   Q_win    [batch][H_q][alpha][d]    the queries of the last alpha positions
 *   The head dimension is contiguous (stride 1) in every tensor; base pointers
 *   and strides are multiples of 16 bytes.  Query head g belongs to KV head
 *   g / (H_q / H_kv).
 *
 * Packed ragged output of one layer
 *   Every KV head of sequence b keeps the same number of rows
 *   c_b = pyramidkv_kept_count(cfg, k_layer, n_b).  Rows are packed sequence
 *   after sequence, head after head:  head h of sequence b owns rows
 *   [off_b + h*c_b, off_b + (h+1)*c_b)  with  off_b = H_kv * sum_{b'<b} c_{b'}.
 *   `indices` holds one int32 per row (the row's original position in its
 *   sequence, ascending inside a head, the alpha window positions last);
 *   k_out / v_out hold the d elements of that row, contiguous.
 */
#ifndef PYRAMIDKV_H_
#define PYRAMIDKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Status codes. */
#define PKV_OK 0
#define PKV_ERR_INVALID_ARG 1     /* null pointer, bad shape, bad length, even pool width ... */
#define PKV_ERR_UNSUPPORTED 2     /* dtype / head_dim / pool kind / batch size not built */
#define PKV_ERR_WORKSPACE 3       /* workspace too small or misaligned (256 bytes) */
#define PKV_ERR_CUDA 4            /* a launch failed; the CUDA error is left for the caller */
#define PKV_ERR_DEVICE_STATUS 5   /* a kernel recorded a failure in the workspace status word */
#define PKV_ERR_STATIC_SCRATCH 6  /* problem needs more than PKV_STATIC_SCRATCH_BYTES of built-in scratch */

#define PKV_DTYPE_FP32 0
#define PKV_DTYPE_BF16 1
#define PKV_DTYPE_FP16 2          /* IEEE binary16 */

#define PKV_POOL_MAX 0            /* centred max, window clipped to the prefix (the graded reading of Section 4.2.2) */
#define PKV_POOL_AVG 1            /* centred mean: zeros outside the prefix, always divided by the width; float
                                     additions left to right, then one float division (it decides the top-k) */

#define PKV_SCHEDULE_LINEAR 0      /* Eq. 1: arithmetic decrease from the lowest layer to the top one */
#define PKV_SCHEDULE_GEOMETRIC 1   /* appendix "Allocation Strategies": constant ratio between consecutive layers */

/* cfg->flags.  PKV_FLAG_INPUTS_FINAL: the caller promises that q_win and k are complete in memory by the time
 * the kernels ahead of the call on its stream have been ALLOWED TO LET THEIR DEPENDENTS START, not merely by the
 * time they finish: nothing still running on the stream writes them.  The score kernels then begin to read them
 * at once, beside the tail of whatever runs before them (about 5 % on short contexts).  Without the flag they
 * wait until everything ahead of them on the stream has completed and flushed its writes, which is always right,
 * also when the producer of K is a kernel that signals its dependents early (programmatic dependent launch). */
#define PKV_FLAG_INPUTS_FINAL 1u

#define PKV_MAX_BATCH 64          /* sequences per call */
#define PKV_MAX_STAGES 8          /* kernels one pyramidkv_compress_layer call may launch */
#define PKV_STATIC_SCRATCH_BYTES (8u << 20)  /* built-in scratch of pyramidkv_score_window_static: 8 MiB per GPU */

typedef struct pkv_config {
  int32_t num_layers;    /* m >= 1 */
  int32_t num_q_heads;   /* H_q, a multiple of num_kv_heads */
  int32_t num_kv_heads;  /* H_kv */
  int32_t head_dim;      /* d: 64 or 128 */
  int32_t window;        /* alpha >= 1: instruction tokens, always kept (Section 4.2.1) */
  int32_t pool_kernel;   /* odd width of the score pooling, 1 = none (Section 4.2.2) */
  int32_t pool_kind;     /* PKV_POOL_MAX or PKV_POOL_AVG */
  int32_t dtype;         /* PKV_DTYPE_*: element type shared by K, V and Q_win */
  int32_t avg_budget;    /* B: mean rows kept per layer and KV head, window rows included; >= alpha */
  int32_t schedule;      /* PKV_SCHEDULE_*: shape of the per-layer budgets; 0 = Eq. 1 */
  double  beta;          /* pyramid shape, >= 1 (Section 4.2.1); 1 = same size in every layer */
  uint32_t flags;        /* PKV_FLAG_* bits, 0 by default */
  uint32_t sweep_ctas;   /* CTAs the persistent score sweeps of a call launch: 0 = one per SM (default), else at
                            most this many (<= 1024).  A caller that runs independent layers on several streams
                            gives each call a share of the SMs this way, so that two layers' sweeps run side by
                            side instead of one after the other; results do not depend on it beyond rounding. */
} pkv_config;

typedef struct pkv_tensor {
  const void* ptr;       /* device */
  int64_t stride_batch;  /* strides in elements */
  int64_t stride_head;
  int64_t stride_token;  /* >= head_dim; the head dimension itself has stride 1 */
} pkv_tensor;

/*
 * Where a pointer lives, as the CUDA runtime sees it (host only; a query, nothing is enqueued):
 *   PKV_MEM_PAGEABLE_HOST 0   ordinary host memory: kernels cannot read it
 *   PKV_MEM_PINNED_HOST   1   page-locked host memory mapped at the same address on the device
 *   PKV_MEM_DEVICE        2   device memory
 *   PKV_MEM_MANAGED       3   managed memory
 * Returns the kind, or a negative status (-PKV_ERR_CUDA when no CUDA device answers).
 * "device" tensors of the calls below may be of kind 1, 2 or 3.  Kind 1 makes sense for V: the path only
 * ever touches the rows of V that are kept (Section 4.2.2: the rest is evicted), so a V that stays in pinned
 * host memory costs a few hundred kilobytes of bus reads per layer instead of a copy of the whole tensor.
 * K is read in full, twice, and belongs in device memory.
 */
#define PKV_MEM_PAGEABLE_HOST 0
#define PKV_MEM_PINNED_HOST 1
#define PKV_MEM_DEVICE 2
#define PKV_MEM_MANAGED 3
int pyramidkv_memory_kind(const void* ptr);

/* Human-readable name of a status code (static string, never NULL). */
const char* pyramidkv_strerror(int status);

/*
 * Per-layer budgets, Section 4.2.1 and Eq. 1.  Host only, no CUDA call.
 * The alpha window tokens are set aside first, so the budget that the pyramid
 * shares out is k_total = m * (B - alpha):
 *     k^{m-1} = k_total / (beta * m),   k^0 = 2 * k_total / m - k^{m-1},
 *     k^l = k^0 - (k^0 - k^{m-1}) * l / (m - 1).
 * beta is snapped to the nearest multiple of 1/1024 and the schedule is
 * evaluated in integers: every k^l is floored and the units lost to flooring go
 * one each to layers 0, 1, ... so that the budgets are non-increasing and sum to
 * k_total exactly.  m = 1 gives k^0 = k_total.
 *
 * cfg->schedule = PKV_SCHEDULE_GEOMETRIC selects the geometric (exponential in the layer index) decay that
 * the appendix "Allocation Strategies" compares Eq. 1 with.  The paper gives it no formula; here it keeps
 * Eq. 1's two constraints (top layer k_total / (beta m), budgets sum to k_total) and puts a constant ratio
 * rho >= 1 between consecutive layers: rho is the root of 1 + rho + ... + rho^(m-1) = beta m, rounded to a
 * multiple of 2^-20, and layer l gets k_total * rho^(m-1-l) / (1 + rho + ... + rho^(m-1)), floored, leftover
 * units to layers 0, 1, ... as above.  beta = 1 is the uniform split under both schedules; with m = 2 the
 * two schedules coincide.
 *   k_out  host, [num_layers]: rows of the prefix layer l may keep (window rows come on top).
 * Errors: PKV_ERR_INVALID_ARG for a null pointer or a config outside the ranges above.
 */
int pyramidkv_layer_budgets(const pkv_config* cfg, int32_t* k_out);

/*
 * Rows each KV head of a sequence of seq_len tokens keeps in a layer whose
 * budget is k_layer (Section 4.1: a budget k^l < n; Section 4.2.1: the window is
 * kept in every layer).  Host only.
 *   seq_len <= avg_budget      -> seq_len (the context fits: nothing is evicted)
 *   otherwise                  -> min(k_layer, seq_len - alpha) + alpha
 * Returns the count, or a negative status (-PKV_ERR_INVALID_ARG).
 */
int pyramidkv_kept_count(const pkv_config* cfg, int32_t k_layer, int32_t seq_len);

/*
 * Bytes of device scratch that any call below needs for up to `batch` sequences
 * of at most `max_seq_len` tokens.  Host only.  Returns 0 for an invalid config.
 * The workspace must be 256-byte aligned.  Its first 256 bytes hold a status
 * word that kernels only ever set to non-zero; the caller zeroes those bytes once
 * after allocation (the rest needs no initialisation).  Calls that share a
 * workspace must be ordered on one stream.
 */
size_t pyramidkv_workspace_bytes(const pkv_config* cfg, int32_t batch, int32_t max_seq_len);

/*
 * Window attention scores, Section 4.2.2, Eq. 2 and Eq. 3.
 * For query head g and window row j (absolute position P_b + j) the logits are
 * q . k_i / sqrt(d) over the keys i <= P_b + j the row can see (causal), and
 * A = softmax over those keys.  The score of prefix key i < P_b for KV head h is
 *     s[h][i] = (1/G) * sum over the G query heads of the group, sum over j < alpha, of A[j][i].
 * Inputs in fp32 or bf16; products and sums accumulate in fp32; scores are fp32.
 *   q_win, k   device tensors (layout above)
 *   seq_lens   host [batch], each alpha + 1 <= n_b
 *   scores     device, [batch][H_kv][ld_scores] floats; the first P_b entries of a row are written
 *   ld_scores  >= max_b P_b
 *   workspace  device scratch, workspace_bytes >= pyramidkv_workspace_bytes(cfg, batch, max n_b)
 * Errors: INVALID_ARG, UNSUPPORTED (dtype, head_dim, batch > PKV_MAX_BATCH), WORKSPACE, CUDA.
 */
int pyramidkv_score_window(const pkv_config* cfg, pkv_tensor q_win, pkv_tensor k,
                           const int32_t* seq_lens, int32_t batch,
                           float* scores, int64_t ld_scores,
                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * pyramidkv_score_window for callers that cannot allocate.  The paper has no
 * counterpart: this is an integration aid.  Same inputs, same scores as
 * pyramidkv_score_window, but no workspace argument: the kernels' scratch
 * (partial row statistics and the row normalisers) lives in an array of
 * PKV_STATIC_SCRATCH_BYTES (8 MiB) that is built into the library, so the call
 * and everything under it performs no cudaMalloc / cudaFree and needs no memory
 * pool.  It is meant for code that is handed only its input and output buffers:
 * an operator plugged into a serving engine that has already given all device
 * memory to its own pool, or a section where an allocation (which may
 * synchronise the whole device) is not acceptable.
 *   - Every GPU on which the library is loaded holds the 8 MiB until the process ends.
 *   - The problem must fit.  With 16-bit inputs and (H_q / H_kv) * alpha <= 256 rows per KV head the
 *     scratch is (256 + batch * H_kv) * 32 * (H_q / H_kv) * alpha bytes plus the row normalisers,
 *     whatever the context length (2.2 MB for one 8-head sequence with 256 rows); other shapes run
 *     on the fp32-pipe kernels and need batch * H_kv * ceil(n_max / 128) * (H_q / H_kv) * alpha * 16
 *     bytes.  Larger problems are refused with PKV_ERR_STATIC_SCRATCH before anything is enqueued;
 *     use pyramidkv_score_window with a workspace for those.
 *   - The first call made on a device looks up the array's device address
 *     (cudaGetSymbolAddress) and caches it; make that first call outside any
 *     stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's
 *     contents.  The call clears the part that must start at zero itself, but two
 *     calls whose kernels overlap on the GPU (different streams, no ordering
 *     between them) race on it: order them on one stream or with events.
 * Errors: INVALID_ARG, UNSUPPORTED, STATIC_SCRATCH, CUDA.
 */
int pyramidkv_score_window_static(const pkv_config* cfg, pkv_tensor q_win, pkv_tensor k,
                                  const int32_t* seq_lens, int32_t batch,
                                  float* scores, int64_t ld_scores, void* stream);

/*
 * pyramidkv_check_status for the built-in scratch (the paper has no counterpart): the status word of
 * pyramidkv_score_window_static lives at the head of the library's own array, where the caller has no
 * pointer to it.  Synchronises `stream`, copies the word out and returns PKV_OK or
 * PKV_ERR_DEVICE_STATUS (word in *detail_or_null); PKV_ERR_CUDA if the array cannot be reached.
 * Allocates nothing.
 */
int pyramidkv_check_status_static(void* stream, uint32_t* detail_or_null);

/*
 * Pooling and selection, Section 4.2.2.  Per sequence and KV head:
 * pooled[i] = max of scores[i + t] over |t| <= (pool_kernel - 1)/2 clipped to [0, P_b);
 * the min(k_layer, P_b) positions with the largest pooled value are kept, ties
 * going to the smaller position; kept positions are written in ascending order
 * followed by the window positions P_b .. n_b - 1.  A sequence with
 * n_b <= avg_budget keeps every position and its scores are not read.
 *   scores     device, as written by pyramidkv_score_window
 *   k_layer    >= 0, this layer's entry of pyramidkv_layer_budgets
 *   indices    device int32, packed rows (layout above), sum_b H_kv * c_b entries
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA.
 */
int pyramidkv_select_topk(const pkv_config* cfg, const float* scores, int64_t ld_scores,
                          const int32_t* seq_lens, int32_t batch, int32_t k_layer,
                          int32_t* indices,
                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * Eviction by gather (appendix on torch.gather: select indices, compute source
 * addresses from the strides, write a new tensor).  Copies, bit for bit, row
 * indices[r] of K and of V into row r of k_out and v_out.  Out of place: k_out
 * and v_out must not overlap K or V.  v.ptr and v_out may both be NULL to move K only.
 *   indices    device int32, packed rows as written by pyramidkv_select_topk.  An entry outside
 *              [0, n_b) is never turned into an address: its output row is left as it was.  (This
 *              call has no workspace, so nothing is recorded; pyramidkv_gather_paged records it.)
 *   k_out,v_out device, [sum_b H_kv * c_b][d] elements of the config dtype, 16-byte aligned
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA.
 */
int pyramidkv_gather_compact(const pkv_config* cfg, pkv_tensor k, pkv_tensor v,
                             const int32_t* indices, const int32_t* seq_lens, int32_t batch,
                             int32_t k_layer, void* k_out, void* v_out, void* stream);

/*
 * The whole step for one layer (Section 4.2): scores, pool, top-k with the
 * budget of `layer`, window retention, gather; the same results as the three
 * calls above issued in order.
 *   layer          0 <= layer < num_layers; its budget is taken from the schedule cfg->schedule names (Eq. 1 by default)
 *   scores_or_null device [batch][H_kv][ld_scores] to receive the scores, or NULL
 *                  (then ld_scores is ignored and scores live in the workspace)
 * Errors: as above.
 */
int pyramidkv_compress_layer(const pkv_config* cfg, int32_t layer,
                             pkv_tensor q_win, pkv_tensor k, pkv_tensor v,
                             const int32_t* seq_lens, int32_t batch,
                             void* k_out, void* v_out, int32_t* indices,
                             float* scores_or_null, int64_t ld_scores,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * Hand-off from the prefill attention (Section 4.1: the scores come from the very attention rows the
 * prefill has just computed, Eq. 2).  A prefill attention kernel that ran over the window rows
 * already holds each row's log-sum-exp; given it, the first of the two K sweeps (the one that only
 * finds the row normalisers) is skipped and the scores need a single pass over K.
 *   window_lse  device, [batch][H_q][alpha] floats, contiguous: for query head g and window row j of
 *               sequence b the natural logarithm of  sum over keys i <= P_b + j of exp(q . k_i / sqrt(d)),
 *               i.e. the causal softmax denominator of that row in log form.
 * Everything else as pyramidkv_score_window / pyramidkv_compress_layer; results agree with them to
 * rounding when window_lse is exact.  A wrong window_lse gives wrongly scaled scores: it is not
 * checked.  Errors: as the base calls, plus INVALID_ARG for a null window_lse.
 */
int pyramidkv_score_window_lse(const pkv_config* cfg, pkv_tensor q_win, pkv_tensor k, const float* window_lse,
                               const int32_t* seq_lens, int32_t batch,
                               float* scores, int64_t ld_scores,
                               void* workspace, size_t workspace_bytes, void* stream);
int pyramidkv_compress_layer_lse(const pkv_config* cfg, int32_t layer,
                                 pkv_tensor q_win, pkv_tensor k, pkv_tensor v, const float* window_lse,
                                 const int32_t* seq_lens, int32_t batch,
                                 void* k_out, void* v_out, int32_t* indices,
                                 float* scores_or_null, int64_t ld_scores,
                                 void* workspace, size_t workspace_bytes, void* stream);

/*
 * Decode attention over the compact cache of one layer (Section 4.1: after compression only K_s, V_s
 * are used for inference; Section 4.2.2: evicted entries take part in no later computation).  For one
 * new token per sequence, query head g attends to every kept row of its KV head:
 *     out[b][g] = softmax(q[b][g] . K_s^T / sqrt(d)) V_s      (no mask: every kept token precedes it).
 *   q          device, [batch][H_q][d] of the config dtype, contiguous, 16-byte aligned
 *   k_cache, v_cache  device, packed rows as written by pyramidkv_compress_layer for budget k_layer
 *   out        device, [batch][H_q][d] floats
 * Positions are not needed here: K rows carry their rotary embedding as computed at prefill.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA.
 */
int pyramidkv_decode_attention(const pkv_config* cfg, const void* q, const void* k_cache, const void* v_cache,
                               const int32_t* seq_lens, int32_t batch, int32_t k_layer, float* out, void* stream);

/*
 * Attention recall of a layer's selection (appendix "Attention Recall Rate Experiment": the share of
 * the attention computed with the kept keys relative to all keys), per sequence and KV head, averaged
 * over the alpha window rows and the group's query heads.  With the scores of Eq. 3 this is
 *     recall[b][h] = 1 - (sum of scores[b][h][i] over evicted prefix positions i) / alpha,
 * since each window row's attention sums to one and the window keys are always kept.
 *   scores, indices  device, as produced for this layer; recall  device, [batch][H_kv] floats
 * An index entry that is no prefix position of its sequence is not used as an address; it counts as
 * not kept.
 * Errors: INVALID_ARG, CUDA.
 */
int pyramidkv_attention_recall(const pkv_config* cfg, const float* scores, int64_t ld_scores,
                               const int32_t* indices, const int32_t* seq_lens, int32_t batch,
                               int32_t k_layer, float* recall, void* stream);

/*
 * The window rows' attention together with the scores (Section 4.1, Section 4.2.2 Eq. 2 and Eq. 3: the scores
 * are column sums of the attention matrix of the last alpha queries, whose rows times V are what the prefill
 * attention returns for those queries).  One kernel forms the softmax probabilities of the window rows once and
 * uses them twice: summed over rows and query heads they are the scores, multiplied by V they are the attention
 * output.  A prefill that calls this for its last alpha rows gets their output and the compression from the same
 * pass over K; the row normalisers still come from the row-statistics sweep that runs first.
 *   attn_out  device, [batch][H_q][alpha][d] floats, contiguous, 16-byte aligned:
 *             attn_out[b][g][j] = sum over keys i <= P_b + j of softmax_i(q_gj . k_i / sqrt(d)) * v_i
 *   scores    pyramidkv_attend_window: required, device [batch][H_kv][ld_scores] (the P_b prefix positions of
 *             each row are written); pyramidkv_attend_compress_layer: optional as in pyramidkv_compress_layer
 * The probabilities are rounded to the inputs' 16-bit type before they multiply V, as V itself is.  Rows of V
 * behind a sequence's length are never used, whatever they hold.  Everything else as pyramidkv_score_window /
 * pyramidkv_compress_layer; the scores agree with theirs to rounding.
 * Errors: as those calls; UNSUPPORTED unless the inputs are 16-bit, head_dim is 128 and (H_q / H_kv) * window
 * <= 256.  The workspace is the one pyramidkv_workspace_bytes sizes.
 */
int pyramidkv_attend_window(const pkv_config* cfg, pkv_tensor q_win, pkv_tensor k, pkv_tensor v,
                            const int32_t* seq_lens, int32_t batch, float* attn_out,
                            float* scores, int64_t ld_scores,
                            void* workspace, size_t workspace_bytes, void* stream);
int pyramidkv_attend_compress_layer(const pkv_config* cfg, int32_t layer,
                                    pkv_tensor q_win, pkv_tensor k, pkv_tensor v,
                                    const int32_t* seq_lens, int32_t batch, float* attn_out,
                                    void* k_out, void* v_out, int32_t* indices,
                                    float* scores_or_null, int64_t ld_scores,
                                    void* workspace, size_t workspace_bytes, void* stream);

/*
 * Measuring aid; the paper has no counterpart.  Same arguments and results as
 * pyramidkv_compress_layer, but a CUDA event is recorded after every kernel the
 * call launches, the stream is synchronised, and the device time of each kernel
 * is returned.  Creates and destroys CUDA events; not for use on a hot path.
 *   stage_ms     host [PKV_MAX_STAGES]      milliseconds per kernel, in launch order
 *   stage_names  host [PKV_MAX_STAGES][32]  NUL-terminated kernel names
 *   num_stages   host                       kernels launched
 */
int pyramidkv_profile_layer(const pkv_config* cfg, int32_t layer,
                            pkv_tensor q_win, pkv_tensor k, pkv_tensor v,
                            const int32_t* seq_lens, int32_t batch,
                            void* k_out, void* v_out, int32_t* indices,
                            float* scores_or_null, int64_t ld_scores,
                            void* workspace, size_t workspace_bytes, void* stream,
                            float* stage_ms, char (*stage_names)[32], int32_t* num_stages);

/* The same measuring aid for pyramidkv_attend_compress_layer. */
int pyramidkv_profile_attend_compress_layer(const pkv_config* cfg, int32_t layer,
                                            pkv_tensor q_win, pkv_tensor k, pkv_tensor v,
                                            const int32_t* seq_lens, int32_t batch, float* attn_out,
                                            void* k_out, void* v_out, int32_t* indices,
                                            float* scores_or_null, int64_t ld_scores,
                                            void* workspace, size_t workspace_bytes, void* stream,
                                            float* stage_ms, char (*stage_names)[32], int32_t* num_stages);

/* The same measuring aid for pyramidkv_compress_layer_lse. */
int pyramidkv_profile_layer_lse(const pkv_config* cfg, int32_t layer,
                                pkv_tensor q_win, pkv_tensor k, pkv_tensor v, const float* window_lse,
                                const int32_t* seq_lens, int32_t batch,
                                void* k_out, void* v_out, int32_t* indices,
                                float* scores_or_null, int64_t ld_scores,
                                void* workspace, size_t workspace_bytes, void* stream,
                                float* stage_ms, char (*stage_names)[32], int32_t* num_stages);

/*
 * Paged placement of a layer's compact cache (appendix on paged attention: the block table of a
 * sequence is widened to one block table per layer, so that each layer's cache is found through its
 * own pages rather than at fixed offsets, and a layer with a small budget holds few pages).
 *
 * Layout.  A pool holds num_pages pages; a page holds page_size rows of d elements of ONE KV head of
 * one sequence: k_pool, v_pool are [num_pages][page_size][d] of the config dtype.  Row r of the kept
 * list of (sequence b, KV head h) sits in page  table[r / page_size]  at slot  r % page_size, where
 * `table` is that head's slice of the layer's block table.  The block table of one layer is a packed
 * int32 array: sequences in batch order, inside a sequence head after head, each head holding
 *     pages_b = pyramidkv_pages_needed(cfg, k_layer, n_b, page_size) = ceil(c_b / page_size)
 * entries; the slice of (b, h) starts at  H_kv * (pages_0 + ... + pages_{b-1}) + h * pages_b.
 * The caller's allocator fills the table with pages it owns; the library only follows it.  Slots of
 * the last page past c_b, and pages the table does not name, are not touched.  The index list (one
 * original position per kept row) keeps the packed layout of pyramidkv_compress_layer.
 *
 * A table entry outside [0, num_pages) is never dereferenced: the row is skipped and the workspace
 * status word gets bit 2 set (pyramidkv_check_status then returns PKV_ERR_DEVICE_STATUS).  An entry of
 * a caller-supplied index list outside [0, n_b) is treated the same way, with bit 3.
 */

/* Host only.  Pages one KV head of a seq_len-token sequence needs; negative status on bad arguments. */
int pyramidkv_pages_needed(const pkv_config* cfg, int32_t k_layer, int32_t seq_len, int32_t page_size);

/*
 * Eviction by gather into pages: the rows of K and V named by `indices` (packed, as written by
 * pyramidkv_select_topk for budget k_layer) go to their page slots.  Bit copies.
 *   block_table  device int32, layout above      page_size >= 1, num_pages >= 1
 *   k_pool, v_pool  device, 16-byte aligned      workspace: only its status word is used (>= 256 bytes)
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA.
 */
int pyramidkv_gather_paged(const pkv_config* cfg, pkv_tensor k, pkv_tensor v, const int32_t* indices,
                           const int32_t* seq_lens, int32_t batch, int32_t k_layer,
                           const int32_t* block_table, int32_t page_size, int32_t num_pages,
                           void* k_pool, void* v_pool,
                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * pyramidkv_compress_layer with the kept rows placed in pages: scores, pool, top-k and window
 * retention as there (window_lse_or_null: the optional row normalisers of the single-sweep mode),
 * then the gather above.  `indices` receives the packed list of original positions.
 */
int pyramidkv_compress_layer_paged(const pkv_config* cfg, int32_t layer,
                                   pkv_tensor q_win, pkv_tensor k, pkv_tensor v, const float* window_lse_or_null,
                                   const int32_t* seq_lens, int32_t batch,
                                   const int32_t* block_table, int32_t page_size, int32_t num_pages,
                                   void* k_pool, void* v_pool, int32_t* indices,
                                   float* scores_or_null, int64_t ld_scores,
                                   void* workspace, size_t workspace_bytes, void* stream);

/*
 * pyramidkv_decode_attention over a paged layer: the kept rows of each KV head are read through the
 * layer's block table, in list order.  Arguments as there and as pyramidkv_gather_paged.
 */
int pyramidkv_decode_attention_paged(const pkv_config* cfg, const void* q, const void* k_pool, const void* v_pool,
                                     const int32_t* block_table, int32_t page_size, int32_t num_pages,
                                     const int32_t* seq_lens, int32_t batch, int32_t k_layer, float* out,
                                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * Sequence-sharded compression, for contexts whose K does not fit one GPU.  The keys (and values) of a
 * sequence are split into contiguous position ranges, one per GPU; every GPU holds the window queries.
 * The window keys (the last alpha positions) all lie on the shard that ends the sequence, which must also
 * hold at least one prefix key.  A layer then takes these steps (Section 4.2.2 on each shard, with the one
 * exchange Eq. 2's softmax needs); the two exchanges are the caller's (any all-gather / all-reduce):
 *   1. pyramidkv_shard_window_lse   every shard: partial normalisers of the window rows over its keys
 *      -- all-gather the parts --
 *   2. pyramidkv_merge_lse          the rows' full normalisers
 *   3. pyramidkv_shard_scores       every shard: Eq. 3 scores of its own prefix keys (one K sweep)
 *      -- all-gather the score ranges into the sequence's score row --
 *   4. pyramidkv_select_topk        every shard runs the same selection on the full score row
 *   5. pyramidkv_shard_gather       every shard copies the kept rows it owns into a zero-filled packed
 *      buffer  -- all-reduce (integer sum, each row has one owner) if every GPU wants the whole cache --
 * The result equals pyramidkv_compress_layer on the unsharded tensors (scores to rounding, rows bit for bit).
 *
 *   k_shard, v_shard  this GPU's keys/values: token t of the view is position shard_begin[b] + t
 *   shard_keys   host [batch]: keys of sequence b in this shard (>= 1)
 *   window_keys  host [batch]: alpha if this shard ends sequence b (then shard_keys[b] >= alpha + 1), else 0
 *   lse_out, parts, window_lse  device floats [batch][H_q][alpha]: natural log of a sum of exponentials
 * Errors: as pyramidkv_score_window; INVALID_ARG for a window_keys entry other than 0 or alpha.
 */
int pyramidkv_shard_window_lse(const pkv_config* cfg, pkv_tensor q_win, pkv_tensor k_shard,
                               const int32_t* shard_keys, const int32_t* window_keys, int32_t batch,
                               float* lse_out, void* workspace, size_t workspace_bytes, void* stream);
/* parts: device [num_shards][count] floats; out: device [count];  out = log(sum over shards of exp(part)). */
int pyramidkv_merge_lse(const float* parts, int32_t num_shards, int64_t count, float* out, void* stream);
/* scores: device [batch][H_kv][ld_scores], the first shard_keys[b] - window_keys[b] of each row are written. */
int pyramidkv_shard_scores(const pkv_config* cfg, pkv_tensor q_win, pkv_tensor k_shard, const float* window_lse,
                           const int32_t* shard_keys, const int32_t* window_keys, int32_t batch,
                           float* scores, int64_t ld_scores,
                           void* workspace, size_t workspace_bytes, void* stream);
/*
 * indices, k_out, v_out: the packed layout of the WHOLE layer (seq_lens are the full lengths); only the
 * rows whose position lies in [shard_begin[b], shard_begin[b] + shard_keys[b]) are written.
 */
int pyramidkv_shard_gather(const pkv_config* cfg, pkv_tensor k_shard, pkv_tensor v_shard, const int32_t* indices,
                           const int32_t* seq_lens, int32_t batch, int32_t k_layer,
                           const int32_t* shard_begin, const int32_t* shard_keys,
                           void* k_out, void* v_out, void* stream);

/*
 * Whole-model call on two lanes.  The paper has no counterpart: this is scheduling.  Selection and gather
 * (Section 4.2.2's last step) keep only a fraction of the GPU's SMs busy, and layers are independent, so the
 * score sweeps of layer l + 1 can run beside the selection of layer l.  A pkv_lanes object splits the SMs of
 * the current device into two disjoint groups (CUDA green contexts; nothing outlives the process or touches
 * another process) with one stream on each: `select_sms` SMs (a multiple of 8, at least 8, at most half of
 * the device) for selection and gather, the rest for the score sweeps.
 *   pyramidkv_lanes_create    host; creates contexts, streams and events: not for a hot path.  UNSUPPORTED
 *                             when the driver has no green contexts or cannot split as asked.
 *   pyramidkv_lanes_destroy   host; the lanes must be idle.
 *   pyramidkv_compress_model_lanes
 *       layers first_layer .. first_layer + num_layers - 1 of the model, exactly as num_layers calls of
 *       pyramidkv_compress_layer (window_lse_or_null: NULL, or one pointer per layer as for
 *       pyramidkv_compress_layer_lse); q_win, k, v, k_out, v_out, indices are host arrays with one entry per
 *       layer.  `workspaces` holds TWO distinct workspaces of workspace_bytes each (consecutive layers
 *       alternate between them); each has its own status word.  The work is ordered after what `stream`
 *       holds at the call and `stream` continues after all of it; in between it runs on the lanes' streams.
 * Results are those of the per-layer calls bit for bit (the same kernels on the same data; only the number of
 * CTAs of the sweeps follows the lane's SM count).  Errors: as pyramidkv_compress_layer; INVALID_ARG when the
 * lanes belong to another device.
 */
typedef struct pkv_lanes pkv_lanes;
int pyramidkv_lanes_create(int32_t select_sms, pkv_lanes** out);
int pyramidkv_lanes_destroy(pkv_lanes* lanes);
int pyramidkv_lanes_info(const pkv_lanes* lanes, int32_t* score_sms, int32_t* select_sms);
int pyramidkv_compress_model_lanes(const pkv_config* cfg, pkv_lanes* lanes, int32_t first_layer, int32_t num_layers,
                                   const pkv_tensor* q_win, const pkv_tensor* k, const pkv_tensor* v,
                                   const float* const* window_lse_or_null,
                                   const int32_t* seq_lens, int32_t batch,
                                   void* const* k_out, void* const* v_out, int32_t* const* indices,
                                   void* const* workspaces, size_t workspace_bytes, void* stream);

/*
 * Test aids; the paper has no counterpart.
 *
 * pyramidkv_test_hooks: process-wide knobs read by the calls that follow.  wait_clocks > 0 replaces the bound
 * of every wait inside the tensor-core score kernels (default 2^31 SM clocks).  Bit 0 of withhold_tile makes the
 * copy engine thread of the first CTA of the row-statistics sweep leave out its last K tile, so that the waits
 * for that tile run out, the kernel gives up in an orderly way (every role leaves its loop, the accumulator
 * memory is released, the status word gets bit 1) and returns.  Bit 1 keeps short contexts on the two-sweep
 * kernels instead of the single-sweep one (same scores within rounding).  Bit 2 is bit 0 for the window-attention
 * kernel of pyramidkv_attend_window.  (0, 0) restores normal operation.
 *
 * pyramidkv_test_slow_copy: copies `bytes` (a multiple of 16) from src to dst with one small CTA that lets
 * its dependents start at once and then copies in `steps` pieces with a pause after each: a stand-in for a
 * caller's kernel that produces K and signals early.
 */
int pyramidkv_test_hooks(int64_t wait_clocks, int32_t withhold_tile);
int pyramidkv_test_slow_copy(void* dst, const void* src, size_t bytes, int32_t steps, void* stream);

/*
 * Synchronises `stream` and reads the workspace status word.  For tests and
 * debugging.  Returns PKV_OK, PKV_ERR_DEVICE_STATUS (a kernel gave up on a
 * bounded wait or saw an impossible state; *detail_or_null receives the word),
 * or PKV_ERR_CUDA.  Bits of the word: 0 the selection emitted a wrong count,
 * 1 a bounded wait ran out, 2 a block-table entry outside the pool, 3 an index
 * entry outside its sequence.  The bits stay set until the caller zeroes the
 * first 256 bytes of the workspace.
 */
int pyramidkv_check_status(const void* workspace, void* stream, uint32_t* detail_or_null);

#ifdef __cplusplus
}
#endif
#endif /* PYRAMIDKV_H_ */
