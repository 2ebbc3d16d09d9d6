/*
 * fastkv.h -- C ABI of the B200 (sm_100a) FastKV token-saliency selection path.
 *
 * One layer's work is four calls on one CUDA stream:
 *
 *   fastkv_score       window-query saliency scores          (Eq. 1, Eq. 2, Sec. 4.2)
 *   fastkv_select_kv   per-KV-group top-k   (KVCompress)      (App. B.1, Alg. 1)
 *   fastkv_select_tsp  layer-level top-k    (HiddenCompress)  (App. B.1, Sec. 4.2)
 *   fastkv_compact     gather of the kept K/V rows, hidden states and position ids
 *                                                             (Alg. 1: C <- update(K, V); x)
 *
 * Conventions
 *   - Every function returns a fastkv_status; nothing throws or aborts.
 *   - Unless a parameter says HOST, every data pointer is DEVICE memory owned by the
 *     caller.  The library allocates no device memory, keeps no pointer after the
 *     enqueued work has run, and does not synchronise (fastkv_device_status and
 *     fastkv_layer_host excepted).  Work is ordered on `stream` (a cudaStream_t
 *     passed as void*; NULL is the legacy default stream).
 *   - bf16 tensors are passed as void*; the innermost dimension is contiguous and
 *     strides are counted in elements.
 *   - Sequences of a batch are packed along the token axis: sequence b owns rows
 *     cu_seqlens[b] .. cu_seqlens[b+1]-1, L_b = cu_seqlens[b+1]-cu_seqlens[b].
 *     Token indices produced and consumed by the library are sequence-local.
 *   - Inputs must be finite.  With NaN/Inf inputs the index sets are unspecified
 *     (but in range).
 */
#ifndef FASTKV_H_
#define FASTKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum fastkv_status {
  FASTKV_OK = 0,
  FASTKV_ERR_INVALID_ARG = 1,   /* NULL where a pointer is required, bad sizes, k out of range ...  */
  FASTKV_ERR_UNSUPPORTED = 2,   /* valid but not built: head_dim, G*w, alignment, device generation */
  FASTKV_ERR_WORKSPACE = 3,     /* workspace NULL, misaligned or smaller than fastkv_workspace_bytes */
  FASTKV_ERR_CUDA = 4,          /* a CUDA call failed; fastkv_last_error() has the text             */
  FASTKV_ERR_DEVICE_TIMEOUT = 5,/* a bounded device-side wait gave up (fastkv_device_status only)   */
  FASTKV_ERR_DEVICE_INDEX = 6   /* an index handed to fastkv_compact was out of range; row skipped  */
} fastkv_status;

enum { FASTKV_POOL_AVG = 0, FASTKV_POOL_MAX = 1 };
enum { FASTKV_GROUP_THEN_POOL = 0, FASTKV_POOL_THEN_GROUP = 1 };
enum { FASTKV_Q_FULL = 0, FASTKV_Q_WINDOW = 1 };

/*
 * Problem statement of one layer (Sec. 4.2, App. B.1): N_I = L_b prompt tokens per
 * sequence, N_obs = window, H = n_q_heads, key/value groups of G = H / n_kv_heads heads
 * (query head h reads KV head h / G).
 */
typedef struct fastkv_shape {
  int32_t batch;            /* B >= 1                                                         */
  int32_t total_len;        /* sum of L_b: rows of the packed k / v / hidden / pos tensors   */
  int32_t max_len;          /* max L_b (HOST knowledge used for grid sizing)                  */
  int32_t n_q_heads;
  int32_t n_kv_heads;
  int32_t head_dim;         /* 64 or 128                                                      */
  int32_t hidden_dim;       /* multiple of 8; only used by fastkv_compact                     */
  int32_t window;           /* w = N_obs (paper: 8); fastkv_score needs G*w <= 64             */
  int32_t pool_kernel;      /* odd, 1..63 (paper: 7)                                          */
  int32_t pool_mode;        /* FASTKV_POOL_AVG | FASTKV_POOL_MAX                              */
  int32_t agg_order;        /* FASTKV_GROUP_THEN_POOL: pool the group-summed score;
                               FASTKV_POOL_THEN_GROUP: pool per query head (Eq. 1), then sum
                               within the group (App. B.1).  Identical for AVG up to rounding */
  int32_t force_window;     /* 1: the last w positions are always kept and are not ranked
                               (Sec. 4.2); 0: plain top-k over all positions                  */
  int32_t q_layout;         /* FASTKV_Q_FULL: q has total_len rows, the library reads rows
                               cu_seqlens[b+1]-w .. cu_seqlens[b+1]-1;
                               FASTKV_Q_WINDOW: q has batch*w rows, sequence b at rows b*w..  */
  float softmax_scale;      /* 0 => 1/sqrt(head_dim)                                          */
  const int32_t* cu_seqlens;/* DEVICE int32[B+1], or NULL when B == 1 (then L = total_len)    */
  int64_t q_stride_tok, q_stride_head;   /* elements; multiples of 8                          */
  int64_t k_stride_tok, k_stride_head;
  int64_t v_stride_tok, v_stride_head;
  int64_t hidden_stride_tok;
} fastkv_shape;

/*
 * How many positions each sequence keeps.  Either the same k for every sequence
 * (k > 0, cu_k == NULL; sequence b writes outputs at offset b*k, total = B*k), or a
 * DEVICE int32[B+1] array of output offsets (k_b = cu_k[b+1]-cu_k[b]) whose last entry
 * the caller repeats on the host in `total`.  With force_window, w <= k_b <= L_b;
 * otherwise 1 <= k_b <= L_b.  The uniform form is validated on the host against
 * max_len only when B == 1; per-sequence violations clamp on the device and raise
 * FASTKV_ERR_DEVICE_INDEX in the status word.
 */
typedef struct fastkv_budget {
  int32_t k;
  int32_t total;
  const int32_t* cu_k;
} fastkv_budget;

/*
 * Bytes of workspace the calls below need for this shape (a multiple of 256): what the scoring
 * kernel that fastkv_score will pick for the shape uses -- per-phase counters, per-CTA softmax
 * statistics and one un-pooled fp32 score row per KV head (per query head with
 * FASTKV_POOL_THEN_GROUP), about 4.5 MB at 131072 tokens of the Llama-3.1-8B head shape -- plus the
 * 256-byte header with the device status word.  The other calls only use the header.
 */
int fastkv_workspace_bytes(const fastkv_shape* shape, size_t* bytes);

/*
 * Saliency scores (Eq. 1 and Eq. 2; Sec. 4.2).  For each sequence, query head h and window
 * row j (query position t_j = L-w+j) the causal softmax attention row over keys 0..t_j is
 * formed, summed over the window, aggregated over each KV group and pooled along the
 * sequence (kernel `pool_kernel`, stride 1, same length; AVG zero-pads and divides by the
 * kernel size, MAX ignores out-of-range positions):
 *   scores_kv [n_kv_heads, total_len] fp32   group-wise score used by KVCompress
 *   scores_tsp[total_len] fp32 or NULL       sum over all heads (Eq. 2 up to the factor 1/H)
 * Sums replace the paper's means; rankings are unchanged.
 * q, k: bf16.  workspace: >= fastkv_workspace_bytes, 256-byte aligned; it also holds the
 * device status word, so pass the same workspace to the other calls of the layer.
 */
int fastkv_score(const fastkv_shape* shape, const void* q, const void* k, float* scores_kv,
                 float* scores_tsp, void* workspace, size_t workspace_bytes, void* stream);

/*
 * KVCompress selection (App. B.1): for every sequence and KV head, the k_b positions with the
 * largest scores_kv, ties to the lower index; with force_window the last w positions are
 * always kept and only the prefix is ranked.  idx_kv is int32 [n_kv_heads, budget.total],
 * sequence-local, strictly ascending within each (head, sequence) segment.
 */
int fastkv_select_kv(const fastkv_shape* shape, const float* scores_kv, const fastkv_budget* budget,
                     int32_t* idx_kv, void* workspace, size_t workspace_bytes, void* stream);

/*
 * HiddenCompress selection (App. B.1, Sec. 4.2): the same rule applied once per sequence to
 * the layer-level score.  idx_tsp is int32 [budget.total].
 */
int fastkv_select_tsp(const fastkv_shape* shape, const float* scores_tsp, const fastkv_budget* budget,
                      int32_t* idx_tsp, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Both selections of a TSP layer in one launch (KVCompress and HiddenCompress, App. B.1): exactly
 * what fastkv_select_kv followed by fastkv_select_tsp produce, but the nine problems of a layer
 * (one per KV head plus the layer-level one) run side by side instead of one call after the other.
 */
int fastkv_select(const fastkv_shape* shape, const float* scores_kv, const fastkv_budget* kv, int32_t* idx_kv,
                  const float* scores_tsp, const fastkv_budget* tsp, int32_t* idx_tsp, void* workspace,
                  size_t workspace_bytes, void* stream);

/*
 * Compaction (Alg. 1: C <- update(K, V); reduced hidden states x).  Byte copies:
 *   k_out[g, j, :]   = k[cu_seqlens[b] + idx_kv[g, j], g, :]     [n_kv_heads, kv.total, head_dim]
 *   v_out likewise                                               (v, v_out may both be NULL)
 *   hidden_out[j, :] = hidden[cu_seqlens[b] + idx_tsp[j], :]     [tsp.total, hidden_dim]
 *   pos_out[j]       = pos_ids[cu_seqlens[b] + idx_tsp[j]]       [tsp.total] int32
 * where b is the sequence that owns output slot j.  Pass idx_tsp == NULL on layers without
 * Token-Selective Propagation; hidden/hidden_out and pos_ids/pos_out may each be NULL.
 * An index outside [0, L_b) is skipped and reported through the status word.
 */
int fastkv_compact(const fastkv_shape* shape, const int32_t* idx_kv, const fastkv_budget* kv,
                   const int32_t* idx_tsp, const fastkv_budget* tsp, const void* k, const void* v,
                   const void* hidden, const int32_t* pos_ids, void* k_out, void* v_out,
                   void* hidden_out, int32_t* pos_out, void* workspace, size_t workspace_bytes,
                   void* stream);

/*
 * Decoding over the compressed cache (what the retained KV of Alg. 1 is kept for; Sec. 3, Sec. 5.3): one new
 * query token per sequence attends to the kept entries of its KV group,
 *   out[b, h, :] = sum_j softmax_j(scale * <q[b, h], K[h / G, j]>) * V[h / G, j, :],  j over sequence b's kept entries.
 * q: bf16 [B, n_q_heads, head_dim]; k_cache, v_cache: bf16 [n_kv_heads, kv.total, head_dim], the k_out / v_out
 * layout of fastkv_compact; out: fp32 [B, n_q_heads, head_dim]; lse (optional): fp32 [B, n_q_heads], natural-log
 * sum of exponentials of each head's logits.  workspace: >= fastkv_decode_attn_workspace_bytes, 256-byte aligned
 * (the status word is not cleared by this call).  head_dim 64 or 128, at most 8 query heads per KV head.
 */
int fastkv_decode_attn_workspace_bytes(const fastkv_shape* shape, size_t* bytes);
int fastkv_decode_attn(const fastkv_shape* shape, const void* q, const void* k_cache, const void* v_cache,
                       const fastkv_budget* kv, float* out, float* lse, void* workspace, size_t workspace_bytes,
                       void* stream);

/*
 * The layer's own causal attention with the saliency scores as a by-product (Alg. 1: the scores are read off
 * Att_l, the attention matrix of the layer that is being computed anyway; App. D.4 times the separate
 * "token importance estimation" pass this call makes unnecessary).  For every sequence b and query head h
 *   out[t, h, :] = sum_{i <= t} softmax_i(scale * <q[t, h], k[i, h / G]>) * v[i, h / G, :]        t = 0 .. L_b - 1
 * and, from the rows t = L_b - w .. L_b - 1 of the same attention matrix, the scores fastkv_score defines:
 *   scores_kv [n_kv_heads, total_len] fp32 (may be NULL: attention only), scores_tsp [total_len] fp32 or NULL.
 * q: bf16, the FULL packed queries [total_len, n_q_heads, head_dim] (shape->q_layout must be FASTKV_Q_FULL);
 * k, v: bf16 [total_len, n_kv_heads, head_dim]; strides as in the shape (multiples of 8 elements);
 * out: bf16, dense [total_len, n_q_heads, head_dim], 16-byte aligned.  Probabilities are rounded to bf16 before
 * they are multiplied with v (fp32 accumulation), the scores are formed from the fp32 logits.
 * workspace: >= fastkv_prefill_workspace_bytes, 256-byte aligned: the header with the status word (cleared by this
 * call), the window rows' logits (n_q_heads x window x total_len fp32) and one un-pooled score row per KV head.
 */
int fastkv_prefill_workspace_bytes(const fastkv_shape* shape, size_t* bytes);
int fastkv_prefill_attention(const fastkv_shape* shape, const void* q, const void* k, const void* v, void* out,
                             float* scores_kv, float* scores_tsp, void* workspace, size_t workspace_bytes,
                             void* stream);

/*
 * Synchronises `stream`, then copies the device status word of `workspace` to the HOST
 * integers *status (a fastkv_status) and *site (which wait or check raised it; 0 if none).
 */
int fastkv_device_status(const void* workspace, void* stream, int32_t* status, int32_t* site);

/*
 * One whole layer step from HOST buffers (the end-to-end path of the bench): copies q, k, v,
 * hidden, pos_ids (HOST, pinned for full speed) into `arena` (DEVICE, caller-owned, at least
 * fastkv_layer_host_arena_bytes), runs score -> select_kv -> select_tsp -> compact on `stream`,
 * copies idx_kv, idx_tsp, k_out, v_out, hidden_out, pos_out back to the HOST outputs and
 * synchronises.  B == 1 or uniform budgets only (budget.cu_k must be NULL); shape->cu_seqlens,
 * if given, is a HOST array here.  k_tsp == 0 skips the TSP part.
 */
int fastkv_layer_host_arena_bytes(const fastkv_shape* shape, int32_t k_kv, int32_t k_tsp,
                                  size_t* bytes);
int fastkv_layer_host(const fastkv_shape* shape, int32_t k_kv, int32_t k_tsp, const void* q,
                      const void* k, const void* v, const void* hidden, const int32_t* pos_ids,
                      int32_t* idx_kv, int32_t* idx_tsp, void* k_out, void* v_out,
                      void* hidden_out, int32_t* pos_out, void* arena, size_t arena_bytes,
                      void* stream);

/*
 * fastkv_score for callers that cannot allocate device memory (no counterpart in the paper:
 * this is a deployment variant, not a step of the method).  Some callers have no workspace to
 * give: a plug-in inside a serving process whose device allocator belongs to the host
 * framework, code that runs where cudaMalloc is not permitted, a minimal C client without an
 * allocator.  This entry point computes exactly what fastkv_score computes, with the scratch
 * memory of the scoring kernels held in a fixed 16 MiB device array inside the library (so
 * every GPU that loads the library carries those 16 MiB until the process exits).  It calls no
 * cudaMalloc, cudaFree or other allocating routine.
 *   - Limit: fastkv_workspace_bytes(shape) must be <= 16 MiB (Llama-3.1-8B head shape: about
 *     500 000 tokens per call); larger shapes return FASTKV_ERR_WORKSPACE and launch nothing.
 *   - The first call on each device looks up the array's device address (the device must be
 *     current); make that first call before starting any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents; the
 *     words that must start at zero are cleared on `stream` by every call.  Two calls whose
 *     GPU work overlaps (different streams, no ordering) race on it: serialise them.
 *   - The device status word lives inside the array; fastkv_score_static_status reads it.
 *     Waits on the device stay bounded as in fastkv_score.
 * q, k, scores_kv, scores_tsp, stream: as for fastkv_score.
 */
int fastkv_score_static(const fastkv_shape* shape, const void* q, const void* k, float* scores_kv,
                        float* scores_tsp, void* stream);
/*
 * fastkv_device_status for the built-in array of the current device (no counterpart in the paper):
 * synchronises `stream`, then copies the status word and site left by the last fastkv_score_static
 * call on this device to the HOST integers.  Allocates nothing.  FASTKV_ERR_INVALID_ARG if
 * fastkv_score_static has not run on this device yet.
 */
int fastkv_score_static_status(void* stream, int32_t* status, int32_t* site);

/*
 * Test and tuning hooks (no counterpart in the paper).  Process-wide, not thread-safe; the
 * defaults (all 0) are what production code wants.  Keys:
 *   "score_path"          0 the library picks the scoring kernel by shape; 1 two kernels with
 *                         fp32 logits buffered in the workspace; 2 persistent kernel that reads K
 *                         a second time from L2; 3 persistent kernel that parks the logits in
 *                         tensor memory (FASTKV_ERR_UNSUPPORTED from the scoring calls when a
 *                         sequence is too long for it).  fastkv_workspace_bytes follows the choice.
 *   "score_partition"     path 3: several (sequence, head) phases side by side, each on its share of
 *                         the CTAs: 0 by shape (batches, and single sequences of middling length);
 *                         1 never; 2 whenever the shape allows it
 *   "fused_heads"         path 2: KV heads scored side by side in one phase (0: by size)
 *   "fused_lead"          path 2: phases the first read may lead the second (0: by size)
 *   "wait_limit_cycles"   clock cycles a device-side wait of the scoring kernels polls before it
 *                         gives up and raises FASTKV_ERR_DEVICE_TIMEOUT (0: about a second)
 *   "extra_publications"  the scoring kernels' second pass waits for this many publications of
 *                         softmax statistics beyond those that will arrive; with a short wait limit
 *                         this makes a bounded wait run out without any fault (timeout test)
 *   "prefill_skip_commit" n > 0: the prefill attention's issuer withholds the signal that S of key tile
 *                         n - 1 is ready (first query tile of every CTA); with a short wait limit the
 *                         softmax warps' bounded wait runs out without any fault (timeout test); 0: off
 *   "time_kernels"        1: record a pair of CUDA events around every kernel the library launches
 *                         (this creates events, and an event between two kernels keeps the second
 *                         from starting under the first one's tail); read with
 *                         fastkv_debug_kernel_time
 * Unknown keys return FASTKV_ERR_INVALID_ARG.
 */
int fastkv_debug_set(const char* key, int64_t value);
/*
 * Sum of the device durations (HOST double, milliseconds) and number of launches recorded for one
 * kernel class since the last query (0 scoring kernel, 1 pooling kernel, 2 selection, 3 compaction,
 * 4 decode attention, 5 prefill attention, 6 window scores); waits for the recorded launches and forgets them.  *name receives a static
 * string.  Any of the three outputs may be NULL.  No counterpart in the paper (measurement aid).
 */
int fastkv_debug_kernel_time(int32_t kernel, double* total_ms, int64_t* launches, const char** name);

/* Text for a fastkv_status; static storage. */
const char* fastkv_status_string(int status);
/* Text of the last FASTKV_ERR_CUDA / argument failure on the calling thread; static storage. */
const char* fastkv_last_error(void);
/* Number of kernels the library has launched from this process (for launch accounting). */
int64_t fastkv_kernel_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* FASTKV_H_ */
