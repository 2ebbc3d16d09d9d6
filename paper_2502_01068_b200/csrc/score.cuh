// Parameter blocks and launchers of the scoring kernels (see score.cu).
#pragma once

#include "common.cuh"

namespace fastkv {

constexpr int kPoolKeys = 256;      // positions produced by one CTA of the pooling kernel
constexpr int kPoolThreads = 256;

struct ScoreParams {
  int batch, total_len, n_kv_heads, group, window;
  int n_rows;                 // G * w query rows per KV head (columns of the accumulator)
  int q_layout;
  int tiles_per_cta;          // 128-key tiles handled by one CTA
  int max_ranges;             // CTAs per (sequence, head) the partial-statistics array is sized for
  float scale_log2;           // softmax scale times log2(e): logits are kept in log2 units
  const int* cu_seqlens;      // device, may be null (single sequence)
  float* logits;              // [Hkv][NPAD][ld_logits], masked entries hold -inf
  long long ld_logits;
  float2* partial;            // [B][Hkv][max_ranges][NPAD] per-CTA (max, sum of exp2)
  float2* final_stats;        // [B][Hkv][NPAD] (row max, 1 / row sum)
  int* counters;              // [B][Hkv] CTAs finished; zero before and after the kernel
  WorkspaceHeader* hdr;
};

struct PoolParams {
  int total_len, n_kv_heads, group, window, npad;
  int pool_kernel, pool_mode, agg_order;
  const int* cu_seqlens;
  const float* logits;
  long long ld_logits;
  const float2* final_stats;
  float* scores_kv;           // [Hkv][ld_scores]
  long long ld_scores;
  float* scores_tsp;          // [total_len] or null
};

// scoring with one HBM pass over K (score_fused.cu): nothing but the per-key sums is written to memory
struct FusedParams {
  int batch, total_len, n_kv_heads, group, window;
  int n_rows;                 // G * w
  int q_layout;
  int per_head;               // 1: write one un-pooled row per query head (POOL_THEN_GROUP)
  float scale_log2;
  const int* cu_seqlens;
  int max_lead;               // phases the HBM pipeline may run ahead of the re-read pipeline
  int heads_per_phase;        // > 0: KV heads of a sequence processed side by side in one phase (forced);
                              // 0: chosen per sequence so that a phase holds about phase_bytes of K
  long long phase_bytes;      // target size of a phase
  long long head_bytes;       // bytes of one key row of one head (head_dim * 2)
  float* a_out;               // [Hkv or Hq][ld_a] un-pooled scores
  long long ld_a;
  float2* partial;            // [phases][CTAs][NPAD]
  int* counters;              // [phases] CTAs that published their statistics (zero before launch)
  WorkspaceHeader* hdr;
  int max_len;                // longest sequence of the batch (host knowledge)
  long long wait_limit;       // cycles a device-side wait may poll before it gives up
  int extra_publications;     // test hook: pass 2 waits for this many publications that never come
  int partition;              // parked kernel: 0 the grid walks the phases together; 1 CTAs dealt out to the sequences
                              // of a batch; 2 to the (sequence, head) pairs (see score_parked.cu)
};

struct PoolRowsParams {
  int total_len, n_kv_heads, group, window, per_head;
  int pool_kernel, pool_mode;
  const int* cu_seqlens;
  const float* a;             // [Hkv or Hq][ld_a] un-pooled scores
  long long ld_a;
  float* scores_kv;
  long long ld_scores;
  float* scores_tsp;
};

cudaError_t launch_score_fused(int head_dim, int npad, const CUtensorMap& tmap_k, const CUtensorMap& tmap_q,
                               const FusedParams& p, int grid, cudaStream_t stream);
// one pass over K, one contraction per tile, logits parked in tensor memory (score_parked.cu)
cudaError_t launch_score_parked(int head_dim, int npad, const CUtensorMap& tmap_k, const CUtensorMap& tmap_q,
                                const FusedParams& p, int grid, cudaStream_t stream);
int parked_slots(int npad);   // tiles of one phase a CTA can park: its tiles per phase must not exceed this
// zeroes `bytes` (a multiple of 4) at `ptr` with a kernel that takes part in the chain of programmatic launches
cudaError_t launch_clear_words(void* ptr, size_t bytes, cudaStream_t stream);
cudaError_t launch_pool_rows(const PoolRowsParams& p, int max_len, int batch, cudaStream_t stream);

cudaError_t launch_score_logits(int head_dim, int npad, const CUtensorMap& tmap_k,
                                const CUtensorMap& tmap_q, const ScoreParams& p, dim3 grid,
                                cudaStream_t stream);
size_t score_pool_smem_bytes(const PoolParams& p);
cudaError_t launch_score_pool(const PoolParams& p, int max_len, int batch, cudaStream_t stream);

}  // namespace fastkv
