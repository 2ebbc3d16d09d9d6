// Parameter blocks and launchers of the prefill attention with the saliency by-product (see prefill_attn.cu).
#pragma once

#include "common.cuh"

namespace fastkv {

struct PrefillParams {
  int batch, total_len, n_q_heads, group, window;
  float scale_log2;           // softmax scale times log2(e)
  const int* cu_seqlens;      // device, may be null (single sequence)
  void* out;                  // bf16 [total_len][n_q_heads][head_dim] with the strides below (elements)
  long long out_stride_tok, out_stride_head;
  float* wlog;                // [n_q_heads][window][ld_w]: scaled logits (log2 units) of the window rows, or null
  long long ld_w;
  float2* wstat;              // [batch][n_q_heads][window]: (reference, sum of exp2(s - reference)) of the window rows
  WorkspaceHeader* hdr;
  long long wait_limit;
  int skip_commit_tile;       // test hook: the first query tile's issuer does not signal that S of this key tile is ready (-1: none)
};

struct WindowScoresParams {
  int total_len, n_q_heads, n_kv_heads, group, window, per_head;
  const int* cu_seqlens;
  const float* wlog;
  long long ld_w;
  const float2* wstat;
  float* a_out;               // [n_kv_heads or n_q_heads][ld_a] un-pooled scores (what the pooling kernel reads)
  long long ld_a;
};

cudaError_t launch_prefill_attn(int head_dim, const CUtensorMap& tmap_q, const CUtensorMap& tmap_k, const CUtensorMap& tmap_v,
                                const PrefillParams& p, int max_len, cudaStream_t stream);
cudaError_t launch_window_scores(const WindowScoresParams& p, int max_len, int batch, cudaStream_t stream);

}  // namespace fastkv
