// Parameter block and launcher of the decode-time attention over the compact cache (see decode_attn.cu).
#pragma once

#include "common.cuh"

namespace fastkv {

constexpr int kDecodeMaxSplits = 64;

struct DecodeParams {
  const uint16_t* q;          // [B][Hq][d] bf16 bits: one new query token per sequence
  // the caches ([Hkv][ld_cache][d] bf16, sequence b at rows cu_k[b] .. or b * k_uniform ..) come as tensor maps
  long long ld_cache;         // kept entries summed over the batch (rows per head of the caches)
  const int* cu_k;            // device, may be null (then k_uniform)
  int k_uniform;
  int n_q_heads, n_kv_heads, group;
  float scale_log2;           // softmax scale times log2(e)
  float* out;                 // [B][Hq][d] fp32
  float* lse;                 // [B][Hq] natural-log sum of exponentials, may be null
  float2* part_ml;            // [B][Hkv][splits][G] per-split (max, sum) in log2 units
  float* part_o;              // [B][Hkv][splits][G][d] per-split unnormalised outputs
  WorkspaceHeader* hdr;
};

size_t decode_workspace_bytes(int batch, int n_kv_heads, int group, int head_dim);
// tmap_k / tmap_v: the caches as (column, head, row) tensors, boxes of 64 columns x 1 head x 16 rows, 128-byte swizzle
// *launches: kernels launched (1 when every (sequence, KV head) has a single split: no merge kernel then)
cudaError_t launch_decode_attn(const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, DecodeParams& p, int head_dim, int batch,
                               int k_max, cudaStream_t stream, int* launches);

}  // namespace fastkv
