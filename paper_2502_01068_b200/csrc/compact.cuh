// Parameter block and launcher of the gather / compaction kernel (see compact.cu).
#pragma once

#include "common.cuh"

namespace fastkv {

// One gather job: dst[head][j][:] = src[(cu_seqlens[b] + idx[head][j]) * tok_stride + head * head_stride ...]
struct GatherJob {
  const uint8_t* src;
  uint8_t* dst;
  const int* idx;             // [heads][ld_idx]
  const int* cu_k;            // output offsets per sequence, may be null (then k_uniform)
  long long src_tok_bytes;    // byte stride between consecutive tokens of src
  long long src_head_bytes;   // byte stride between heads of src
  long long ld_idx;
  int heads;
  int rows;                   // kept positions summed over the batch (per head)
  int row_chunks;             // 16-byte chunks per row
  int k_uniform;
  const int* pos_src;         // optional int32 side channel gathered with head 0 rows
  int* pos_dst;
  int rows_per_chunk;         // rows copied per 8 KB chunk (short rows), or 1
  int pieces_per_row;         // chunks per row (rows longer than a chunk), or 1
  long long first_chunk;      // chunks [first_chunk, next job's first_chunk) belong to this job
};

struct CompactParams {
  GatherJob job[3];
  int n_jobs;
  long long total_chunks;
  int batch;
  int total_len;
  const int* cu_seqlens;
  WorkspaceHeader* hdr;
};

cudaError_t launch_compact(CompactParams& p, cudaStream_t stream);

}  // namespace fastkv
