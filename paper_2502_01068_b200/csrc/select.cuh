// Parameter block and launcher of the top-k selection kernel (see select.cu).
#pragma once

#include "common.cuh"

namespace fastkv {

struct SelectParams {
  const float* scores;        // [rows][ld_scores]
  long long ld_scores;
  int* idx;                   // [rows][ld_idx], sequence-local positions, ascending per segment
  long long ld_idx;
  const int* cu_seqlens;      // device, may be null
  const int* cu_k;            // device output offsets, may be null (then k_uniform)
  int k_uniform;
  int total_len;
  int window;
  int force_window;
  WorkspaceHeader* hdr;
};

cudaError_t launch_select(const SelectParams& p, int n_rows, int batch, int max_len, cudaStream_t stream);

}  // namespace fastkv
