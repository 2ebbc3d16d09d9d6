// Parameter block and launcher of the top-k selection kernel (see select.cu).
#pragma once

#include "common.cuh"

namespace fastkv {

// One set of score rows selected under one budget (the KV heads, or the single TSP row).
struct SelectSet {
  const float* scores;        // [rows][ld_scores]
  long long ld_scores;
  int* idx;                   // [rows][ld_idx], sequence-local positions, ascending per segment
  long long ld_idx;
  const int* cu_k;            // device output offsets, may be null (then k_uniform)
  int k_uniform;
  int n_rows;
};

struct SelectParams {
  SelectSet set[2];           // grid rows 0 .. set[0].n_rows-1 belong to set 0, the rest to set 1
  const int* cu_seqlens;      // device, may be null
  int total_len;
  int window;
  int force_window;
  WorkspaceHeader* hdr;
};

cudaError_t launch_select(const SelectParams& p, int batch, int max_len, cudaStream_t stream);

}  // namespace fastkv
