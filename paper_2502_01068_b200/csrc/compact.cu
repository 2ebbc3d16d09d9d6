// Compaction of the kept K/V rows, hidden states and position ids (Alg. 1: C <- update(K, V);
// the reduced hidden states x).  Pure byte movement: every row is copied with 16-byte vector
// loads and stores, several independent loads in flight per thread before the first store.
#include "compact.cuh"

namespace fastkv {

namespace {

constexpr int kGatherThreads = 256;
constexpr int kGatherWarps = kGatherThreads / 32;
constexpr int kUnroll = 4;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
               "r"(v.w)
               : "memory");
}

// sequence that owns output slot j: the last b with cu_k[b] <= j
__device__ __forceinline__ int owner_of_slot(const int* cu_k, int k_uniform, int batch, int j) {
  if (batch == 1) return 0;
  if (cu_k == nullptr) return j / k_uniform;
  int lo = 0, hi = batch;            // invariant: cu_k[lo] <= j < cu_k[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (cu_k[mid] <= j) lo = mid; else hi = mid;
  }
  return lo;
}

}  // namespace

__global__ void __launch_bounds__(kGatherThreads) compact_rows_kernel(const CompactParams p) {
  pdl_wait();                  // the indices come from the kernel before this one
  pdl_launch_dependents();
  int ji = 0;
  while (ji + 1 < p.n_jobs && static_cast<int>(blockIdx.x) >= p.job[ji + 1].first_block) ++ji;
  const GatherJob& job = p.job[ji];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunks = job.row_chunks;
  const long long total_rows = static_cast<long long>(job.heads) * job.rows;
  // a warp copies `rows_per_step` rows at a time: narrow rows share a warp, wide rows loop
  const int lanes_per_row = chunks >= 32 ? 32 : (chunks > 16 ? 32 : (chunks > 8 ? 16 : (chunks > 4 ? 8 : 4)));
  const int rows_per_step = 32 / lanes_per_row;
  const int sub = lane / lanes_per_row, lane_in_row = lane % lanes_per_row;
  const long long warp_global = static_cast<long long>(blockIdx.x - job.first_block) * kGatherWarps + warp;
  const long long warp_count = static_cast<long long>(job.n_blocks) * kGatherWarps;

  for (long long r0 = warp_global * rows_per_step; r0 < total_rows; r0 += warp_count * rows_per_step) {
    const long long r = r0 + sub;
    if (r >= total_rows) continue;
    const int head = static_cast<int>(r / job.rows);
    const int j = static_cast<int>(r - static_cast<long long>(head) * job.rows);
    const int b = owner_of_slot(job.cu_k, job.k_uniform, p.batch, j);
    const int row0 = p.cu_seqlens ? p.cu_seqlens[b] : 0;
    const int L = p.cu_seqlens ? p.cu_seqlens[b + 1] - row0 : p.total_len;
    const int i = job.idx[static_cast<long long>(head) * job.ld_idx + j];
    if (i < 0 || i >= L) {           // never read outside the sequence: skip the row and report it
      if (lane_in_row == 0) raise_status(p.hdr, FASTKV_ERR_DEVICE_INDEX, SITE_COMPACT_INDEX);
      continue;
    }
    const long long tok = static_cast<long long>(row0) + i;
    const uint4* src = reinterpret_cast<const uint4*>(job.src + tok * job.src_tok_bytes +
                                                      head * job.src_head_bytes);
    uint4* dst = reinterpret_cast<uint4*>(job.dst) + r * chunks;
    if (job.src != nullptr) {
      for (int c0 = lane_in_row; c0 < chunks; c0 += lanes_per_row * kUnroll) {
        uint4 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
          if (c0 + u * lanes_per_row < chunks) v[u] = ld_stream(src + c0 + u * lanes_per_row);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
          if (c0 + u * lanes_per_row < chunks) st_stream(dst + c0 + u * lanes_per_row, v[u]);
      }
    }
    if (job.pos_src != nullptr && head == 0 && lane_in_row == 0) job.pos_dst[j] = job.pos_src[tok];
  }
}

cudaError_t launch_compact(CompactParams& p, cudaStream_t stream) {
  // blocks are shared out among the jobs in proportion to the bytes they move
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) sms = v;
  }
  const int budget = sms * 8;
  double bytes[3] = {0, 0, 0}, total = 0;
  for (int i = 0; i < p.n_jobs; ++i) {
    bytes[i] = static_cast<double>(p.job[i].heads) * p.job[i].rows * (p.job[i].row_chunks * 16.0 + 4.0);
    total += bytes[i];
  }
  if (total <= 0) return cudaSuccess;
  int first = 0;
  for (int i = 0; i < p.n_jobs; ++i) {
    const GatherJob& j = p.job[i];
    const int lanes_per_row = j.row_chunks >= 32 ? 32 : (j.row_chunks > 16 ? 32 : (j.row_chunks > 8 ? 16 : (j.row_chunks > 4 ? 8 : 4)));
    const long long steps = (static_cast<long long>(j.heads) * j.rows * lanes_per_row + 31) / 32;
    long long want = static_cast<long long>(budget * (bytes[i] / total) + 0.999);
    const long long cap = (steps + kGatherWarps - 1) / kGatherWarps;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    p.job[i].first_block = first;
    p.job[i].n_blocks = static_cast<int>(want);
    first += static_cast<int>(want);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(first);
  cfg.blockDim = dim3(kGatherThreads);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  fill_pdl_attribute(&attr[0]);
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, compact_rows_kernel, static_cast<const CompactParams&>(p));
}

}  // namespace fastkv
