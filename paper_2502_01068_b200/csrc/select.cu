// Top-k token selection (KVCompress / HiddenCompress, App. B.1; window rule of Sec. 4.2).
//
// One thread-block cluster per problem (one score row of one sequence).  The k-th largest
// candidate score is found exactly by a most-significant-digit-first radix search on the
// order-preserving integer image of the fp32 scores (4 passes of 8 bits); per-CTA digit
// histograms are merged through distributed shared memory.  The kept positions are then
// written in ascending order by an index-ordered stream compaction: every candidate above
// the threshold, plus the lowest-index candidates equal to it until the budget is met --
// which is exactly "rank by (score descending, index ascending), keep the first k".  With
// force_window the last w positions are appended unranked.
#include <cooperative_groups.h>

#include "select.cuh"

namespace cg = cooperative_groups;

namespace fastkv {

namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kBins = 256;

// Monotone map fp32 -> uint32 (larger float <=> larger integer); -0 is folded onto +0 so that
// equal scores compare equal.
__device__ __forceinline__ uint32_t order_key(float x) {
  uint32_t u = __float_as_uint(x);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct SelShared {
  int hist[kBins * 32];          // lane-private digit counters: hist[bin * 32 + lane]
  int block_hist[2][kBins];      // this CTA's histogram, double-buffered by pass parity
  int warp_tot[2][kSelWarps];
  int counts[2];                 // this CTA's (#above threshold, #equal to threshold)
  int digit, k_rem;
};

}  // namespace

template <int CLUSTER>
__global__ void __launch_bounds__(kSelThreads, 1) select_topk_kernel(const SelectParams p) {
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ SelShared sh;
  const int rank = static_cast<int>(cluster.block_rank());
  const int row = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  const int row0 = p.cu_seqlens ? p.cu_seqlens[b] : 0;
  const int L = p.cu_seqlens ? p.cu_seqlens[b + 1] - row0 : p.total_len;
  const int out0 = p.cu_k ? p.cu_k[b] : b * p.k_uniform;
  int k = p.cu_k ? p.cu_k[b + 1] - out0 : p.k_uniform;
  const int w = p.force_window ? p.window : 0;
  const float* S = p.scores + static_cast<size_t>(row) * p.ld_scores + row0;
  int* out = p.idx + static_cast<size_t>(row) * p.ld_idx + out0;

  // budget outside [w, L]: clamp so that writes stay inside this sequence's output segment,
  // and report it (the whole cluster takes the same branch: k, L, w are uniform)
  if (L < w || k < w || k > L) {
    if (rank == 0 && tid == 0) raise_status(p.hdr, FASTKV_ERR_DEVICE_INDEX, SITE_SELECT_BUDGET);
    if (L < w || k < w) return;
    k = L;
  }
  const int n_cand = L - w;          // ranked positions: [0, n_cand)
  const int k_sel = k - w;           // how many of them are kept
  // contiguous chunk of this CTA, contiguous sub-chunk of this thread (index order = rank order)
  const int chunk = (n_cand + CLUSTER - 1) / CLUSTER;
  const int c_begin = min(n_cand, rank * chunk), c_end = min(n_cand, c_begin + chunk);
  const int per_thread = (chunk + kSelThreads - 1) / kSelThreads;
  const int t_begin = min(c_end, c_begin + tid * per_thread), t_end = min(c_end, t_begin + per_thread);

  uint32_t prefix = 0;
  int k_rem = k_sel;
  if (k_sel > 0) {
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      for (int i = tid; i < kBins * 32; i += kSelThreads) sh.hist[i] = 0;
      __syncthreads();
      for (int i = c_begin + tid; i < c_end; i += kSelThreads) {
        const uint32_t u = order_key(S[i]);
        const bool match = (pass == 0) || ((u ^ prefix) >> (shift + 8)) == 0;
        if (match) atomicAdd(&sh.hist[((u >> shift) & 0xFFu) * 32 + lane], 1);
      }
      __syncthreads();
      {
        // 4 threads per bin, each sums 8 lane counters
        const int bin = tid >> 2, part = tid & 3;
        int s = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) s += sh.hist[bin * 32 + ((part * 8 + i + bin) & 31)];
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        if (part == 0) sh.block_hist[pass & 1][bin] = s;
      }
      cluster.sync();
      if (warp == 0) {
        // cluster-wide histogram, 8 bins per lane, highest bins first: lane 0 owns bins 255..248
        int cnt[8], tot = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int bin = 255 - (lane * 8 + i);
          int c = 0;
          for (int r = 0; r < CLUSTER; ++r)
            c += cluster.map_shared_rank(&sh.block_hist[pass & 1][0], r)[bin];
          cnt[i] = c;
          tot += c;
        }
        int incl = tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += v;
        }
        int above = incl - tot;          // candidates in higher bins than this lane's
        if (above < k_rem && k_rem <= incl) {   // exactly one lane holds the k_rem-th largest
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            if (above < k_rem && k_rem <= above + cnt[i]) {
              sh.digit = 255 - (lane * 8 + i);
              sh.k_rem = k_rem - above;
            }
            above += cnt[i];
          }
        }
      }
      __syncthreads();
      prefix |= static_cast<uint32_t>(sh.digit) << shift;
      k_rem = sh.k_rem;
      __syncthreads();
    }
  }
  // prefix = image of the threshold score tau; k_rem = how many candidates equal to tau are kept
  const uint32_t tau = prefix;
  const int need_eq = (k_sel > 0) ? k_rem : 0;

  // per-thread counts over its contiguous sub-chunk
  int n_gt = 0, n_eq = 0;
  if (k_sel > 0) {
    for (int i = t_begin; i < t_end; ++i) {
      const uint32_t u = order_key(S[i]);
      n_gt += (u > tau);
      n_eq += (u == tau);
    }
  }
  // block-wide exclusive scans of both counts (packed: candidates per CTA < 2^31 / 2)
  int gt_excl, eq_excl, gt_block, eq_block;
  {
    int gi = n_gt, ei = n_eq;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int a = __shfl_up_sync(0xffffffffu, gi, o), e = __shfl_up_sync(0xffffffffu, ei, o);
      if (lane >= o) { gi += a; ei += e; }
    }
    if (lane == 31) { sh.warp_tot[0][warp] = gi; sh.warp_tot[1][warp] = ei; }
    __syncthreads();
    if (warp == 0) {
      int a = sh.warp_tot[0][lane], e = sh.warp_tot[1][lane];
      const int a0 = a, e0 = e;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int va = __shfl_up_sync(0xffffffffu, a, o), ve = __shfl_up_sync(0xffffffffu, e, o);
        if (lane >= o) { a += va; e += ve; }
      }
      sh.warp_tot[0][lane] = a - a0;
      sh.warp_tot[1][lane] = e - e0;
      if (lane == 31) { sh.counts[0] = a; sh.counts[1] = e; }
    }
    __syncthreads();
    gt_excl = sh.warp_tot[0][warp] + gi - n_gt;
    eq_excl = sh.warp_tot[1][warp] + ei - n_eq;
    gt_block = sh.counts[0];
    eq_block = sh.counts[1];
  }
  cluster.sync();
  // candidates kept by lower-ranked CTAs (they hold lower indices)
  int eq_before = 0, kept_before = 0;
  for (int r = 0; r < rank; ++r) {
    const int* c = cluster.map_shared_rank(&sh.counts[0], r);
    const int g_r = c[0], e_r = c[1];
    kept_before += g_r + max(0, min(e_r, need_eq - eq_before));
    eq_before += e_r;
  }
  (void)gt_block; (void)eq_block;
  if (k_sel > 0) {
    int eq_rank = eq_before + eq_excl;                       // rank of my first tau-valued candidate
    const int eq_kept_before_me = min(eq_rank, need_eq) - min(eq_before, need_eq);
    int pos = kept_before + gt_excl + eq_kept_before_me;
    for (int i = t_begin; i < t_end; ++i) {
      const uint32_t u = order_key(S[i]);
      bool keep = u > tau;
      if (u == tau) { keep = eq_rank < need_eq; ++eq_rank; }
      if (keep) out[pos++] = i;
    }
  }
  if (rank == 0 && tid < w) out[k_sel + tid] = n_cand + tid;   // the window, always kept
  cluster.sync();   // no CTA may exit while others still read its shared memory
}

cudaError_t launch_select(const SelectParams& p, int n_rows, int batch, cudaStream_t stream) {
  constexpr int kCluster = 8;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kCluster, n_rows, batch);
  cfg.blockDim = dim3(kSelThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kCluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, select_topk_kernel<kCluster>, p);
}

}  // namespace fastkv
