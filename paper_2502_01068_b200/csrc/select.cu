// Top-k token selection (KVCompress / HiddenCompress, App. B.1; window rule of Sec. 4.2).
//
// One thread-block cluster per problem (one score row of one sequence).  The k-th largest
// candidate score is found exactly by a most-significant-digit-first radix search on the
// order-preserving integer image of the fp32 scores (4 passes of 8 bits); every CTA adds its
// digit histogram into every CTA's copy of the cluster's histogram with remote shared-memory
// atomics (nothing waits for them), so after the pass's cluster barrier the sum is local.  The kept positions are then
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

struct alignas(16) SelShared {
  int hist[kBins * 32];          // lane-private digit counters: hist[bin * 32 + lane]
  int total_hist[2][kBins];      // the cluster's histogram of a pass (every CTA adds into it), double-buffered by pass parity
  int warp_tot[2][kSelWarps];
  alignas(8) int counts[16][2];  // per CTA of the cluster: (#above threshold, #equal to threshold), written by that CTA
  int digit, k_rem;
};

}  // namespace

// Every thread owns `per` consecutive candidates of its CTA's chunk, so index order is thread order
// and the ordered compaction at the end needs no warp votes, only one scan of per-thread counts.
// ITEMS > 0: per = ITEMS and the candidates (converted once) stay in registers for all passes.
// ITEMS == 0: any chunk size; every pass re-reads the scores (they are L2 resident).
template <int CLUSTER, int ITEMS, int THREADS>
__global__ void __launch_bounds__(THREADS, 1) select_topk_kernel(const SelectParams p) {
  constexpr int kWarps = THREADS / 32;
  constexpr int kPerBin = THREADS / kBins;         // threads that share one bin in the histogram reduction
  static_assert(THREADS % kBins == 0 && kPerBin >= 1 && kPerBin <= 4, "256, 512 or 1024 threads");
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ SelShared sh;
  constexpr bool CACHED = ITEMS > 0;
  constexpr int R = CACHED ? ITEMS : 1;
  const int rank = static_cast<int>(cluster.block_rank());
  const bool second = static_cast<int>(blockIdx.y) >= p.set[0].n_rows;
  const SelectSet& ps = p.set[second ? 1 : 0];
  const int row = static_cast<int>(blockIdx.y) - (second ? p.set[0].n_rows : 0), b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  for (int i = tid; i < 2 * kBins; i += THREADS) (&sh.total_hist[0][0])[i] = 0;
  cluster.sync();              // nobody adds into a histogram that is not cleared yet (overlaps the previous kernel's tail)
  pdl_wait();                  // the scores come from the kernel before this one
  pdl_launch_dependents();
  const int row0 = p.cu_seqlens ? p.cu_seqlens[b] : 0;
  const int L = p.cu_seqlens ? p.cu_seqlens[b + 1] - row0 : p.total_len;
  const int out0 = ps.cu_k ? ps.cu_k[b] : b * ps.k_uniform;
  int k = ps.cu_k ? ps.cu_k[b + 1] - out0 : ps.k_uniform;
  const int w = p.force_window ? p.window : 0;
  const float* S = ps.scores + static_cast<size_t>(row) * ps.ld_scores + row0;
  int* out = ps.idx + static_cast<size_t>(row) * ps.ld_idx + out0;

  // budget outside [w, L]: clamp so that writes stay inside this sequence's output segment,
  // and report it (the whole cluster takes the same branch: k, L, w are uniform)
  if (L < w || k < w || k > L) {
    if (rank == 0 && tid == 0) raise_status(p.hdr, FASTKV_ERR_DEVICE_INDEX, SITE_SELECT_BUDGET);
    if (L < w || k < w) return;
    k = L;
  }
  const int n_cand = L - w;          // ranked positions: [0, n_cand)
  const int k_sel = k - w;           // how many of them are kept
  // contiguous chunk per CTA, `per` consecutive candidates per thread
  const int chunk = ((n_cand + CLUSTER - 1) / CLUSTER + 3) & ~3;   // multiple of 4: keeps 16-byte alignment
  const int c_begin = min(n_cand, rank * chunk), c_end = min(n_cand, c_begin + chunk);
  const int per = CACHED ? ITEMS : (chunk + THREADS - 1) / THREADS;
  const int t_begin = min(c_end, c_begin + tid * per), t_end = min(c_end, t_begin + per);
  const int n_mine = t_end - t_begin;

  uint32_t key[R];
  uint32_t live = 0;                 // bit r: candidate r exists and still matches the threshold's prefix
  if (CACHED) {
    const float* mine = S + t_begin;
    if (n_mine == R && R % 4 == 0 && (reinterpret_cast<uintptr_t>(mine) & 15u) == 0) {
#pragma unroll
      for (int r = 0; r < R; r += 4) {                 // 16-byte loads: a thread's candidates are contiguous
        const float4 v = __ldg(reinterpret_cast<const float4*>(mine + r));
        key[r] = order_key(v.x); key[r + 1] = order_key(v.y); key[r + 2] = order_key(v.z); key[r + 3] = order_key(v.w);
      }
    } else {
#pragma unroll
      for (int r = 0; r < R; ++r) key[r] = (r < n_mine) ? order_key(__ldg(mine + r)) : 0u;
    }
    live = n_mine >= 32 ? 0xffffffffu : ((1u << n_mine) - 1u);
  }

  uint32_t prefix = 0;
  int k_rem = k_sel;
  if (k_sel > 0) {
    for (int i = tid; i < kBins * 32; i += THREADS) sh.hist[i] = 0;
    __syncthreads();
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      if (CACHED) {
        if (live != 0) {               // after two passes almost nobody is left
#pragma unroll
          for (int r = 0; r < R; ++r)
            if ((live >> r) & 1u) atomicAdd(&sh.hist[((key[r] >> shift) & 0xFFu) * 32 + lane], 1);
        }
      } else {
        for (int i = t_begin; i < t_end; ++i) {
          const uint32_t u = order_key(__ldg(S + i));
          const bool match = (pass == 0) || ((u ^ prefix) >> (shift + 8)) == 0;
          if (match) atomicAdd(&sh.hist[((u >> shift) & 0xFFu) * 32 + lane], 1);
        }
      }
      __syncthreads();
      {
        // kPerBin threads per bin, each sums (and clears for the next pass) its share of the 32 lane counters
        const int bin = tid / kPerBin, part = tid % kPerBin;
        int sum = 0;
#pragma unroll
        for (int i = 0; i < 32 / kPerBin; ++i) {
          int* c = &sh.hist[bin * 32 + ((part * (32 / kPerBin) + i + bin) & 31)];
          sum += *c;
          *c = 0;
        }
        if (kPerBin >= 2) sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        if (kPerBin >= 4) sum += __shfl_xor_sync(0xffffffffu, sum, 2);
        if (part == 0 && sum != 0) {   // non-empty bins go to every CTA of the cluster
#pragma unroll
          for (int r = 0; r < CLUSTER; ++r) atomicAdd(cluster.map_shared_rank(&sh.total_hist[pass & 1][bin], r), sum);
        }
      }
      cluster.sync();
      if (warp == 0) {
        // 8 bins per lane, highest bins first: lane 0 owns bins 255..248
        int cnt[8], tot = 0;
        const int4 lo = *reinterpret_cast<const int4*>(&sh.total_hist[pass & 1][248 - lane * 8]);
        const int4 hi = *reinterpret_cast<const int4*>(&sh.total_hist[pass & 1][252 - lane * 8]);
        cnt[0] = hi.w; cnt[1] = hi.z; cnt[2] = hi.y; cnt[3] = hi.x;
        cnt[4] = lo.w; cnt[5] = lo.z; cnt[6] = lo.y; cnt[7] = lo.x;
#pragma unroll
        for (int i = 0; i < 8; ++i) tot += cnt[i];
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
      if (tid < kBins) sh.total_hist[pass & 1][tid] = 0;   // for the pass after next; nobody adds into it before the next barrier
      const uint32_t digit = static_cast<uint32_t>(sh.digit);
      prefix |= digit << shift;
      k_rem = sh.k_rem;
      if (CACHED && live != 0) {       // keep only the candidates that share the threshold's digit
        uint32_t still = 0;
#pragma unroll
        for (int r = 0; r < R; ++r) still |= (((key[r] >> shift) & 0xFFu) == digit ? 1u : 0u) << r;
        live &= still;
      }
    }
  }
  // prefix = image of the threshold score tau; k_rem = how many candidates equal to tau are kept
  const uint32_t tau = prefix;
  const int need_eq = (k_sel > 0) ? k_rem : 0;

  // this thread's candidates above / equal to tau
  int n_gt = 0, n_eq = 0;
  if (k_sel > 0) {
    if (CACHED) {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        n_gt += (r < n_mine && key[r] > tau) ? 1 : 0;
        n_eq += (r < n_mine && key[r] == tau) ? 1 : 0;
      }
    } else {
      for (int i = t_begin; i < t_end; ++i) {
        const uint32_t u = order_key(__ldg(S + i));
        n_gt += (u > tau) ? 1 : 0;
        n_eq += (u == tau) ? 1 : 0;
      }
    }
  }
  // exclusive scans in thread order: within the warp, then over the 32 warps
  int gt_incl = n_gt, eq_incl = n_eq;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int va = __shfl_up_sync(0xffffffffu, gt_incl, o), ve = __shfl_up_sync(0xffffffffu, eq_incl, o);
    if (lane >= o) { gt_incl += va; eq_incl += ve; }
  }
  if (lane == 31) { sh.warp_tot[0][warp] = gt_incl; sh.warp_tot[1][warp] = eq_incl; }
  __syncthreads();
  if (warp == 0) {
    int a = lane < kWarps ? sh.warp_tot[0][lane] : 0, e = lane < kWarps ? sh.warp_tot[1][lane] : 0;
    const int a0 = a, e0 = e;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int va = __shfl_up_sync(0xffffffffu, a, o), ve = __shfl_up_sync(0xffffffffu, e, o);
      if (lane >= o) { a += va; e += ve; }
    }
    sh.warp_tot[0][lane] = a - a0;
    sh.warp_tot[1][lane] = e - e0;
    // this CTA's totals go to every CTA of the cluster (remote stores; the barrier below makes them visible)
    const int a_tot = __shfl_sync(0xffffffffu, a, 31), e_tot = __shfl_sync(0xffffffffu, e, 31);
    if (lane < CLUSTER) *reinterpret_cast<int2*>(cluster.map_shared_rank(&sh.counts[rank][0], lane)) = make_int2(a_tot, e_tot);
  }
  __syncthreads();
  const int gt_excl = sh.warp_tot[0][warp] + gt_incl - n_gt, eq_excl = sh.warp_tot[1][warp] + eq_incl - n_eq;
  cluster.sync();
  // candidates kept by lower-ranked CTAs (they hold lower indices)
  int g_r[CLUSTER], e_r[CLUSTER];
#pragma unroll
  for (int r = 0; r < CLUSTER; ++r) {
    g_r[r] = sh.counts[r][0];
    e_r[r] = sh.counts[r][1];
  }
  int eq_before = 0, kept_before = 0;
#pragma unroll
  for (int r = 0; r < CLUSTER; ++r) {
    if (r < rank) {
      kept_before += g_r[r] + max(0, min(e_r[r], need_eq - eq_before));
      eq_before += e_r[r];
    }
  }
  if (k_sel > 0 && n_gt + n_eq > 0) {
    int eq_rank = eq_before + eq_excl;                       // rank of this thread's first tau-valued candidate
    int pos = kept_before + gt_excl + min(eq_rank, need_eq) - min(eq_before, need_eq);
    if (CACHED) {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (r < n_mine) {
          const uint32_t u = key[r];
          const bool is_eq = u == tau;
          if (u > tau || (is_eq && eq_rank < need_eq)) out[pos++] = t_begin + r;
          eq_rank += is_eq ? 1 : 0;
        }
      }
    } else {
      for (int i = t_begin; i < t_end; ++i) {
        const uint32_t u = order_key(__ldg(S + i));
        const bool is_eq = u == tau;
        if (u > tau || (is_eq && eq_rank < need_eq)) out[pos++] = i;
        eq_rank += is_eq ? 1 : 0;
      }
    }
  }
  if (rank == 0)
    for (int i = tid; i < w; i += THREADS) out[k_sel + i] = n_cand + i;   // the window, always kept
  // nobody touches another CTA's shared memory after the last barrier above: a CTA may end on its own
}

namespace {

template <int CLUSTER, int ITEMS, int THREADS>
cudaError_t launch_select_t(const SelectParams& p, int batch, cudaStream_t stream) {
  if (CLUSTER > 8) {
    static PerDeviceOnce configured;      // launch attributes are per device
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (!configured.done(dev)) {
      e = cudaFuncSetAttribute(select_topk_kernel<CLUSTER, ITEMS, THREADS>,
                               cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
      if (e != cudaSuccess) return e;
      configured.set(dev);
    }
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(CLUSTER, p.set[0].n_rows + p.set[1].n_rows, batch);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CLUSTER;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  fill_pdl_attribute(&attr[1]);
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, select_topk_kernel<CLUSTER, ITEMS, THREADS>, p);
}

}  // namespace

template <int CLUSTER, int THREADS>
static cudaError_t launch_select_c(const SelectParams& p, int batch, int max_len, cudaStream_t stream) {
  const long long per_cta = (static_cast<long long>(max_len) + CLUSTER - 1) / CLUSTER;
  if (per_cta <= 4 * THREADS) return launch_select_t<CLUSTER, 4, THREADS>(p, batch, stream);
  if (per_cta <= 8 * THREADS) return launch_select_t<CLUSTER, 8, THREADS>(p, batch, stream);
  if (per_cta <= 16 * THREADS) return launch_select_t<CLUSTER, 16, THREADS>(p, batch, stream);
  if (per_cta <= 32 * THREADS) return launch_select_t<CLUSTER, 32, THREADS>(p, batch, stream);
  return launch_select_t<CLUSTER, 0, THREADS>(p, batch, stream);
}

cudaError_t launch_select(const SelectParams& p, int batch, int max_len, cudaStream_t stream) {
  // Long sequences: 8-CTA clusters of 1024 threads, with which every problem of a layer (KV heads plus the
  // TSP row) is resident at once on a 148-SM part.  Short sequences are bound by the fixed cost of the CTA
  // and cluster barriers, so they use 256-thread CTAs (16 candidates per thread) in clusters as small as
  // the length allows.  The per-thread register cache is picked from the longest sequence.
  if (max_len <= 16 * 256) return launch_select_c<1, 256>(p, batch, max_len, stream);
  if (max_len <= 2 * 16 * 256) return launch_select_c<2, 256>(p, batch, max_len, stream);
  if (max_len <= 4 * 16 * 256) return launch_select_c<4, 256>(p, batch, max_len, stream);
  if (max_len <= 8 * 16 * 256) return launch_select_c<8, 256>(p, batch, max_len, stream);
  // Batches: every problem (a score row of a sequence) is a cluster; with many of them, smaller clusters keep the
  // whole launch in one wave of a 148-SM part (1024-thread CTAs: one per SM) as long as a CTA's share still fits
  // the register cache (32 candidates per thread): 72 problems x 8 CTAs take four waves, x 2 one.
  const int problems = (p.set[0].n_rows + p.set[1].n_rows) * batch;
  int cluster = 8;
  while (cluster > 1 && problems * cluster > 148 && (max_len + cluster / 2 - 1) / (cluster / 2) <= 32 * 1024) cluster /= 2;
  if (cluster == 4) return launch_select_c<4, 1024>(p, batch, max_len, stream);
  if (cluster == 2) return launch_select_c<2, 1024>(p, batch, max_len, stream);
  if (cluster == 1) return launch_select_c<1, 1024>(p, batch, max_len, stream);
  return launch_select_c<8, 1024>(p, batch, max_len, stream);
}

}  // namespace fastkv
