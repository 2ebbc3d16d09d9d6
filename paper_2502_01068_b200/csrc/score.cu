// Window-query saliency scoring (Eq. 1 and Eq. 2 of the paper; Sec. 4.2).
//
// Kernel 1 (score_logits_kernel): the only dense contraction of the path.  For one KV head and a
// run of 128-key tiles, logits S^T = K_tile . Q_g^T are formed on the tcgen05 tensor cores: the
// A operand is the K tile (128 keys x head_dim, bf16, staged by TMA with the 128-byte swizzle),
// the B operand the G*w window-query rows of the head's GQA group, the fp32 accumulator lives in
// tensor memory with one key per lane and one query row per column.  Epilogue warps read the
// accumulator, scale it into log2 units, apply the causal mask of the window, store the logits
// and keep a running (max, sum of exponentials) per query row.  The last CTA of each
// (sequence, head) merges the per-CTA statistics into the softmax normaliser of every row.
//
// Kernel 2 (score_pool_kernel): p = exp2(s - M_r) / l_r, summed over the window rows of each
// query head (Eq. 1, inner sum), aggregated over the GQA group (App. B.1) and pooled along the
// sequence (Eq. 1, Pooling), plus the sum over all heads used at the TSP layer (Eq. 2).
#include "score.cuh"

namespace fastkv {

namespace {

constexpr int kTileKeys = 128;
constexpr int kHalfBytes = kTileKeys * 128;   // one 64-column half of a K tile: 128 rows x 128 B
constexpr int kEpilogueWarps = 4;
constexpr int kScoreThreads = 32 * (2 + kEpilogueWarps);

template <int D, int NPAD>
struct ScoreCfg {
  static constexpr int KH = D / 64;
  static constexpr int kStageBytes = KH * kHalfBytes;
  static constexpr int kQBytes = KH * NPAD * 128;
  static constexpr int kStages = (D == 128) ? 3 : 4;
  static constexpr int kAcc = (NPAD == 32) ? 4 : 2;
  static constexpr int kTmemCols = kAcc * NPAD;          // 128: a power of two >= 32
  static constexpr int kBarBytes = 256;
  static constexpr int kSmemBytes = 1024 /*alignment slack*/ + kStages * kStageBytes + kQBytes +
                                    kBarBytes + kEpilogueWarps * NPAD * 8;
};

struct ScoreBarriers {
  uint64_t full[6];
  uint64_t empty[6];
  uint64_t acc_full[4];
  uint64_t acc_empty[4];
  uint64_t q_full;
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(ScoreBarriers) <= 256, "barrier block");

}  // namespace

template <int D, int NPAD>
__global__ void __launch_bounds__(kScoreThreads, 2)
score_logits_kernel(const __grid_constant__ CUtensorMap tmap_k,
                    const __grid_constant__ CUtensorMap tmap_q, const ScoreParams p) {
  using Cfg = ScoreCfg<D, NPAD>;
  const int g = blockIdx.x, range = blockIdx.y, b = blockIdx.z;
  const int row0 = p.cu_seqlens ? p.cu_seqlens[b] : 0;
  const int L = p.cu_seqlens ? p.cu_seqlens[b + 1] - row0 : p.total_len;
  if (L < p.window) {   // nothing defined for this sequence; fastkv_score documents the rule
    if (threadIdx.x == 0 && range == 0 && g == 0)
      raise_status(p.hdr, FASTKV_ERR_INVALID_ARG, SITE_SCORE_SHORT_SEQUENCE);
    return;
  }
  const int ntiles = (L + kTileKeys - 1) / kTileKeys;
  const int t_begin = range * p.tiles_per_cta;
  if (t_begin >= ntiles) return;
  const int t_end = min(ntiles, t_begin + p.tiles_per_cta);
  const int nranges = (ntiles + p.tiles_per_cta - 1) / p.tiles_per_cta;
  const int n_my_tiles = t_end - t_begin;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* smem_k = smem;                                        // kStages x kStageBytes
  uint8_t* smem_q = smem + Cfg::kStages * Cfg::kStageBytes;      // kQBytes (1024-aligned)
  ScoreBarriers* bars = reinterpret_cast<ScoreBarriers*>(smem_q + Cfg::kQBytes);
  float2* warp_stats = reinterpret_cast<float2*>(reinterpret_cast<uint8_t*>(bars) + Cfg::kBarBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::kStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
    for (int a = 0; a < Cfg::kAcc; ++a) {
      mbar_init(&bars->acc_full[a], 1);
      mbar_init(&bars->acc_empty[a], kEpilogueWarps);
    }
    mbar_init(&bars->q_full, 1);
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tma_prefetch_desc(&tmap_k);
    tma_prefetch_desc(&tmap_q);
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, Cfg::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;
  volatile int* abort_flag = &bars->abort_flag;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      const uint64_t pol_stream = l2_policy_evict_first();
      const uint64_t pol_keep = l2_policy_evict_last();
      const int q_row0 = (p.q_layout == FASTKV_Q_WINDOW) ? b * p.window : row0 + L - p.window;
      mbar_arrive_expect_tx(&bars->q_full, Cfg::KH * p.n_rows * 128);
      for (int h = 0; h < Cfg::KH; ++h)
        tma_load_3d(smem_q + h * NPAD * 128, &tmap_q, &bars->q_full, h * 64, g * p.group, q_row0,
                    pol_keep);
      for (int it = 0; it < n_my_tiles; ++it) {
        const int s = it % Cfg::kStages;
        const uint32_t ph = (it / Cfg::kStages) & 1;
        if (!mbar_wait_bounded(&bars->empty[s], ph ^ 1, abort_flag, p.hdr, SITE_SCORE_TMA_EMPTY)) break;
        mbar_arrive_expect_tx(&bars->full[s], Cfg::kStageBytes);
        for (int h = 0; h < Cfg::KH; ++h)
          tma_load_3d(smem_k + s * Cfg::kStageBytes + h * kHalfBytes, &tmap_k, &bars->full[s],
                      h * 64, g, row0 + (t_begin + it) * kTileKeys, pol_stream);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16_f32(kTileKeys, NPAD);
      bool ok = mbar_wait_bounded(&bars->q_full, 0, abort_flag, p.hdr, SITE_SCORE_MMA_QFULL);
      const uint32_t q_addr = smem_u32(smem_q);
      for (int it = 0; ok && it < n_my_tiles; ++it) {
        const int s = it % Cfg::kStages, a = it % Cfg::kAcc;
        const uint32_t ph = (it / Cfg::kStages) & 1, aph = (it / Cfg::kAcc) & 1;
        ok = mbar_wait_bounded(&bars->acc_empty[a], aph ^ 1, abort_flag, p.hdr, SITE_SCORE_MMA_ACC_EMPTY) &&
             mbar_wait_bounded(&bars->full[s], ph, abort_flag, p.hdr, SITE_SCORE_MMA_FULL);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t k_addr = smem_u32(smem_k + s * Cfg::kStageBytes);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint64_t adesc = umma_desc_k_sw128(k_addr + (kk >> 2) * kHalfBytes + (kk & 3) * 32);
          const uint64_t bdesc = umma_desc_k_sw128(q_addr + (kk >> 2) * NPAD * 128 + (kk & 3) * 32);
          tc_mma_bf16(tmem_base + a * NPAD, adesc, bdesc, idesc, kk > 0 ? 1u : 0u);
        }
        tc_commit(&bars->empty[s]);      // the stage may be refilled once these MMAs have read it
        tc_commit(&bars->acc_full[a]);   // the accumulator is complete
      }
    }
  } else {
    // ---------------- epilogue: logits, causal mask, running row statistics ----------------
    const int quarter = warp & 3;                   // TMEM lanes this warp may read
    const int key_in_tile = quarter * 32 + lane;
    float m[NPAD], l[NPAD];
#pragma unroll
    for (int n = 0; n < NPAD; ++n) { m[n] = -INFINITY; l[n] = 0.0f; }
    const int n_rows = p.n_rows, G = p.group;
    const int win_start = L - p.window;
    float* const lg = p.logits + static_cast<size_t>(g) * NPAD * p.ld_logits + row0;
    bool ok = true;
    for (int it = 0; ok && it < n_my_tiles; ++it) {
      const int a = it % Cfg::kAcc;
      const uint32_t aph = (it / Cfg::kAcc) & 1;
      ok = mbar_wait_bounded(&bars->acc_full[a], aph, abort_flag, p.hdr, SITE_SCORE_EPI_ACC_FULL);
      ok = __all_sync(0xffffffffu, ok);   // the tensor-memory loads below need the whole warp
      if (!ok) break;
      tc_fence_after_sync();
      const int key = (t_begin + it) * kTileKeys + key_in_tile;
      const bool tile_unmasked = (t_begin + it + 1) * kTileKeys <= win_start;
#pragma unroll
      for (int c = 0; c < NPAD / 32; ++c) {
        float acc[32];
        tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + a * NPAD + c * 32, acc);
        if (c == NPAD / 32 - 1) {      // all columns of this accumulator are in registers
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars->acc_empty[a]);
        }
        const int n_valid = n_rows - c * 32;
        float* const lg_c = lg + static_cast<size_t>(c * 32) * p.ld_logits + key;
        if (tile_unmasked) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (i < n_valid) lg_c[static_cast<size_t>(i) * p.ld_logits] = acc[i] * p.scale_log2;
          stats_update_unmasked<32>(acc, m + c * 32, l + c * 32, p.scale_log2, n_valid);
        } else if (key < L) {
          uint32_t visible = 0;                          // causal: key i <= t_j, j = n / G
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (i < n_valid && key <= win_start + (c * 32 + i) / G) visible |= 1u << i;
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (i < n_valid)
              lg_c[static_cast<size_t>(i) * p.ld_logits] = ((visible >> i) & 1u) ? acc[i] * p.scale_log2 : -INFINITY;
          stats_update_masked<32>(acc, m + c * 32, l + c * 32, p.scale_log2, n_valid, visible);
        } else {
          stats_update_masked<32>(acc, m + c * 32, l + c * 32, p.scale_log2, n_valid, 0u);   // warp-uniform call
        }
      }
    }
    // merge the 32 lanes of this warp: lane r ends up with row r (and r + 32) of the warp's stats
#pragma unroll
    for (int c = 0; c < NPAD / 32; ++c) {
      stats_transpose_merge<32>(m + c * 32, l + c * 32, lane);
      warp_stats[quarter * NPAD + c * 32 + lane] = make_float2(m[c * 32], l[c * 32]);
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }

  // per-CTA statistics -> global; the last CTA of this (sequence, head) builds the normaliser
  float2* const part = p.partial + (static_cast<size_t>(b) * p.n_kv_heads + g) * p.max_ranges * NPAD;
  if (threadIdx.x < NPAD) {
    const int n = threadIdx.x;
    float mm = -INFINITY;
    for (int q = 0; q < kEpilogueWarps; ++q) mm = fmaxf(mm, warp_stats[q * NPAD + n].x);
    float ll = 0.0f;
    for (int q = 0; q < kEpilogueWarps; ++q) {
      const float2 s = warp_stats[q * NPAD + n];
      if (s.x != -INFINITY) ll += s.y * ex2(s.x - mm);
    }
    part[static_cast<size_t>(range) * NPAD + n] = make_float2(mm, ll);
    __threadfence();
  }
  __shared__ int is_last;
  __syncthreads();
  if (threadIdx.x == 0) {
    const int done = atomicAdd(&p.counters[b * p.n_kv_heads + g], 1);
    is_last = (done == nranges - 1);
  }
  __syncthreads();
  if (is_last) {
    // 128 threads: row n = t % NPAD, CTAs r = t / NPAD, + 128 / NPAD, ...; the partitions are then
    // combined in a fixed order, so the result does not depend on which CTA came last
    __shared__ float2 merge_buf[128];
    constexpr int kParts = 128 / NPAD;
    const int t = threadIdx.x;
    if (t < 128) {
      __threadfence();
      merge_buf[t] = merge_partials(part, NPAD, t % NPAD, t / NPAD, kParts, nranges);
    }
    __syncthreads();
    if (t < NPAD) {
      float mm = -INFINITY, ll = 0.0f;
#pragma unroll
      for (int q = 0; q < kParts; ++q) merge_stats(mm, ll, merge_buf[q * NPAD + t].x, merge_buf[q * NPAD + t].y);
      float2 out = make_float2(0.0f, 0.0f);
      if (t < p.n_rows && ll > 0.0f && *abort_flag == 0) out = make_float2(mm, 1.0f / ll);
      p.final_stats[(static_cast<size_t>(b) * p.n_kv_heads + g) * NPAD + t] = out;
      if (t == 0) p.counters[b * p.n_kv_heads + g] = 0;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Kernel 2: normalise, window/group sums, pooling, TSP sum.
// One CTA produces kPoolKeys consecutive positions of one sequence for all KV heads; it first
// fills shared memory with the un-pooled scores of those positions plus a halo of p/2 on each
// side (rows = KV heads for GROUP_THEN_POOL, query heads for POOL_THEN_GROUP), then pools.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kPoolThreads)
score_pool_kernel(const PoolParams p) {
  extern __shared__ float sm[];
  const int b = blockIdx.y;
  const int row0 = p.cu_seqlens ? p.cu_seqlens[b] : 0;
  const int L = p.cu_seqlens ? p.cu_seqlens[b + 1] - row0 : p.total_len;
  const int k0 = blockIdx.x * kPoolKeys;
  if (k0 >= L || L < p.window) return;
  const int r = p.pool_kernel >> 1;
  const int span = kPoolKeys + 2 * r;                 // positions k0-r .. k0+kPoolKeys+r-1
  const int Hkv = p.n_kv_heads, G = p.group, w = p.window, npad = p.npad;
  const bool per_head = p.agg_order == FASTKV_POOL_THEN_GROUP;
  const int rows = per_head ? Hkv * G : Hkv;
  float* stat_m = sm;                                 // [Hkv * npad]
  float* stat_il = sm + Hkv * npad;                   // [Hkv * npad]
  float* un = sm + 2 * Hkv * npad;                    // [rows][span]
  for (int i = threadIdx.x; i < Hkv * npad; i += blockDim.x) {
    const float2 s = p.final_stats[static_cast<size_t>(b) * Hkv * npad + i];
    stat_m[i] = s.x;
    stat_il[i] = s.y;
  }
  __syncthreads();
  for (int item = threadIdx.x; item < Hkv * span; item += blockDim.x) {
    const int g = item / span, o = item - g * span;
    const int key = k0 - r + o;
    float acc_g = 0.0f;
    const bool inside = key >= 0 && key < L;
    const float* lg = p.logits + static_cast<size_t>(g) * npad * p.ld_logits + row0 + key;
    for (int hl = 0; hl < G; ++hl) {
      float acc_h = 0.0f;
      if (inside) {
        for (int j = 0; j < w; ++j) {                 // Eq. 1: sum over the window rows
          const int n = j * G + hl;
          const float x = __ldcs(lg + static_cast<size_t>(n) * p.ld_logits);
          acc_h += ex2(x - stat_m[g * npad + n]) * stat_il[g * npad + n];
        }
      }
      if (per_head) un[(g * G + hl) * span + o] = acc_h; else acc_g += acc_h;
    }
    if (!per_head) un[g * span + o] = acc_g;
  }
  __syncthreads();
  const float inv_p = 1.0f / static_cast<float>(p.pool_kernel);
  for (int o = threadIdx.x; o < kPoolKeys; o += blockDim.x) {
    const int key = k0 + o;
    if (key >= L) break;
    float tsp = 0.0f;
    for (int g = 0; g < Hkv; ++g) {
      float s_g = 0.0f;
      const int sub = per_head ? G : 1;
      for (int hl = 0; hl < sub; ++hl) {
        const float* x = un + (g * sub + hl) * span + o;   // x[0..2r] = positions key-r .. key+r
        float v;
        if (p.pool_mode == FASTKV_POOL_AVG) {
          v = 0.0f;
          for (int t = 0; t <= 2 * r; ++t) v += x[t];      // out-of-range entries hold 0
          v *= inv_p;
        } else {
          v = 0.0f;                                         // scores are >= 0: 0 = "no entry"
          for (int t = 0; t <= 2 * r; ++t) v = fmaxf(v, x[t]);
        }
        s_g += v;
      }
      p.scores_kv[static_cast<size_t>(g) * p.ld_scores + row0 + key] = s_g;
      tsp += s_g;
    }
    if (p.scores_tsp) p.scores_tsp[row0 + key] = tsp;
  }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
template <int D, int NPAD>
static cudaError_t launch_logits_t(const CUtensorMap& tk, const CUtensorMap& tq, const ScoreParams& p,
                                   dim3 grid, cudaStream_t stream) {
  using Cfg = ScoreCfg<D, NPAD>;
  static PerDeviceOnce configured;   // per device; idempotent attribute, a race only repeats the call
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (!configured.done(dev)) {
    e = cudaFuncSetAttribute(score_logits_kernel<D, NPAD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Cfg::kSmemBytes);
    if (e != cudaSuccess) return e;
    configured.set(dev);
  }
  score_logits_kernel<D, NPAD><<<grid, kScoreThreads, Cfg::kSmemBytes, stream>>>(tk, tq, p);
  return cudaGetLastError();
}

cudaError_t launch_score_logits(int head_dim, int npad, const CUtensorMap& tk, const CUtensorMap& tq,
                                const ScoreParams& p, dim3 grid, cudaStream_t stream) {
  if (head_dim == 128 && npad == 32) return launch_logits_t<128, 32>(tk, tq, p, grid, stream);
  if (head_dim == 128 && npad == 64) return launch_logits_t<128, 64>(tk, tq, p, grid, stream);
  if (head_dim == 64 && npad == 32) return launch_logits_t<64, 32>(tk, tq, p, grid, stream);
  if (head_dim == 64 && npad == 64) return launch_logits_t<64, 64>(tk, tq, p, grid, stream);
  return cudaErrorInvalidValue;
}

size_t score_pool_smem_bytes(const PoolParams& p) {
  const int rows = p.agg_order == FASTKV_POOL_THEN_GROUP ? p.n_kv_heads * p.group : p.n_kv_heads;
  return sizeof(float) * (2 * static_cast<size_t>(p.n_kv_heads) * p.npad +
                          static_cast<size_t>(rows) * (kPoolKeys + 2 * (p.pool_kernel >> 1)));
}

cudaError_t launch_score_pool(const PoolParams& p, int max_len, int batch, cudaStream_t stream) {
  const size_t smem = score_pool_smem_bytes(p);
  if (smem > 48 * 1024) {          // rare (many heads, wide pooling window): opt in on every such launch
    cudaError_t e = cudaFuncSetAttribute(score_pool_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem));
    if (e != cudaSuccess) return e;
  }
  dim3 grid((max_len + kPoolKeys - 1) / kPoolKeys, batch);
  score_pool_kernel<<<grid, kPoolThreads, smem, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace fastkv
