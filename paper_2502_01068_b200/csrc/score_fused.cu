// Window-query saliency scoring, single pass over K (Eq. 1 inner term; Sec. 4.2).
//
// One persistent CTA per SM (cooperative launch, so all CTAs are resident).  The work is cut into
// phases, one per (sequence, KV head); in a phase every CTA owns a run of consecutive 128-key
// tiles.  The logits of a CTA's tiles stay in tensor memory between the two things that need them:
//
//   pass 1  (warp group A) running (max, sum of exp2) per query row over the CTA's tiles; the
//           CTAs' statistics meet in global memory, counted by one counter per phase;
//   pass 2  (warp group B) once every CTA of the phase has published, merge the statistics into
//           the softmax normaliser (fixed order: identical in every CTA), then
//           p = exp2(s - M_r) / l_r summed over the window rows (and the GQA group) of each key,
//           read again from tensor memory -- K is streamed from HBM exactly once and no logit is
//           ever written to memory.
//
// Tensor memory (512 columns) is a ring of accumulator slots: the MMA warp fills a slot, group A
// reads it, group B reads it again and hands it back.  All tiles a CTA owns in one phase must be
// in the ring at once (up to 16 tiles of 32 query rows), and the next phase's MMAs start as soon
// as group B frees slots, so the TMA stream of K runs ahead of both passes.  Every wait (mbarrier
// or counter) is bounded and ends in a status word instead of a hang.
#include "score.cuh"

namespace fastkv {

namespace {

constexpr int kTileKeys = 128;
constexpr int kHalfBytes = kTileKeys * 128;
constexpr int kGroupWarps = 4;                 // warps per epilogue group (one per tensor-memory lane quarter)
constexpr int kFusedThreads = 32 * (2 + 2 * kGroupWarps);

template <int D, int NPAD>
struct FusedCfg {
  static constexpr int KH = D / 64;
  static constexpr int kStageBytes = KH * kHalfBytes;
  static constexpr int kQBytes = KH * NPAD * 128;
  static constexpr int kStages = (D == 128) ? (NPAD == 32 ? 6 : 5) : 8;
  static constexpr int kSlots = 512 / NPAD;              // accumulators in tensor memory (a ring)
  static constexpr int kTmemCols = 512;
  static constexpr int kBarBytes = 512;
  static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + 2 * kQBytes + kBarBytes +
                                    kGroupWarps * NPAD * 8 + NPAD * 8 + kGroupWarps * 32 * 8;
};

struct FusedBarriers {
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t q_full[2];
  uint64_t q_empty[2];
  uint64_t acc_full[16];
  uint64_t acc_free[16];
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(FusedBarriers) <= 512, "barrier block");

template <int ID>
__device__ __forceinline__ void group_sync() { asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(kGroupWarps * 32) : "memory"); }

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_add(int* p, int v) {
  asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

template <int GG>
__device__ __forceinline__ void add_heads(const float (&pr)[32], float (&a_h)[8]) {
#pragma unroll
  for (int x = 0; x < 32; ++x) a_h[x % GG] += pr[x];
}

// what one CTA does in one phase
struct PhaseWork {
  int b, g, row0, L, t0, n, nact;
};

__device__ __forceinline__ PhaseWork phase_work(const FusedParams& p, int phase, int cta, int ncta) {
  PhaseWork w;
  w.b = phase / p.n_kv_heads;
  w.g = phase - w.b * p.n_kv_heads;
  w.row0 = p.cu_seqlens ? p.cu_seqlens[w.b] : 0;
  w.L = p.cu_seqlens ? p.cu_seqlens[w.b + 1] - w.row0 : p.total_len;
  if (w.L < p.window) { w.t0 = 0; w.n = 0; w.nact = 0; return w; }
  const int ntiles = (w.L + kTileKeys - 1) / kTileKeys;
  int per = (ntiles + ncta - 1) / ncta;
  if (per > p.slots) per = p.slots;                 // host guarantees ntiles <= ncta * slots
  w.nact = (ntiles + per - 1) / per;
  w.t0 = cta * per;
  w.n = max(0, min(per, ntiles - w.t0));
  return w;
}

}  // namespace

template <int D, int NPAD>
__global__ void __launch_bounds__(kFusedThreads, 1)
score_fused_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_q,
                   const FusedParams p) {
  using Cfg = FusedCfg<D, NPAD>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* smem_k = smem;
  uint8_t* smem_q = smem + Cfg::kStages * Cfg::kStageBytes;           // two buffers of kQBytes
  FusedBarriers* bars = reinterpret_cast<FusedBarriers*>(smem_q + 2 * Cfg::kQBytes);
  float2* warp_stats = reinterpret_cast<float2*>(reinterpret_cast<uint8_t*>(bars) + Cfg::kBarBytes);
  float2* norm = warp_stats + kGroupWarps * NPAD;                     // [NPAD] (row max, 1 / row sum)
  float2* merge_buf = norm + NPAD;                                    // [128] partial merges

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, ncta = gridDim.x;
  const int n_phases = p.batch * p.n_kv_heads;

  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::kStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&bars->q_full[i], 1); mbar_init(&bars->q_empty[i], 1); }
    for (int i = 0; i < Cfg::kSlots; ++i) { mbar_init(&bars->acc_full[i], 1); mbar_init(&bars->acc_free[i], kGroupWarps); }
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
      int it = 0, u = 0;
      bool ok = true;
      for (int phase = 0; ok && phase < n_phases; ++phase) {
        const PhaseWork w = phase_work(p, phase, cta, ncta);
        if (w.n == 0) continue;
        const int h = u & 1;
        if (u >= 2) ok = mbar_wait_bounded(&bars->q_empty[h], ((u >> 1) - 1) & 1, abort_flag, p.hdr, SITE_FUSED_Q_EMPTY);
        if (!ok) break;
        const int q_row0 = (p.q_layout == FASTKV_Q_WINDOW) ? w.b * p.window : w.row0 + w.L - p.window;
        mbar_arrive_expect_tx(&bars->q_full[h], Cfg::KH * p.n_rows * 128);
        for (int c = 0; c < Cfg::KH; ++c)
          tma_load_3d(smem_q + h * Cfg::kQBytes + c * NPAD * 128, &tmap_q, &bars->q_full[h], c * 64,
                      w.g * p.group, q_row0, pol_keep);
        for (int i = 0; i < w.n; ++i, ++it) {
          const int s = it % Cfg::kStages;
          ok = mbar_wait_bounded(&bars->empty[s], ((it / Cfg::kStages) & 1) ^ 1, abort_flag, p.hdr, SITE_FUSED_EMPTY);
          if (!ok) break;
          mbar_arrive_expect_tx(&bars->full[s], Cfg::kStageBytes);
          for (int c = 0; c < Cfg::KH; ++c)
            tma_load_3d(smem_k + s * Cfg::kStageBytes + c * kHalfBytes, &tmap_k, &bars->full[s], c * 64, w.g,
                        w.row0 + (w.t0 + i) * kTileKeys, pol_stream);
        }
        ++u;
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: accumulators form a ring of kSlots tensor-memory slots ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16_f32(kTileKeys, NPAD);
      int it = 0, u = 0, seq = 0;
      bool ok = true;
      for (int phase = 0; ok && phase < n_phases; ++phase) {
        const PhaseWork w = phase_work(p, phase, cta, ncta);
        if (w.n == 0) continue;
        const int h = u & 1;
        ok = mbar_wait_bounded(&bars->q_full[h], (u >> 1) & 1, abort_flag, p.hdr, SITE_FUSED_Q_FULL);
        if (!ok) break;
        const uint32_t q_addr = smem_u32(smem_q + h * Cfg::kQBytes);
        for (int i = 0; i < w.n; ++i, ++it) {
          const int s = it % Cfg::kStages, slot = (seq + i) % Cfg::kSlots, use = (seq + i) / Cfg::kSlots;
          ok = mbar_wait_bounded(&bars->acc_free[slot], (use & 1) ^ 1, abort_flag, p.hdr, SITE_FUSED_ACC_FREE) &&
               mbar_wait_bounded(&bars->full[s], (it / Cfg::kStages) & 1, abort_flag, p.hdr, SITE_FUSED_FULL);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t k_addr = smem_u32(smem_k + s * Cfg::kStageBytes);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint64_t adesc = umma_desc_k_sw128(k_addr + (kk >> 2) * kHalfBytes + (kk & 3) * 32);
            const uint64_t bdesc = umma_desc_k_sw128(q_addr + (kk >> 2) * NPAD * 128 + (kk & 3) * 32);
            tc_mma_bf16(tmem_base + slot * NPAD, adesc, bdesc, idesc, kk > 0 ? 1u : 0u);
          }
          tc_commit(&bars->empty[s]);
          tc_commit(&bars->acc_full[slot]);
        }
        if (ok) tc_commit(&bars->q_empty[h]);
        seq += w.n + 1;                                  // the phase's tiles plus its statistics slot
        ++u;
      }
    }
  } else if (warp < 2 + kGroupWarps) {
    // ---------------- group A: pass 1 ----------------
    // Per tile: e = exp2(s - m) with a per-(lane, row) reference m, written back over the logits;
    // l += e.  m is the row's first logit and moves only when a logit exceeds it by more than the
    // slack (rare); then l and the e already stored for the phase's earlier tiles are rescaled,
    // so that at the end of the phase every stored e of a lane is relative to its final m.
    const int quarter = warp & 3;
    const int key_in_tile = quarter * 32 + lane;
    const int at = threadIdx.x - 64;                    // 0..127 within the group
    const int n_rows = p.n_rows, G = p.group;
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    int seq = 0;
    bool ok = true;
    for (int phase = 0; ok && phase < n_phases; ++phase) {
      const PhaseWork w = phase_work(p, phase, cta, ncta);
      if (w.n == 0) continue;
      float m[NPAD], l[NPAD];
      const int win_start = w.L - p.window;
      for (int i = 0; i < w.n; ++i) {
        const int slot = (seq + i) % Cfg::kSlots, use = (seq + i) / Cfg::kSlots;
        ok = mbar_wait_bounded(&bars->acc_full[slot], use & 1, abort_flag, p.hdr, SITE_FUSED_ACC_FULL);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after_sync();
        const int key = (w.t0 + i) * kTileKeys + key_in_tile;
        const bool tile_unmasked = (w.t0 + i + 1) * kTileKeys <= win_start;
#pragma unroll
        for (int c = 0; c < NPAD / 32; ++c) {
          float e[32];
          const uint32_t taddr = lane_base + slot * NPAD + c * 32;
          tmem_ld_32x32(taddr, e);
          const int n_valid = n_rows - c * 32;
          uint32_t visible = 0xffffffffu;                // causal: key i <= t_j, j = n / G
          if (!tile_unmasked) {
            visible = 0;
            if (key < w.L) {
#pragma unroll
              for (int x = 0; x < 32; ++x)
                if (x < n_valid && key <= win_start + (c * 32 + x) / G) visible |= 1u << x;
            }
          }
          float* const mc = m + c * 32;
          float* const lc = l + c * 32;
          if (i == 0) {
#pragma unroll
            for (int x = 0; x < 32; ++x) {
              const bool vis = (visible >> x) & 1u;
              mc[x] = vis ? e[x] * p.scale_log2 : -INFINITY;
              e[x] = vis ? 1.0f : 0.0f;
              lc[x] = e[x];
            }
          } else {
            bool need = false;                           // s - m is +inf while m = -inf
#pragma unroll
            for (int x = 0; x < 32; ++x)
              need |= (x < n_valid) && ((visible >> x) & 1u) && (fmaf(e[x], p.scale_log2, -mc[x]) > kLazyMaxSlackLog2);
            if (__any_sync(0xffffffffu, need)) {         // rare: some reference moves up to its new logit
              float fac[32];
#pragma unroll
              for (int x = 0; x < 32; ++x) {
                const float sx = e[x] * p.scale_log2;
                const bool mv = (x < n_valid) && ((visible >> x) & 1u) && (sx - mc[x] > kLazyMaxSlackLog2);
                fac[x] = (mv && mc[x] != -INFINITY) ? ex2(mc[x] - sx) : 1.0f;      // 2^(m_old - m_new)
                mc[x] = mv ? sx : mc[x];
                lc[x] *= fac[x];
              }
              for (int j = 0; j < i; ++j) {              // earlier tiles of the phase: e *= 2^(m_old - m_new)
                const uint32_t tj = lane_base + ((seq + j) % Cfg::kSlots) * NPAD + c * 32;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  float old[8];
                  tmem_ld_32x8(tj + q * 8, old);
#pragma unroll
                  for (int x = 0; x < 8; ++x) old[x] *= fac[q * 8 + x];
                  tmem_st_32x8(tj + q * 8, old);
                }
              }
            }
#pragma unroll
            for (int x = 0; x < 32; ++x) {
              e[x] = ((visible >> x) & 1u) ? ex2(fmaf(e[x], p.scale_log2, -mc[x])) : 0.0f;
              lc[x] += e[x];
            }
          }
          tmem_st_32x32(taddr, e);
        }
      }
      if (!ok) break;
      // the lane's final references go into the phase's statistics slot for group B
      const int sslot = (seq + w.n) % Cfg::kSlots, suse = (seq + w.n) / Cfg::kSlots;
      ok = mbar_wait_bounded(&bars->acc_free[sslot], (suse & 1) ^ 1, abort_flag, p.hdr, SITE_FUSED_ACC_FREE);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after_sync();
#pragma unroll
      for (int c = 0; c < NPAD / 32; ++c)
        tmem_st_32x32(lane_base + sslot * NPAD + c * 32, *reinterpret_cast<const float(*)[32]>(m + c * 32));
      tmem_wait_st();
      tc_fence_before_sync();
      // lanes -> warp: after the butterfly lane r holds row c * 32 + r in entry c * 32
#pragma unroll
      for (int c = 0; c < NPAD / 32; ++c) {
        stats_transpose_merge(m + c * 32, l + c * 32, lane);
        warp_stats[quarter * NPAD + c * 32 + lane] = make_float2(m[c * 32], l[c * 32]);
      }
      group_sync<1>();
      if (at < NPAD) {                                   // warps -> CTA, publish
        float mm = -INFINITY, ll = 0.0f;
#pragma unroll
        for (int q = 0; q < kGroupWarps; ++q) merge_stats(mm, ll, warp_stats[q * NPAD + at].x, warp_stats[q * NPAD + at].y);
        p.partial[(static_cast<size_t>(phase) * ncta + cta) * NPAD + at] = make_float2(mm, ll);
      }
      group_sync<1>();                                   // also: warp_stats may be rewritten next phase
      if (at == 0) {
        red_release_add(p.counters + phase, 1);          // release: cumulative over the barrier
        mbar_arrive(&bars->acc_full[sslot]);             // keeps this slot's full/free parities in step
      }
      seq += w.n + 1;
    }
  } else {
    // ---------------- group B: pass 2 ----------------
    // Once every CTA of the phase has published: merge the statistics into (M_r, 1 / l_r), turn the
    // lane's references into factors f = 2^(m - M_r) / l_r, and sum e * f over the window rows (and
    // the group) of each key.  No exponential per logit here.
    const int quarter = warp & 3;
    const int key_in_tile = quarter * 32 + lane;
    const int bt = threadIdx.x - 64 - kGroupWarps * 32;   // 0..127 within the group
    const int n_rows = p.n_rows, G = p.group;
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    constexpr int kParts = kGroupWarps * 32 / NPAD;
    int seq = 0;
    for (int phase = 0; phase < n_phases; ++phase) {
      const PhaseWork w = phase_work(p, phase, cta, ncta);
      if (w.n == 0) continue;
      if (bt == 0) {
        const int* ctr = p.counters + phase;
        if (ld_acquire(ctr) < w.nact) {
          const long long t0 = clock64();
          unsigned spins = 0;
          while (ld_acquire(ctr) < w.nact) {
            if ((++spins & 0x3Fu) == 0 && (*abort_flag || clock64() - t0 > kWaitLimitCycles)) {
              *abort_flag = 1;
              raise_status(p.hdr, FASTKV_ERR_DEVICE_TIMEOUT, SITE_FUSED_FLAG);
              break;
            }
          }
        }
      }
      group_sync<2>();
      if (*abort_flag) break;
      // the softmax normaliser of the phase, merged in a fixed order (the same in every CTA)
      merge_buf[bt] = merge_partials(p.partial + static_cast<size_t>(phase) * ncta * NPAD, NPAD, bt % NPAD, bt / NPAD,
                                     kParts, w.nact);
      group_sync<2>();
      if (bt < NPAD) {
        float mm = -INFINITY, ll = 0.0f;
#pragma unroll
        for (int q = 0; q < kParts; ++q) merge_stats(mm, ll, merge_buf[q * NPAD + bt].x, merge_buf[q * NPAD + bt].y);
        norm[bt] = (bt < n_rows && ll > 0.0f) ? make_float2(mm, 1.0f / ll) : make_float2(0.0f, 0.0f);
      }
      group_sync<2>();
      tc_fence_after_sync();
      const int sslot = (seq + w.n) % Cfg::kSlots;
      float f[NPAD];
#pragma unroll
      for (int c = 0; c < NPAD / 32; ++c) {
        float mref[32];
        tmem_ld_32x32(lane_base + sslot * NPAD + c * 32, mref);
#pragma unroll
        for (int x = 0; x < 32; ++x) {
          const float2 st = norm[c * 32 + x];
          f[c * 32 + x] = (c * 32 + x < n_rows) ? ex2(mref[x] - st.x) * st.y : 0.0f;   // m = -inf gives 0
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->acc_free[sslot]);
      for (int i = 0; i < w.n; ++i) {
        const int slot = (seq + i) % Cfg::kSlots;
        const int key = (w.t0 + i) * kTileKeys + key_in_tile;
        float a_g = 0.0f;
        float a_h[8];                                    // per query head of the group (G in {1,2,4,8})
#pragma unroll
        for (int q = 0; q < 8; ++q) a_h[q] = 0.0f;
#pragma unroll
        for (int c = 0; c < NPAD / 32; ++c) {
          float pr[32];
          tmem_ld_32x32(lane_base + slot * NPAD + c * 32, pr);
          if (c == NPAD / 32 - 1) {                      // the slot is in registers: hand it back
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->acc_free[slot]);
          }
          const int n_valid = n_rows - c * 32;
#pragma unroll
          for (int x = 0; x < 32; ++x) pr[x] = (x < n_valid) ? pr[x] * f[c * 32 + x] : 0.0f;
          if (!p.per_head) {
#pragma unroll
            for (int x = 0; x < 32; x += 4) a_g += (pr[x] + pr[x + 1]) + (pr[x + 2] + pr[x + 3]);
          } else {                                       // row n = j * G + hl and G divides 32
            switch (G) {
              case 1: add_heads<1>(pr, a_h); break;
              case 2: add_heads<2>(pr, a_h); break;
              case 4: add_heads<4>(pr, a_h); break;
              default: add_heads<8>(pr, a_h); break;
            }
          }
        }
        if (key < w.L) {
          if (p.per_head) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
              if (q < G) p.a_out[static_cast<size_t>(w.g * G + q) * p.ld_a + w.row0 + key] = a_h[q];
          } else {
            p.a_out[static_cast<size_t>(w.g) * p.ld_a + w.row0 + key] = a_g;
          }
        }
      }
      group_sync<2>();                                   // norm / merge_buf are rewritten next phase
      seq += w.n + 1;
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------
// Pooling of the un-pooled scores a[rows][L] written by pass 2 (Eq. 1 Pooling, App. B.1 group
// aggregation, Eq. 2): rows = KV heads (GROUP_THEN_POOL) or query heads (POOL_THEN_GROUP).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kPoolThreads) pool_rows_kernel(const PoolRowsParams p) {
  extern __shared__ float sm[];
  const int b = blockIdx.y;
  const int row0 = p.cu_seqlens ? p.cu_seqlens[b] : 0;
  const int L = p.cu_seqlens ? p.cu_seqlens[b + 1] - row0 : p.total_len;
  const int k0 = blockIdx.x * kPoolKeys;
  if (k0 >= L || L < p.window) return;
  const int r = p.pool_kernel >> 1;
  const int span = kPoolKeys + 2 * r;
  const int sub = p.per_head ? p.group : 1;
  const int rows = p.n_kv_heads * sub;
  for (int item = threadIdx.x; item < rows * span; item += blockDim.x) {
    const int row = item / span, o = item - row * span;
    const int key = k0 - r + o;
    sm[item] = (key >= 0 && key < L) ? __ldg(p.a + static_cast<size_t>(row) * p.ld_a + row0 + key) : 0.0f;
  }
  __syncthreads();
  const float inv_p = 1.0f / static_cast<float>(p.pool_kernel);
  for (int o = threadIdx.x; o < kPoolKeys; o += blockDim.x) {
    const int key = k0 + o;
    if (key >= L) break;
    float tsp = 0.0f;
    for (int g = 0; g < p.n_kv_heads; ++g) {
      float s_g = 0.0f;
      for (int hl = 0; hl < sub; ++hl) {
        const float* x = sm + (g * sub + hl) * span + o;     // x[0..2r] = positions key-r .. key+r
        float v = 0.0f;
        if (p.pool_mode == FASTKV_POOL_AVG) {
          for (int t = 0; t <= 2 * r; ++t) v += x[t];        // out-of-range entries hold 0
          v *= inv_p;
        } else {
          for (int t = 0; t <= 2 * r; ++t) v = fmaxf(v, x[t]);   // scores are >= 0: 0 = "no entry"
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
int fused_slots(int npad) { return 512 / npad - 1; }   // one slot per phase carries the lanes' references

template <int D, int NPAD>
static cudaError_t launch_fused_t(const CUtensorMap& tk, const CUtensorMap& tq, const FusedParams& p, int grid,
                                  cudaStream_t stream) {
  using Cfg = FusedCfg<D, NPAD>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(score_fused_kernel<D, NPAD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         Cfg::kSmemBytes);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  void* args[] = {const_cast<CUtensorMap*>(&tk), const_cast<CUtensorMap*>(&tq), const_cast<FusedParams*>(&p)};
  return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(score_fused_kernel<D, NPAD>), dim3(grid),
                                     dim3(kFusedThreads), args, Cfg::kSmemBytes, stream);
}

cudaError_t launch_score_fused(int head_dim, int npad, const CUtensorMap& tk, const CUtensorMap& tq,
                               const FusedParams& p, int grid, cudaStream_t stream) {
  if (head_dim == 128 && npad == 32) return launch_fused_t<128, 32>(tk, tq, p, grid, stream);
  if (head_dim == 128 && npad == 64) return launch_fused_t<128, 64>(tk, tq, p, grid, stream);
  if (head_dim == 64 && npad == 32) return launch_fused_t<64, 32>(tk, tq, p, grid, stream);
  if (head_dim == 64 && npad == 64) return launch_fused_t<64, 64>(tk, tq, p, grid, stream);
  return cudaErrorInvalidValue;
}

cudaError_t launch_pool_rows(const PoolRowsParams& p, int max_len, int batch, cudaStream_t stream) {
  const int rows = p.n_kv_heads * (p.per_head ? p.group : 1);
  const size_t smem = sizeof(float) * static_cast<size_t>(rows) * (kPoolKeys + 2 * (p.pool_kernel >> 1));
  static size_t configured = 48 * 1024;
  if (smem > configured) {
    cudaError_t e = cudaFuncSetAttribute(pool_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  dim3 grid((max_len + kPoolKeys - 1) / kPoolKeys, batch);
  pool_rows_kernel<<<grid, kPoolThreads, smem, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace fastkv
