// Window-query saliency scoring with one HBM pass over K (Eq. 1 inner term; Sec. 4.2).
//
// One persistent CTA per SM (cooperative launch, so all CTAs are resident).  The work is cut into
// phases, one per (sequence, KV head); in a phase every CTA owns a run of consecutive 128-key
// tiles.  Two tile pipelines run side by side in every CTA, each with its own TMA ring, its own
// tcgen05 MMA issuer and its own ring of tensor-memory accumulators:
//
//   pipeline 1  streams the CTA's K tiles from HBM, forms the logits S^T = K_tile . Q_g^T and keeps
//               a running (max, sum of exp2) per query row (warp group A); the CTAs' statistics of
//               a phase meet in global memory, counted by one counter per phase;
//   pipeline 2  follows one or two phases behind: once every CTA of the phase has published, it
//               merges the statistics into the softmax normaliser (fixed order: identical in every
//               CTA), loads the same K tiles again -- they are still in L2 -- recomputes the logits
//               on the idle tensor cores and sums p = exp2(s - M_r) / l_r over the window rows
//               (and the GQA group) of each key (warp group B).
//
// Nothing but the final per-key sums is written to memory, HBM sees K once, and neither pipeline
// holds anything across the grid-wide dependency except L2 lines, so the HBM stream of pipeline 1
// never waits for other CTAs.  Pipeline 1 is throttled to stay at most kMaxLead phases ahead of
// pipeline 2 so that the re-read really hits L2.  Every wait (mbarrier, counter, flag) is bounded
// and ends in a status word instead of a hang.
#include "score.cuh"

namespace fastkv {

namespace {

constexpr int kTileKeys = 128;
constexpr int kHalfBytes = kTileKeys * 128;
constexpr int kGroupWarps = 8;                 // warps per epilogue group: 4 lane quarters x 2 column halves
constexpr int kCtrlWarps = 4;                  // TMA 1, MMA 1, TMA 2, MMA 2
constexpr int kFusedThreads = 32 * (kCtrlWarps + 2 * kGroupWarps);
constexpr int kAcc = 4;                        // accumulators per pipeline

template <int D, int NPAD>
struct FusedCfg {
  static constexpr int KH = D / 64;
  static constexpr int kStageBytes = KH * kHalfBytes;
  static constexpr int kQBytes = KH * NPAD * 128;
  static constexpr int kStages1 = (D == 128) ? 3 : 6;                       // HBM stream
  static constexpr int kStages2 = (D == 128) ? (NPAD == 32 ? 3 : 2) : 4;    // L2 re-read
  static constexpr int kTmemCols = 2 * kAcc * NPAD;                         // 256 or 512
  static constexpr int kBarBytes = 512;
  static constexpr int kSmemBytes = 1024 + (kStages1 + kStages2) * kStageBytes + 3 * kQBytes + kBarBytes +
                                    4 * NPAD * 8 + NPAD * 8 + kGroupWarps * 32 * 8 + NPAD * 4;
};

struct FusedBarriers {
  uint64_t full1[6], empty1[6];
  uint64_t full2[4], empty2[4];
  uint64_t q1_full[2], q1_empty[2], q2_full[2], q2_empty[2];
  uint64_t acc1_full[kAcc], acc1_empty[kAcc], acc2_full[kAcc], acc2_empty[kAcc];
  uint64_t mma_done[2];
  uint32_t tmem_base;
  int abort_flag;
  int p1_done;                 // phases (this CTA took part in) whose pass 1 is published
  int p2_done;                 // ... whose pass 2 is finished
};
static_assert(sizeof(FusedBarriers) <= 512, "barrier block");

template <int ID>
__device__ __forceinline__ void group_sync() { asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(kGroupWarps * 32) : "memory"); }


// Bounded wait until *flag (shared memory, written by another warp of the CTA) reaches `target`.
__device__ __forceinline__ bool wait_smem_counter(volatile int* flag, int target, volatile int* abort_flag,
                                                  WorkspaceHeader* hdr, int site, long long limit) {
  if (*flag >= target) return true;
  if (*abort_flag) return false;
  const long long t0 = clock64();
  unsigned spins = 0;
  while (*flag < target) {
    if ((++spins & 0x3Fu) == 0 && (*abort_flag || clock64() - t0 > limit)) {
      *abort_flag = 1;
      raise_status(hdr, FASTKV_ERR_DEVICE_TIMEOUT, site);
      return false;
    }
  }
  return true;
}

template <int GG>
__device__ __forceinline__ void add_heads(const float (&pr)[16], float (&a_h)[8]) {
#pragma unroll
  for (int x = 0; x < 16; ++x) a_h[x % GG] += pr[x];
}

// What one CTA does in one phase.  A phase covers a few KV heads of one sequence -- as many as keep it
// near `phase_bytes` of K, so short sequences get fewer, fuller phases and fewer grid-wide
// dependencies; the CTAs are split evenly among those heads, and within a head every CTA owns a run
// of consecutive tiles.  Every role of every CTA walks the same sequence of phases.
struct PhaseWork {
  int b, g, row0, L, t0, n, nact;
  int stat;                    // index of the (sequence, head) statistics: b * n_kv_heads + g
  int c;                       // this CTA's index among the CTAs of its head
};

struct PhaseIter {
  int b, g0;                   // next phase: sequence b, heads g0 .. g0 + hp - 1
};

__device__ __forceinline__ bool next_phase(const FusedParams& p, PhaseIter& it, int cta, int ncta, PhaseWork& w) {
  if (it.b >= p.batch) return false;
  w.b = it.b;
  w.row0 = p.cu_seqlens ? p.cu_seqlens[w.b] : 0;
  w.L = p.cu_seqlens ? p.cu_seqlens[w.b + 1] - w.row0 : p.total_len;
  // heads per phase of this sequence: the same arithmetic in every thread that walks the phases
  long long hp = p.phase_bytes / (static_cast<long long>(w.L > 0 ? w.L : 1) * p.head_bytes);
  if (p.heads_per_phase > 0) hp = p.heads_per_phase;        // forced
  if (hp > p.n_kv_heads) hp = p.n_kv_heads;
  if (hp > ncta) hp = ncta;
  if (hp < 1) hp = 1;
  const int g0 = it.g0;
  it.g0 += static_cast<int>(hp);
  if (it.g0 >= p.n_kv_heads) { it.g0 = 0; ++it.b; }
  const int ctas_per_head = ncta / static_cast<int>(hp);
  const int hi = cta / ctas_per_head;
  w.c = cta - hi * ctas_per_head;
  w.g = g0 + hi;
  w.stat = w.b * p.n_kv_heads + w.g;
  if (hi >= hp || w.g >= p.n_kv_heads || w.L < p.window) { w.t0 = 0; w.n = 0; w.nact = 0; return true; }
  const int ntiles = (w.L + kTileKeys - 1) / kTileKeys;
  const int per = (ntiles + ctas_per_head - 1) / ctas_per_head;
  w.nact = (ntiles + per - 1) / per;
  w.t0 = w.c * per;
  w.n = max(0, min(per, ntiles - w.t0));
  return true;
}

}  // namespace

static_assert(FusedCfg<128, 32>::kSmemBytes <= 232448 && FusedCfg<128, 64>::kSmemBytes <= 232448 &&
              FusedCfg<64, 32>::kSmemBytes <= 232448 && FusedCfg<64, 64>::kSmemBytes <= 232448,
              "dynamic shared memory per CTA");

template <int D, int NPAD>
__global__ void __launch_bounds__(kFusedThreads, 1)
score_fused_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_q,
                   const FusedParams p) {
  using Cfg = FusedCfg<D, NPAD>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* smem_k1 = smem;
  uint8_t* smem_k2 = smem_k1 + Cfg::kStages1 * Cfg::kStageBytes;
  uint8_t* smem_q1 = smem_k2 + Cfg::kStages2 * Cfg::kStageBytes;      // two buffers of kQBytes
  uint8_t* smem_q2 = smem_q1 + 2 * Cfg::kQBytes;                      // one buffer of kQBytes
  FusedBarriers* bars = reinterpret_cast<FusedBarriers*>(smem_q2 + Cfg::kQBytes);
  float2* warp_stats = reinterpret_cast<float2*>(reinterpret_cast<uint8_t*>(bars) + Cfg::kBarBytes);   // [4][NPAD]
  float2* norm = warp_stats + 4 * NPAD;                               // [NPAD] (row max, 1 / row sum)
  float2* merge_buf = norm + NPAD;                                    // [256] partial merges
  int* row_j = reinterpret_cast<int*>(merge_buf + kGroupWarps * 32);  // [NPAD] window row j = n / G of query row n
  constexpr int CPW = NPAD / 2;                                       // accumulator columns per epilogue warp

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, ncta = gridDim.x;
  const long long limit = p.wait_limit;

  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::kStages1; ++s) { mbar_init(&bars->full1[s], 1); mbar_init(&bars->empty1[s], 1); }
    for (int s = 0; s < Cfg::kStages2; ++s) { mbar_init(&bars->full2[s], 1); mbar_init(&bars->empty2[s], 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->q1_full[i], 1); mbar_init(&bars->q1_empty[i], 1);
      mbar_init(&bars->q2_full[i], 1); mbar_init(&bars->q2_empty[i], 1);
    }
    for (int i = 0; i < kAcc; ++i) {
      mbar_init(&bars->acc1_full[i], 1); mbar_init(&bars->acc1_empty[i], kGroupWarps);   // every warp of the group
      mbar_init(&bars->acc2_full[i], 1); mbar_init(&bars->acc2_empty[i], 4);             // the four warps of one set
    }
    mbar_init(&bars->mma_done[0], 1);
    mbar_init(&bars->mma_done[1], 1);
    bars->abort_flag = 0;
    bars->p1_done = 0;
    bars->p2_done = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tma_prefetch_desc(&tmap_k);
    tma_prefetch_desc(&tmap_q);
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, Cfg::kTmemCols);
    tmem_relinquish();
  }
  if (threadIdx.x >= 64 && threadIdx.x < 64 + NPAD) row_j[threadIdx.x - 64] = (threadIdx.x - 64) / p.group;   // divide once
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;
  volatile int* abort_flag = &bars->abort_flag;
  pdl_launch_dependents();     // the pooling kernel may be brought up; it waits for this grid to finish

  if (warp == 0 || warp == 2) {
    // ---------------- TMA producers (warp 0: pipeline 1 from HBM, warp 2: pipeline 2 from L2) ----------------
    if (lane == 0) {
      const bool second = warp == 2;
      const uint64_t pol_k = second ? l2_policy_evict_first() : l2_policy_evict_last();
      const uint64_t pol_q = l2_policy_evict_last();
      uint8_t* const ring = second ? smem_k2 : smem_k1;
      uint8_t* const qbuf = second ? smem_q2 : smem_q1;
      uint64_t* const full = second ? bars->full2 : bars->full1;
      uint64_t* const empty = second ? bars->empty2 : bars->empty1;
      uint64_t* const q_full = second ? bars->q2_full : bars->q1_full;
      uint64_t* const q_empty = second ? bars->q2_empty : bars->q1_empty;
      const int stages = second ? Cfg::kStages2 : Cfg::kStages1;
      const int nq = second ? 1 : 2;                     // Q buffers of the pipeline
      int it = 0, u = 0, uq = 0;
      bool ok = true;
      PhaseIter pit = {0, 0};
      PhaseWork w;
      while (ok && next_phase(p, pit, cta, ncta, w)) {
        if (w.n == 0) continue;
        // pipeline 2 re-reads what pipeline 1 of this CTA has finished with; pipeline 1 stays close
        // enough ahead for those tiles to be still in L2
        if (second) ok = wait_smem_counter(&bars->p1_done, u + 1, abort_flag, p.hdr, SITE_FUSED_P1_DONE, limit);
        else if (u >= p.max_lead) ok = wait_smem_counter(&bars->p2_done, u - p.max_lead + 1, abort_flag, p.hdr, SITE_FUSED_P2_DONE, limit);
        const int h = u % nq;
        if (ok && u >= nq) ok = mbar_wait_bounded(&q_empty[h], ((u / nq) - 1) & 1, abort_flag, p.hdr, SITE_FUSED_Q_EMPTY, limit);
        if (!ok) break;
        const int q_row0 = (p.q_layout == FASTKV_Q_WINDOW) ? w.b * p.window : w.row0 + w.L - p.window;
        mbar_arrive_expect_tx(&q_full[h], Cfg::KH * p.n_rows * 128);
        for (int c = 0; c < Cfg::KH; ++c)
          tma_load_3d(qbuf + h * Cfg::kQBytes + c * NPAD * 128, &tmap_q, &q_full[h], c * 64, w.g * p.group, q_row0,
                      pol_q);
        ++uq;
        for (int i = 0; i < w.n; ++i, ++it) {
          const int s = it % stages;
          ok = mbar_wait_bounded(&empty[s], ((it / stages) & 1) ^ 1, abort_flag, p.hdr, SITE_FUSED_EMPTY, limit);
          if (!ok) break;
          mbar_arrive_expect_tx(&full[s], Cfg::kStageBytes);
          for (int c = 0; c < Cfg::KH; ++c)
            tma_load_3d(ring + s * Cfg::kStageBytes + c * kHalfBytes, &tmap_k, &full[s], c * 64, w.g,
                        w.row0 + (w.t0 + i) * kTileKeys, pol_k);
        }
        ++u;
      }
      // No copy may still be writing this CTA's shared memory when the CTA ends: wait for the last
      // load of every stage and query buffer, whatever the abort flag says.
      for (int s = 0; s < stages && s < it; ++s) {
        const int last = it - 1 - ((it - 1 - s) % stages);
        mbar_wait_drain(&full[s], (last / stages) & 1, p.hdr, SITE_PARKED_DRAIN, limit);
      }
      for (int h = 0; h < nq && h < uq; ++h) {
        const int last = uq - 1 - ((uq - 1 - h) % nq);
        mbar_wait_drain(&q_full[h], (last / nq) & 1, p.hdr, SITE_PARKED_DRAIN, limit);
      }
    }
  } else if (warp == 1 || warp == 3) {
    // ---------------- MMA issuers (warp 1: pipeline 1, warp 3: pipeline 2) ----------------
    if (lane == 0) {
      const bool second = warp == 3;
      constexpr uint32_t idesc = umma_idesc_bf16_f32(kTileKeys, NPAD);
      uint8_t* const ring = second ? smem_k2 : smem_k1;
      uint8_t* const qbuf = second ? smem_q2 : smem_q1;
      uint64_t* const full = second ? bars->full2 : bars->full1;
      uint64_t* const empty = second ? bars->empty2 : bars->empty1;
      uint64_t* const q_full = second ? bars->q2_full : bars->q1_full;
      uint64_t* const q_empty = second ? bars->q2_empty : bars->q1_empty;
      uint64_t* const acc_full = second ? bars->acc2_full : bars->acc1_full;
      uint64_t* const acc_empty = second ? bars->acc2_empty : bars->acc1_empty;
      const int stages = second ? Cfg::kStages2 : Cfg::kStages1;
      const int nq = second ? 1 : 2;
      const uint32_t acc_base = tmem_base + (second ? kAcc * NPAD : 0);
      int it = 0, u = 0;
      bool ok = true;
      PhaseIter pit = {0, 0};
      PhaseWork w;
      while (ok && next_phase(p, pit, cta, ncta, w)) {
        if (w.n == 0) continue;
        const int h = u % nq;
        ok = mbar_wait_bounded(&q_full[h], (u / nq) & 1, abort_flag, p.hdr, SITE_FUSED_Q_FULL, limit);
        if (!ok) break;
        const uint32_t q_addr = smem_u32(qbuf + h * Cfg::kQBytes);
        for (int i = 0; i < w.n; ++i, ++it) {
          const int s = it % stages, a = it % kAcc;
          ok = mbar_wait_bounded(&acc_empty[a], ((it / kAcc) & 1) ^ 1, abort_flag, p.hdr, SITE_FUSED_ACC_FREE, limit) &&
               mbar_wait_bounded(&full[s], (it / stages) & 1, abort_flag, p.hdr, SITE_FUSED_FULL, limit);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t k_addr = smem_u32(ring + s * Cfg::kStageBytes);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint64_t adesc = umma_desc_k_sw128(k_addr + (kk >> 2) * kHalfBytes + (kk & 3) * 32);
            const uint64_t bdesc = umma_desc_k_sw128(q_addr + (kk >> 2) * NPAD * 128 + (kk & 3) * 32);
            tc_mma_bf16(acc_base + a * NPAD, adesc, bdesc, idesc, kk > 0 ? 1u : 0u);
          }
          tc_commit(&empty[s]);
          tc_commit(&acc_full[a]);
        }
        if (ok) tc_commit(&q_empty[h]);
        ++u;
      }
      // every contraction issued above has finished before tensor memory is released
      if (it > 0) {
        tc_commit(&bars->mma_done[second ? 1 : 0]);
        mbar_wait_drain(&bars->mma_done[second ? 1 : 0], 0, p.hdr, SITE_PARKED_DRAIN, limit);
      }
    }
  } else if (warp < kCtrlWarps + kGroupWarps) {
    // ---------------- group A: pass 1, running (max, sum of exp2) per query row; publish per phase ----------------
    // 8 warps: warp (quarter, half) owns tensor-memory lanes 32 * quarter .. +31 (one key per lane)
    // and the accumulator columns (query rows) half * CPW .. +CPW-1.
    const int gw = warp - kCtrlWarps;
    const int quarter = warp & 3, half = gw >> 2;
    const int key_in_tile = quarter * 32 + lane;
    const int at = threadIdx.x - kCtrlWarps * 32;       // 0..255 within the group
    const int n_rows = p.n_rows;
    const int col0 = half * CPW;                         // first query row of this warp
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + col0;
    int it = 0, u = 0;
    bool ok = true;
    PhaseIter pit = {0, 0};
    PhaseWork w;
    while (next_phase(p, pit, cta, ncta, w)) {           // an aborted CTA still walks every phase: see group_sync
      if (w.n == 0) {
        // a sequence shorter than the observation window has no defined scores: say so once
        if (w.L < p.window && cta == 0 && at == 0) raise_status(p.hdr, FASTKV_ERR_INVALID_ARG, SITE_SCORE_SHORT_SEQUENCE);
        continue;
      }
      float m[CPW], l[CPW];
#pragma unroll
      for (int n = 0; n < CPW; ++n) { m[n] = -INFINITY; l[n] = 0.0f; }
      const int win_start = w.L - p.window;
      for (int i = 0; i < w.n; ++i, ++it) {
        const int a = it % kAcc;
        if (ok) ok = mbar_wait_bounded(&bars->acc1_full[a], (it / kAcc) & 1, abort_flag, p.hdr, SITE_FUSED_ACC_FULL, limit);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) continue;                               // aborted: no more waiting or computing
        tc_fence_after_sync();
        const int key = (w.t0 + i) * kTileKeys + key_in_tile;
        const bool tile_unmasked = (w.t0 + i + 1) * kTileKeys <= win_start;
#pragma unroll
        for (int c = 0; c < CPW / 16; ++c) {
          float acc[16];
          tmem_ld_32x16(lane_base + a * NPAD + c * 16, acc);
          if (c == CPW / 16 - 1) {                       // this warp's part of the accumulator is in registers
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->acc1_empty[a]);
          }
          const int n_valid = n_rows - col0 - c * 16;
          if (tile_unmasked) {
            if (i == 0) stats_init_unmasked<16>(acc, m + c * 16, l + c * 16, p.scale_log2, n_valid);
            else stats_update_unmasked<16>(acc, m + c * 16, l + c * 16, p.scale_log2, n_valid);
          } else {
            uint32_t visible = 0;                        // causal: key i <= t_j, j = n / G
            if (key < w.L) {
#pragma unroll
              for (int x = 0; x < 16; ++x)
                if (x < n_valid && key <= win_start + row_j[col0 + c * 16 + x]) visible |= 1u << x;
            }
            stats_update_masked<16>(acc, m + c * 16, l + c * 16, p.scale_log2, n_valid, visible);
          }
        }
      }
      // lanes -> warp: after the butterfly lanes r and r + 16 hold row col0 + c * 16 + r in entry c * 16
#pragma unroll
      for (int c = 0; c < CPW / 16; ++c) {
        stats_transpose_merge<16>(m + c * 16, l + c * 16, lane);
        if (lane < 16) warp_stats[quarter * NPAD + col0 + c * 16 + lane] = make_float2(m[c * 16], l[c * 16]);
      }
      group_sync<1>();
      if (at < NPAD) {                                   // lane quarters -> CTA, publish
        float mm = -INFINITY, ll = 0.0f;
#pragma unroll
        for (int q = 0; q < 4; ++q) merge_stats(mm, ll, warp_stats[q * NPAD + at].x, warp_stats[q * NPAD + at].y);
        p.partial[(static_cast<size_t>(w.stat) * ncta + w.c) * NPAD + at] = make_float2(mm, ll);
      }
      group_sync<1>();                                   // also: warp_stats may be rewritten next phase
      ++u;
      if (at == 0) {
        red_release_add(p.counters + w.stat, 1);         // release: cumulative over the barrier
        bars->p1_done = u;                               // pipeline 2 may re-read this phase's tiles
      }
    }
  } else {
    // ---------------- group B: pass 2, normalise and sum over window rows / group ----------------
    // Two sets of four warps (one per tensor-memory lane quarter) take alternate tiles, so two tiles
    // are in flight and one set's waits and stores overlap the other set's exponentials.  A warp
    // handles all query rows of its 32 keys; the normaliser is read from shared memory (broadcast).
    const int gw = warp - kCtrlWarps - kGroupWarps;
    const int quarter = warp & 3, set = gw >> 2;
    const int key_in_tile = quarter * 32 + lane;
    const int bt = threadIdx.x - (kCtrlWarps + kGroupWarps) * 32;   // 0..255 within the group
    const int n_rows = p.n_rows, G = p.group;
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + kAcc * NPAD;
    constexpr int kParts = kGroupWarps * 32 / NPAD;
    int it = 0, u = 0;
    bool ok = true;
    PhaseIter pit = {0, 0};
    PhaseWork w;
    while (next_phase(p, pit, cta, ncta, w)) {
      if (w.n == 0) continue;
      // every CTA that owns tiles of this phase has published its statistics?
      if (bt == 0 && !*abort_flag) {
        const int* ctr = p.counters + w.stat;
        const int target = w.nact + p.extra_publications;
        if (ld_acquire(ctr) < target) {
          const long long t0 = clock64();
          unsigned spins = 0;
          while (ld_acquire(ctr) < target) {
            if ((++spins & 0x3Fu) == 0 && (*abort_flag || clock64() - t0 > limit)) {
              *abort_flag = 1;
              raise_status(p.hdr, FASTKV_ERR_DEVICE_TIMEOUT, SITE_FUSED_FLAG);
              break;
            }
          }
        }
      }
      group_sync<2>();
      if (*abort_flag) ok = false;                       // every warp still reaches every barrier below
      // the softmax normaliser of the phase, merged in a fixed order (the same in every CTA)
      merge_buf[bt] = merge_partials(p.partial + static_cast<size_t>(w.stat) * ncta * NPAD, NPAD, bt % NPAD, bt / NPAD,
                                     kParts, w.nact);
      group_sync<2>();
      if (bt < NPAD) {
        float mm = -INFINITY, ll = 0.0f;
#pragma unroll
        for (int q = 0; q < kParts; ++q) merge_stats(mm, ll, merge_buf[q * NPAD + bt].x, merge_buf[q * NPAD + bt].y);
        // (-row max, 1 / row sum); rows beyond G * w contribute nothing
        norm[bt] = (bt < n_rows && ll > 0.0f) ? make_float2(-mm, 1.0f / ll) : make_float2(0.0f, 0.0f);
      }
      group_sync<2>();
      const int win_start = w.L - p.window;
      for (int i = 0; i < w.n; ++i, ++it) {
        if ((it & 1) != set) continue;                   // the other set's tile
        const int a = it % kAcc;
        if (ok) ok = mbar_wait_bounded(&bars->acc2_full[a], (it / kAcc) & 1, abort_flag, p.hdr, SITE_FUSED_ACC_FULL, limit);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) continue;
        tc_fence_after_sync();
        const int key = (w.t0 + i) * kTileKeys + key_in_tile;
        const bool tile_unmasked = (w.t0 + i + 1) * kTileKeys <= win_start;
        float a_g = 0.0f;
        float a_h[8];                                    // per query head of the group (G in {1,2,4,8})
#pragma unroll
        for (int q = 0; q < 8; ++q) a_h[q] = 0.0f;
#pragma unroll
        for (int c = 0; c < NPAD / 16; ++c) {
          float pr[16];
          tmem_ld_32x16(lane_base + a * NPAD + c * 16, pr);
          if (c == NPAD / 16 - 1) {                      // the accumulator is in registers: hand it back
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->acc2_empty[a]);
          }
          const int n_valid = n_rows - c * 16;
#pragma unroll
          for (int x = 0; x < 16; ++x) {
            const float2 st = norm[c * 16 + x];
            pr[x] = (x < n_valid) ? ex2(fmaf(pr[x], p.scale_log2, st.x)) * st.y : 0.0f;
          }
          if (!tile_unmasked) {                          // causal: key i <= t_j, j = n / G
#pragma unroll
            for (int x = 0; x < 16; ++x)
              if (x < n_valid && key > win_start + row_j[c * 16 + x]) pr[x] = 0.0f;
          }
          if (!p.per_head) {
#pragma unroll
            for (int x = 0; x < 16; x += 4) a_g += (pr[x] + pr[x + 1]) + (pr[x + 2] + pr[x + 3]);
          } else {                                       // row n = j * G + hl and G divides 16
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
      ++u;
      if (bt == 0) bars->p2_done = u;                    // lets pipeline 1 move further ahead
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
  pdl_wait();                  // the un-pooled scores come from the scoring kernel before this one
  pdl_launch_dependents();     // (after the wait: letting the selection kernel queue up earlier costs short steps 1.5 us)
  const int b = blockIdx.y;
  const int row0 = p.cu_seqlens ? p.cu_seqlens[b] : 0;
  const int L = p.cu_seqlens ? p.cu_seqlens[b + 1] - row0 : p.total_len;
  const int k0 = blockIdx.x * kPoolKeys;
  if (k0 >= L || L < p.window) return;
  const int r = p.pool_kernel >> 1;
  const int span = kPoolKeys + 2 * r;
  const int sub = p.per_head ? p.group : 1;
  const int rows = p.n_kv_heads * sub;
  // each thread fetches its position(s) for every row; eight rows' loads are in flight together
  for (int o = threadIdx.x; o < span; o += blockDim.x) {
    const int key = k0 - r + o;
    const bool inside = key >= 0 && key < L;
    const float* src = p.a + row0 + key;
#pragma unroll 8
    for (int row = 0; row < rows; ++row) {
      const float* s0 = src + static_cast<size_t>(row) * p.ld_a;
      sm[row * span + o] = inside ? __ldg(s0) : 0.0f;
    }
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

template <int D, int NPAD>
static cudaError_t launch_fused_t(const CUtensorMap& tk, const CUtensorMap& tq, const FusedParams& p, int grid,
                                  cudaStream_t stream) {
  using Cfg = FusedCfg<D, NPAD>;
  static PerDeviceOnce configured;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (!configured.done(dev)) {
    e = cudaFuncSetAttribute(score_fused_kernel<D, NPAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes);
    if (e != cudaSuccess) return e;
    configured.set(dev);
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
  if (smem > 48 * 1024) {          // rare (many heads, wide pooling window): opt in on every such launch
    cudaError_t e = cudaFuncSetAttribute(pool_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem));
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((max_len + kPoolKeys - 1) / kPoolKeys, batch);
  cfg.blockDim = dim3(kPoolThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  fill_pdl_attribute(&attr[0]);
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, pool_rows_kernel, p);
}

}  // namespace fastkv
