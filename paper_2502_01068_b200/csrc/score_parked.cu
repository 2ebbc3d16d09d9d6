// Window-query saliency scoring with one pass over K and one contraction per key tile (Eq. 1 inner
// term; Sec. 4.2): the logits of a tile stay parked in tensor memory until the softmax statistics
// of their row are known, then they are normalised and summed in place.
//
// One persistent CTA per SM (cooperative launch: every CTA is resident).  The work is cut into
// phases, one per (sequence, KV head); in every phase CTA c owns the same run of consecutive
// 128-key tiles of the sequence.  Per CTA:
//
//   producer   one thread streams the K tiles (and the G*w window-query rows of the phase) into a
//              ring of shared-memory stages with TMA;
//   issuer     one thread forms S^T = K_tile . Q_g^T with tcgen05.mma (M = 128 keys, N = query
//              rows, fp32) into the next slot of a ring that covers all of tensor memory
//              (16 slots of 32 columns, or 8 of 64); a slot is not recycled by the issuer, it is
//              handed back by pass 2;
//   pass 1     (eight warps, one key per lane) reads each new slot, turns every logit into
//              e = exp2(s - ref) against the thread's own reference for that query row, adds e to
//              the row's running sum and writes e back over the logit; at the end of the phase the
//              thread's references and the warp's (max, sum) per row go to shared memory.  The
//              reference of a row is the first logit the thread saw; it moves (and the e already
//              parked for this phase are rescaled) only if a logit exceeds it by more than 64
//              binary orders of magnitude;
//   publisher  (one warp) writes the CTA's (max, sum) per row of a finished phase to global memory and
//              bumps the phase's counter, so that publication never waits behind anything else; between
//              publications it watches the counter of the oldest phase not yet collected and, once
//              every CTA has published, brings all CTAs' statistics of that phase into shared memory
//              with one bulk copy -- while pass 2 is still busy with the phase before;
//   pass 2     (four warps, one per tensor-memory lane quarter) waits for the collected statistics
//              of the phase, merges them in a fixed order (identical in every CTA:
//              deterministic) into the softmax normaliser of every row, forms one weight per
//              (key lane, query row), f = exp2(ref - M_r) / l_r, and then only needs a multiply-add
//              per parked value: the score of a key is the sum of e * f over its window rows and
//              GQA group.  It writes the per-key sums and frees the slots.
// Pass 1 hands its results on through mbarriers only: it never waits for its own slowest warp.
//
// K crosses the memory system once and is contracted once; the only grid-wide dependency (the
// statistics of a phase) is hidden behind the next phases as long as a CTA's tiles of two phases
// fit in the ring.  A phase must fit in the ring on its own (tiles per CTA <= slots), else the
// issuer would wait for slots that only the end of the phase can free: the host checks this and
// the kernel re-checks it before touching any barrier.
//
// Every wait is bounded.  A wait that gives up raises the status word and the CTA-wide abort flag;
// from then on every role runs through the rest of its loops without waiting or computing, so all
// warps still meet at every named barrier and at the final __syncthreads, copies in flight are
// waited for, and tensor memory is released.
#include "score.cuh"

namespace fastkv {

namespace {

constexpr int kTileKeys = 128;
constexpr int kHalfBytes = kTileKeys * 128;
// warp roles; any four consecutive warps cover the four tensor-memory lane quarters (quarter = warp % 4)
constexpr int kCtrlWarps = 3;                  // producer, issuer, publisher of the softmax statistics
constexpr int kPass1Warps = 8;                 // 4 lane quarters x 2 halves of the query rows
constexpr int kPass2Warps = 4;                 // 4 lane quarters
constexpr int kPass2Threads = 32 * kPass2Warps;
constexpr int kParkedThreads = 32 * (kCtrlWarps + kPass1Warps + kPass2Warps);   // 15 warps: at most 4 per scheduler
constexpr int kMaxStages = 8;
constexpr int kMaxSlots = 16;
constexpr int kMaxCtas = 148;                  // CTAs whose statistics the collection buffer holds
// Pass 1 keeps e = exp2(s - ref) with the row's first logit as the reference; the reference only moves
// when a logit exceeds it by more than this many binary orders of magnitude (e and its row sums stay far
// inside the fp32 range: e <= 2^64, at most 2^20-odd terms per sum).
constexpr float kRefSlackLog2 = 64.0f;

template <int D, int NPAD>
struct ParkedCfg {
  static constexpr int KH = D / 64;
  static constexpr int kStageBytes = KH * kHalfBytes;
  static constexpr int kQBytes = KH * NPAD * 128;
  static constexpr int kStages = (D == 128) ? 3 : 6;
  // with 32 query rows all CTAs' statistics of a phase (37 KB) are collected in shared memory by the
  // publisher warp; with 64 rows there is no room and pass 2 reads them from global memory itself
  static constexpr bool kCollect = NPAD == 32;
  static constexpr int kCollectBytes = kCollect ? kMaxCtas * NPAD * 8 : 0;
  static constexpr int kSlots = 512 / NPAD;                 // tensor memory: 512 columns
  static constexpr int kBarBytes = 1024;
  static constexpr int kRefBytes = NPAD * kTileKeys * 4;    // one reference per (query row, key lane)
  static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + 2 * kQBytes + 2 * kRefBytes + kBarBytes +
                                    2 * 4 * NPAD * 8 /*warp_stats*/ + NPAD * 8 /*norm*/ +
                                    2 * kPass2Threads * 8 /*merge_buf*/ + NPAD * 4 /*row_j*/ + kCollectBytes;
};

struct ParkedBarriers {
  uint64_t full[kMaxStages], empty[kMaxStages];
  uint64_t q_full[2], q_empty[2];
  uint64_t slot_full[kMaxSlots], slot_free[kMaxSlots];
  uint64_t mma_done;
  uint64_t ref_free[2];        // pass 2 has finished with the references of a phase
  uint64_t stats_ready[2];     // pass 1 has written its warps' statistics of a phase
  uint64_t stats_free[2];      // ... and the publisher has read them
  uint64_t coll_full;          // all CTAs' statistics of a phase have landed in shared memory
  uint64_t coll_free;          // ... and pass 2 has merged them
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(ParkedBarriers) <= 1024, "barrier block");

// barrier of the pass-2 group (the only named barrier of the kernel)
__device__ __forceinline__ void pass2_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kPass2Threads) : "memory");
}

// Merges the per-CTA statistics of two adjacent query rows (n2, n2 + 1) over CTAs first, first + stride, ...
// in a fixed order, with up to twenty 16-byte loads in flight.  part[r * npad + n] = (max, sum) of row n in CTA r.
__device__ __forceinline__ void merge_partials_2rows(const float2* part, int npad, int n2, int first, int stride,
                                                     int count, float2& out0, float2& out1) {
  float m0 = -INFINITY, l0 = 0.0f, m1 = -INFINITY, l1 = 0.0f;
  for (int r0 = first; r0 < count; r0 += stride * 20) {
    float4 v[20];
#pragma unroll
    for (int j = 0; j < 20; ++j) {
      const int r = r0 + j * stride;
      v[j] = (r < count) ? __ldcg(reinterpret_cast<const float4*>(&part[static_cast<size_t>(r) * npad + n2]))
                         : make_float4(-INFINITY, 0.0f, -INFINITY, 0.0f);
    }
#pragma unroll
    for (int j = 0; j < 20; ++j) {
      merge_stats(m0, l0, v[j].x, v[j].y);
      merge_stats(m1, l1, v[j].z, v[j].w);
    }
  }
  out0 = make_float2(m0, l0);
  out1 = make_float2(m1, l1);
}

// The same merge from the copy of all CTAs' statistics in shared memory.
__device__ __forceinline__ void merge_collected_2rows(const float2* part, int npad, int n2, int first, int stride,
                                                      int count, float2& out0, float2& out1) {
  float m0 = -INFINITY, l0 = 0.0f, m1 = -INFINITY, l1 = 0.0f;
  for (int r = first; r < count; r += stride) {
    const float4 v = *reinterpret_cast<const float4*>(&part[r * npad + n2]);
    merge_stats(m0, l0, v.x, v.y);
    merge_stats(m1, l1, v.z, v.w);
  }
  out0 = make_float2(m0, l0);
  out1 = make_float2(m1, l1);
}

// global -> shared bulk copy (16-byte aligned, size a multiple of 16) that completes on an mbarrier
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(smem_dst)),
               "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

template <int GG>
__device__ __forceinline__ void add_heads(const float (&pr)[32], float (&a_h)[8]) {
#pragma unroll
  for (int x = 0; x < 32; ++x) a_h[x % GG] += pr[x];
}

// What one CTA does in one phase (one KV head of one sequence).
struct PhaseWork {
  int b, g, row0, L, t0, n, nact, stat;
};

struct PhaseIter {
  int b, g;
};

// Every role of every CTA walks the same list of phases with the same arithmetic.
__device__ __forceinline__ bool next_phase(const FusedParams& p, PhaseIter& it, int cta, int ncta, PhaseWork& w) {
  if (it.b >= p.batch) return false;
  w.b = it.b;
  w.g = it.g;
  if (++it.g >= p.n_kv_heads) { it.g = 0; ++it.b; }
  w.row0 = p.cu_seqlens ? p.cu_seqlens[w.b] : 0;
  w.L = p.cu_seqlens ? p.cu_seqlens[w.b + 1] - w.row0 : p.total_len;
  w.stat = w.b * p.n_kv_heads + w.g;
  if (w.L < p.window) { w.t0 = 0; w.n = 0; w.nact = 0; return true; }
  const int ntiles = (w.L + kTileKeys - 1) / kTileKeys;
  const int per = (ntiles + ncta - 1) / ncta;
  w.nact = (ntiles + per - 1) / per;
  w.t0 = cta * per;
  w.n = max(0, min(per, ntiles - w.t0));
  return true;
}

}  // namespace

static_assert(ParkedCfg<128, 32>::kSmemBytes <= 232448 && ParkedCfg<128, 64>::kSmemBytes <= 232448 &&
              ParkedCfg<64, 32>::kSmemBytes <= 232448 && ParkedCfg<64, 64>::kSmemBytes <= 232448,
              "dynamic shared memory per CTA");

template <int D, int NPAD>
__global__ void __launch_bounds__(kParkedThreads, 1)
score_parked_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_q,
                    const FusedParams p) {
  using Cfg = ParkedCfg<D, NPAD>;
  constexpr int kStages = Cfg::kStages, kSlots = Cfg::kSlots;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* smem_k = smem;
  uint8_t* smem_q = smem_k + kStages * Cfg::kStageBytes;              // two buffers of kQBytes
  float* smem_ref = reinterpret_cast<float*>(smem_q + 2 * Cfg::kQBytes);   // [2][NPAD][128]: pass 1's references
  ParkedBarriers* bars = reinterpret_cast<ParkedBarriers*>(smem_q + 2 * Cfg::kQBytes + 2 * Cfg::kRefBytes);
  float2* warp_stats = reinterpret_cast<float2*>(reinterpret_cast<uint8_t*>(bars) + Cfg::kBarBytes);   // [2][4][NPAD]
  float2* norm = warp_stats + 2 * 4 * NPAD;                           // [NPAD] (-row max, 1 / row sum)
  float2* merge_buf = norm + NPAD;                                    // [256] partial merges
  int* row_j = reinterpret_cast<int*>(merge_buf + 2 * kPass2Threads); // [NPAD] window row j = n / G of query row n
  float2* collected = reinterpret_cast<float2*>(row_j + NPAD);        // [CTAs][NPAD] (16-byte aligned)
  constexpr int CPW = NPAD / 2;                                       // accumulator columns per pass-1 warp

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, ncta = gridDim.x;
  const long long limit = p.wait_limit;

  // A phase that does not fit in the slot ring could never complete: refuse before any barrier exists.
  if ((((p.max_len + kTileKeys - 1) / kTileKeys) + ncta - 1) / ncta > kSlots || ncta > kMaxCtas) {
    if (cta == 0 && threadIdx.x == 0) raise_status(p.hdr, FASTKV_ERR_UNSUPPORTED, SITE_PARKED_RING);
    return;
  }

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&bars->q_full[i], 1); mbar_init(&bars->q_empty[i], 1); }
    for (int i = 0; i < kSlots; ++i) {
      mbar_init(&bars->slot_full[i], 1);
      mbar_init(&bars->slot_free[i], kPass2Warps);   // every pass-2 warp reads its lane quarter of the slot
    }
    mbar_init(&bars->mma_done, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->ref_free[i], kPass2Warps);
      mbar_init(&bars->stats_ready[i], kPass1Warps);
      mbar_init(&bars->stats_free[i], 1);
    }
    mbar_init(&bars->coll_full, 1);
    mbar_init(&bars->coll_free, 1);
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tma_prefetch_desc(&tmap_k);
    tma_prefetch_desc(&tmap_q);
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, 512);
    tmem_relinquish();
  }
  if (threadIdx.x >= 64 && threadIdx.x < 64 + NPAD) row_j[threadIdx.x - 64] = (threadIdx.x - 64) / p.group;   // divide once
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;
  volatile int* abort_flag = &bars->abort_flag;
  pdl_launch_dependents();     // the pooling kernel may be brought up; it waits for this grid to finish

  if (warp == 0) {
    // ---------------- producer: K tiles (and the phase's query rows) by TMA ----------------
    if (lane == 0) {
      const uint64_t pol_k = l2_policy_evict_first();      // K is read exactly once
      const uint64_t pol_q = l2_policy_evict_last();
      int T = 0, u = 0, uq = 0;
      bool ok = true;
      PhaseIter pit = {0, 0};
      PhaseWork w;
      while (ok && next_phase(p, pit, cta, ncta, w)) {
        if (w.n == 0) continue;
        const int h = u & 1;
        if (u >= 2) ok = mbar_wait_bounded(&bars->q_empty[h], ((u >> 1) - 1) & 1, abort_flag, p.hdr, SITE_FUSED_Q_EMPTY, limit);
        if (!ok) break;
        const int q_row0 = (p.q_layout == FASTKV_Q_WINDOW) ? w.b * p.window : w.row0 + w.L - p.window;
        mbar_arrive_expect_tx(&bars->q_full[h], Cfg::KH * p.n_rows * 128);
        for (int c = 0; c < Cfg::KH; ++c)
          tma_load_3d(smem_q + h * Cfg::kQBytes + c * NPAD * 128, &tmap_q, &bars->q_full[h], c * 64, w.g * p.group,
                      q_row0, pol_q);
        ++uq;
        for (int i = 0; i < w.n; ++i, ++T) {
          const int s = T % kStages;
          ok = mbar_wait_bounded(&bars->empty[s], ((T / kStages) & 1) ^ 1, abort_flag, p.hdr, SITE_FUSED_EMPTY, limit);
          if (!ok) break;
          mbar_arrive_expect_tx(&bars->full[s], Cfg::kStageBytes);
          for (int c = 0; c < Cfg::KH; ++c)
            tma_load_3d(smem_k + s * Cfg::kStageBytes + c * kHalfBytes, &tmap_k, &bars->full[s], c * 64, w.g,
                        w.row0 + (w.t0 + i) * kTileKeys, pol_k);
        }
        ++u;
      }
      // No copy may still be writing this CTA's shared memory when the CTA ends: wait for the last
      // load of every stage and of every query buffer, whatever the abort flag says.
      for (int s = 0; s < kStages && s < T; ++s) {
        const int last = T - 1 - ((T - 1 - s) % kStages);           // last tile that used stage s
        mbar_wait_drain(&bars->full[s], (last / kStages) & 1, p.hdr, SITE_PARKED_DRAIN, limit);
      }
      for (int h = 0; h < 2 && h < uq; ++h) {
        const int last = uq - 1 - ((uq - 1 - h) & 1);
        mbar_wait_drain(&bars->q_full[h], (last >> 1) & 1, p.hdr, SITE_PARKED_DRAIN, limit);
      }
    }
  } else if (warp == 1) {
    // ---------------- issuer: one tcgen05.mma chain per tile into the next ring slot ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16_f32(kTileKeys, NPAD);
      int T = 0, u = 0;
      bool ok = true;
      PhaseIter pit = {0, 0};
      PhaseWork w;
      while (ok && next_phase(p, pit, cta, ncta, w)) {
        if (w.n == 0) continue;
        const int h = u & 1;
        ok = mbar_wait_bounded(&bars->q_full[h], (u >> 1) & 1, abort_flag, p.hdr, SITE_FUSED_Q_FULL, limit);
        if (!ok) break;
        const uint32_t q_addr = smem_u32(smem_q + h * Cfg::kQBytes);
        for (int i = 0; i < w.n; ++i, ++T) {
          const int s = T % kStages, a = T % kSlots;
          ok = mbar_wait_bounded(&bars->slot_free[a], ((T / kSlots) & 1) ^ 1, abort_flag, p.hdr, SITE_FUSED_ACC_FREE, limit) &&
               mbar_wait_bounded(&bars->full[s], (T / kStages) & 1, abort_flag, p.hdr, SITE_FUSED_FULL, limit);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t k_addr = smem_u32(smem_k + s * Cfg::kStageBytes);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint64_t adesc = umma_desc_k_sw128(k_addr + (kk >> 2) * kHalfBytes + (kk & 3) * 32);
            const uint64_t bdesc = umma_desc_k_sw128(q_addr + (kk >> 2) * NPAD * 128 + (kk & 3) * 32);
            tc_mma_bf16(tmem_base + a * NPAD, adesc, bdesc, idesc, kk > 0 ? 1u : 0u);
          }
          tc_commit(&bars->empty[s]);
          tc_commit(&bars->slot_full[a]);
        }
        if (ok) tc_commit(&bars->q_empty[h]);
        ++u;
      }
      // every contraction issued above has finished before tensor memory is released
      if (T > 0) {
        tc_commit(&bars->mma_done);
        mbar_wait_drain(&bars->mma_done, 0, p.hdr, SITE_PARKED_DRAIN, limit);
      }
    }
  } else if (warp == 2) {
    // ---------------- publisher: this CTA's row statistics of each finished phase go to global memory; ----------------
    // ---------------- collector: all CTAs' statistics of a complete phase come back into shared memory ----------------
    // Two walks over the phase list, `pw` for publication and `cw` for collection; whichever has something to
    // do goes first, so a publication never waits behind a collection and the other way round.
    int pu = 0, cu = 0;                                  // phases with tiles here: published / collected
    bool ok = true;
    PhaseIter pit = {0, 0}, cit = {0, 0};
    PhaseWork pw, cw;
    bool have_p = next_phase(p, pit, cta, ncta, pw), have_c = Cfg::kCollect && next_phase(p, cit, cta, ncta, cw);
    while (have_p && pw.n == 0) have_p = next_phase(p, pit, cta, ncta, pw);
    while (have_c && cw.n == 0) have_c = next_phase(p, cit, cta, ncta, cw);
    long long t0 = clock64();
    unsigned spins = 0;
    while (have_p || have_c) {
      bool progress = false;
      if (have_p) {
        const int buf = pu & 1;
        int ready = 1;
        if (ok && lane == 0) ready = mbar_try_wait(&bars->stats_ready[buf], (pu >> 1) & 1) ? 1 : 0;
        ready = __shfl_sync(0xffffffffu, ready, 0);
        if (ready) {                                     // (an aborted CTA publishes without waiting: nobody hangs on it)
          __syncwarp();
          const float2* ws = warp_stats + buf * 4 * NPAD;
#pragma unroll
          for (int n = lane; n < NPAD; n += 32) {        // lane quarters -> CTA
            float mm = -INFINITY, ll = 0.0f;
#pragma unroll
            for (int q = 0; q < 4; ++q) merge_stats(mm, ll, ws[q * NPAD + n].x, ws[q * NPAD + n].y);
            p.partial[(static_cast<size_t>(pw.stat) * ncta + cta) * NPAD + n] = make_float2(mm, ll);
          }
          __syncwarp();
          if (lane == 0) {
            red_release_add(p.counters + pw.stat, 1);    // release: cumulative over the warp's stores
            mbar_arrive(&bars->stats_free[buf]);
          }
          ++pu;
          do have_p = next_phase(p, pit, cta, ncta, pw); while (have_p && pw.n == 0);
          progress = true;
        }
      }
      if (have_c && !ok) have_c = false;                 // aborted: nothing more is collected
      if (have_c && cu < pu) {
        int ready = 0;
        if (lane == 0)                                   // the buffer is free again and every CTA has published?
          ready = (mbar_try_wait(&bars->coll_free, (cu & 1) ^ 1) &&
                   ld_acquire(p.counters + cw.stat) >= cw.nact + p.extra_publications) ? 1 : 0;
        ready = __shfl_sync(0xffffffffu, ready, 0);
        if (ready) {
          if (lane == 0) {
            // the other CTAs' stores (generic proxy, acquired above) are read by the copy engine
            asm volatile("fence.proxy.async;" ::: "memory");
            const uint32_t bytes = static_cast<uint32_t>(cw.nact) * NPAD * 8;
            mbar_arrive_expect_tx(&bars->coll_full, bytes);
            bulk_load(collected, p.partial + static_cast<size_t>(cw.stat) * ncta * NPAD, bytes, &bars->coll_full);
          }
          ++cu;
          do have_c = next_phase(p, cit, cta, ncta, cw); while (have_c && cw.n == 0);
          progress = true;
        }
      }
      if (progress) {
        t0 = clock64();
        spins = 0;
      } else if ((++spins & 0x3Fu) == 0 && ok) {
        int give_up = 0;
        if (lane == 0) {
          if (*abort_flag) give_up = 1;
          else if (clock64() - t0 > limit) {
            *abort_flag = 1;
            raise_status(p.hdr, FASTKV_ERR_DEVICE_TIMEOUT, have_c && cu < pu ? SITE_FUSED_FLAG : SITE_PARKED_STATS);
            give_up = 1;
          }
        }
        if (__shfl_sync(0xffffffffu, give_up, 0)) ok = false;
      }
    }
    // the last collection issued has landed before the CTA ends, whether pass 2 consumed it or not
    if (lane == 0 && cu > 0) mbar_wait_drain(&bars->coll_full, (cu - 1) & 1, p.hdr, SITE_PARKED_DRAIN, limit);
  } else if (warp < kCtrlWarps + kPass1Warps) {
    // ---------------- pass 1: logits -> e = exp2(s - ref), row sums ----------------
    // warp (quarter, half) owns tensor-memory lanes 32 * quarter .. +31 (one key per lane) and the
    // accumulator columns (query rows) half * CPW .. +CPW-1.
    const int gw = warp - kCtrlWarps;
    const int quarter = warp & 3, half = gw >> 2;
    const int key_in_tile = quarter * 32 + lane;
    const int n_rows = p.n_rows;
    const int col0 = half * CPW;
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + col0;
    int T = 0, u = 0;
    bool ok = true;
    PhaseIter pit = {0, 0};
    PhaseWork w;
    while (next_phase(p, pit, cta, ncta, w)) {
      if (w.n == 0) {
        // a sequence shorter than the observation window has no defined scores: say so once
        if (w.L < p.window && cta == 0 && gw == 0 && lane == 0)
          raise_status(p.hdr, FASTKV_ERR_INVALID_ARG, SITE_SCORE_SHORT_SEQUENCE);
        continue;
      }
      float m[CPW], l[CPW];                              // this thread's reference and sum of e per query row
#pragma unroll
      for (int n = 0; n < CPW; ++n) { m[n] = -INFINITY; l[n] = 0.0f; }
      const int win_start = w.L - p.window;
      const int T0 = T;                                  // first tile of the phase
      for (int i = 0; i < w.n; ++i, ++T) {
        const int a = T % kSlots;
        if (ok) ok = mbar_wait_bounded(&bars->slot_full[a], (T / kSlots) & 1, abort_flag, p.hdr, SITE_FUSED_ACC_FULL, limit);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) continue;                               // aborted: run through the loops without work
        tc_fence_after_sync();
        const int key = (w.t0 + i) * kTileKeys + key_in_tile;
        const bool tile_unmasked = (w.t0 + i + 1) * kTileKeys <= win_start;
#pragma unroll
        for (int c = 0; c < CPW / 16; ++c) {
          float v[16];
          tmem_ld_32x16(lane_base + a * NPAD + c * 16, v);
          const int n_valid = n_rows - col0 - c * 16;
          float* const mc = m + c * 16;
          float* const lc = l + c * 16;
          bool general = !tile_unmasked || i == 0;
          if (!general) {
            // common case: no logit is far above its reference, one exp2 per logit and nothing else
            float x[16];
            bool far = false;
#pragma unroll
            for (int r = 0; r < 16; ++r) {
              x[r] = fmaf(v[r], p.scale_log2, -mc[r]);
              far |= (r < n_valid) && (x[r] > kRefSlackLog2);
            }
            general = __any_sync(0xffffffffu, far);
            if (!general) {
#pragma unroll
              for (int r = 0; r < 16; ++r) {
                const float e = (r < n_valid) ? ex2(x[r]) : 0.0f;
                lc[r] += e;
                v[r] = e;
              }
            }
          }
          if (general) {
            // first tile of the phase, a tile that overlaps the observation window (causal mask), or a
            // logit far above its reference: per row, start / keep / move the reference
            uint32_t visible = 0xFFFFu;
            if (!tile_unmasked) {
              visible = 0;
              if (key < w.L) {
#pragma unroll
                for (int r = 0; r < 16; ++r)
                  if (r < n_valid && key <= win_start + row_j[col0 + c * 16 + r]) visible |= 1u << r;
              }
            }
            float fac[16];
            bool moved = false;
#pragma unroll
            for (int r = 0; r < 16; ++r) {
              fac[r] = 1.0f;
              if (r >= n_valid || !((visible >> r) & 1u)) { v[r] = 0.0f; continue; }
              const float sl = v[r] * p.scale_log2;
              if (mc[r] == -INFINITY) {                  // first logit of the row: it becomes the reference
                mc[r] = sl; lc[r] = 1.0f; v[r] = 1.0f;
              } else {
                const float x = sl - mc[r];
                if (x > kRefSlackLog2) {                 // move the reference up to this logit
                  fac[r] = ex2(-x);
                  lc[r] = lc[r] * fac[r] + 1.0f;
                  mc[r] = sl; v[r] = 1.0f;
                  moved = true;
                } else {
                  const float e = ex2(x);
                  lc[r] += e;
                  v[r] = e;
                }
              }
            }
            if (__any_sync(0xffffffffu, moved)) {        // rescale what this warp parked earlier in the phase
              tmem_wait_st();
              for (int Tp = T0; Tp < T; ++Tp) {
                float old[16];
                const uint32_t addr = lane_base + (Tp % kSlots) * NPAD + c * 16;
                tmem_ld_32x16(addr, old);
#pragma unroll
                for (int r = 0; r < 16; ++r) old[r] *= fac[r];
                tmem_st_32x16(addr, old);
              }
            }
          }
          tmem_st_32x16(lane_base + a * NPAD + c * 16, v);
        }
      }
      // this thread's references go to pass 2, the warp's (max, sum) per row to the statistics group, as
      // soon as they are done with the buffers of the phase before last
      const int buf = u & 1;
      if (ok && u >= 2)
        ok = mbar_wait_bounded(&bars->ref_free[buf], ((u >> 1) - 1) & 1, abort_flag, p.hdr, SITE_PARKED_REF, limit) &&
             mbar_wait_bounded(&bars->stats_free[buf], ((u >> 1) - 1) & 1, abort_flag, p.hdr, SITE_PARKED_STATS, limit);
      float* const ref_out = smem_ref + (buf * NPAD + col0) * kTileKeys + key_in_tile;
#pragma unroll
      for (int n = 0; n < CPW; ++n) ref_out[n * kTileKeys] = m[n];
      // lanes -> warp: after the butterfly lanes r and r + 16 hold row col0 + c * 16 + r in entry c * 16
#pragma unroll
      for (int c = 0; c < CPW / 16; ++c) {
        stats_transpose_merge<16>(m + c * 16, l + c * 16, lane);
        if (lane < 16) warp_stats[(buf * 4 + quarter) * NPAD + col0 + c * 16 + lane] = make_float2(m[c * 16], l[c * 16]);
      }
      tmem_wait_st();                                    // the parked e are read by pass 2 once the statistics are merged
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->stats_ready[buf]);
      ++u;
    }
  } else {
    // ---------------- pass 2: merge the statistics, weight the parked e, sum over window rows / group ----------------
    // One warp per tensor-memory lane quarter; a warp handles all query rows of its 32 keys.
    const int quarter = warp & 3;
    const int key_in_tile = quarter * 32 + lane;
    const int pt = threadIdx.x - (kCtrlWarps + kPass1Warps) * 32;    // 0..127 within the group
    const int n_rows = p.n_rows, G = p.group;
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    constexpr int kTPL = NPAD / 2;                       // threads per CTA's line of statistics: two rows each
    constexpr int kParts = kPass2Threads / kTPL;
    int T = 0, u = 0;
    bool ok = true;
    PhaseIter pit = {0, 0};
    PhaseWork w;
    while (next_phase(p, pit, cta, ncta, w)) {           // an aborted CTA still walks every phase: see pass2_sync
      if (w.n == 0) continue;
      const int buf = u & 1;
      if (Cfg::kCollect) {
        // all CTAs' statistics of the phase are in shared memory (the publisher warp saw to it)
        // (twice the limit: a publication that never comes is reported by the collector, which watches for it)
        if (ok) ok = mbar_wait_bounded(&bars->coll_full, u & 1, abort_flag, p.hdr, SITE_PARKED_NORM, 2 * limit);
        const int n2 = 2 * (pt % kTPL), part = pt / kTPL;
        float2 r0, r1;
        merge_collected_2rows(collected, NPAD, n2, part, kParts, w.nact, r0, r1);
        merge_buf[part * NPAD + n2] = r0;
        merge_buf[part * NPAD + n2 + 1] = r1;
      } else {
        // every CTA that owns tiles of this phase has published its statistics?
        if (pt == 0 && !*abort_flag) {
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
        pass2_sync();
        // the softmax normaliser of the phase, merged in a fixed order (the same in every CTA)
        const int n2 = 2 * (pt % kTPL), part = pt / kTPL;
        float2 r0, r1;
        merge_partials_2rows(p.partial + static_cast<size_t>(w.stat) * ncta * NPAD, NPAD, n2, part, kParts, w.nact, r0, r1);
        merge_buf[part * NPAD + n2] = r0;
        merge_buf[part * NPAD + n2 + 1] = r1;
      }
      pass2_sync();
      if (*abort_flag) ok = false;
      if (Cfg::kCollect && pt == 0) mbar_arrive(&bars->coll_free);   // the buffer may take the next phase
      if (pt < NPAD) {
        float mm = -INFINITY, ll = 0.0f;
#pragma unroll
        for (int q = 0; q < kParts; ++q) merge_stats(mm, ll, merge_buf[q * NPAD + pt].x, merge_buf[q * NPAD + pt].y);
        // (-row max, 1 / row sum); rows beyond G * w contribute nothing
        norm[pt] = (pt < n_rows && ll > 0.0f) ? make_float2(-mm, 1.0f / ll) : make_float2(0.0f, 0.0f);
      }
      pass2_sync();
      tc_fence_after_sync();
      // one weight per query row for this thread's key lane: f = exp2(ref - M) / l (ref = -inf: nothing parked)
      float* const ref_in = smem_ref + (buf * NPAD) * kTileKeys + key_in_tile;
      float f[NPAD == 32 ? 32 : 1];
      if (NPAD == 32) {
#pragma unroll
        for (int r = 0; r < 32; ++r) {
          const float2 st = norm[r];
          f[r] = ex2(ref_in[r * kTileKeys] + st.x) * st.y;
        }
      } else {                                           // many rows: the weights replace this thread's references
        for (int r = 0; r < NPAD; ++r) {
          const float2 st = norm[r];
          ref_in[r * kTileKeys] = ex2(ref_in[r * kTileKeys] + st.x) * st.y;
        }
      }
      for (int i = 0; i < w.n; ++i, ++T) {
        const int a = T % kSlots;
        if (ok) ok = mbar_wait_bounded(&bars->slot_full[a], (T / kSlots) & 1, abort_flag, p.hdr, SITE_FUSED_ACC_FULL, limit);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) continue;
        tc_fence_after_sync();
        const int key = (w.t0 + i) * kTileKeys + key_in_tile;
        float a_g = 0.0f;
        float a_h[8];                                    // per query head of the group (G in {1,2,4,8})
#pragma unroll
        for (int q = 0; q < 8; ++q) a_h[q] = 0.0f;
#pragma unroll
        for (int c = 0; c < NPAD / 32; ++c) {
          float pr[32];
          tmem_ld_32x32(lane_base + a * NPAD + c * 32, pr);
          if (c == NPAD / 32 - 1) {                      // the slot is in registers: hand it back to the issuer
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->slot_free[a]);
          }
#pragma unroll
          for (int x = 0; x < 32; ++x)
            pr[x] *= (NPAD == 32) ? f[x % (NPAD == 32 ? 32 : 1)] : ref_in[(c * 32 + x) * kTileKeys];
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
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->ref_free[buf]);  // pass 1 may overwrite this phase's references
      pass2_sync();                                      // norm / merge_buf are rewritten next phase
      ++u;
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------

int parked_slots(int npad) { return 512 / npad; }

template <int D, int NPAD>
static cudaError_t launch_parked_t(const CUtensorMap& tk, const CUtensorMap& tq, const FusedParams& p, int grid,
                                   cudaStream_t stream) {
  using Cfg = ParkedCfg<D, NPAD>;
  static PerDeviceOnce configured;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (!configured.done(dev)) {
    e = cudaFuncSetAttribute(score_parked_kernel<D, NPAD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Cfg::kSmemBytes);
    if (e != cudaSuccess) return e;
    configured.set(dev);
  }
  void* args[] = {const_cast<CUtensorMap*>(&tk), const_cast<CUtensorMap*>(&tq), const_cast<FusedParams*>(&p)};
  return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(score_parked_kernel<D, NPAD>), dim3(grid),
                                     dim3(kParkedThreads), args, Cfg::kSmemBytes, stream);
}

cudaError_t launch_score_parked(int head_dim, int npad, const CUtensorMap& tk, const CUtensorMap& tq,
                                const FusedParams& p, int grid, cudaStream_t stream) {
  if (head_dim == 128 && npad == 32) return launch_parked_t<128, 32>(tk, tq, p, grid, stream);
  if (head_dim == 128 && npad == 64) return launch_parked_t<128, 64>(tk, tq, p, grid, stream);
  if (head_dim == 64 && npad == 32) return launch_parked_t<64, 32>(tk, tq, p, grid, stream);
  if (head_dim == 64 && npad == 64) return launch_parked_t<64, 64>(tk, tq, p, grid, stream);
  return cudaErrorInvalidValue;
}

}  // namespace fastkv
