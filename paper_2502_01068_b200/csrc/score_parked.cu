// Window-query saliency scoring with one pass over K and one contraction per key tile (Eq. 1 inner
// term; Sec. 4.2): the logits of a tile stay parked in tensor memory until the softmax statistics
// of their row are known, then they are normalised and summed in place.
//
// One persistent CTA per SM (cooperative launch: every CTA is resident).  The work is cut into
// phases, one per (sequence, KV head); in every phase CTA c owns the same run of consecutive
// 128-key tiles of the sequence.  Either the whole grid walks the phases one after the other, or
// (partition mode: batches, short sequences) several phases run side by side, each on its own share
// of the CTAs.  Per CTA:
//
//   producer   one thread streams the K tiles (and the G*w window-query rows of the phase) into a
//              ring of shared-memory stages with TMA;
//   issuer     one thread forms S^T = K_tile . Q_g^T with tcgen05.mma (M = 128 keys, N = query
//              rows, fp32) into the next slot of a ring that covers all of tensor memory
//              (16 slots of 32 columns, or 8 of 64); a slot is not recycled by the issuer, it is
//              handed back by pass 2;
//   pass 1     (eight warps, one key per lane) reads each new slot, turns every logit into
//              e = exp2(s - ref) against the warp's reference for that query row, adds e to the
//              thread's running sum of the row and writes e back over the logit; at the
//              end of the phase the warp's references and its (reference, sum) per row go to shared
//              memory.  The reference of a row is the largest logit of the warp's first tile; it
//              moves (and the e already parked for this phase are rescaled) only if a logit exceeds
//              it by more than 64 binary orders of magnitude;
//   publisher  (one warp) writes the CTA's (max, sum) per row of a finished phase to global memory and
//              bumps the phase's counter, so that publication never waits behind anything else;
//   pass 2     (four warps, one per tensor-memory lane quarter) waits until every CTA of the phase
//              has published, merges the statistics in a fixed order (identical in every CTA:
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
constexpr int kRefBufs = 4;                    // phases whose references may be waiting for pass 2
constexpr int kMaxPartUnits = 512;             // (sequence, KV head) pairs a partitioned launch may have (waves <= units)
// Pass 1 keeps e = exp2(s - ref) with the row's first logit as the reference; the reference only moves
// when a logit exceeds it by more than this many binary orders of magnitude (e and its row sums stay far
// inside the fp32 range: e <= 2^64, at most 2^20-odd terms per sum).
constexpr float kRefSlackLog2 = 64.0f;

template <int D, int NPAD>
struct ParkedCfg {
  static constexpr int KH = D / 64;
  static constexpr int kStageBytes = KH * kHalfBytes;
  static constexpr int kQBytes = KH * NPAD * 128;
  static constexpr int kStages = (D == 128) ? 5 : 8;
  static constexpr int kSlots = 512 / NPAD;                 // tensor memory: 512 columns
  static constexpr int kBarBytes = 1024;
  static constexpr int kRefBytes = kRefBufs * 4 * NPAD * 4; // one reference per (phase in flight, lane quarter, query row)
  static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + 2 * kQBytes + kRefBytes + kBarBytes +
                                    2 * 4 * NPAD * 8 /*warp_stats*/ + NPAD * 8 /*norm*/ +
                                    2 * kPass2Threads * 8 /*merge_buf*/ + NPAD * 4 /*row_j*/ + (kMaxPartUnits + 1) * 20 /*part_tab*/;
};

struct ParkedBarriers {
  uint64_t full[kMaxStages], empty[kMaxStages];
  uint64_t q_full[2], q_empty[2];
  uint64_t slot_full[kMaxSlots], slot_free[kMaxSlots];
  uint64_t mma_done;
  uint64_t ref_free[kRefBufs]; // pass 2 has finished with the references of a phase
  uint64_t stats_ready[2];     // pass 1 has written its warps' statistics of a phase
  uint64_t stats_free[2];      // ... and the publisher has read them
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

// Sums of sixteen values per lane over the 32 lanes of a warp: fifteen exchanges that halve the rows a
// lane holds, then one between lanes r and r + 16; afterwards both hold the sum of row r in v[0].
__device__ __forceinline__ void transpose_sum16(float* v, int lane) {
#pragma unroll
  for (int o = 8; o >= 1; o >>= 1) {
    const bool upper = (lane & o) != 0;
#pragma unroll
    for (int i = 0; i < o; ++i) {
      const float send = upper ? v[i] : v[i + o];
      const float keep = upper ? v[i + o] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
    }
  }
  v[0] += __shfl_xor_sync(0xffffffffu, v[0], 16);
}

template <int GG>
__device__ __forceinline__ void add_heads(const float (&pr)[32], float (&a_h)[8]) {
#pragma unroll
  for (int x = 0; x < 32; ++x) a_h[x % GG] += pr[x];
}

// What one CTA does in one phase (one KV head of one sequence).
struct PhaseWork {
  int b, g, row0, L, t0, n, nact, stat;
  int slot;        // this CTA's number among the CTAs that share the phase: where its statistics go
};

struct PhaseIter {
  int b, g;
};

// Partition mode.  Units of work -- a whole sequence (all its KV heads, one after the other: p.partition == 1,
// batches) or one KV head of a sequence (p.partition == 2, a single sequence of middling length) -- are taken
// in waves of consecutive units; within a wave the CTAs of the grid are dealt out to the wave's units in
// proportion to their length: this CTA is number `cta` of the `ncta` that share the unit and sees no other
// unit of the wave.  The units of a wave are scored side by side, every CTA has tiles in every phase, and a
// statistics exchange involves only the CTAs of one unit.  That is what batches and shorter sequences want (a
// grid-wide phase per head would cost sequences x heads exchanges, or leave most CTAs without a tile); a
// single long sequence is better off with the whole grid on one head at a time and two phases in the ring.
// One entry per wave, worked out once per CTA and kept in shared memory.
struct PartEntry {
  int b, g;        // the CTA's unit in this wave (g < 0: every head of b in turn); b == kPartIdle: none; kPartEnd: no more waves
  int cta, ncta;   // its number among the CTAs of that unit, and how many they are
  int per;         // tiles per CTA the deal came out at (at most the ring)
};
constexpr int kPartIdle = -2, kPartEnd = -3;

__device__ __forceinline__ int seq_tiles(const FusedParams& p, int b) {
  const int row0 = p.cu_seqlens ? p.cu_seqlens[b] : 0;
  const int L = p.cu_seqlens ? p.cu_seqlens[b + 1] - row0 : p.total_len;
  return L < p.window ? 0 : (L + kTileKeys - 1) / kTileKeys;       // a sequence shorter than the window has no scores
}

// The same arithmetic in every CTA.  Waves are filled greedily: a unit joins the wave while the wave's
// units still fit the grid at `ring` tiles per CTA (one unit always does: the host checked the longest
// sequence); inside a wave the smallest number of tiles per CTA that fits is used.  Run by one thread.
__device__ void fill_part_table(const FusedParams& p, int cta, int ncta, int ring, PartEntry* tab) {
  const int H = p.partition == 2 ? p.n_kv_heads : 1, units = p.batch * H;
  int u0 = 0, r = 0;
  while (u0 < units) {
    int u1 = u0, need = 0, total = 0;
    while (u1 < units) {
      const int t = seq_tiles(p, u1 / H), n = (t + ring - 1) / ring;
      if (u1 > u0 && need + n > ncta) break;
      need += n;
      total += t;
      ++u1;
    }
    int per = max(1, (total + ncta - 1) / ncta);
    while (true) {
      int n = 0;
      for (int u = u0; u < u1; ++u) n += (seq_tiles(p, u / H) + per - 1) / per;
      if (n <= ncta) break;
      ++per;
    }
    PartEntry e = {kPartIdle, 0, 0, 0, per};                          // a CTA left over in this wave
    int first = 0;
    for (int u = u0; u < u1; ++u) {
      const int n = (seq_tiles(p, u / H) + per - 1) / per;
      if (cta >= first && cta < first + n) e = {u / H, p.partition == 2 ? u % H : -1, cta - first, n, per};
      first += n;
    }
    tab[r++] = e;
    u0 = u1;
  }
  tab[r] = {kPartEnd, 0, 0, 0, 0};
}

// Every role of every CTA walks the same list of phases with the same arithmetic.
template <bool PART>
__device__ __forceinline__ bool next_phase(const FusedParams& p, PhaseIter& it, int cta, int ncta, const PartEntry* tab,
                                           PhaseWork& w) {
  int per_fixed = 0;
  if (PART) {                                              // this CTA's unit of the wave: one head, or all heads in turn
    PartEntry e = tab[it.b];                               // (it.b counts waves here)
    while (e.b == kPartIdle || (e.b >= 0 && it.g >= (e.g < 0 ? p.n_kv_heads : 1))) {
      e = tab[++it.b];
      it.g = 0;
    }
    if (e.b == kPartEnd) return false;
    w.b = e.b;
    w.g = e.g < 0 ? it.g : e.g;
    ++it.g;
    cta = e.cta;
    ncta = e.ncta;
    per_fixed = e.per;
  } else {
    if (it.b >= p.batch) return false;
    w.b = it.b;
    w.g = it.g;
    if (++it.g >= p.n_kv_heads) { it.g = 0; ++it.b; }
  }
  if (PART) w.slot = cta;
  w.row0 = p.cu_seqlens ? p.cu_seqlens[w.b] : 0;
  w.L = p.cu_seqlens ? p.cu_seqlens[w.b + 1] - w.row0 : p.total_len;
  w.stat = w.b * p.n_kv_heads + w.g;
  if (w.L < p.window) { w.t0 = 0; w.n = 0; w.nact = 0; return true; }
  const int ntiles = (w.L + kTileKeys - 1) / kTileKeys;
  const int per = per_fixed > 0 ? per_fixed : (ntiles + ncta - 1) / ncta;
  w.nact = (ntiles + per - 1) / per;
  w.t0 = cta * per;
  w.n = max(0, min(per, ntiles - w.t0));
  return true;
}

}  // namespace

static_assert(ParkedCfg<128, 32>::kSmemBytes <= 232448 && ParkedCfg<128, 64>::kSmemBytes <= 232448 &&
              ParkedCfg<64, 32>::kSmemBytes <= 232448 && ParkedCfg<64, 64>::kSmemBytes <= 232448,
              "dynamic shared memory per CTA");

template <int D, int NPAD, bool PART>
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
  float* smem_ref = reinterpret_cast<float*>(smem_q + 2 * Cfg::kQBytes);   // [kRefBufs][4][NPAD]: pass 1's references
  ParkedBarriers* bars = reinterpret_cast<ParkedBarriers*>(reinterpret_cast<uint8_t*>(smem_ref) + Cfg::kRefBytes);
  float2* warp_stats = reinterpret_cast<float2*>(reinterpret_cast<uint8_t*>(bars) + Cfg::kBarBytes);   // [2][4][NPAD]
  float2* norm = warp_stats + 2 * 4 * NPAD;                           // [NPAD] (-row max, 1 / row sum)
  float2* merge_buf = norm + NPAD;                                    // [256] partial merges
  int* row_j = reinterpret_cast<int*>(merge_buf + 2 * kPass2Threads); // [NPAD] window row j = n / G of query row n
  PartEntry* part_tab = reinterpret_cast<PartEntry*>(row_j + NPAD);   // [waves + 1], partition mode only
  constexpr int CPW = NPAD / 2;                                       // accumulator columns per pass-1 warp

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, ncta = gridDim.x;
  const long long limit = p.wait_limit;

  if (PART && cta == 0 && threadIdx.x == 0) {
    // a sequence shorter than the observation window has no defined scores (and no CTA): say so once
    for (int b = 0; b < p.batch; ++b)
      if (seq_tiles(p, b) == 0) raise_status(p.hdr, FASTKV_ERR_INVALID_ARG, SITE_SCORE_SHORT_SEQUENCE);
  }
  // A phase that does not fit in the slot ring could never complete: refuse before any barrier exists.
  if ((((p.max_len + kTileKeys - 1) / kTileKeys) + ncta - 1) / ncta > kSlots) {
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
    for (int i = 0; i < kRefBufs; ++i) mbar_init(&bars->ref_free[i], kPass2Warps);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->stats_ready[i], kPass1Warps);
      mbar_init(&bars->stats_free[i], 1);
    }
    bars->abort_flag = 0;
    if (PART) fill_part_table(p, cta, ncta, kSlots, part_tab);
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
  // Everything above overlapped the end of the kernel before this one in the stream (the launch allows it);
  // from here on global memory is read and written: K and Q, the counters the clearing kernel zeroed, and
  // the un-pooled scores the previous call's pooling kernel may still be reading.
  pdl_wait();

  if (warp == 0) {
    // ---------------- producer: K tiles (and the phase's query rows) by TMA ----------------
    // (the producer and the issuer wait with a poll every ~50 ns: a hot polling loop takes issue slots from the
    //  pass-1 warps on their schedulers)
    if (lane == 0) {
      const uint64_t pol_k = l2_policy_evict_first();      // K is read exactly once
      const uint64_t pol_q = l2_policy_evict_last();
      int T = 0, u = 0, uq = 0;
      bool ok = true;
      PhaseIter pit = {0, 0};
      PhaseWork w;
      while (ok && next_phase<PART>(p, pit, cta, ncta, part_tab, w)) {
        if (w.n == 0) continue;
        const int h = u & 1;
        if (u >= 2) ok = mbar_wait_nap(&bars->q_empty[h], ((u >> 1) - 1) & 1, abort_flag, p.hdr, SITE_FUSED_Q_EMPTY, limit);
        if (!ok) break;
        const int q_row0 = (p.q_layout == FASTKV_Q_WINDOW) ? w.b * p.window : w.row0 + w.L - p.window;
        mbar_arrive_expect_tx(&bars->q_full[h], Cfg::KH * p.n_rows * 128);
        for (int c = 0; c < Cfg::KH; ++c)
          tma_load_3d(smem_q + h * Cfg::kQBytes + c * NPAD * 128, &tmap_q, &bars->q_full[h], c * 64, w.g * p.group,
                      q_row0, pol_q);
        ++uq;
        for (int i = 0; i < w.n; ++i, ++T) {
          const int s = T % kStages;
          ok = mbar_wait_nap(&bars->empty[s], ((T / kStages) & 1) ^ 1, abort_flag, p.hdr, SITE_FUSED_EMPTY, limit);
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
      while (ok && next_phase<PART>(p, pit, cta, ncta, part_tab, w)) {
        if (w.n == 0) continue;
        const int h = u & 1;
        ok = mbar_wait_nap(&bars->q_full[h], (u >> 1) & 1, abort_flag, p.hdr, SITE_FUSED_Q_FULL, limit);
        if (!ok) break;
        const uint32_t q_addr = smem_u32(smem_q + h * Cfg::kQBytes);
        for (int i = 0; i < w.n; ++i, ++T) {
          const int s = T % kStages, a = T % kSlots;
          ok = mbar_wait_nap(&bars->slot_free[a], ((T / kSlots) & 1) ^ 1, abort_flag, p.hdr, SITE_FUSED_ACC_FREE, limit) &&
               mbar_wait_nap(&bars->full[s], (T / kStages) & 1, abort_flag, p.hdr, SITE_FUSED_FULL, limit);
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
    // ---------------- publisher: this CTA's row statistics of each finished phase go to global memory ----------------
    int u = 0;
    bool ok = true;
    PhaseIter pit = {0, 0};
    PhaseWork w;
    while (next_phase<PART>(p, pit, cta, ncta, part_tab, w)) {
      if (w.n == 0) continue;
      const int buf = u & 1;
      if (ok) ok = mbar_wait_bounded(&bars->stats_ready[buf], (u >> 1) & 1, abort_flag, p.hdr, SITE_PARKED_STATS, limit);
      ok = __all_sync(0xffffffffu, ok);
      const float2* ws = warp_stats + buf * 4 * NPAD;
#pragma unroll
      for (int n = lane; n < NPAD; n += 32) {            // lane quarters -> CTA
        float mm = -INFINITY, ll = 0.0f;
#pragma unroll
        for (int q = 0; q < 4; ++q) merge_stats(mm, ll, ws[q * NPAD + n].x, ws[q * NPAD + n].y);
        p.partial[(static_cast<size_t>(w.stat) * ncta + (PART ? w.slot : cta)) * NPAD + n] = make_float2(mm, ll);
      }
      __syncwarp();
      if (lane == 0) {
        red_release_add(p.counters + w.stat, 1);         // release: cumulative over the warp's stores
        mbar_arrive(&bars->stats_free[buf]);
      }
      ++u;
    }
  } else if (warp < kCtrlWarps + kPass1Warps) {
    // ---------------- pass 1: logits -> e = exp2(s - ref), row sums ----------------
    // warp (quarter, half) owns tensor-memory lanes 32 * quarter .. +31 (one key per lane) and the
    // accumulator columns (query rows) half * CPW .. +CPW-1.  The reference m[] of a row is the same in
    // all lanes of the warp; the sums l[] are the thread's own.
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
    while (next_phase<PART>(p, pit, cta, ncta, part_tab, w)) {
      if (w.n == 0) {
        // a sequence shorter than the observation window has no defined scores: say so once
        if (w.L < p.window && cta == 0 && gw == 0 && lane == 0)
          raise_status(p.hdr, FASTKV_ERR_INVALID_ARG, SITE_SCORE_SHORT_SEQUENCE);
        continue;
      }
      float m[CPW], l[CPW];                              // the warp's reference and this thread's sum of e per query row
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
          bool general = !tile_unmasked;
          if (!general && i == 0) {
            // first tile of the phase, every key visible: lane 0's logit starts the row's reference
#pragma unroll
            for (int r = 0; r < 16; ++r) {
              const float first = __shfl_sync(0xffffffffu, v[r] * p.scale_log2, 0);
              if (r < n_valid) mc[r] = first;
            }
          }
          if (!general && n_valid >= 16) {
            // common case: every row in use, no logit far above its reference: one multiply-add, one exp2
            // and one add per logit, and a maximum to find out
            float x[16];
#pragma unroll
            for (int r = 0; r < 16; ++r) x[r] = fmaf(v[r], p.scale_log2, -mc[r]);
            const float top = fmaxf(fmaxf(fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3])), fmaxf(fmaxf(x[4], x[5]), fmaxf(x[6], x[7]))),
                                    fmaxf(fmaxf(fmaxf(x[8], x[9]), fmaxf(x[10], x[11])), fmaxf(fmaxf(x[12], x[13]), fmaxf(x[14], x[15]))));
            general = __any_sync(0xffffffffu, top > kRefSlackLog2);
            if (!general) {
#pragma unroll
              for (int r = 0; r < 16; ++r) {
                const float e = ex2(x[r]);
                lc[r] += e;
                v[r] = e;
              }
            }
          } else if (!general) {
            // the same with unused (padding) rows among the sixteen
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
            // a tile that overlaps the observation window (causal mask), or a logit far above its reference:
            // per row, start / keep / move the warp's reference
            uint32_t visible = 0xFFFFu;
            if (!tile_unmasked) {
              visible = 0;
              if (key < w.L) {
#pragma unroll
                for (int r = 0; r < 16; ++r)
                  if (r < n_valid && key <= win_start + row_j[col0 + c * 16 + r]) visible |= 1u << r;
              }
            }
            float sl[16], xm[16];
#pragma unroll
            for (int r = 0; r < 16; ++r) {
              sl[r] = (r < n_valid && ((visible >> r) & 1u)) ? v[r] * p.scale_log2 : -INFINITY;
              xm[r] = sl[r];
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) {
#pragma unroll
              for (int r = 0; r < 16; ++r) xm[r] = fmaxf(xm[r], __shfl_xor_sync(0xffffffffu, xm[r], off));
            }
            float fac[16];
            bool moved = false;                          // the same in every lane: xm and mc are
#pragma unroll
            for (int r = 0; r < 16; ++r) {
              fac[r] = 1.0f;
              if (xm[r] == -INFINITY) { v[r] = 0.0f; continue; }     // nothing of this row is visible to the warp here
              if (mc[r] == -INFINITY) {
                mc[r] = xm[r];                           // first logits of the row: the largest becomes the reference
              } else if (xm[r] - mc[r] > kRefSlackLog2) {            // move the reference up
                fac[r] = ex2(mc[r] - xm[r]);
                lc[r] *= fac[r];
                mc[r] = xm[r];
                moved = true;
              }
              const float e = ex2(sl[r] - mc[r]);        // exp2(-inf) = 0 for a masked key
              lc[r] += e;
              v[r] = e;
            }
            if (moved) {                                 // rescale what this warp parked earlier in the phase
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
      // the warp's references go to pass 2, its (reference, sum) per row to the publisher, as soon as
      // they are done with the buffers of earlier phases
      const int buf = u & 1, rbuf = u % kRefBufs;
      if (ok && u >= kRefBufs)
        ok = mbar_wait_bounded(&bars->ref_free[rbuf], ((u / kRefBufs) - 1) & 1, abort_flag, p.hdr, SITE_PARKED_REF, limit);
      if (ok && u >= 2)
        ok = mbar_wait_bounded(&bars->stats_free[buf], ((u >> 1) - 1) & 1, abort_flag, p.hdr, SITE_PARKED_STATS, limit);
      float* const ref_out = smem_ref + (rbuf * 4 + quarter) * NPAD + col0;
      if (lane == 0) {
#pragma unroll
        for (int n = 0; n < CPW; ++n) ref_out[n] = m[n];
      }
      __syncwarp();
      // lanes -> warp: the reference of a row is the same in all lanes, so its sums just add up; after
      // the butterfly lanes r and r + 16 hold the sum of row col0 + c * 16 + r in entry c * 16
#pragma unroll
      for (int c = 0; c < CPW / 16; ++c) {
        transpose_sum16(l + c * 16, lane);
        if (lane < 16)
          warp_stats[(buf * 4 + quarter) * NPAD + col0 + c * 16 + lane] = make_float2(ref_out[c * 16 + lane], l[c * 16]);
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
    while (next_phase<PART>(p, pit, cta, ncta, part_tab, w)) {           // an aborted CTA still walks every phase: see pass2_sync
      if (w.n == 0) continue;
      const int rbuf = u % kRefBufs;
      {
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
      if (pt < NPAD) {
        float mm = -INFINITY, ll = 0.0f;
#pragma unroll
        for (int q = 0; q < kParts; ++q) merge_stats(mm, ll, merge_buf[q * NPAD + pt].x, merge_buf[q * NPAD + pt].y);
        // (-row max, 1 / row sum); rows beyond G * w contribute nothing
        norm[pt] = (pt < n_rows && ll > 0.0f) ? make_float2(-mm, 1.0f / ll) : make_float2(0.0f, 0.0f);
      }
      pass2_sync();
      tc_fence_after_sync();
      // one weight per query row for this warp's keys: f = exp2(ref - M) / l (ref = -inf: nothing parked)
      float* const ref_in = smem_ref + (rbuf * 4 + quarter) * NPAD;
      float f[NPAD == 32 ? 32 : 1];
      if (NPAD == 32) {
        const float2 st = norm[lane];
        const float mine = ex2(ref_in[lane] + st.x) * st.y;
#pragma unroll
        for (int r = 0; r < 32; ++r) f[r] = __shfl_sync(0xffffffffu, mine, r);
      } else {                                           // many rows: the weights replace the warp's references
        for (int r = lane; r < NPAD; r += 32) {
          const float2 st = norm[r];
          ref_in[r] = ex2(ref_in[r] + st.x) * st.y;
        }
        __syncwarp();
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
          if (!p.per_head) {
            float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f;      // four chains of multiply-adds, fixed order
#pragma unroll
            for (int x = 0; x < 32; x += 4) {
              s0 = fmaf(pr[x], (NPAD == 32) ? f[x % (NPAD == 32 ? 32 : 1)] : ref_in[c * 32 + x], s0);
              s1 = fmaf(pr[x + 1], (NPAD == 32) ? f[(x + 1) % (NPAD == 32 ? 32 : 1)] : ref_in[c * 32 + x + 1], s1);
              s2 = fmaf(pr[x + 2], (NPAD == 32) ? f[(x + 2) % (NPAD == 32 ? 32 : 1)] : ref_in[c * 32 + x + 2], s2);
              s3 = fmaf(pr[x + 3], (NPAD == 32) ? f[(x + 3) % (NPAD == 32 ? 32 : 1)] : ref_in[c * 32 + x + 3], s3);
            }
            a_g += (s0 + s1) + (s2 + s3);
          } else {                                       // row n = j * G + hl and G divides 32
#pragma unroll
            for (int x = 0; x < 32; ++x)
              pr[x] *= (NPAD == 32) ? f[x % (NPAD == 32 ? 32 : 1)] : ref_in[c * 32 + x];
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
      if (lane == 0) mbar_arrive(&bars->ref_free[rbuf]); // pass 1 may overwrite this phase's references
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

// Zeroes the workspace header and the phase counters ahead of the scoring kernel.  A kernel rather than a
// memset so that it can sit in the chain of programmatic launches: it comes up while the kernel before it
// is still running and lets the scoring kernel come up behind it.
__global__ void clear_words_kernel(uint32_t* words, int n) {
  pdl_launch_dependents();
  pdl_wait();
  for (int i = threadIdx.x; i < n; i += blockDim.x) words[i] = 0u;
}

cudaError_t launch_clear_words(void* ptr, size_t bytes, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(1);
  cfg.blockDim = dim3(256);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  fill_pdl_attribute(&attr[0]);
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, clear_words_kernel, static_cast<uint32_t*>(ptr), static_cast<int>(bytes / 4));
}

template <int D, int NPAD, bool PART>
static cudaError_t launch_parked_t(const CUtensorMap& tk, const CUtensorMap& tq, const FusedParams& p, int grid,
                                   cudaStream_t stream) {
  using Cfg = ParkedCfg<D, NPAD>;
  static PerDeviceOnce configured;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (!configured.done(dev)) {
    e = cudaFuncSetAttribute(score_parked_kernel<D, NPAD, PART>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Cfg::kSmemBytes);
    if (e != cudaSuccess) return e;
    configured.set(dev);
  }
  void* args[] = {const_cast<CUtensorMap*>(&tk), const_cast<CUtensorMap*>(&tq), const_cast<FusedParams*>(&p)};
  // cooperative (every CTA resident: they wait on one another) and, where the driver takes both attributes
  // together, programmatic as well: the kernel's set-up then overlaps the end of the kernel before it
  static PerDeviceOnce no_overlap;
  if (!no_overlap.done(dev)) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kParkedThreads);
    cfg.dynamicSmemBytes = Cfg::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    fill_pdl_attribute(&attr[1]);
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    e = cudaLaunchKernelExC(&cfg, reinterpret_cast<const void*>(score_parked_kernel<D, NPAD, PART>), args);
    if (e == cudaSuccess) return e;
    if (e != cudaErrorNotSupported && e != cudaErrorInvalidValue) return e;
    cudaGetLastError();          // the combination is refused: from now on plain cooperative launches
    no_overlap.set(dev);
  }
  return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(score_parked_kernel<D, NPAD, PART>), dim3(grid),
                                     dim3(kParkedThreads), args, Cfg::kSmemBytes, stream);
}

cudaError_t launch_score_parked(int head_dim, int npad, const CUtensorMap& tk, const CUtensorMap& tq,
                                const FusedParams& p, int grid, cudaStream_t stream) {
  if (p.partition) {
    if (head_dim == 128 && npad == 32) return launch_parked_t<128, 32, true>(tk, tq, p, grid, stream);
    if (head_dim == 128 && npad == 64) return launch_parked_t<128, 64, true>(tk, tq, p, grid, stream);
    if (head_dim == 64 && npad == 32) return launch_parked_t<64, 32, true>(tk, tq, p, grid, stream);
    if (head_dim == 64 && npad == 64) return launch_parked_t<64, 64, true>(tk, tq, p, grid, stream);
    return cudaErrorInvalidValue;
  }
  if (head_dim == 128 && npad == 32) return launch_parked_t<128, 32, false>(tk, tq, p, grid, stream);
  if (head_dim == 128 && npad == 64) return launch_parked_t<128, 64, false>(tk, tq, p, grid, stream);
  if (head_dim == 64 && npad == 32) return launch_parked_t<64, 32, false>(tk, tq, p, grid, stream);
  if (head_dim == 64 && npad == 64) return launch_parked_t<64, 64, false>(tk, tq, p, grid, stream);
  return cudaErrorInvalidValue;
}

}  // namespace fastkv
