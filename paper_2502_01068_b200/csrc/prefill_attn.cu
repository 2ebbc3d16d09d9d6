// Causal prefill attention of a whole prompt that hands out the saliency scores as a by-product
// (Alg. 1: the TSP layer's own attention produces Att_l; Sec. 4.2 / App. D.4: the token importance
// estimation is otherwise a separate pass over Q_window x K).
//
// One CTA per (pair of 128-query tiles A and B, query head); it walks the key tiles 0 .. tile of its last query:
//
//   producer   one thread: the two Q tiles once, then K and V tiles into two-stage rings by TMA (both query
//              tiles use every K / V tile: half the shared-memory fills per flop);
//   issuers    one warp per query tile (on two warp schedulers: issuing a contraction holds up the other warps
//              of the issuer's scheduler), walking its loop as a whole warp with one elected lane per
//              instruction.  Per key tile j a tile's issuer issues one block: O += P_(j-1) V_(j-1) with P (bf16,
//              packed two keys per column) read from tensor memory and V as an MN-major operand from shared
//              memory (the V tile is used as TMA delivers it, keys x d with d contiguous), then S = Q K_j^T
//              (tcgen05.mma, 128 x 128 x d, fp32 in tensor memory).  Contractions of one thread execute in order,
//              so S_j overwrites the tile's S / P columns only after the contraction that read P_(j-1) from
//              them, and the softmax of key tile j finds O complete up to j - 1 -- no barrier for either.  The
//              two tiles' blocks alternate on the tensor cores (A(0) B(0) A(1) B(1) ..., a turn barrier each
//              way), which keeps the two softmaxes half a period apart: one tile's exponentials run under the
//              other's contractions.  Left alone the two tiles fall into step and take turns waiting;
//   softmax    eight warps per query tile, two threads per query row (tensor-memory lane = row; the two warps
//              that share a lane quarter take 64 keys of the tile each and exchange their maxima through
//              shared memory at one named barrier per tile): online softmax in log2 units with a lazily raised
//              reference (the row's reference moves, and its O row is rescaled, only when a logit exceeds it by
//              more than 8 binary orders of magnitude).  The logits stay in tensor memory and are read twice,
//              32 at a time (maximum, then exponentials): 96 registers per thread let 19 warps share the SM.
//              P is rounded to bf16 and stored into the first half of the thread's own S columns (columns it
//              has read already); at the end O / l -> bf16 -> global memory.
//
// Tensor memory (512 columns): S (and P inside it) of tile A at 0, of tile B at 128; O of A at 256, of B at 256 + d.
//
// The by-product: the threads whose query row is one of the last w of its sequence (the observation
// window) also store their scaled logits of every key (fp32, log2 units) and, at the end, their
// (reference, sum); window_scores_kernel turns these into Eq. 1's inner term summed over the window
// and the GQA group, in the layout the pooling kernel of the scoring path reads.  No second pass over
// K: what is added to the attention is w fp32 rows per query head.
//
// Every wait is bounded; a wait that gives up raises the status word and the CTA-wide abort flag, the
// roles stop issuing work, copies and contractions in flight are waited for, tensor memory is released.
#include "prefill_attn.cuh"

namespace fastkv {

namespace {

constexpr int kBM = 128;                       // queries per query tile; a CTA has two of them
constexpr int kBN = 128;                       // keys per tile
constexpr int kCtrlWarps = 3;                  // producer, issuer of query tile A, issuer of query tile B
constexpr int kSoftmaxWarps = 8;               // per query tile
constexpr int kAttnThreads = (kCtrlWarps + 2 * kSoftmaxWarps) * 32;
constexpr int kChunkBytes = 128 * 128;         // 128 rows x 64 bf16: one swizzled column chunk of a tile
constexpr float kRescaleSlackLog2 = 8.0f;

template <int D>
struct AttnCfg {
  static constexpr int KH = D / 64;
  static constexpr int kTileBytes = KH * kChunkBytes;     // Q, K or V tile
  static constexpr int kKvStages = 2;
  // two Q tiles, the K and V rings, the barriers, what the two halves of a row exchange ([tile][2][2][128] floats)
  static constexpr int kSmemBytes = (2 + 2 * kKvStages) * kTileBytes + 256 + 2 * 2 * 2 * kBM * 4;
};

struct AttnBarriers {
  uint64_t q_full;
  uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2];   // empty: both issuers are done with the stage
  uint64_t s_full[2];           // per query tile: S = Q K^T of the current key tile is in tensor memory
  uint64_t p_full[2];           // per query tile: every softmax warp has stored its part of P
  uint64_t o_done[2];           // per query tile: every contraction its issuer started has finished
  uint64_t turn[2];             // turn[x]: the other tile's issuer has issued the block that goes before x's next one
  uint32_t tmem_base;
  int abort_flag;
};

// MN-major operand tile as TMA writes it (rows of 128 bytes = 64 elements of the MN dimension, one row per
// K index, 128-byte swizzle): 64-element MN chunks are `chunk_bytes` apart (leading byte offset), groups of
// eight K rows 1024 bytes apart (stride byte offset).
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t smem_addr, uint32_t chunk_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((chunk_bytes >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

// D[tmem] (+)= A[tmem] * B[smem]: A is read from tensor memory (lane = row, two bf16 per 32-bit column)
__device__ __forceinline__ void tc_mma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// True in exactly one lane of the (converged) warp.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred != 0;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

}  // namespace

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
prefill_attn_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                    const __grid_constant__ CUtensorMap tmap_v, const PrefillParams p) {
  using Cfg = AttnCfg<D>;
  extern __shared__ __align__(1024) uint8_t smem[];       // the tiles need 1024-byte alignment (128-byte swizzle atoms)
  uint8_t* sQ = smem;                                     // two query tiles
  constexpr int NS = Cfg::kKvStages;
  uint8_t* sK = sQ + 2 * Cfg::kTileBytes;                 // NS stages
  uint8_t* sV = sK + NS * Cfg::kTileBytes;                // NS stages
  AttnBarriers* bars = reinterpret_cast<AttnBarriers*>(sV + NS * Cfg::kTileBytes);
  float* xch_all = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(bars) + 256);   // [tile][2][2][128]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Launch order (blockIdx.x fastest): when K and V of all heads fit in L2 together, all query heads fastest, then
  // the pairs of query tiles, longest rows first -- every head's long CTAs start before anybody's short ones.  For
  // long prompts the heads of one GQA group fastest, then the pairs, then the KV heads: what runs at the same time
  // works on one or two KV heads' K and V, which stay in L2.
  const int heads_x = static_cast<int>(gridDim.x);                 // n_q_heads or group
  const int per_z = p.n_q_heads / heads_x;                         // 1 or n_kv_heads
  const int b = blockIdx.z / per_z, h = (blockIdx.z - b * per_z) * heads_x + blockIdx.x, g = h / p.group;
  const int row0 = p.cu_seqlens ? p.cu_seqlens[b] : 0;
  const int L = p.cu_seqlens ? p.cu_seqlens[b + 1] - row0 : p.total_len;
  const int n_pairs = (L + 2 * kBM - 1) / (2 * kBM);
  const int qp = n_pairs - 1 - static_cast<int>(blockIdx.y);       // the longest rows first
  if (qp < 0) return;                                              // (uniform per CTA, before any barrier)
  if (smem_u32(smem) & 1023u) {                                    // never seen; would garble every tile
    if (threadIdx.x == 0) raise_status(p.hdr, FASTKV_ERR_UNSUPPORTED, SITE_ATTN_Q);
    return;
  }
  const int q0 = qp * 2 * kBM;
  const bool b_active = q0 + kBM < L;                              // the sequence may end inside query tile A
  // key tiles of each query tile (causal): A sees 0 .. 2 qp, B one more; the rings carry the longer list
  const int n_key_a = 2 * qp + 1, n_key_b = b_active ? 2 * qp + 2 : 0;
  const int n_tiles = b_active ? n_key_b : n_key_a;
  const long long limit = p.wait_limit;

  if (threadIdx.x == 0) {
    mbar_init(&bars->q_full, 1);
    for (int i = 0; i < NS; ++i) {
      mbar_init(&bars->k_full[i], 1); mbar_init(&bars->k_empty[i], 2);
      mbar_init(&bars->v_full[i], 1); mbar_init(&bars->v_empty[i], 2);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->s_full[i], 1);
      mbar_init(&bars->p_full[i], kSoftmaxWarps);
      mbar_init(&bars->o_done[i], 1);
      mbar_init(&bars->turn[i], 1);
    }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tma_prefetch_desc(&tmap_q);
    tma_prefetch_desc(&tmap_k);
    tma_prefetch_desc(&tmap_v);
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;
  volatile int* abort_flag = &bars->abort_flag;
  pdl_launch_dependents();
  pdl_wait();

  if (warp == 0) {
    // ---------------- producer ----------------
    if (lane == 0) {
      const uint64_t pol_q = l2_policy_evict_first();      // a Q tile is read by one CTA
      const uint64_t pol_kv = l2_policy_evict_last();      // K / V tiles are read by every later pair of query tiles
      mbar_arrive_expect_tx(&bars->q_full, (b_active ? 2 : 1) * Cfg::kTileBytes);
      for (int x = 0; x < (b_active ? 2 : 1); ++x)
        for (int c = 0; c < Cfg::KH; ++c)
          tma_load_3d(sQ + x * Cfg::kTileBytes + c * kChunkBytes, &tmap_q, &bars->q_full, c * 64, h, row0 + q0 + x * kBM, pol_q);
      bool ok = true;
      int issued = 0;
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int s = j % NS;
        const uint32_t par = (j / NS) & 1;
        ok = mbar_wait_parked(&bars->k_empty[s], par ^ 1, abort_flag, p.hdr, SITE_ATTN_RING, limit);
        if (!ok) break;
        mbar_arrive_expect_tx(&bars->k_full[s], Cfg::kTileBytes);
        for (int c = 0; c < Cfg::KH; ++c)
          tma_load_3d(sK + s * Cfg::kTileBytes + c * kChunkBytes, &tmap_k, &bars->k_full[s], c * 64, g, row0 + j * kBN, pol_kv);
        ok = mbar_wait_parked(&bars->v_empty[s], par ^ 1, abort_flag, p.hdr, SITE_ATTN_RING, limit);
        if (!ok) {                                          // K of this tile is in flight, V is not
          mbar_wait_drain(&bars->k_full[s], par, p.hdr, SITE_ATTN_DRAIN, limit);
          break;
        }
        mbar_arrive_expect_tx(&bars->v_full[s], Cfg::kTileBytes);
        for (int c = 0; c < Cfg::KH; ++c)
          tma_load_3d(sV + s * Cfg::kTileBytes + c * kChunkBytes, &tmap_v, &bars->v_full[s], c * 64, g, row0 + j * kBN, pol_kv);
        issued = j + 1;
      }
      // nothing may still be landing in shared memory when the CTA ends
      mbar_wait_drain(&bars->q_full, 0, p.hdr, SITE_ATTN_DRAIN, limit);
      for (int j = max(0, issued - NS); j < issued; ++j) {
        mbar_wait_drain(&bars->k_full[j % NS], (j / NS) & 1, p.hdr, SITE_ATTN_DRAIN, limit);
        mbar_wait_drain(&bars->v_full[j % NS], (j / NS) & 1, p.hdr, SITE_ATTN_DRAIN, limit);
      }
    }
  } else if (warp < kCtrlWarps) {
    // ---------------- issuer of one query tile ----------------
    // A query tile's contractions come from one thread and therefore execute in the order S(0), O += P V (0), S(1),
    // O += P V (1), ...: S of the next key tile overwrites the tile's S / P columns only after the contraction that
    // read P from them, and the softmax of key tile j finds O complete up to j - 1, with no barrier for either.
    // The two tiles' issuers sit on two warp schedulers (issuing a contraction holds up the other warps of the
    // issuer's scheduler); each walks its loop as a whole warp, one elected lane issues; its waits poll every ~50 ns
    // (a hot polling loop takes the scheduler's issue slots, a suspended wait wakes 0.5 kcycles late).
    const int x = warp - 1;
    const int nk = x == 0 ? n_key_a : n_key_b;
    constexpr uint32_t idesc_s = umma_idesc_bf16_f32(kBM, kBN);
    constexpr uint32_t idesc_o = umma_idesc_bf16_f32(kBM, D) | (1u << 16);      // B (V) is MN-major
    const uint32_t q_addr = smem_u32(sQ + x * Cfg::kTileBytes);
    const uint32_t s_tmem = tmem_base + x * kBN, o_tmem = tmem_base + 256 + x * D;
    bool ok = true;
    int committed = 0;
    auto first = [&](int j) {                              // S = Q K_j^T (the caller has seen K_j arrive)
      const int ks = j % NS;
      const uint64_t a0 = umma_desc_k_sw128(q_addr), b0 = umma_desc_k_sw128(smem_u32(sK + ks * Cfg::kTileBytes));
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {                // 64-element chunk kk / 4, 32 bytes per step inside it
        const uint64_t step = static_cast<uint64_t>(((kk >> 2) * kChunkBytes + (kk & 3) * 32) >> 4);
        if (elect_one()) tc_mma_bf16(s_tmem, a0 + step, b0 + step, idesc_s, kk > 0 ? 1u : 0u);
      }
      if (elect_one()) {
        tc_commit(&bars->k_empty[ks]);
        if (!(x == 0 && j == p.skip_commit_tile)) tc_commit(&bars->s_full[x]);   // (test hook: a completion that is never signalled)
      }
      ++committed;
    };
    auto second = [&](int j) {                             // O (+)= P_j V_j
      const int s = j % NS;
      // one descriptor per tile; a step further along K only moves its start-address field (units of 16 bytes).
      // P: each half of a row keeps its 64 keys, packed, in the first 32 of its own 64 S columns
      const uint64_t b0 = umma_desc_mn_sw128(smem_u32(sV + s * Cfg::kTileBytes), kChunkBytes);
#pragma unroll
      for (int kk = 0; kk < kBN / 16; ++kk)                // 16 keys = 8 packed columns of P, 2048 bytes of V per step
        if (elect_one())
          tc_mma_bf16_ts(o_tmem, s_tmem + (kk >> 2) * 64 + (kk & 3) * 8, b0 + static_cast<uint64_t>(kk * (2048 >> 4)), idesc_o,
                         (j > 0 || kk > 0) ? 1u : 0u);
      if (elect_one()) tc_commit(&bars->v_empty[s]);
      ++committed;
    };
    if (nk > 0) {
      ok = mbar_wait_nap(&bars->q_full, 0, abort_flag, p.hdr, SITE_ATTN_Q, limit);
      ok = __all_sync(0xffffffffu, ok);
    }
    // Block jb of a tile = [O += P V of key tile jb - 1] [S of key tile jb].  The two tiles' blocks alternate on the
    // tensor cores -- A(0) B(0) A(1) B(1) ... -- which keeps the two softmaxes half a period apart: one tile's
    // exponentials run under the other's contractions (left alone, the two tiles fall into step, want the tensor
    // cores at the same time and the special-function unit at the same time, and each waits while the other works).
    int jb = 0;
    for (; nk > 0 && jb <= nk && ok; ++jb) {
      if (jb < nk) {                                       // K of the block's S: long there when P arrives
        ok = mbar_wait_nap(&bars->k_full[jb % NS], (jb / NS) & 1, abort_flag, p.hdr, SITE_ATTN_K, limit);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      if (jb > 0) {
        ok = mbar_wait_nap(&bars->v_full[(jb - 1) % NS], ((jb - 1) / NS) & 1, abort_flag, p.hdr, SITE_ATTN_V, limit) &&
             mbar_wait_nap(&bars->p_full[x], (jb - 1) & 1, abort_flag, p.hdr, SITE_ATTN_P, limit);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      if (b_active) {
        if (x == 0 && jb >= 1) ok = mbar_wait_nap(&bars->turn[0], (jb - 1) & 1, abort_flag, p.hdr, SITE_ATTN_S, limit);
        if (x == 1 && jb <= n_key_a) ok = mbar_wait_nap(&bars->turn[1], jb & 1, abort_flag, p.hdr, SITE_ATTN_S, limit);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      tc_fence_after_sync();
      if (jb > 0) second(jb - 1);
      if (jb < nk) first(jb);
      if (b_active && elect_one()) mbar_arrive(&bars->turn[x ^ 1]);
    }
    const bool all_issued = ok && jb > nk;
    // key tiles this query tile does not use (A has one fewer than B; a tile past the end of the sequence uses none):
    // the stage still counts two releases
    for (int jj = (nk == 0 || all_issued) ? nk : n_tiles; jj < n_tiles; ++jj) {
      const int s = jj % NS;
      bool fine = mbar_wait_nap(&bars->k_full[s], (jj / NS) & 1, abort_flag, p.hdr, SITE_ATTN_K, limit);
      fine = __all_sync(0xffffffffu, fine);
      if (!fine) break;
      if (lane == 0) mbar_arrive(&bars->k_empty[s]);
      fine = mbar_wait_nap(&bars->v_full[s], (jj / NS) & 1, abort_flag, p.hdr, SITE_ATTN_V, limit);
      fine = __all_sync(0xffffffffu, fine);
      if (!fine) break;
      if (lane == 0) mbar_arrive(&bars->v_empty[s]);
    }
    // every contraction issued has finished before tensor memory is released (and O is complete)
    if (committed > 0) {
      if (elect_one()) tc_commit(&bars->o_done[x]);
      __syncwarp();
      mbar_wait_drain(&bars->o_done[x], 0, p.hdr, SITE_ATTN_DRAIN, limit);
    }
  } else {
    // ---------------- softmax: eight warps per query tile, two threads per query row, 64 keys of the tile each ----------------
    const int gw = warp - kCtrlWarps;
    const int x = gw >> 3, g8 = gw & 7;                   // query tile; warp of the tile
    const int quarter = warp & 3, half = g8 >> 2;         // a tile's warps cover the four lane quarters twice
    const int nk = x == 0 ? n_key_a : n_key_b;
    const int r = quarter * 32 + lane;                    // row of the tile = tensor-memory lane
    const int t = q0 + x * kBM + r;                       // query position in its sequence
    const int t_eff = min(t, L - 1);                      // rows past the end repeat the last row (never stored)
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    const uint32_t s_addr = lane_addr + x * kBN + half * 64;          // this thread's 64 S columns; P goes into the first 32
    const uint32_t o_addr = lane_addr + 256 + x * D + half * (D / 2); // this thread's D / 2 columns of O
    float* const xch = xch_all + x * (2 * 2 * kBM);
    const int jw = t - (L - p.window);                    // window row index, if 0 <= jw < w
    const bool is_window = p.wlog != nullptr && jw >= 0 && t < L;
    float* const wlog_row = is_window ? p.wlog + (static_cast<size_t>(h) * p.window + jw) * p.ld_w + row0 : nullptr;
    constexpr int HN = kBN / 2;                           // keys per thread and tile
    auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(1 + x * 4 + (g8 & 3)) : "memory"); };
    float m_ref = -INFINITY, l = 0.0f;                    // the reference is the same in both threads of a row; l is this half's
    bool ok = true;
    // Both warps of a pair walk every tile and meet at the pair's barrier once per tile whatever happens: a
    // warp whose wait gave up skips the work of the tile, never the barrier.
    for (int j = 0; j < nk; ++j) {
      const int s = j & 1;
      if (ok) ok = mbar_wait_bounded(&bars->s_full[x], j & 1, abort_flag, p.hdr, SITE_ATTN_SFULL, limit);
      ok = __all_sync(0xffffffffu, ok);
      const int key0 = j * kBN + half * HN;
      const bool diagonal = key0 + HN - 1 > t_eff;        // some keys of this half are not visible to this row
      float half_max = -INFINITY;
      if (ok) {
        tc_fence_after_sync();
        // first reading of this half of the row: its maximum (the row stays in tensor memory: a thread holds 32 of
        // its 64 logits at a time)
#pragma unroll
        for (int c = 0; c < HN / 32; ++c) {
          float v[32];
          tmem_ld_32x32(s_addr + c * 32, v);
          if (diagonal) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = key0 + c * 32 + i <= t_eff ? v[i] : -INFINITY;
          }
          float mx[4] = {v[0], v[1], v[2], v[3]};
#pragma unroll
          for (int i = 4; i < 32; i += 4) {
            mx[0] = fmaxf(mx[0], v[i]); mx[1] = fmaxf(mx[1], v[i + 1]); mx[2] = fmaxf(mx[2], v[i + 2]); mx[3] = fmaxf(mx[3], v[i + 3]);
          }
          half_max = fmaxf(half_max, fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])));
        }
      }
      xch[(s * 2 + half) * kBM + r] = half_max;
      pair_sync();
      if (!ok) continue;
      const float tile_max = fmaxf(half_max, xch[(s * 2 + (half ^ 1)) * kBM + r]) * p.scale_log2;   // the scale is positive
      // the reference moves only when the tile's maximum is far above it (or at the first tile)
      const bool move = tile_max > m_ref + kRescaleSlackLog2;
      const float alpha = move ? ex2(m_ref - tile_max) : 1.0f;     // 0 at the first tile
      if (move) { m_ref = tile_max; l *= alpha; }
      if (j >= 1 && __any_sync(0xffffffffu, move)) {
        // O is rescaled, each half its own columns.  It is complete up to key tile j - 1: the contraction that
        // produced this S was issued after the one that added tile j - 1, by the same thread.
#pragma unroll
        for (int c = 0; c < D / 64; ++c) {
          float o[32];
          tmem_ld_32x32(o_addr + c * 32, o);
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] *= alpha;
          tmem_st_32x32(o_addr + c * 32, o);
        }
        tmem_wait_st();
      }
      // second reading: p = exp2(s * scale - ref), the row sum, P in bf16 for the second contraction: two keys per
      // 32-bit column, this thread's 64 keys in the first 32 of its own 64 S columns (columns it has read already)
      const float neg_ref = -m_ref;
      float ls[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
      for (int c = 0; c < HN / 32; ++c) {
        float v[32];
        tmem_ld_32x32(s_addr + c * 32, v);
        if (diagonal) {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = key0 + c * 32 + i <= t_eff ? v[i] : -INFINITY;
        }
        if (is_window) {                                   // by-product: this row's logits (log2 units), masked = -inf
          float* const dst = wlog_row + key0 + c * 32;
          if (key0 + c * 32 + 32 <= L && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              *reinterpret_cast<float4*>(dst + i) = make_float4(v[i] * p.scale_log2, v[i + 1] * p.scale_log2,
                                                                v[i + 2] * p.scale_log2, v[i + 3] * p.scale_log2);
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (key0 + c * 32 + i < L) dst[i] = v[i] * p.scale_log2;
          }
        }
        float packed[16];
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float e0 = ex2(fmaf(v[i], p.scale_log2, neg_ref));      // exp2(-inf) = 0 for a masked key
          const float e1 = ex2(fmaf(v[i + 1], p.scale_log2, neg_ref));
          ls[i & 2] += e0;
          ls[(i & 2) + 1] += e1;
          packed[i / 2] = __uint_as_float(pack_bf16(e0, e1));
        }
        tmem_st_32x16(s_addr + c * 16, packed);
      }
      l += (ls[0] + ls[1]) + (ls[2] + ls[3]);
      tmem_wait_st();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->p_full[x]);
    }
    if (nk > 0) {
      // the finished row: the halves' sums meet, O / l -> bf16, each half its own columns
      const int xb = nk & 1;                              // the exchange buffer the last tile did not use
      xch[(xb * 2 + half) * kBM + r] = l;
      pair_sync();
      l += xch[(xb * 2 + (half ^ 1)) * kBM + r];
      if (ok) ok = mbar_wait_bounded(&bars->o_done[x], 0, abort_flag, p.hdr, SITE_ATTN_ODONE, limit);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        tc_fence_after_sync();
        const float inv_l = 1.0f / l;
        uint8_t* const orow = reinterpret_cast<uint8_t*>(p.out) +
                              (static_cast<size_t>(row0 + t) * p.out_stride_tok + static_cast<size_t>(h) * p.out_stride_head) * 2 +
                              half * D;                      // D / 2 elements of 2 bytes
#pragma unroll
        for (int c = 0; c < D / 64; ++c) {
          float o[32];
          tmem_ld_32x32(o_addr + c * 32, o);
          if (t < L) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              uint4 w4;
              w4.x = pack_bf16(o[u * 8 + 0] * inv_l, o[u * 8 + 1] * inv_l);
              w4.y = pack_bf16(o[u * 8 + 2] * inv_l, o[u * 8 + 3] * inv_l);
              w4.z = pack_bf16(o[u * 8 + 4] * inv_l, o[u * 8 + 5] * inv_l);
              w4.w = pack_bf16(o[u * 8 + 6] * inv_l, o[u * 8 + 7] * inv_l);
              *reinterpret_cast<uint4*>(orow + c * 64 + u * 16) = w4;
            }
          }
        }
        if (is_window && half == 0) p.wstat[(static_cast<size_t>(b) * p.n_q_heads + h) * p.window + jw] = make_float2(m_ref, l);
      }
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
// Eq. 1's inner term from the window rows' logits: for key i of KV head g,
//   a[g, i] = sum over the query heads h of the group and the window rows j with i <= L - w + j of
//             exp2(s[h, j, i] - ref[h, j]) / l[h, j]
// (one row per query head instead with per_head).  One thread per key and KV head; G * w <= 64.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) window_scores_kernel(const WindowScoresParams p) {
  __shared__ float2 st[64];                                // (reference, 1 / sum) of the group's G * w window rows
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.z, g = blockIdx.y;
  const int row0 = p.cu_seqlens ? p.cu_seqlens[b] : 0;
  const int L = p.cu_seqlens ? p.cu_seqlens[b + 1] - row0 : p.total_len;
  if (L < p.window) return;
  const int G = p.group, w = p.window;
  if (threadIdx.x < G * w) {
    const float2 v = p.wstat[(static_cast<size_t>(b) * p.n_q_heads + g * G) * w + threadIdx.x];
    st[threadIdx.x] = make_float2(v.x, 1.0f / v.y);
  }
  __syncthreads();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= L) return;
  const int first_j = max(0, i - (L - w));                 // causal: key i is visible to window rows j >= i - (L - w)
  float a_g = 0.0f;
  for (int hl = 0; hl < G; ++hl) {
    const float* src = p.wlog + (static_cast<size_t>(g * G + hl) * w) * p.ld_w + row0 + i;
    float a_h = 0.0f;
#pragma unroll 8
    for (int j = 0; j < w; ++j) {
      const float s = j >= first_j ? __ldg(src + static_cast<size_t>(j) * p.ld_w) : -INFINITY;
      const float2 rf = st[hl * w + j];
      a_h += ex2(s - rf.x) * rf.y;
    }
    if (p.per_head) p.a_out[static_cast<size_t>(g * G + hl) * p.ld_a + row0 + i] = a_h;
    a_g += a_h;
  }
  if (!p.per_head) p.a_out[static_cast<size_t>(g) * p.ld_a + row0 + i] = a_g;
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------

template <int D>
static cudaError_t launch_attn_t(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                                 const PrefillParams& p, int max_len, cudaStream_t stream) {
  using Cfg = AttnCfg<D>;
  static PerDeviceOnce configured;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (!configured.done(dev)) {
    e = cudaFuncSetAttribute(prefill_attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes);
    if (e != cudaSuccess) return e;
    configured.set(dev);
  }
  cudaLaunchConfig_t cfg = {};
  const int n_kv_heads = p.n_q_heads / p.group;
  const long long kv_bytes = 2ll * p.total_len * n_kv_heads * D * 2;           // K and V of every head
  const bool all_heads_first = kv_bytes <= (64ll << 20);                       // they stay in L2 whatever runs together
  cfg.gridDim = all_heads_first ? dim3(p.n_q_heads, (max_len + 2 * kBM - 1) / (2 * kBM), p.batch)
                                : dim3(p.group, (max_len + 2 * kBM - 1) / (2 * kBM), p.batch * n_kv_heads);
  cfg.blockDim = dim3(kAttnThreads);
  cfg.dynamicSmemBytes = Cfg::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  fill_pdl_attribute(&attr[0]);
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, prefill_attn_kernel<D>, tq, tk, tv, p);
}

cudaError_t launch_prefill_attn(int head_dim, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                                const PrefillParams& p, int max_len, cudaStream_t stream) {
  if (head_dim == 128) return launch_attn_t<128>(tq, tk, tv, p, max_len, stream);
  if (head_dim == 64) return launch_attn_t<64>(tq, tk, tv, p, max_len, stream);
  return cudaErrorInvalidValue;
}

cudaError_t launch_window_scores(const WindowScoresParams& p, int max_len, int batch, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((max_len + 255) / 256, p.n_kv_heads, batch);
  cfg.blockDim = dim3(256);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  fill_pdl_attribute(&attr[0]);
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, window_scores_kernel, p);
}

}  // namespace fastkv
