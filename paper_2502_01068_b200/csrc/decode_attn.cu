// Decode-time attention of one new query token over the compressed KV cache that fastkv_compact
// leaves behind ([Hkv, kept, d] per sequence): the stage the retained KV of Alg. 1 exists for.
//
// Memory-bound: every kept K and V row is read once (4 * d bytes per kept entry and KV head) for G <= 8
// query rows per KV head.  The two products are far too small for the 128-row tcgen05 tiles, but on the
// CUDA cores they cost ~100 instructions per kept entry and the kernel was issue-bound at 0.43 of the copy
// rate; so they run as warp-level m16n8k16 bf16 tensor-core products, whose only job here is to cut the
// instruction count (~7 per kept entry).
//
// Split-KV: one CTA (eight warps; four for batches with more pairs than SMs) per (key range, KV head, sequence), and
// inside the CTA every warp works on its own: it
// owns a ring of shared-memory stages (16 kept entries of K and of V each) that one lane fills with tiled
// TMA copies (boxes of 16 rows x 64 elements in the 128-byte swizzle, which makes the 8x8 matrix loads
// conflict-free; one bulk copy per padded row instead was bound by the ~100 cycles each copy takes to
// issue), and runs its own online softmax.  No CTA-wide barrier in the loop.
//   S  [heads x 16 keys] = Q K^T : A = the group's queries (rows >= 8 are zero), B = K rows as stored;
//   O^T[d x heads]      += V^T P^T: A = V rows through the transposing matrix load, B = P, which is
//                          exactly the layout the first product leaves S in (no exchange between lanes).
// P goes in as two bf16 terms (value and rounding remainder), so the result carries fp32-level error.
// The warps of a CTA merge through shared memory at the end; a second small kernel merges the splits.
#include "decode_attn.cuh"

namespace fastkv {

namespace {

constexpr int kDecStages = 3;       // stages per warp: two chunks in flight while one is consumed
// Warps per CTA: 8 (one CTA per SM) when the launch has fewer (key range, KV head, sequence) triples than SMs can hold
// that way, 4 (two CTAs per SM) for batches with more pairs than that: the launch then runs as one wave.
constexpr int kDecChunk = 16;       // kept entries per stage: the K extent of the second product
constexpr int kDecHeads = 8;        // query heads per KV head, padded: the N extent of the second product

// Four 8x8 matrices of 16-bit elements; lane l gives the address of row l % 8 of matrix l / 8.
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
// D[16x8] += A[16x16] B[16x8], bf16 operands, fp32 accumulators.
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// Two floats to bf16 (round to nearest even): `lo` in the low half.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

template <int D, int kDecWarps>
struct DecCfg {
  static constexpr int kBoxes = D / 64;                               // 64-element (128-byte) column blocks of a row
  static constexpr int kBoxBytes = kDecChunk * 128;                   // one box: 16 rows x 128 bytes, swizzled
  static constexpr int kHalfBytes = kBoxes * kBoxBytes;               // K (or V) rows of one stage
  static constexpr int kStageBytes = 2 * kHalfBytes;
  static constexpr int kRingBytes = kDecWarps * kDecStages * kStageBytes;
  static constexpr int kMergeBytes = kDecWarps * kDecHeads * (D + 2) * 4;   // the warps' outputs and (max, sum)
  static constexpr int kSmem = (kRingBytes > kMergeBytes ? kRingBytes : kMergeBytes) + 1024;   // the swizzle atom is 1024 bytes
};

}  // namespace

template <int D, int kDecWarps>
__global__ void __launch_bounds__(32 * kDecWarps)
decode_attn_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v, const DecodeParams p) {
  using Cfg = DecCfg<D, kDecWarps>;
  constexpr int kDecThreads = 32 * kDecWarps;
  constexpr int KS = D / 16;                    // 16-wide steps over the head dimension (first product)
  constexpr int MT = D / 16;                    // 16-row tiles of the head dimension (second product)
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  __shared__ uint64_t full[kDecWarps][kDecStages];
  __shared__ int abort_flag;

  const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int quad = lane >> 2, c = lane & 3;     // fragment coordinates: row (or column) quad, element pair c
  const int G = p.group, n_splits = gridDim.x;
  const int seg0 = p.cu_k ? p.cu_k[b] : b * p.k_uniform;
  const int kept = p.cu_k ? p.cu_k[b + 1] - seg0 : p.k_uniform;
  // the CTA's range of chunks, dealt to its warps round robin
  const int n_chunks_all = (kept + kDecChunk - 1) / kDecChunk;
  const int per = (n_chunks_all + n_splits - 1) / n_splits;
  const int c0 = split * per, c1 = min(n_chunks_all, c0 + per);
  const int my_chunks = c1 - c0 > warp ? (c1 - c0 - warp + kDecWarps - 1) / kDecWarps : 0;
  const size_t part = ((static_cast<size_t>(b) * p.n_kv_heads + g) * n_splits + split) * G;

  if (t == 0) {
    tma_prefetch_desc(&tmap_k);
    tma_prefetch_desc(&tmap_v);
  }
  pdl_wait();
  if (lane == 0) {
    for (int i = 0; i < kDecStages; ++i) mbar_init(&full[warp][i], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (t == 0) abort_flag = 0;
  __syncthreads();
  pdl_launch_dependents();   // the merge kernel may take its place now; it waits for this grid to end before it reads

  // A fragments of the group's queries: head `quad` (absent heads are zero), elements 2c, 2c + 1 and 2c + 8, 2c + 9
  // of every 16-wide step; the fragment's rows 8..15 are zero
  uint32_t qa[KS][2];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    qa[ks][0] = qa[ks][1] = 0u;
    if (quad < G) {
      const uint16_t* qp = p.q + (static_cast<size_t>(b) * p.n_q_heads + g * G + quad) * D + ks * 16 + c * 2;
      qa[ks][0] = static_cast<uint32_t>(qp[0]) | (static_cast<uint32_t>(qp[1]) << 16);
      qa[ks][1] = static_cast<uint32_t>(qp[8]) | (static_cast<uint32_t>(qp[9]) << 16);
    }
  }
  // O^T: tile mt holds (d = mt * 16 + quad, heads 2c, 2c + 1) in [0], [1] and (d + 8, same heads) in [2], [3]
  float o[MT][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int e = 0; e < 4; ++e) o[mt][e] = 0.0f;
  float m_run = -INFINITY;                      // of head `quad` (the four lanes of a quad hold equal copies)
  float l_part = 0.0f;                          // this lane's share of the head's sum of exponentials

  uint8_t* const ring_ptr = smem + warp * kDecStages * Cfg::kStageBytes;
  const uint32_t ring = smem_u32(ring_ptr);
  const uint64_t policy = l2_policy_evict_first();      // every kept row is read once
  // Lane 0: the K and V rows of this warp's i-th chunk, one box per 64 columns.  Rows past the end of the cache
  // arrive as zeros; rows past the end of this sequence are another sequence's (finite, and masked below).
  auto issue = [&](int i) {
    const int r0 = seg0 + (c0 + warp + i * kDecWarps) * kDecChunk;
    uint64_t* bar = &full[warp][i % kDecStages];
    uint8_t* stage = ring_ptr + (i % kDecStages) * Cfg::kStageBytes;
    mbar_arrive_expect_tx(bar, Cfg::kStageBytes);
#pragma unroll
    for (int x = 0; x < Cfg::kBoxes; ++x) {
      tma_load_3d(stage + x * Cfg::kBoxBytes, &tmap_k, bar, x * 64, g, r0, policy);
      tma_load_3d(stage + Cfg::kHalfBytes + x * Cfg::kBoxBytes, &tmap_v, bar, x * 64, g, r0, policy);
    }
  };
  int issued = 0;                      // lane 0: chunks whose copies have been started
  if (lane == 0)
    for (; issued < kDecStages - 1 && issued < my_chunks; ++issued) issue(issued);
  // swizzled address of a 16-byte piece: (row, piece) sits at row * 128 + ((piece ^ (row & 7)) * 16); every matrix
  // load below takes its eight rows from one group of eight, so row & 7 is lane & 7
  const uint32_t row7 = lane & 7;
  bool ok = true;
  int done = 0;                        // chunks consumed
  for (int i = 0; i < my_chunks; ++i) {
    if (lane == 0 && i + kDecStages - 1 < my_chunks) issue(issued++);   // that stage was consumed last iteration
    ok = mbar_wait_bounded(&full[warp][i % kDecStages], (i / kDecStages) & 1, &abort_flag, p.hdr, SITE_DECODE_WAIT);
    if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
    const uint32_t ks_addr = ring + (i % kDecStages) * Cfg::kStageBytes;
    const uint32_t vs_addr = ks_addr + Cfg::kHalfBytes;
    const int rows = min(kDecChunk, kept - (c0 + warp + i * kDecWarps) * kDecChunk);
    if (rows < kDecChunk) {
      // the last chunk of the sequence: the rows past its end belong to the next sequence (or are the zero fill
      // past the cache).  Their logits are masked below, but a zero probability does not silence a NaN or an
      // infinity in V, so those V rows are cleared: nothing of another sequence can reach this one's output.
      uint8_t* vs = ring_ptr + (i % kDecStages) * Cfg::kStageBytes + Cfg::kHalfBytes;
      for (int j = lane; j < Cfg::kBoxes * (kDecChunk - rows) * 8; j += 32) {
        const int x = j / ((kDecChunk - rows) * 8), rem = j - x * (kDecChunk - rows) * 8;
        *reinterpret_cast<uint4*>(vs + x * Cfg::kBoxBytes + rows * 128 + rem * 16) = make_uint4(0u, 0u, 0u, 0u);
      }
      __syncwarp();
    }
    // ---- S = Q K^T: two tiles of 8 keys; lane holds (head quad, keys nt * 8 + 2c, + 1) in s[nt][0], [1] ----
    float s[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) s[nt][e] = 0.0f;
    }
#pragma unroll
    for (int ks2 = 0; ks2 < KS / 2; ++ks2) {
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        uint32_t kb[4];                // B fragments of two 16-wide steps: K rows as stored, 8 keys x 32 elements
        const uint32_t piece = (ks2 & 1) * 4 + (lane >> 3);     // of the 128-byte row of box ks2 / 2
        ldmatrix_x4(kb, ks_addr + (ks2 >> 1) * Cfg::kBoxBytes + (nt * 8 + row7) * 128 + ((piece ^ row7) << 4));
        mma_16816(s[nt], qa[2 * ks2][0], 0u, qa[2 * ks2][1], 0u, kb[0], kb[1]);
        mma_16816(s[nt], qa[2 * ks2 + 1][0], 0u, qa[2 * ks2 + 1][1], 0u, kb[2], kb[3]);
      }
    }
    float sv[4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e)
        sv[nt * 2 + e] = (nt * 8 + c * 2 + e < rows) ? s[nt][e] * p.scale_log2 : -INFINITY;
    // ---- online softmax of head `quad`: its 16 keys sit in the four lanes of the quad ----
    float mx = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float m_new = fmaxf(m_run, mx);          // finite: the chunk has at least one key
    const float alpha = ex2(m_run - m_new);        // first chunk: 2^-inf = 0
    float pr[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) pr[e] = ex2(sv[e] - m_new);   // keys past the end: 0
    l_part = l_part * alpha + ((pr[0] + pr[1]) + (pr[2] + pr[3]));
    m_run = m_new;
    // ---- O^T = O^T * alpha + V^T P^T ----
    if (__any_sync(0xffffffffu, alpha != 1.0f)) {  // the running maxima settle after a few chunks
      const float a0 = __shfl_sync(0xffffffffu, alpha, 8 * c), a1 = __shfl_sync(0xffffffffu, alpha, 8 * c + 4);
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        o[mt][0] *= a0; o[mt][1] *= a1; o[mt][2] *= a0; o[mt][3] *= a1;
      }
    }
    // B fragments of P^T (keys x heads) are the S fragments as they stand; value and rounding remainder
    const uint32_t ph0 = pack_bf16x2(pr[0], pr[1]), ph1 = pack_bf16x2(pr[2], pr[3]);
    const uint32_t pl0 = pack_bf16x2(pr[0] - __uint_as_float(ph0 << 16), pr[1] - __uint_as_float(ph0 & 0xffff0000u));
    const uint32_t pl1 = pack_bf16x2(pr[2] - __uint_as_float(ph1 << 16), pr[3] - __uint_as_float(ph1 & 0xffff0000u));
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      uint32_t va[4];                  // A fragment of V^T: 16 elements of the head dimension x 16 keys
      const uint32_t piece = (mt & 3) * 2 + ((lane >> 3) & 1);  // of the 128-byte row of box mt / 4
      ldmatrix_x4_trans(va, vs_addr + (mt >> 2) * Cfg::kBoxBytes + ((lane >> 4) * 8 + row7) * 128 + ((piece ^ row7) << 4));
      mma_16816(o[mt], va[0], va[1], va[2], va[3], ph0, ph1);
      mma_16816(o[mt], va[0], va[1], va[2], va[3], pl0, pl1);
    }
    __syncwarp();                                  // every lane is done with the stage before it is refilled
    done = i + 1;
  }
  if (lane == 0)                                   // after a wait that gave up: no copy may still be in flight
    for (int j = done; j < issued; ++j)
      mbar_wait_drain(&full[warp][j % kDecStages], (j / kDecStages) & 1, p.hdr, SITE_DECODE_WAIT);
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 1);
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 2);
  // ---- the warps of the CTA merge through shared memory (the rings are idle: every copy was waited for) ----
  __syncthreads();
  float* mo = reinterpret_cast<float*>(smem);                                  // [warps][8 heads][D]
  float2* mml = reinterpret_cast<float2*>(mo + kDecWarps * kDecHeads * D);     // [warps][8 heads]
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    float* row0 = mo + (warp * kDecHeads + 2 * c) * D + mt * 16 + quad;
    row0[0] = o[mt][0]; row0[D] = o[mt][1]; row0[8] = o[mt][2]; row0[D + 8] = o[mt][3];
  }
  if (c == 0) mml[warp * kDecHeads + quad] = make_float2(ok ? m_run : -INFINITY, ok ? l_part : 0.0f);
  __syncthreads();
  for (int i = t; i < G * D; i += kDecThreads) {
    const int h = i / D, col = i - h * D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, mml[w * kDecHeads + h].x);
    float L = 0.0f, acc = 0.0f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) {
      const float2 ml = mml[w * kDecHeads + h];
      const float f = ml.x == -INFINITY ? 0.0f : ex2(ml.x - M);        // warps without keys weigh nothing
      L = fmaf(ml.y, f, L);
      acc = fmaf(mo[(w * kDecHeads + h) * D + col], f, acc);
    }
    if (n_splits == 1) {
      // the only split of this (sequence, KV head): the result is final, no merge kernel follows
      const size_t row = static_cast<size_t>(b) * p.n_q_heads + g * G + h;
      p.out[row * D + col] = L > 0.0f ? acc / L : 0.0f;
      if (p.lse != nullptr && col == 0) p.lse[row] = (M + log2f(L)) * 0.6931471805599453f;
    } else {
      if (col == 0) p.part_ml[part + h] = make_float2(M, L);
      p.part_o[(part + h) * D + col] = acc;
    }
  }
}

// Merges the splits of one (sequence, query head): out = sum_s o_s 2^(m_s - M) / sum_s l_s 2^(m_s - M).
// The per-split factors are built once in shared memory; the sums over splits are fixed-order loops with
// several independent loads in flight.
template <int D>
__global__ void __launch_bounds__(D) decode_combine_kernel(const DecodeParams p, int n_splits) {
  __shared__ float f_s[kDecodeMaxSplits];
  __shared__ float l_s[kDecodeMaxSplits];
  pdl_wait();
  const int h = blockIdx.x, b = blockIdx.y, t = threadIdx.x;
  const int G = p.group, g = h / G, hl = h - g * G;
  const size_t base = (static_cast<size_t>(b) * p.n_kv_heads + g) * n_splits;
  if (t < n_splits) {
    const float2 ml = p.part_ml[(base + t) * G + hl];
    f_s[t] = ml.x;
    l_s[t] = ml.y;
  }
  __syncthreads();
  float M = -INFINITY;
  for (int s = 0; s < n_splits; ++s) M = fmaxf(M, f_s[s]);
  __syncthreads();
  if (t < n_splits) f_s[t] = (f_s[t] == -INFINITY) ? 0.0f : ex2(f_s[t] - M);     // empty splits weigh nothing
  __syncthreads();
  float L = 0.0f, acc = 0.0f;
  for (int s = 0; s < n_splits; ++s) L = fmaf(l_s[s], f_s[s], L);
  const float* o = p.part_o + (base * G + hl) * D + t;
#pragma unroll 16
  for (int s = 0; s < n_splits; ++s) acc = fmaf(__ldg(o + static_cast<size_t>(s) * G * D), f_s[s], acc);
  p.out[(static_cast<size_t>(b) * p.n_q_heads + h) * D + t] = L > 0.0f ? acc / L : 0.0f;
  if (p.lse != nullptr && t == 0) p.lse[static_cast<size_t>(b) * p.n_q_heads + h] = (M + log2f(L)) * 0.6931471805599453f;
}

size_t decode_workspace_bytes(int batch, int n_kv_heads, int group, int head_dim) {
  const size_t parts = static_cast<size_t>(batch) * n_kv_heads * kDecodeMaxSplits * group;
  return sizeof(WorkspaceHeader) + (parts * sizeof(float2) + 255) / 256 * 256 + parts * head_dim * sizeof(float);
}

template <int D, int kDecWarps>
static cudaError_t launch_decode_w(const CUtensorMap& tk, const CUtensorMap& tv, DecodeParams& p, int batch, int k_max,
                                   cudaStream_t stream, int* launches, int* capacity_out) {
  constexpr int kSmem = DecCfg<D, kDecWarps>::kSmem;
  constexpr int kDecThreads = 32 * kDecWarps;
  // launch attributes and occupancy are per device: cached by device ordinal
  static PerDeviceOnce configured;
  static int capacity_of[PerDeviceOnce::kMaxDevices];
  int dev = 0;
  cudaError_t e0 = cudaGetDevice(&dev);
  if (e0 != cudaSuccess) return e0;
  if (dev < 0 || dev >= PerDeviceOnce::kMaxDevices) return cudaErrorInvalidDevice;
  if (!configured.done(dev)) {
    cudaError_t e = cudaFuncSetAttribute(decode_attn_kernel<D, kDecWarps>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    // one wave: as many splits as keep every CTA resident at once
    int sms = 148, per_sm = 1;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_attn_kernel<D, kDecWarps>, kDecThreads, kSmem) != cudaSuccess || per_sm < 1)
      per_sm = 1;
    capacity_of[dev] = sms * per_sm;
    configured.set(dev);
  }
  const int capacity = capacity_of[dev];
  if (capacity_out != nullptr) {                 // only asked how many CTAs this shape of CTA keeps resident
    *capacity_out = capacity;
    return cudaSuccess;
  }
  int splits = capacity / (batch * p.n_kv_heads);
  const int chunks = (k_max + kDecChunk - 1) / kDecChunk;
  const int useful = (chunks + kDecWarps - 1) / kDecWarps;      // at least one chunk per warp
  if (splits > useful) splits = useful;
  if (splits > kDecodeMaxSplits) splits = kDecodeMaxSplits;
  if (splits < 1) splits = 1;
  decode_attn_kernel<D, kDecWarps><<<dim3(splits, p.n_kv_heads, batch), kDecThreads, kSmem, stream>>>(tk, tv, p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  *launches = 1;
  if (splits == 1) return cudaSuccess;          // the split kernel wrote the output itself
  *launches = 2;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.n_q_heads, batch);
  cfg.blockDim = dim3(D);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  fill_pdl_attribute(&attr[0]);
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_combine_kernel<D>, static_cast<const DecodeParams&>(p), splits);
}

template <int D>
static cudaError_t launch_decode_d(const CUtensorMap& tk, const CUtensorMap& tv, DecodeParams& p, int batch, int k_max,
                                   cudaStream_t stream, int* launches) {
  int big = 0;
  cudaError_t e = launch_decode_w<D, 8>(tk, tv, p, batch, k_max, stream, launches, &big);
  if (e != cudaSuccess) return e;
  // more (KV head, sequence) pairs than one-CTA-per-SM holds: the small CTAs, two per SM, keep the launch in one wave
  if (batch * p.n_kv_heads > big) return launch_decode_w<D, 4>(tk, tv, p, batch, k_max, stream, launches, nullptr);
  return launch_decode_w<D, 8>(tk, tv, p, batch, k_max, stream, launches, nullptr);
}

cudaError_t launch_decode_attn(const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, DecodeParams& p, int head_dim, int batch,
                               int k_max, cudaStream_t stream, int* launches) {
  *launches = 0;
  if (head_dim == 128) return launch_decode_d<128>(tmap_k, tmap_v, p, batch, k_max, stream, launches);
  if (head_dim == 64) return launch_decode_d<64>(tmap_k, tmap_v, p, batch, k_max, stream, launches);
  return cudaErrorInvalidValue;
}

}  // namespace fastkv
