// Decode-time attention of one new query token over the compressed KV cache that fastkv_compact
// leaves behind ([Hkv, kept, d] per sequence): the stage the retained KV of Alg. 1 exists for.
//
// Memory-bound (every kept K and V row is read once, 4 * d bytes per kept entry and KV head) with G <= 8
// query rows per KV head, so it runs on the CUDA cores.  Split-KV: one CTA per (key range, KV head,
// sequence), and inside the CTA every warp works on its own: it owns a ring of shared-memory stages
// that one lane fills with bulk copies (16 kept entries of K and of V per stage: they are contiguous in
// the compact layout), keeps its slice of the group's queries and of the output in registers (the 32
// lanes split the head dimension), and runs its own online softmax.  No CTA-wide barrier in the loop.
// Per round of 32 / GP keys (GP = group size padded to 2, 4 or 8) the lanes' partial dot products are
// summed by a transposing butterfly (31 exchanges for 32 values; lane r ends up with key r / GP, head
// r % GP), the probabilities are broadcast back by shuffles for the P.V product.  The warps of a CTA
// merge through shared memory at the end; a second small kernel merges the splits.
#include "decode_attn.cuh"

namespace fastkv {

namespace {

constexpr int kDecStages = 3;       // stages per warp: two chunks in flight while one is consumed
constexpr int kMaxGroup = 8;
// Warps per CTA and kept entries per stage: a stage holds at least one round of 32 / GP keys; with small stages
// sixteen warps fit one SM's shared memory and hide each other's shuffle and exponential latencies.
template <int GP> struct DecShape {
  static constexpr int kWarps = GP >= 4 ? 16 : 8;
  static constexpr int kChunk = GP >= 4 ? 8 : 16;
};

__device__ __forceinline__ void bulk_load_1d(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(smem_dst)),
      "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

// Sum of v[i] over the 32 lanes for every i = 0..31: on return lane r holds the total of v[r] in v[0].
__device__ __forceinline__ void transpose_sum32(float (&v)[32], int lane) {
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) {
    const bool upper = (lane & o) != 0;
#pragma unroll
    for (int i = 0; i < o; ++i) {
      const float send = upper ? v[i] : v[i + o];
      const float keep = upper ? v[i + o] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
    }
  }
}

template <int D, int GP>
struct DecCfg {
  static constexpr int kDecWarps = DecShape<GP>::kWarps, kDecChunk = DecShape<GP>::kChunk;
  static constexpr int kRowBytes = D * 2;
  static constexpr int kHalfBytes = kDecChunk * kRowBytes;            // K (or V) rows of one stage
  static constexpr int kStageBytes = 2 * kHalfBytes;
  static constexpr int kRingBytes = kDecWarps * kDecStages * kStageBytes;
  static constexpr int kMergeBytes = kDecWarps * GP * (D + 2) * 4;    // the warps' outputs and (max, sum)
  static constexpr int kSmem = (kRingBytes > kMergeBytes ? kRingBytes : kMergeBytes) + 128;
};

}  // namespace

template <int D, int GP>
__global__ void __launch_bounds__(32 * DecShape<GP>::kWarps) decode_attn_kernel(const DecodeParams p) {
  using Cfg = DecCfg<D, GP>;
  constexpr int kDecWarps = Cfg::kDecWarps, kDecChunk = Cfg::kDecChunk, kDecThreads = 32 * kDecWarps;
  constexpr int EPL = D / 32;                   // elements of the head dimension per lane
  constexpr int KPR = 32 / GP;                  // keys per round
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~static_cast<uintptr_t>(127));
  __shared__ uint64_t full[kDecWarps][kDecStages];
  __shared__ int abort_flag;

  const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int G = p.group, n_splits = gridDim.x;
  const int seg0 = p.cu_k ? p.cu_k[b] : b * p.k_uniform;
  const int kept = p.cu_k ? p.cu_k[b + 1] - seg0 : p.k_uniform;
  // the CTA's range of chunks, dealt to its warps round robin
  const int n_chunks_all = (kept + kDecChunk - 1) / kDecChunk;
  const int per = (n_chunks_all + n_splits - 1) / n_splits;
  const int c0 = split * per, c1 = min(n_chunks_all, c0 + per);
  const int my_chunks = c1 - c0 > warp ? (c1 - c0 - warp + kDecWarps - 1) / kDecWarps : 0;
  const size_t part = ((static_cast<size_t>(b) * p.n_kv_heads + g) * n_splits + split) * G;

  pdl_wait();
  if (lane == 0) {
    for (int i = 0; i < kDecStages; ++i) mbar_init(&full[warp][i], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (t == 0) abort_flag = 0;
  __syncthreads();

  // this lane's slice of the group's queries, in fp32, multiplied by scale * log2(e); absent heads are zero
  float q[GP][EPL];
#pragma unroll
  for (int h = 0; h < GP; ++h) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const uint16_t bits = h < G ? p.q[(static_cast<size_t>(b) * p.n_q_heads + g * G + h) * D + lane * EPL + e] : 0;
      q[h][e] = __uint_as_float(static_cast<uint32_t>(bits) << 16) * p.scale_log2;
    }
  }
  float o[GP][EPL];
#pragma unroll
  for (int h = 0; h < GP; ++h)
#pragma unroll
    for (int e = 0; e < EPL; ++e) o[h][e] = 0.0f;
  float m_run = -INFINITY, l_run = 0.0f;        // of head lane % GP (the lanes of one head hold equal copies)

  const uint8_t* k_head = reinterpret_cast<const uint8_t*>(p.k_cache) + (static_cast<size_t>(g) * p.ld_cache + seg0) * Cfg::kRowBytes;
  const uint8_t* v_head = reinterpret_cast<const uint8_t*>(p.v_cache) + (static_cast<size_t>(g) * p.ld_cache + seg0) * Cfg::kRowBytes;
  uint8_t* const ring = smem + warp * kDecStages * Cfg::kStageBytes;
  auto issue = [&](int i) {            // lane 0: one bulk copy for the K rows and one for the V rows of this warp's i-th chunk
    const int r0 = (c0 + warp + i * kDecWarps) * kDecChunk, rows = min(kDecChunk, kept - r0);
    const uint32_t bytes = static_cast<uint32_t>(rows) * Cfg::kRowBytes;
    uint64_t* bar = &full[warp][i % kDecStages];
    uint8_t* stage = ring + (i % kDecStages) * Cfg::kStageBytes;
    mbar_arrive_expect_tx(bar, 2 * bytes);
    bulk_load_1d(stage, k_head + static_cast<size_t>(r0) * Cfg::kRowBytes, bytes, bar);
    bulk_load_1d(stage + Cfg::kHalfBytes, v_head + static_cast<size_t>(r0) * Cfg::kRowBytes, bytes, bar);
  };
  int issued = 0;                      // lane 0: chunks whose copies have been started
  if (lane == 0)
    for (; issued < kDecStages - 1 && issued < my_chunks; ++issued) issue(issued);
  bool ok = true;
  int done = 0;                        // chunks consumed
  for (int i = 0; i < my_chunks; ++i) {
    if (lane == 0 && i + kDecStages - 1 < my_chunks) issue(issued++);   // that stage was consumed last iteration
    ok = mbar_wait_bounded(&full[warp][i % kDecStages], (i / kDecStages) & 1, &abort_flag, p.hdr, SITE_DECODE_WAIT);
    if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
    const uint8_t* ks = ring + (i % kDecStages) * Cfg::kStageBytes;
    const uint8_t* vs = ks + Cfg::kHalfBytes;
    const int rows = min(kDecChunk, kept - (c0 + warp + i * kDecWarps) * kDecChunk);
#pragma unroll
    for (int r0 = 0; r0 < kDecChunk; r0 += KPR) {
      if (r0 >= rows) break;                       // warp-uniform
      // ---- S = Q K^T for KPR keys: every lane its slice of the head dimension, then the transposing sum ----
      float s[32];
#pragma unroll
      for (int kk = 0; kk < KPR; ++kk) {
        float kf[EPL];
        if (EPL == 4) {
          const uint2 w = *reinterpret_cast<const uint2*>(ks + (r0 + kk) * Cfg::kRowBytes + lane * 8);
          kf[0] = __uint_as_float(w.x << 16); kf[1] = __uint_as_float(w.x & 0xffff0000u);
          kf[2 % EPL] = __uint_as_float(w.y << 16); kf[3 % EPL] = __uint_as_float(w.y & 0xffff0000u);
        } else {
          const uint32_t w = *reinterpret_cast<const uint32_t*>(ks + (r0 + kk) * Cfg::kRowBytes + lane * 4);
          kf[0] = __uint_as_float(w << 16); kf[1 % EPL] = __uint_as_float(w & 0xffff0000u);
        }
#pragma unroll
        for (int h = 0; h < GP; ++h) {
          float a = 0.0f;
#pragma unroll
          for (int e = 0; e < EPL; ++e) a = fmaf(kf[e], q[h][e], a);
          s[kk * GP + h] = a;
        }
      }
      transpose_sum32(s, lane);
      // lane r: key r0 + r / GP, head r % GP
      float sv = (r0 + lane / GP < rows) ? s[0] : -INFINITY;
      // ---- online softmax of the head: the lanes of one head are GP apart ----
      float mx = sv;
#pragma unroll
      for (int off = GP; off < 32; off <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
      const float m_new = fmaxf(m_run, mx);        // finite: the round has at least one key
      const float alpha = ex2(m_run - m_new);      // first round: 2^-inf = 0
      const float pr = ex2(sv - m_new);            // keys past the end: 0
      float ps = pr;
#pragma unroll
      for (int off = GP; off < 32; off <<= 1) ps += __shfl_xor_sync(0xffffffffu, ps, off);
      l_run = l_run * alpha + ps;
      m_run = m_new;
      // ---- O = O * alpha + P V: every lane its slice of the head dimension ----
#pragma unroll
      for (int h = 0; h < GP; ++h) {
        const float ah = __shfl_sync(0xffffffffu, alpha, h);
#pragma unroll
        for (int e = 0; e < EPL; ++e) o[h][e] *= ah;
      }
#pragma unroll
      for (int kk = 0; kk < KPR; ++kk) {
        if (r0 + kk >= rows) break;                // rows past the end were never copied: their bytes are not data
        float vf[EPL];
        if (EPL == 4) {
          const uint2 w = *reinterpret_cast<const uint2*>(vs + (r0 + kk) * Cfg::kRowBytes + lane * 8);
          vf[0] = __uint_as_float(w.x << 16); vf[1] = __uint_as_float(w.x & 0xffff0000u);
          vf[2 % EPL] = __uint_as_float(w.y << 16); vf[3 % EPL] = __uint_as_float(w.y & 0xffff0000u);
        } else {
          const uint32_t w = *reinterpret_cast<const uint32_t*>(vs + (r0 + kk) * Cfg::kRowBytes + lane * 4);
          vf[0] = __uint_as_float(w << 16); vf[1 % EPL] = __uint_as_float(w & 0xffff0000u);
        }
#pragma unroll
        for (int h = 0; h < GP; ++h) {
          const float ph = __shfl_sync(0xffffffffu, pr, kk * GP + h);
#pragma unroll
          for (int e = 0; e < EPL; ++e) o[h][e] = fmaf(ph, vf[e], o[h][e]);
        }
      }
    }
    __syncwarp();                                  // every lane is done with the stage before lane 0 refills it
    done = i + 1;
  }
  if (lane == 0)                                   // after a wait that gave up: no copy may still be in flight
    for (int j = done; j < issued; ++j)
      mbar_wait_drain(&full[warp][j % kDecStages], (j / kDecStages) & 1, p.hdr, SITE_DECODE_WAIT);
  // ---- the warps of the CTA merge through shared memory (the rings are idle: every copy was waited for) ----
  __syncthreads();
  float* mo = reinterpret_cast<float*>(smem);                          // [warps][GP][D]
  float2* mml = reinterpret_cast<float2*>(mo + kDecWarps * GP * D);    // [warps][GP]
#pragma unroll
  for (int h = 0; h < GP; ++h)
#pragma unroll
    for (int e = 0; e < EPL; ++e) mo[(warp * GP + h) * D + lane * EPL + e] = o[h][e];
  if (lane < GP) mml[warp * GP + lane] = make_float2(ok ? m_run : -INFINITY, ok ? l_run : 0.0f);
  __syncthreads();
  for (int i = t; i < G * D; i += kDecThreads) {
    const int h = i / D, c = i - h * D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, mml[w * GP + h].x);
    float L = 0.0f, acc = 0.0f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) {
      const float2 ml = mml[w * GP + h];
      const float f = ml.x == -INFINITY ? 0.0f : ex2(ml.x - M);        // warps without keys weigh nothing
      L = fmaf(ml.y, f, L);
      acc = fmaf(mo[(w * GP + h) * D + c], f, acc);
    }
    if (c == 0) p.part_ml[part + h] = make_float2(M, L);
    p.part_o[(part + h) * D + c] = acc;
  }
  pdl_launch_dependents();
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

template <int D, int GP>
static cudaError_t launch_decode_t(DecodeParams& p, int batch, int k_max, cudaStream_t stream) {
  constexpr int kSmem = DecCfg<D, GP>::kSmem;
  constexpr int kDecWarps = DecShape<GP>::kWarps, kDecChunk = DecShape<GP>::kChunk, kDecThreads = 32 * kDecWarps;
  // launch attributes and occupancy are per device: cached by device ordinal
  static PerDeviceOnce configured;
  static int capacity_of[PerDeviceOnce::kMaxDevices];
  int dev = 0;
  cudaError_t e0 = cudaGetDevice(&dev);
  if (e0 != cudaSuccess) return e0;
  if (dev < 0 || dev >= PerDeviceOnce::kMaxDevices) return cudaErrorInvalidDevice;
  if (!configured.done(dev)) {
    cudaError_t e = cudaFuncSetAttribute(decode_attn_kernel<D, GP>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    // one wave: as many splits as keep every CTA resident at once
    int sms = 148, per_sm = 1;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_attn_kernel<D, GP>, kDecThreads, kSmem) != cudaSuccess || per_sm < 1)
      per_sm = 1;
    capacity_of[dev] = sms * per_sm;
    configured.set(dev);
  }
  const int capacity = capacity_of[dev];
  int splits = capacity / (batch * p.n_kv_heads);
  const int chunks = (k_max + kDecChunk - 1) / kDecChunk;
  const int useful = (chunks + kDecWarps - 1) / kDecWarps;      // at least one chunk per warp
  if (splits > useful) splits = useful;
  if (splits > kDecodeMaxSplits) splits = kDecodeMaxSplits;
  if (splits < 1) splits = 1;
  decode_attn_kernel<D, GP><<<dim3(splits, p.n_kv_heads, batch), kDecThreads, kSmem, stream>>>(p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
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
static cudaError_t launch_decode_d(DecodeParams& p, int batch, int k_max, cudaStream_t stream) {
  if (p.group <= 2) return launch_decode_t<D, 2>(p, batch, k_max, stream);    // one head: the second one is a zero query
  if (p.group <= 4) return launch_decode_t<D, 4>(p, batch, k_max, stream);
  return launch_decode_t<D, 8>(p, batch, k_max, stream);
}

cudaError_t launch_decode_attn(DecodeParams& p, int head_dim, int batch, int k_max, cudaStream_t stream) {
  if (head_dim == 128) return launch_decode_d<128>(p, batch, k_max, stream);
  if (head_dim == 64) return launch_decode_d<64>(p, batch, k_max, stream);
  return cudaErrorInvalidValue;
}

}  // namespace fastkv
