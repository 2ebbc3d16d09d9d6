// Decode-time attention of one new query token over the compressed KV cache that fastkv_compact
// leaves behind ([Hkv, kept, d] per sequence): the stage the retained KV of Alg. 1 exists for.
//
// Memory-bound (every kept K and V row is read once, 4 * d bytes per kept entry and KV head) with G
// query rows per KV head, so it runs on the CUDA cores: split-KV, one CTA per (key range, KV head,
// sequence).  K/V chunks of 128 kept entries are contiguous in the compact layout and are pulled into
// a three-deep ring of shared-memory stages with one bulk copy each.  For Q.K^T the d / 8 lanes that
// share a key each take 16 bytes of its row and keep their slice of the group's queries in registers
// (one shuffle reduction per key and head); an online softmax keeps per-head (max, sum); for the P.V
// product thread t owns output dimension t.  A second small kernel
// merges the splits.
#include "decode_attn.cuh"

namespace fastkv {

namespace {

constexpr int kDecThreads = 128;
constexpr int kDecChunk = 64;       // kept entries per shared-memory stage
constexpr int kDecStages = 3;       // stages in flight (K and V of 64 entries each): 96 KB, two CTAs per SM
constexpr int kMaxGroup = 8;

__device__ __forceinline__ void bulk_load_1d(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(smem_dst)),
      "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

}  // namespace

template <int D>
__global__ void __launch_bounds__(kDecThreads) decode_attn_kernel(const DecodeParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~static_cast<uintptr_t>(127));
  constexpr int kStageBytes = kDecChunk * D * 2;
  uint8_t* k_stage = smem;                                   // [stages][chunk][D] bf16
  uint8_t* v_stage = smem + kDecStages * kStageBytes;        // [stages][chunk][D] bf16 each
  float* q_s = reinterpret_cast<float*>(smem + 2 * kDecStages * kStageBytes);      // [G][D], scaled, log2 units
  float* p_s = q_s + kMaxGroup * D;                                    // [chunk][kMaxGroup]
  float* s_s = p_s + kDecChunk * kMaxGroup;                            // [chunk][kMaxGroup] raw logits of the chunk
  float* scratch = s_s + kDecChunk * kMaxGroup;                        // [4 * kMaxGroup]
  __shared__ uint64_t full[kDecStages];
  __shared__ int abort_flag;

  const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int G = p.group, n_splits = gridDim.x;
  const int seg0 = p.cu_k ? p.cu_k[b] : b * p.k_uniform;
  const int kept = p.cu_k ? p.cu_k[b + 1] - seg0 : p.k_uniform;
  const int per = ((kept + n_splits - 1) / n_splits + kDecChunk - 1) / kDecChunk * kDecChunk;   // whole chunks
  const int j0 = split * per, j1 = min(kept, j0 + per);
  const size_t part = ((static_cast<size_t>(b) * p.n_kv_heads + g) * n_splits + split) * G;

  pdl_wait();
  if (t == 0) {
    for (int i = 0; i < kDecStages; ++i) mbar_init(&full[i], 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  // the group's queries, in fp32, multiplied by scale * log2(e)
  for (int i = t; i < kMaxGroup * D; i += kDecThreads) {
    const int h = i / D, c = i - h * D;
    const uint16_t bits = h < G ? p.q[(static_cast<size_t>(b) * p.n_q_heads + g * G + h) * D + c] : 0;
    q_s[i] = __uint_as_float(static_cast<uint32_t>(bits) << 16) * p.scale_log2;      // absent heads: zeros
  }
  for (int i = t; i < kDecChunk * kMaxGroup; i += kDecThreads) p_s[i] = 0.0f;   // columns of absent heads stay 0
  __syncthreads();

  float m_run[kMaxGroup], l_t[kMaxGroup], o[kMaxGroup];
#pragma unroll
  for (int h = 0; h < kMaxGroup; ++h) { m_run[h] = -INFINITY; l_t[h] = 0.0f; o[h] = 0.0f; }

  const uint8_t* k_head = reinterpret_cast<const uint8_t*>(p.k_cache) + (static_cast<size_t>(g) * p.ld_cache + seg0) * D * 2;
  const uint8_t* v_head = reinterpret_cast<const uint8_t*>(p.v_cache) + (static_cast<size_t>(g) * p.ld_cache + seg0) * D * 2;
  const int n_chunks = j1 > j0 ? (j1 - j0 + kDecChunk - 1) / kDecChunk : 0;
  auto issue = [&](int c) {            // thread 0: one bulk copy for the K rows and one for the V rows of chunk c
    const int r0 = j0 + c * kDecChunk, rows = min(kDecChunk, j1 - r0);
    const uint32_t bytes = static_cast<uint32_t>(rows) * D * 2;
    mbar_arrive_expect_tx(&full[c % kDecStages], 2 * bytes);
    bulk_load_1d(k_stage + (c % kDecStages) * kStageBytes, k_head + static_cast<size_t>(r0) * D * 2, bytes, &full[c % kDecStages]);
    bulk_load_1d(v_stage + (c % kDecStages) * kStageBytes, v_head + static_cast<size_t>(r0) * D * 2, bytes, &full[c % kDecStages]);
  };
  if (t == 0)
    for (int c = 0; c < kDecStages - 1 && c < n_chunks; ++c) issue(c);
  bool ok = true;
  for (int c = 0; c < n_chunks; ++c) {
    if (t == 0 && c + kDecStages - 1 < n_chunks) issue(c + kDecStages - 1);   // that stage was released by the barrier below
    ok = mbar_wait_bounded(&full[c % kDecStages], (c / kDecStages) & 1, &abort_flag, p.hdr, SITE_DECODE_WAIT);
    if (!__syncthreads_and(ok)) break;
    const int rows = min(kDecChunk, j1 - j0 - c * kDecChunk);
    // ---- S = Q K^T: D / 8 lanes share a key (16 bytes of the row each), the warps share the chunk's keys ----
    constexpr int kLanesPerKey = D / 8, kKeysPerIter = 32 / kLanesPerKey, kKeysPerWarp = kDecChunk / 4;
    {
      const int sub = lane / kLanesPerKey, cc = lane % kLanesPerKey;
      for (int h0 = 0; h0 < G; h0 += 4) {                  // four query heads at a time (register budget)
        float qr[4][8];
#pragma unroll
        for (int hh = 0; hh < 4; ++hh) {
          const float4 qa = *reinterpret_cast<const float4*>(q_s + (h0 + hh) * D + cc * 8);
          const float4 qb = *reinterpret_cast<const float4*>(q_s + (h0 + hh) * D + cc * 8 + 4);
          qr[hh][0] = qa.x; qr[hh][1] = qa.y; qr[hh][2] = qa.z; qr[hh][3] = qa.w;
          qr[hh][4] = qb.x; qr[hh][5] = qb.y; qr[hh][6] = qb.z; qr[hh][7] = qb.w;
        }
        for (int it = 0; it < kKeysPerWarp / kKeysPerIter; ++it) {
          const int kk = warp * kKeysPerWarp + it * kKeysPerIter + sub;      // key of this lane group
          const uint4 kv = *reinterpret_cast<const uint4*>(k_stage + (c % kDecStages) * kStageBytes + kk * D * 2 + cc * 16);
          const uint32_t w[4] = {kv.x, kv.y, kv.z, kv.w};
          float kf[8];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            kf[2 * e] = __uint_as_float(w[e] << 16);
            kf[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
          }
          float acc[4];
#pragma unroll
          for (int hh = 0; hh < 4; ++hh) {
            float a = 0.0f;
#pragma unroll
            for (int e = 0; e < 8; ++e) a = fmaf(kf[e], qr[hh][e], a);
#pragma unroll
            for (int off = kLanesPerKey / 2; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
            acc[hh] = a;
          }
          if (cc == 0) {
#pragma unroll
            for (int hh = 0; hh < 4; ++hh)
              if (h0 + hh < G) s_s[kk * kMaxGroup + h0 + hh] = (kk < rows) ? acc[hh] : -INFINITY;
          }
        }
      }
    }
    __syncthreads();
    const int key = t & (kDecChunk - 1), hsel = t >> 6;      // softmax: thread t takes key t % 64, heads h % 2 == t / 64
    float s[kMaxGroup];
#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h) s[h] = (h < G && (h & 1) == hsel) ? s_s[key * kMaxGroup + h] : -INFINITY;
    // ---- online softmax per head: chunk max (one reduction round for all heads), rescale factor, probabilities ----
    float alpha[kMaxGroup];
#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h) {
      float v = s[h];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
      if (lane == 0) scratch[warp * kMaxGroup + h] = v;
    }
    __syncthreads();
#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h) {
      alpha[h] = 1.0f;
      if (h < G) {
        const float m_chunk = fmaxf(fmaxf(scratch[h], scratch[kMaxGroup + h]), fmaxf(scratch[2 * kMaxGroup + h], scratch[3 * kMaxGroup + h]));
        const float m_new = fmaxf(m_run[h], m_chunk);
        alpha[h] = ex2(m_run[h] - m_new);                    // first chunk: 2^-inf = 0
        const float pr = ex2(s[h] - m_new);                  // rows past the end and other threads' heads: 0
        if ((h & 1) == hsel) p_s[key * kMaxGroup + h] = pr;
        l_t[h] = l_t[h] * alpha[h] + pr;
        m_run[h] = m_new;
      }
    }
    __syncthreads();
    // ---- O = O * alpha + P V: thread t owns output dimension t ----
    if (t < D) {
#pragma unroll
      for (int h = 0; h < kMaxGroup; ++h) o[h] *= alpha[h];
      const uint16_t* vcol = reinterpret_cast<const uint16_t*>(v_stage + (c % kDecStages) * kStageBytes) + t;
      if (G <= 4) {
#pragma unroll 8
        for (int j = 0; j < rows; ++j) {
          const float vf = __uint_as_float(static_cast<uint32_t>(vcol[j * D]) << 16);
          const float4 pa = *reinterpret_cast<const float4*>(p_s + j * kMaxGroup);
          o[0] = fmaf(pa.x, vf, o[0]); o[1] = fmaf(pa.y, vf, o[1]); o[2] = fmaf(pa.z, vf, o[2]); o[3] = fmaf(pa.w, vf, o[3]);
        }
      } else {
#pragma unroll 4
        for (int j = 0; j < rows; ++j) {
          const float vf = __uint_as_float(static_cast<uint32_t>(vcol[j * D]) << 16);
          const float4 pa = *reinterpret_cast<const float4*>(p_s + j * kMaxGroup);
          const float4 pb = *reinterpret_cast<const float4*>(p_s + j * kMaxGroup + 4);
          o[0] = fmaf(pa.x, vf, o[0]); o[1] = fmaf(pa.y, vf, o[1]); o[2] = fmaf(pa.z, vf, o[2]); o[3] = fmaf(pa.w, vf, o[3]);
          o[4] = fmaf(pb.x, vf, o[4]); o[5] = fmaf(pb.y, vf, o[5]); o[6] = fmaf(pb.z, vf, o[6]); o[7] = fmaf(pb.w, vf, o[7]);
        }
      }
    }
    __syncthreads();                                         // stage (c & 1) and p_s may be overwritten
  }
  // ---- this split's (max, sum, unnormalised output) per head ----
#pragma unroll
  for (int h = 0; h < kMaxGroup; ++h) {
    if (h < G) {
      float l = l_t[h];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
      if (lane == 0) scratch[warp * kMaxGroup + h] = l;
    }
  }
  __syncthreads();
#pragma unroll
  for (int h = 0; h < kMaxGroup; ++h) {
    if (h < G) {
      if (t == 0)
        p.part_ml[part + h] = make_float2(ok ? m_run[h] : -INFINITY,
                                          scratch[h] + scratch[kMaxGroup + h] + scratch[2 * kMaxGroup + h] + scratch[3 * kMaxGroup + h]);
      if (t < D) p.part_o[(part + h) * D + t] = o[h];
    }
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

template <int D>
static cudaError_t launch_decode_t(DecodeParams& p, int batch, int k_max, cudaStream_t stream) {
  constexpr int kSmem = 2 * kDecStages * kDecChunk * D * 2 + kMaxGroup * D * 4 + 2 * kDecChunk * kMaxGroup * 4 + 4 * kMaxGroup * 4 + 128;
  // launch attributes and occupancy are per device: cached by device ordinal
  static PerDeviceOnce configured;
  static int capacity_of[PerDeviceOnce::kMaxDevices];
  int dev = 0;
  cudaError_t e0 = cudaGetDevice(&dev);
  if (e0 != cudaSuccess) return e0;
  if (dev < 0 || dev >= PerDeviceOnce::kMaxDevices) return cudaErrorInvalidDevice;
  if (!configured.done(dev)) {
    cudaError_t e = cudaFuncSetAttribute(decode_attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    // one wave: as many splits as keep every CTA resident at once, at least one chunk per split
    int sms = 148, per_sm = 1;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_attn_kernel<D>, kDecThreads, kSmem) != cudaSuccess || per_sm < 1)
      per_sm = 1;
    capacity_of[dev] = sms * per_sm;
    configured.set(dev);
  }
  const int capacity = capacity_of[dev];
  int splits = capacity / (batch * p.n_kv_heads);
  const int chunks = (k_max + kDecChunk - 1) / kDecChunk;
  if (splits > chunks) splits = chunks;
  if (splits > kDecodeMaxSplits) splits = kDecodeMaxSplits;
  if (splits < 1) splits = 1;
  decode_attn_kernel<D><<<dim3(splits, p.n_kv_heads, batch), kDecThreads, kSmem, stream>>>(p);
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

cudaError_t launch_decode_attn(DecodeParams& p, int head_dim, int batch, int k_max, cudaStream_t stream) {
  if (head_dim == 128) return launch_decode_t<128>(p, batch, k_max, stream);
  if (head_dim == 64) return launch_decode_t<64>(p, batch, k_max, stream);
  return cudaErrorInvalidValue;
}

}  // namespace fastkv
