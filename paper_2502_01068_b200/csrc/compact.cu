// Compaction of the kept K/V rows, hidden states and position ids (Alg. 1: C <- update(K, V);
// the reduced hidden states x).  Pure byte movement, done with the bulk-copy engine: every warp
// owns a small ring of 8 KB shared-memory stages; the kept rows of a chunk are pulled in with
// cp.async.bulk (one copy per row, issued by the lane that resolved the row's index) and, because
// kept rows are contiguous in the output, pushed out again with a single bulk store per chunk.
// No data passes through registers; several chunks per warp are in flight at any time.
#include "compact.cuh"

namespace fastkv {

namespace {

constexpr int kChunkBytes = 8192;
constexpr int kStages = 4;                 // chunks in flight per warp
constexpr int kCompactWarps = 7;                 // 7 x 4 x 8 KB = 224 KB of shared memory per CTA
constexpr int kCompactThreads = kCompactWarps * 32;
constexpr int kCompactSmem = kCompactWarps * kStages * kChunkBytes + 1024;

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(smem_dst)),
      "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_u32(smem_src)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// sequence that owns output slot j: the last b with cu_k[b] <= j
__device__ __forceinline__ int owner_of_slot(const int* cu_k, int k_uniform, int batch, int j) {
  if (batch == 1) return 0;
  if (cu_k == nullptr) return j / k_uniform;
  int lo = 0, hi = batch;            // invariant: cu_k[lo] <= j < cu_k[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (cu_k[mid] <= j) lo = mid; else hi = mid;
  }
  return lo;
}

}  // namespace

__global__ void __launch_bounds__(kCompactThreads, 1) compact_rows_kernel(const CompactParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~static_cast<uintptr_t>(127));
  __shared__ uint64_t full[kCompactWarps][kStages];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t* const ring = smem + warp * kStages * kChunkBytes;
  if (lane == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(&full[warp][s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __shared__ int abort_flag;
  if (threadIdx.x == 0) abort_flag = 0;
  __syncthreads();
  pdl_wait();                  // the indices come from the kernel before this one
  pdl_launch_dependents();

  const long long gw = static_cast<long long>(blockIdx.x) * kCompactWarps + warp;
  const long long n_warps = static_cast<long long>(gridDim.x) * kCompactWarps;
  const long long my_chunks = gw < p.total_chunks ? (p.total_chunks - gw + n_warps - 1) / n_warps : 0;

  // Issue the loads of this warp's c-th chunk into stage c % kStages (warp-collective); returns what
  // lane 0 needs to store the chunk later.
  struct Pending { uint8_t* dst; uint32_t bytes; uint32_t valid; uint32_t row_bytes; };
  auto issue = [&](long long c) -> Pending {
    const long long chunk = gw + c * n_warps;
    int ji = 0;
    while (ji + 1 < p.n_jobs && chunk >= p.job[ji + 1].first_chunk) ++ji;
    const GatherJob& job = p.job[ji];
    const long long lc = chunk - job.first_chunk;
    const int s = static_cast<int>(c % kStages);
    uint8_t* const stage = ring + s * kChunkBytes;
    const long long row_bytes = static_cast<long long>(job.row_chunks) * 16;
    long long r;                       // output row of this lane
    uint32_t bytes, src_off = 0;       // bytes this lane copies, offset inside the source row
    bool active;
    if (job.pieces_per_row > 1) {      // long rows: one piece of one row per chunk, lane 0 copies it
      r = lc / job.pieces_per_row;
      src_off = static_cast<uint32_t>(lc - r * job.pieces_per_row) * kChunkBytes;
      bytes = static_cast<uint32_t>(min(static_cast<long long>(kChunkBytes), row_bytes - src_off));
      active = lane == 0;
    } else {                           // short rows: up to 32 rows per chunk, one per lane
      r = lc * job.rows_per_chunk + lane;
      bytes = static_cast<uint32_t>(row_bytes);
      active = lane < job.rows_per_chunk && r < static_cast<long long>(job.heads) * job.rows;
    }
    const uint8_t* src = nullptr;
    bool valid = false;
    if (active) {
      const int head = static_cast<int>(r / job.rows);
      const int j = static_cast<int>(r - static_cast<long long>(head) * job.rows);
      const int b = owner_of_slot(job.cu_k, job.k_uniform, p.batch, j);
      const int row0 = p.cu_seqlens ? p.cu_seqlens[b] : 0;
      const int L = p.cu_seqlens ? p.cu_seqlens[b + 1] - row0 : p.total_len;
      const int i = job.idx[static_cast<long long>(head) * job.ld_idx + j];
      if (i < 0 || i >= L) {           // never read outside the sequence: skip the row and report it
        raise_status(p.hdr, FASTKV_ERR_DEVICE_INDEX, SITE_COMPACT_INDEX);
      } else {
        valid = true;
        const long long tok = static_cast<long long>(row0) + i;
        src = job.src + tok * job.src_tok_bytes + head * job.src_head_bytes + src_off;
        if (job.pos_src != nullptr && head == 0 && src_off == 0) job.pos_dst[j] = job.pos_src[tok];
      }
    }
    const uint32_t vmask = __ballot_sync(0xffffffffu, valid && job.src != nullptr);
    const uint32_t amask = __ballot_sync(0xffffffffu, active);
    const uint32_t bytes0 = __shfl_sync(0xffffffffu, bytes, 0);          // every row of a chunk has this size
    const long long r_first = __shfl_sync(0xffffffffu, r, 0);
    const uint32_t off_first = __shfl_sync(0xffffffffu, src_off, 0);
    Pending pend;
    pend.valid = vmask;
    pend.row_bytes = bytes0;
    pend.dst = job.dst + r_first * row_bytes + off_first;
    pend.bytes = (vmask == amask) ? static_cast<uint32_t>(__popc(amask)) * bytes0 : 0u;   // 0: store row by row
    // one phase of the stage's barrier per chunk, even when nothing is loaded
    if (lane == 0) mbar_arrive_expect_tx(&full[warp][s], static_cast<uint32_t>(__popc(vmask)) * bytes0);
    __syncwarp();
    if (valid && job.src != nullptr)
      bulk_load(stage + (job.pieces_per_row > 1 ? 0u : lane * bytes0), src, bytes0, &full[warp][s]);
    return pend;
  };

  Pending pending[kStages];
  constexpr int kAhead = kStages - 2;      // loads in flight per warp; one more stage is being stored
  const long long prologue = my_chunks < kAhead ? my_chunks : kAhead;
  for (long long c = 0; c < prologue; ++c) pending[c % kStages] = issue(c);
  for (long long c = 0; c < my_chunks; ++c) {
    const long long ahead = c + kAhead;
    if (ahead < my_chunks) {
      // that stage was stored two chunks ago: all but the latest store must have read their stage
      if (lane == 0) bulk_wait_read<1>();
      __syncwarp();
      pending[ahead % kStages] = issue(ahead);
    }
    const int s = static_cast<int>(c % kStages);
    const Pending pend = pending[s];
    if (lane == 0) {
      const bool ok = mbar_wait_bounded(&full[warp][s], static_cast<uint32_t>((c / kStages) & 1), &abort_flag, p.hdr,
                                        SITE_COMPACT_WAIT);
      if (ok && pend.valid != 0) {
        uint8_t* const stage = ring + s * kChunkBytes;
        if (pend.bytes != 0) {
          bulk_store(pend.dst, stage, pend.bytes);      // every row of the chunk is there: one store
        } else {
          for (int i = 0; i < 32; ++i)                    // some row was skipped: store the others one by one
            if ((pend.valid >> i) & 1u) bulk_store(pend.dst + i * pend.row_bytes, stage + i * pend.row_bytes, pend.row_bytes);
        }
      }
      bulk_commit();
    }
    __syncwarp();
  }
  if (lane == 0) bulk_wait_all();
}

cudaError_t launch_compact(CompactParams& p, cudaStream_t stream) {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) sms = v;
  }
  long long first = 0;
  for (int i = 0; i < p.n_jobs; ++i) {
    GatherJob& j = p.job[i];
    const long long row_bytes = static_cast<long long>(j.row_chunks) * 16;
    const long long rows = static_cast<long long>(j.heads) * j.rows;
    if (row_bytes > kChunkBytes) {
      j.pieces_per_row = static_cast<int>((row_bytes + kChunkBytes - 1) / kChunkBytes);
      j.rows_per_chunk = 1;
    } else {
      j.pieces_per_row = 1;
      long long rpc = row_bytes > 0 ? kChunkBytes / row_bytes : 32;
      j.rows_per_chunk = static_cast<int>(rpc > 32 ? 32 : (rpc < 1 ? 1 : rpc));
    }
    j.first_chunk = first;
    first += j.pieces_per_row > 1 ? rows * j.pieces_per_row : (rows + j.rows_per_chunk - 1) / j.rows_per_chunk;
  }
  p.total_chunks = first;
  if (first == 0) return cudaSuccess;
  static PerDeviceOnce configured;        // launch attributes are per device
  if (!configured.done(dev)) {
    cudaError_t e = cudaFuncSetAttribute(compact_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kCompactSmem);
    if (e != cudaSuccess) return e;
    configured.set(dev);
  }
  long long blocks = (first + kCompactWarps - 1) / kCompactWarps;
  if (blocks > sms) blocks = sms;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(blocks));
  cfg.blockDim = dim3(kCompactThreads);
  cfg.dynamicSmemBytes = kCompactSmem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  fill_pdl_attribute(&attr[0]);
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, compact_rows_kernel, static_cast<const CompactParams&>(p));
}

}  // namespace fastkv
