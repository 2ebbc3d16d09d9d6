// Shared device helpers of the FastKV sm_100a kernels: bounded mbarrier waits, TMA bulk
// tensor loads, tcgen05 (5th-generation tensor core) wrappers and the workspace header.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/fastkv.h"

namespace fastkv {

// ---- workspace header (first 256 bytes of every workspace) -------------------------------
// word 0: device status (a fastkv_status), word 1: site id of the first failure.
struct WorkspaceHeader {
  int status;
  int site;
  int reserved[62];
};
static_assert(sizeof(WorkspaceHeader) == 256, "header is one 256-byte block");

enum Site : int {
  SITE_NONE = 0,
  SITE_SCORE_TMA_EMPTY = 1,
  SITE_SCORE_MMA_FULL = 2,
  SITE_SCORE_MMA_ACC_EMPTY = 3,
  SITE_SCORE_EPI_ACC_FULL = 4,
  SITE_SCORE_MMA_QFULL = 5,
  SITE_SCORE_SHORT_SEQUENCE = 6,
  SITE_FUSED_EMPTY = 8,
  SITE_FUSED_FULL = 9,
  SITE_FUSED_Q_EMPTY = 10,
  SITE_FUSED_Q_FULL = 11,
  SITE_FUSED_ACC_FREE = 12,
  SITE_FUSED_ACC_FULL = 13,
  SITE_FUSED_FLAG = 14,
  SITE_FUSED_P1_DONE = 15,
  SITE_FUSED_P2_DONE = 18,
  SITE_COMPACT_INDEX = 16,
  SITE_COMPACT_WAIT = 19,
  SITE_DECODE_WAIT = 20,
  SITE_SELECT_BUDGET = 17,
  SITE_PARKED_RING = 21,
  SITE_PARKED_DRAIN = 22,
  SITE_PARKED_REF = 23,
  SITE_PARKED_STATS = 24,
  SITE_PARKED_NORM = 25,
  SITE_ATTN_RING = 26,
  SITE_ATTN_DRAIN = 27,
  SITE_ATTN_Q = 28,
  SITE_ATTN_K = 29,
  SITE_ATTN_V = 30,
  SITE_ATTN_P = 31,
  SITE_ATTN_S = 32,
  SITE_ATTN_SFULL = 33,
  SITE_ATTN_PFREE = 34,
  SITE_ATTN_ODONE = 35,
};

// Records `text` as the calling thread's last error (see fastkv_last_error) and returns `status`.
int report_error(int status, const char* text);

__device__ __forceinline__ void raise_status(WorkspaceHeader* hdr, int status, int site) {
  if (hdr != nullptr && atomicCAS(&hdr->status, 0, status) == 0) hdr->site = site;
}

// ---- programmatic dependent launch -----------------------------------------------------------
// Kernels of one layer step are chained on a stream.  A kernel launched with the programmatic
// stream serialization attribute may start while its predecessor drains; pdl_wait() blocks until
// the predecessor has completed and its writes are visible (a no-op for an ordinary launch), and
// pdl_launch_dependents() tells the scheduler that the successor may be brought up.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- shared-memory addresses ---------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier -----------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Every wait in these kernels is bounded: after `limit` cycles of polling (about a second by default)
// the waiter records where it gave up, raises the CTA-wide abort flag and returns false; a waiter that
// finds the flag already raised returns false at once.  Callers then run through the rest of their
// loops without waiting or computing, so the kernel always terminates and the context stays usable.
// `abort_flag` lives in shared memory.
constexpr long long kWaitLimitCycles = 1ll << 31;

__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity,
                                                  volatile int* abort_flag, WorkspaceHeader* hdr,
                                                  int site, long long limit = kWaitLimitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  if (*abort_flag) return false;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 0xFFu) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit) {
        *abort_flag = 1;
        raise_status(hdr, FASTKV_ERR_DEVICE_TIMEOUT, site);
        return false;
      }
    }
  }
}

// The wait of a control warp (a producer, an issuer).  A control warp waits most of the time, and a polling loop takes
// issue slots from the compute warps that share its scheduler: the wait is left to the hardware instead, which
// suspends the thread until the phase completes or the hinted time has passed.  Bounded like every other wait.
#ifndef FASTKV_PARK_NS
#define FASTKV_PARK_NS 1000
#endif
__device__ __forceinline__ bool mbar_wait_parked(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                 WorkspaceHeader* hdr, int site, long long limit) {
  const long long t0 = clock64();
  while (true) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(static_cast<uint32_t>(FASTKV_PARK_NS))
        : "memory");
    if (ok) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) {
      *abort_flag = 1;
      raise_status(hdr, FASTKV_ERR_DEVICE_TIMEOUT, site);
      return false;
    }
  }
}

// The wait of an issuing warp whose wake-up is on the critical path: a suspended thread (above) resumes some
// 0.5 kcycles after the phase completes; a poll every ~50 ns answers within ~0.1 kcycles and still leaves the
// scheduler's issue slots to the compute warps.  Bounded like every other wait.
__device__ __forceinline__ bool mbar_wait_nap(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                              WorkspaceHeader* hdr, int site, long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    __nanosleep(50);
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) {
      *abort_flag = 1;
      raise_status(hdr, FASTKV_ERR_DEVICE_TIMEOUT, site);
      return false;
    }
  }
}

// The wait a role uses for its own copies or contractions still in flight before it leaves: bounded
// like every other wait, but it does not give up just because the CTA is aborting.
__device__ __forceinline__ bool mbar_wait_drain(uint64_t* bar, uint32_t parity, WorkspaceHeader* hdr, int site,
                                                long long limit = kWaitLimitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 0xFFu) == 0 && clock64() - t0 > limit) {
      raise_status(hdr, FASTKV_ERR_DEVICE_TIMEOUT, site);
      return false;
    }
  }
}

// ---- global-memory publication between CTAs ---------------------------------------------------
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_add(int* p, int v) {
  asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// ---- TMA (cp.async.bulk.tensor): plain per-CTA loads only --------------------------------------
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
// 3-D tiled load global -> shared; completion is signalled on `bar` as transaction bytes.
// c0 (innermost, elements) times the element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* map, uint64_t* bar,
                                            int c0, int c1, int c2, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4, %5}], [%2], %6;"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)),
        "r"(c0), "r"(c1), "r"(c2), "l"(policy)
      : "memory");
}

// ---- tcgen05: tensor memory and MMA ----------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                   smem_u32(smem_result)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// Arrives on `bar` once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   smem_u32(bar))
               : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 x bf16 -> fp32, issued by one thread.
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc,
                                            uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Shared-memory matrix descriptor for a K-major operand tile stored as rows of 128 bytes with
// the 128-byte swizzle (what a TMA box of 64 bf16 x rows with SWIZZLE_128B writes): groups of
// 8 rows are 1024 bytes apart (stride byte offset); descriptor version 1 (Blackwell).
__device__ __forceinline__ uint64_t umma_desc_k_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);        // start address, bits 0-13
  d |= static_cast<uint64_t>(1) << 16;                            // leading byte offset (unused)
  d |= static_cast<uint64_t>(1024 >> 4) << 32;                    // stride byte offset, bits 32-45
  d |= static_cast<uint64_t>(1) << 46;                            // version = 1
  d |= static_cast<uint64_t>(2) << 61;                            // layout: SWIZZLE_128B
  return d;
}
// Instruction descriptor: kind::f16, A = B = bf16 (K-major), D = fp32, M x N tile.
__host__ __device__ constexpr uint32_t umma_idesc_bf16_f32(int m, int n) {
  return (1u << 4)                       // D format fp32
         | (1u << 7)                     // A format bf16
         | (1u << 10)                    // B format bf16
         | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}
// 32 lanes x 32 consecutive fp32 columns of tensor memory -> 32 registers per thread
// (thread = lane of its warp's quarter, register i = column i).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
        "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");   // load and wait in one statement: the registers are valid when it ends
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// 32 registers per thread -> 32 lanes x 32 consecutive fp32 columns of tensor memory.
__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const float (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
        "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])),
        "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15])), "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])),
        "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])), "r"(__float_as_uint(v[20])),
        "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
        "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])),
        "r"(__float_as_uint(v[27])), "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])),
        "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
}
// 32 lanes x 16 consecutive fp32 columns -> 16 registers per thread
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// 16 registers per thread -> 32 lanes x 16 consecutive fp32 columns of tensor memory
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const float (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
        "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])),
        "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15]))
      : "memory");
}

// 8-column variants (used where registers are scarce)
__device__ __forceinline__ void tmem_ld_32x8(uint32_t taddr, float (&v)[8]) {
  uint32_t r[8];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st_32x8(uint32_t taddr, const float (&v)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr),
               "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
               "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
               "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7]))
               : "memory");
}
__device__ __forceinline__ void tmem_wait_st() {
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Online-softmax statistics (max m, sum l of exp2(x - m)) of two disjoint sets of logits combine as
// m = max(m1, m2), l = l1 * 2^(m1 - m) + l2 * 2^(m2 - m); an empty set is (-inf, 0).
__device__ __forceinline__ void merge_stats(float& m, float& l, float m2, float l2) {
  if (m2 == -INFINITY) return;
  const float mn = fmaxf(m, m2);
  l = l * ex2(m - mn) + l2 * ex2(m2 - mn);     // m == -inf gives 2^-inf = 0 times l = 0
  m = mn;
}

// Running softmax statistics of one thread over N query rows (one new logit per row):
// s_x = acc[x] * scale.  The running max may lag the true max by up to kLazyMaxSlackLog2 (log2
// units): in the common case no row needs rescaling anywhere in the warp and the update is one
// exp2 per element, straight-line code with N independent dependency chains.
constexpr float kLazyMaxSlackLog2 = 8.0f;

template <int N>
__device__ __forceinline__ void stats_update_unmasked(const float (&acc)[N], float* m, float* l, float scale,
                                                      int n_valid) {
  bool need = false;
#pragma unroll
  for (int x = 0; x < N; ++x) need |= (x < n_valid) && (fmaf(acc[x], scale, -m[x]) > kLazyMaxSlackLog2);
  if (__any_sync(0xffffffffu, need)) {             // some row's max moved: exact update, two exp2
#pragma unroll
    for (int x = 0; x < N; ++x) {
      if (x < n_valid) {
        const float s = acc[x] * scale;
        const float mn = fmaxf(m[x], s);
        l[x] = l[x] * ex2(m[x] - mn) + ex2(s - mn);
        m[x] = mn;
      }
    }
  } else {
#pragma unroll
    for (int x = 0; x < N; ++x)
      if (x < n_valid) l[x] += ex2(fmaf(acc[x], scale, -m[x]));
  }
}

// Same, for the tiles that overlap the observation window: row x sees the key only if visible[x].
template <int N>
__device__ __forceinline__ void stats_update_masked(const float (&acc)[N], float* m, float* l, float scale,
                                                    int n_valid, uint32_t visible) {
#pragma unroll
  for (int x = 0; x < N; ++x) {
    if (x < n_valid) {
      const float s = ((visible >> x) & 1u) ? acc[x] * scale : -INFINITY;
      const float mn = fmaxf(m[x], s);
      const float ref = (mn == -INFINITY) ? 0.0f : mn;      // nothing seen yet: keep (m, l) = (-inf, 0)
      l[x] = l[x] * ex2(m[x] - ref) + ex2(s - ref);
      m[x] = mn;
    }
  }
}

// The first logit of each row starts the statistics without any exp2: (m, l) = (s, 1).
template <int N>
__device__ __forceinline__ void stats_init_unmasked(const float (&acc)[N], float* m, float* l, float scale,
                                                    int n_valid) {
#pragma unroll
  for (int x = 0; x < N; ++x) {
    if (x < n_valid) {
      m[x] = acc[x] * scale;
      l[x] = 1.0f;
    }
  }
}

// Transposing butterfly over the 32 lanes of a warp: on entry every lane holds statistics (m[x], l[x])
// of rows x = 0..N-1 (N = 16 or 32) for its own keys; on return lane r holds in (m[0], l[0]) the
// statistics of row r % N merged over all 32 lanes.  N - 1 (+1) exchanges of a pair instead of
// N x 5 shuffle reductions.
template <int N>
__device__ __forceinline__ void stats_transpose_merge(float* m, float* l, int lane) {
#pragma unroll
  for (int o = N / 2; o >= 1; o >>= 1) {
    const bool upper = (lane & o) != 0;
#pragma unroll
    for (int i = 0; i < o; ++i) {
      // this lane keeps row i (lower) or i + o (upper) of the current 2*o rows and sends the other
      const float send_m = upper ? m[i] : m[i + o], send_l = upper ? l[i] : l[i + o];
      float keep_m = upper ? m[i + o] : m[i], keep_l = upper ? l[i + o] : l[i];
      const float got_m = __shfl_xor_sync(0xffffffffu, send_m, o);
      const float got_l = __shfl_xor_sync(0xffffffffu, send_l, o);
      merge_stats(keep_m, keep_l, got_m, got_l);
      m[i] = keep_m;
      l[i] = keep_l;
    }
  }
  if (N == 16) {                                   // lanes r and r + 16 hold the two halves of row r
    const float got_m = __shfl_xor_sync(0xffffffffu, m[0], 16);
    const float got_l = __shfl_xor_sync(0xffffffffu, l[0], 16);
    float a_m = (lane & 16) ? got_m : m[0], a_l = (lane & 16) ? got_l : l[0];      // lower lane's half first:
    const float b_m = (lane & 16) ? m[0] : got_m, b_l = (lane & 16) ? l[0] : got_l;  // same order on both lanes
    merge_stats(a_m, a_l, b_m, b_l);
    m[0] = a_m;
    l[0] = a_l;
  }
}

// Merges `count` per-CTA statistics of row n (part[r * npad + n], r = first, first + stride, ...) in
// a fixed order, with twenty independent loads in flight at a time.
__device__ __forceinline__ float2 merge_partials(const float2* part, int npad, int n, int first, int stride,
                                                 int count) {
  float m = -INFINITY, l = 0.0f;
  for (int r0 = first; r0 < count; r0 += stride * 20) {
    float2 v[20];
#pragma unroll
    for (int j = 0; j < 20; ++j) {
      const int r = r0 + j * stride;
      v[j] = (r < count) ? __ldcg(&part[static_cast<size_t>(r) * npad + n]) : make_float2(-INFINITY, 0.0f);
    }
#pragma unroll
    for (int j = 0; j < 20; ++j) merge_stats(m, l, v[j].x, v[j].y);
  }
  return make_float2(m, l);
}

// "Done once per device" flag for launch attributes (they are per device, and one process may
// drive several): indexed by the device ordinal.
struct PerDeviceOnce {
  static constexpr int kMaxDevices = 64;
  unsigned char flag[kMaxDevices] = {};
  bool done(int dev) const { return dev >= 0 && dev < kMaxDevices && flag[dev] != 0; }
  void set(int dev) { if (dev >= 0 && dev < kMaxDevices) flag[dev] = 1; }
};

// Launch configuration shared by the kernels that follow another kernel of the step.
inline void fill_pdl_attribute(cudaLaunchAttribute* attr) {
  attr->id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr->val.programmaticStreamSerializationAllowed = 1;
}

}  // namespace fastkv
