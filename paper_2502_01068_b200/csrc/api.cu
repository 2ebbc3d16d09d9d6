// C ABI of the FastKV selection path: argument validation, workspace carving, TMA descriptor
// encoding and kernel launches.  Declarations and contracts live in include/fastkv.h.
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "compact.cuh"
#include "decode_attn.cuh"
#include "prefill_attn.cuh"
#include "score.cuh"
#include "select.cuh"

namespace fastkv {
namespace {

thread_local char g_last_error[512] = "";
std::atomic<long long> g_launches{0};

int fail(int status, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_last_error, sizeof g_last_error, fmt, ap);
  va_end(ap);
  return status;
}

int cuda_fail(cudaError_t e, const char* what) {
  return fail(FASTKV_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int npad_for(int n_rows) { return n_rows <= 32 ? 32 : 64; }

// ---- test and tuning hooks (fastkv_debug_set) ------------------------------------------------------
enum ScorePath { PATH_AUTO = 0, PATH_BUFFERED = 1, PATH_REREAD = 2, PATH_PARKED = 3 };
struct DebugConfig {
  int score_path = PATH_AUTO;
  int fused_heads = 0;              // two-pipeline kernel: KV heads side by side in a phase (0 = by size)
  int fused_lead = 0;               // two-pipeline kernel: phases pass 1 may lead pass 2 (0 = by size)
  long long wait_limit_cycles = 0;  // 0 = the default of about a second
  int extra_publications = 0;       // pass 2 waits for publications that never come (timeout test)
  int score_partition = 0;          // parked kernel's partition mode: 0 = by shape, 1 = never, 2 = whenever it can run
  int prefill_skip_commit = 0;      // prefill attention: n > 0: key tile n - 1's "S ready" signal is withheld (timeout test)
};
DebugConfig g_debug;

// ---- optional per-kernel timing ("time_kernels" hook): a pair of events around every launch ----------
enum KernelId { KID_SCORE = 0, KID_POOL = 1, KID_SELECT = 2, KID_COMPACT = 3, KID_DECODE = 4, KID_PREFILL = 5,
                KID_WINDOW_SCORES = 6, KID_COUNT = 7 };
const char* const kKernelNames[KID_COUNT] = {"score", "pool", "select", "compact", "decode_attn", "prefill_attn",
                                             "window_scores"};
struct KernelTimes {
  bool on = false;
  std::mutex mu;
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> ev[KID_COUNT];
};
KernelTimes g_times;

struct TimedLaunch {          // records an event before and (in the destructor) after one kernel launch
  int id;
  cudaStream_t stream;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  TimedLaunch(int id_, cudaStream_t s) : id(id_), stream(s) {
    if (!g_times.on) return;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) { e0 = e1 = nullptr; return; }
    cudaEventRecord(e0, stream);
  }
  ~TimedLaunch() {
    if (e0 == nullptr) return;
    cudaEventRecord(e1, stream);
    std::lock_guard<std::mutex> lock(g_times.mu);
    g_times.ev[id].emplace_back(e0, e1);
  }
};

// ---- workspace layout --------------------------------------------------------------------------
struct Layout {
  int npad, tiles_per_cta, max_ranges;
  long long ld_logits;
  size_t off_counters, off_final, off_partial, off_logits, b_bytes, zero_bytes;   // buffered path
  // persistent one-HBM-pass kernels (score_parked.cu, score_fused.cu): same header, their own carving of the rest
  bool fused_shape_ok;        // the shape is one the persistent kernels are built for
  int f_rows;                 // un-pooled rows written by pass 2 (KV heads or query heads)
  size_t f_off_counters, f_off_partial, f_off_a, f_zero_bytes, f_bytes;
  int path;                   // the ScorePath fastkv_score takes for this shape; -1: the forced path cannot run it
  bool partition;             // a batch the parked kernel can score with its sequences side by side
  size_t bytes;               // workspace that path needs
};

constexpr int kFusedMaxCtas = 148;      // SMs of a B200: one persistent CTA each

// Tiles of the longest sequence one CTA parks per phase when `ctas` persistent CTAs share it.
int parked_tiles_per_cta(int max_len, int ctas) {
  const int ntiles = (max_len + 127) / 128;
  return (ntiles + ctas - 1) / ctas;
}

// The parked kernel's partition mode (several (sequence, head) phases side by side, each on its share of the
// CTAs, in waves that fit the grid at one ring of tiles per CTA) can run whenever the longest sequence alone
// fits the ring and the table of waves fits its shared memory.
bool partition_ok(const fastkv_shape& s, int ctas, int slots) {
  return static_cast<long long>(s.batch) * s.n_kv_heads <= 512 && parked_tiles_per_cta(s.max_len, ctas) <= slots;
}

Layout make_layout(const fastkv_shape& s) {
  Layout l;
  const int G = s.n_q_heads / s.n_kv_heads;
  l.npad = npad_for(G * s.window);
  const long long max_tiles = (static_cast<long long>(s.max_len) + 127) / 128;
  // about four waves of two co-resident CTAs per SM on a 148-SM part, at least two tiles per CTA
  long long tpc = (max_tiles * s.n_kv_heads * s.batch + 1183) / 1184;
  if (tpc < 2) tpc = 2;
  if (tpc > 32) tpc = 32;
  l.tiles_per_cta = static_cast<int>(tpc);
  l.max_ranges = static_cast<int>((max_tiles + tpc - 1) / tpc);
  if (l.max_ranges < 1) l.max_ranges = 1;
  l.ld_logits = static_cast<long long>(round_up(static_cast<size_t>(s.total_len), 64));
  size_t off = sizeof(WorkspaceHeader);
  l.off_counters = off;
  off += round_up(sizeof(int) * s.batch * s.n_kv_heads, 256);
  l.zero_bytes = off;                       // header + counters are cleared by fastkv_score
  l.off_final = off;
  off += round_up(sizeof(float2) * s.batch * s.n_kv_heads * l.npad, 256);
  l.off_partial = off;
  off += round_up(sizeof(float2) * static_cast<size_t>(s.batch) * s.n_kv_heads * l.max_ranges * l.npad, 256);
  l.off_logits = off;
  off += round_up(sizeof(float) * static_cast<size_t>(s.n_kv_heads) * l.npad * l.ld_logits, 256);
  l.b_bytes = off;

  const int phases = s.batch * s.n_kv_heads;
  const bool per_head = s.agg_order == FASTKV_POOL_THEN_GROUP;
  l.fused_shape_ok = !per_head || G == 1 || G == 2 || G == 4 || G == 8;
  l.f_rows = per_head ? s.n_q_heads : s.n_kv_heads;
  off = sizeof(WorkspaceHeader);
  l.f_off_counters = off;
  off += round_up(sizeof(int) * phases, 256);
  l.f_zero_bytes = off;                     // header + per-phase counters are cleared by fastkv_score
  l.f_off_partial = off;
  off += round_up(sizeof(float2) * static_cast<size_t>(phases) * kFusedMaxCtas * l.npad, 256);
  l.f_off_a = off;
  off += round_up(sizeof(float) * static_cast<size_t>(l.f_rows) * l.ld_logits, 256);
  l.f_bytes = off;
  // Which kernel scores this shape (measured on a B200 with the Llama-3.1-8B head shape, kernel alone, re-read /
  // parked / parked with partition, us: 17.9 / 35.0 / 18.7 at 8K, 30.9 / 45.0 / 27.5 at 32K, 52.0 / 54.3 / 41.6 at
  // 64K, 83.5 / 61.9 / 59.2 at 96K, 89.9 / 60.8 / 68.3 at 128K, 122.9 / 90.0 / 96.8 at 200K, 180.9 / 131.8 / 137.7 at
  // 300K).  A single sequence: below 24K tokens the kernel that reads K a second time from L2 (no per-phase
  // exchange to pay); up to six tiles per CTA and head the parked kernel with its heads side by side; up to the
  // ring (16 tiles per CTA: 303K tokens) the parked kernel with the whole grid on one head at a time; beyond the
  // ring the re-read kernel again.  Batches: see below.  The buffered two-kernel path serves the remaining shapes.
  const int per = parked_tiles_per_cta(s.max_len, kFusedMaxCtas), slots = parked_slots(l.npad);
  // batches: sequences side by side, in as few waves as fit the ring (the ring then holds one phase, not two, but
  // every CTA streams all the time, there are waves x n_kv_heads phases instead of batch x n_kv_heads, and a
  // statistics exchange involves the CTAs of one sequence only)
  const long long batch_per = (static_cast<long long>(s.total_len) / 128 + kFusedMaxCtas - 1) / kFusedMaxCtas;
  // Partition mode: batches with enough work (sequences x heads exchanges are what it removes: 189 against 266 us
  // on the ragged config), and single sequences short enough that a grid-wide phase per head leaves CTAs without
  // tiles, one head per share of the CTAs (kernel alone, re-read / parked / parked with partition: 30.9 / 45.0 /
  // 27.5 us at 32K, 52.0 / 54.3 / 41.6 at 64K, 83.5 / 61.9 / 59.2 at 96K, 89.9 / 60.8 / 68.3 at 128K; below 24K
  // the re-read kernel is as fast).
  const bool partition_wanted = s.batch >= 2 ? batch_per >= 6 : (s.max_len >= 24576 && per <= 6);
  l.partition = partition_ok(s, kFusedMaxCtas, slots) &&
                (g_debug.score_partition == 2 || (g_debug.score_partition == 0 && partition_wanted));
  switch (g_debug.score_path) {
    case PATH_BUFFERED: l.path = PATH_BUFFERED; break;
    case PATH_REREAD: l.path = l.fused_shape_ok ? PATH_REREAD : PATH_BUFFERED; break;
    case PATH_PARKED:
      // forced: batches take the partition mode whenever it can run (the grid-wide walk needs the same ring)
      if (g_debug.score_partition != 1 && s.batch >= 2 && partition_ok(s, kFusedMaxCtas, slots)) l.partition = true;
      l.path = !l.fused_shape_ok ? PATH_BUFFERED : (per <= slots ? PATH_PARKED : -1);
      break;
    default:
      l.path = !l.fused_shape_ok ? PATH_BUFFERED
               : l.partition || (s.batch == 1 && per >= 7 && per <= slots) ? PATH_PARKED : PATH_REREAD;
      break;
  }
  l.bytes = l.path == PATH_BUFFERED ? l.b_bytes : l.f_bytes;
  return l;
}

// ---- validation ---------------------------------------------------------------------------------
int check_shape(const fastkv_shape* s, bool for_score) {
  if (s == nullptr) return fail(FASTKV_ERR_INVALID_ARG, "shape is NULL");
  if (s->batch < 1) return fail(FASTKV_ERR_INVALID_ARG, "batch must be >= 1");
  if (s->total_len < 1 || s->max_len < 1 || s->max_len > s->total_len)
    return fail(FASTKV_ERR_INVALID_ARG, "need 1 <= max_len <= total_len");
  if (s->batch > 1 && s->cu_seqlens == nullptr)
    return fail(FASTKV_ERR_INVALID_ARG, "cu_seqlens is required when batch > 1");
  if (s->batch == 1 && s->max_len != s->total_len)
    return fail(FASTKV_ERR_INVALID_ARG, "batch == 1 needs max_len == total_len");
  if (s->n_kv_heads < 1 || s->n_q_heads < 1 || s->n_q_heads % s->n_kv_heads != 0)
    return fail(FASTKV_ERR_INVALID_ARG, "n_q_heads must be a positive multiple of n_kv_heads");
  if (s->window < 1) return fail(FASTKV_ERR_INVALID_ARG, "window must be >= 1");
  if (s->batch == 1 && s->window > s->total_len)
    return fail(FASTKV_ERR_INVALID_ARG, "window exceeds the sequence length");
  if (s->force_window != 0 && s->force_window != 1)
    return fail(FASTKV_ERR_INVALID_ARG, "force_window must be 0 or 1");
  if (!for_score) return FASTKV_OK;
  if (s->pool_kernel < 1 || (s->pool_kernel & 1) == 0)
    return fail(FASTKV_ERR_INVALID_ARG, "pool_kernel must be odd and >= 1");
  if (s->pool_kernel > 63) return fail(FASTKV_ERR_UNSUPPORTED, "pool_kernel > 63 is not built");
  if (s->pool_mode != FASTKV_POOL_AVG && s->pool_mode != FASTKV_POOL_MAX)
    return fail(FASTKV_ERR_INVALID_ARG, "unknown pool_mode");
  if (s->agg_order != FASTKV_GROUP_THEN_POOL && s->agg_order != FASTKV_POOL_THEN_GROUP)
    return fail(FASTKV_ERR_INVALID_ARG, "unknown agg_order");
  if (s->q_layout != FASTKV_Q_FULL && s->q_layout != FASTKV_Q_WINDOW)
    return fail(FASTKV_ERR_INVALID_ARG, "unknown q_layout");
  if (!(s->softmax_scale >= 0.0f) || std::isinf(s->softmax_scale))
    return fail(FASTKV_ERR_INVALID_ARG, "softmax_scale must be finite and >= 0");
  if (s->head_dim != 64 && s->head_dim != 128)
    return fail(FASTKV_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
  const int n_rows = s->n_q_heads / s->n_kv_heads * s->window;
  if (n_rows > 64) return fail(FASTKV_ERR_UNSUPPORTED, "G * window > 64 is not built");
  if (s->n_q_heads / s->n_kv_heads > 256 || s->window > 256)
    return fail(FASTKV_ERR_UNSUPPORTED, "TMA box limit: G and window must be <= 256");
  if (s->q_stride_tok % 8 || s->q_stride_head % 8 || s->k_stride_tok % 8 || s->k_stride_head % 8)
    return fail(FASTKV_ERR_UNSUPPORTED, "q/k strides must be multiples of 8 elements (16 bytes)");
  if (s->q_stride_head < s->head_dim || s->k_stride_head < s->head_dim ||
      s->q_stride_tok < s->head_dim || s->k_stride_tok < s->head_dim)
    return fail(FASTKV_ERR_INVALID_ARG, "q/k strides are smaller than head_dim");
  return FASTKV_OK;
}

int check_workspace(const void* ws, size_t ws_bytes, size_t need) {
  if (ws == nullptr) return fail(FASTKV_ERR_WORKSPACE, "workspace is NULL");
  if (reinterpret_cast<uintptr_t>(ws) % 256) return fail(FASTKV_ERR_WORKSPACE, "workspace must be 256-byte aligned");
  if (ws_bytes < need) return fail(FASTKV_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", ws_bytes, need);
  return FASTKV_OK;
}

int check_budget(const fastkv_shape* s, const fastkv_budget* b, const char* name) {
  if (b == nullptr) return fail(FASTKV_ERR_INVALID_ARG, "%s budget is NULL", name);
  const int w = s->force_window ? s->window : 0;
  if (b->cu_k == nullptr) {
    if (b->k < 1 || b->k < w) return fail(FASTKV_ERR_INVALID_ARG, "%s: k must be >= max(1, window)", name);
    if (b->k > s->max_len) return fail(FASTKV_ERR_INVALID_ARG, "%s: k exceeds the sequence length", name);
    if (static_cast<long long>(b->k) * s->batch != b->total)
      return fail(FASTKV_ERR_INVALID_ARG, "%s: total must equal batch * k", name);
  } else {
    if (b->total < 1) return fail(FASTKV_ERR_INVALID_ARG, "%s: total must be >= 1", name);
  }
  return FASTKV_OK;
}

// ---- TMA descriptors ------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor [rows][heads][dim] with element strides; box = box_rows x box_heads x 64 columns
int encode_bf16_3d(CUtensorMap* map, const void* base, int dim, int heads, long long rows,
                   long long stride_head, long long stride_tok, int box_heads, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return fail(FASTKV_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  if (reinterpret_cast<uintptr_t>(base) % 16) return fail(FASTKV_ERR_UNSUPPORTED, "tensor base must be 16-byte aligned");
  cuuint64_t dims[3] = {static_cast<cuuint64_t>(dim), static_cast<cuuint64_t>(heads), static_cast<cuuint64_t>(rows)};
  cuuint64_t strides[2] = {static_cast<cuuint64_t>(stride_head) * 2, static_cast<cuuint64_t>(stride_tok) * 2};
  cuuint32_t box[3] = {64, static_cast<cuuint32_t>(box_heads), static_cast<cuuint32_t>(box_rows)};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(FASTKV_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(r));
  return FASTKV_OK;
}

// Persistent CTAs the single-pass scoring kernel may use: one per SM, capped at the count the
// workspace is carved for; 0 if the device cannot be queried or has no cooperative launch.
// (cached per device ordinal: one process may drive several GPUs)
int fused_grid() {
  static int ctas[PerDeviceOnce::kMaxDevices];
  static PerDeviceOnce known;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= PerDeviceOnce::kMaxDevices) return 0;
  if (!known.done(dev)) {
    int sms = 0, coop = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop)
      ctas[dev] = 0;
    else
      ctas[dev] = sms < kFusedMaxCtas ? sms : kFusedMaxCtas;
    known.set(dev);
  }
  return ctas[dev];
}

int check_device() {
  static int ok[PerDeviceOnce::kMaxDevices];
  static PerDeviceOnce known;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
  if (dev < 0 || dev >= PerDeviceOnce::kMaxDevices) return fail(FASTKV_ERR_UNSUPPORTED, "device ordinal out of range");
  if (!known.done(dev)) {
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
    ok[dev] = (major == 10) ? 1 : 0;
    known.set(dev);
  }
  if (!ok[dev]) return fail(FASTKV_ERR_UNSUPPORTED, "this library is built for sm_100a (B200) only");
  return FASTKV_OK;
}

}  // namespace

// Lets the other translation units of the library leave their message where fastkv_last_error()
// finds it.
int report_error(int status, const char* text) { return fail(status, "%s", text); }

}  // namespace fastkv

using namespace fastkv;

extern "C" {

int fastkv_workspace_bytes(const fastkv_shape* shape, size_t* bytes) {
  int rc = check_shape(shape, true);
  if (rc) return rc;
  if (bytes == nullptr) return fail(FASTKV_ERR_INVALID_ARG, "bytes is NULL");
  const Layout lay = make_layout(*shape);
  if (lay.path < 0) return fail(FASTKV_ERR_UNSUPPORTED, "the forced scoring path cannot run this shape");
  *bytes = lay.bytes;
  return FASTKV_OK;
}

int fastkv_debug_set(const char* key, int64_t value) {
  if (key == nullptr) return fail(FASTKV_ERR_INVALID_ARG, "debug_set: key is NULL");
  if (!std::strcmp(key, "score_path")) {
    if (value < PATH_AUTO || value > PATH_PARKED) return fail(FASTKV_ERR_INVALID_ARG, "debug_set: score_path is 0..3");
    g_debug.score_path = static_cast<int>(value);
  } else if (!std::strcmp(key, "fused_heads")) {
    g_debug.fused_heads = static_cast<int>(value < 0 ? 0 : value);
  } else if (!std::strcmp(key, "fused_lead")) {
    g_debug.fused_lead = static_cast<int>(value < 0 ? 0 : value);
  } else if (!std::strcmp(key, "wait_limit_cycles")) {
    g_debug.wait_limit_cycles = value < 0 ? 0 : value;
  } else if (!std::strcmp(key, "score_partition")) {
    if (value < 0 || value > 2) return fail(FASTKV_ERR_INVALID_ARG, "debug_set: score_partition is 0..2");
    g_debug.score_partition = static_cast<int>(value);
  } else if (!std::strcmp(key, "prefill_skip_commit")) {
    g_debug.prefill_skip_commit = static_cast<int>(value < 0 ? 0 : value);
  } else if (!std::strcmp(key, "extra_publications")) {
    g_debug.extra_publications = static_cast<int>(value < 0 ? 0 : value);
  } else if (!std::strcmp(key, "time_kernels")) {
    g_times.on = value != 0;
  } else {
    return fail(FASTKV_ERR_INVALID_ARG, "debug_set: unknown key '%s'", key);
  }
  return FASTKV_OK;
}

int fastkv_debug_kernel_time(int32_t kernel, double* total_ms, int64_t* launches, const char** name) {
  if (kernel < 0 || kernel >= KID_COUNT) return fail(FASTKV_ERR_INVALID_ARG, "debug_kernel_time: kernel is 0..%d", KID_COUNT - 1);
  std::lock_guard<std::mutex> lock(g_times.mu);
  double ms = 0.0;
  int64_t n = 0;
  for (auto& pr : g_times.ev[kernel]) {
    float t = 0.0f;
    if (cudaEventSynchronize(pr.second) == cudaSuccess && cudaEventElapsedTime(&t, pr.first, pr.second) == cudaSuccess) {
      ms += t;
      ++n;
    }
    cudaEventDestroy(pr.first);
    cudaEventDestroy(pr.second);
  }
  g_times.ev[kernel].clear();
  if (total_ms) *total_ms = ms;
  if (launches) *launches = n;
  if (name) *name = kKernelNames[kernel];
  return FASTKV_OK;
}

int fastkv_score(const fastkv_shape* shape, const void* q, const void* k, float* scores_kv,
                 float* scores_tsp, void* workspace, size_t workspace_bytes, void* stream_) {
  int rc = check_shape(shape, true);
  if (rc) return rc;
  if (q == nullptr || k == nullptr || scores_kv == nullptr)
    return fail(FASTKV_ERR_INVALID_ARG, "q, k and scores_kv are required");
  const Layout lay = make_layout(*shape);
  if (lay.path < 0) return fail(FASTKV_ERR_UNSUPPORTED, "the forced scoring path cannot run this shape");
  if ((rc = check_workspace(workspace, workspace_bytes, lay.bytes))) return rc;
  if ((rc = check_device())) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const fastkv_shape& s = *shape;
  const int G = s.n_q_heads / s.n_kv_heads;
  uint8_t* ws = static_cast<uint8_t*>(workspace);

  CUtensorMap tmap_k, tmap_q;
  if ((rc = encode_bf16_3d(&tmap_k, k, s.head_dim, s.n_kv_heads, s.total_len, s.k_stride_head,
                           s.k_stride_tok, 1, 128)))
    return rc;
  const long long q_rows = s.q_layout == FASTKV_Q_WINDOW ? static_cast<long long>(s.batch) * s.window : s.total_len;
  if ((rc = encode_bf16_3d(&tmap_q, q, s.head_dim, s.n_q_heads, q_rows, s.q_stride_head, s.q_stride_tok,
                           G, s.window)))
    return rc;

  const float scale = s.softmax_scale > 0.0f ? s.softmax_scale : 1.0f / std::sqrt(static_cast<float>(s.head_dim));
  const float scale_log2 = scale * 1.4426950408889634f;
  WorkspaceHeader* hdr = reinterpret_cast<WorkspaceHeader*>(ws);
  cudaError_t e;
  if (lay.path != PATH_BUFFERED) {
    // ---- one HBM pass over K: persistent kernel, one CTA per SM ----
    const int ctas = fused_grid();
    if (ctas <= 0) return fail(FASTKV_ERR_UNSUPPORTED, "the device offers no cooperative launch");
    const bool parked = lay.path == PATH_PARKED;
    const bool partition = parked && lay.partition && partition_ok(s, ctas, parked_slots(lay.npad));
    if (parked && !partition && parked_tiles_per_cta(s.max_len, ctas) > parked_slots(lay.npad))
      return fail(FASTKV_ERR_UNSUPPORTED, "this device has too few SMs to park a phase of this length");
    e = parked ? launch_clear_words(ws, lay.f_zero_bytes, stream) : cudaMemsetAsync(ws, 0, lay.f_zero_bytes, stream);
    if (e != cudaSuccess) return cuda_fail(e, "clearing the workspace header");
    FusedParams fp;
    fp.batch = s.batch; fp.total_len = s.total_len; fp.n_kv_heads = s.n_kv_heads; fp.group = G;
    fp.window = s.window; fp.n_rows = G * s.window; fp.q_layout = s.q_layout;
    fp.per_head = s.agg_order == FASTKV_POOL_THEN_GROUP;
    fp.scale_log2 = scale_log2; fp.cu_seqlens = s.cu_seqlens;
    fp.a_out = reinterpret_cast<float*>(ws + lay.f_off_a); fp.ld_a = lay.ld_logits;
    // A phase is sized to about one head of a 128K-token sequence (33.5 MB of K): shorter sequences put several
    // heads side by side in a phase, so that there are fewer grid-wide dependencies per byte.  Pass 1 may lead pass 2
    // by as many phases as keep about 110 MB of K between the two reads: that is what stays in the 126 MB L2.
    fp.heads_per_phase = g_debug.fused_heads;
    fp.phase_bytes = 35000000;
    fp.head_bytes = static_cast<long long>(s.head_dim) * 2;
    double longest_phase = static_cast<double>(s.max_len) * s.head_dim * 2.0;     // bytes of the largest phase
    const double hp_longest = fp.heads_per_phase > 0 ? fp.heads_per_phase : fp.phase_bytes / longest_phase;
    if (hp_longest >= 1.0) longest_phase *= static_cast<int>(hp_longest < s.n_kv_heads ? hp_longest : s.n_kv_heads);
    fp.max_lead = g_debug.fused_lead > 0 ? g_debug.fused_lead : static_cast<int>(110e6 / longest_phase);
    if (fp.max_lead > (1 << 20)) fp.max_lead = 1 << 20;
    if (fp.max_lead < 2) fp.max_lead = 2;
    fp.partial = reinterpret_cast<float2*>(ws + lay.f_off_partial);
    fp.counters = reinterpret_cast<int*>(ws + lay.f_off_counters);
    fp.hdr = hdr;
    fp.max_len = s.max_len;
    fp.wait_limit = g_debug.wait_limit_cycles > 0 ? g_debug.wait_limit_cycles : kWaitLimitCycles;
    fp.extra_publications = g_debug.extra_publications;
    fp.partition = partition ? (s.batch >= 2 ? 1 : 2) : 0;
    {
      TimedLaunch timed(KID_SCORE, stream);
      e = parked ? launch_score_parked(s.head_dim, lay.npad, tmap_k, tmap_q, fp, ctas, stream)
                 : launch_score_fused(s.head_dim, lay.npad, tmap_k, tmap_q, fp, ctas, stream);
    }
    if (e != cudaSuccess) return cuda_fail(e, parked ? "score_parked_kernel launch" : "score_fused_kernel launch");
    ++g_launches;
    PoolRowsParams rp;
    rp.total_len = s.total_len; rp.n_kv_heads = s.n_kv_heads; rp.group = G; rp.window = s.window;
    rp.per_head = fp.per_head; rp.pool_kernel = s.pool_kernel; rp.pool_mode = s.pool_mode;
    rp.cu_seqlens = s.cu_seqlens; rp.a = fp.a_out; rp.ld_a = lay.ld_logits;
    rp.scores_kv = scores_kv; rp.ld_scores = s.total_len; rp.scores_tsp = scores_tsp;
    if (sizeof(float) * static_cast<size_t>(lay.f_rows) * (kPoolKeys + s.pool_kernel) > 200 * 1024)
      return fail(FASTKV_ERR_UNSUPPORTED, "heads x pool halo do not fit the pooling kernel's shared memory");
    {
      TimedLaunch timed(KID_POOL, stream);
      e = launch_pool_rows(rp, s.max_len, s.batch, stream);
    }
    if (e != cudaSuccess) return cuda_fail(e, "pool_rows_kernel launch");
    ++g_launches;
    return FASTKV_OK;
  }

  // ---- two kernels with buffered logits: devices without cooperative launch, or on request ----
  e = cudaMemsetAsync(ws, 0, lay.zero_bytes, stream);
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(workspace header)");

  ScoreParams sp;
  sp.batch = s.batch; sp.total_len = s.total_len; sp.n_kv_heads = s.n_kv_heads; sp.group = G;
  sp.window = s.window; sp.n_rows = G * s.window; sp.q_layout = s.q_layout;
  sp.tiles_per_cta = lay.tiles_per_cta; sp.max_ranges = lay.max_ranges;
  sp.scale_log2 = scale_log2;
  sp.cu_seqlens = s.cu_seqlens;
  sp.logits = reinterpret_cast<float*>(ws + lay.off_logits);
  sp.ld_logits = lay.ld_logits;
  sp.partial = reinterpret_cast<float2*>(ws + lay.off_partial);
  sp.final_stats = reinterpret_cast<float2*>(ws + lay.off_final);
  sp.counters = reinterpret_cast<int*>(ws + lay.off_counters);
  sp.hdr = hdr;
  dim3 grid(s.n_kv_heads, lay.max_ranges, s.batch);
  {
    TimedLaunch timed(KID_SCORE, stream);
    e = launch_score_logits(s.head_dim, lay.npad, tmap_k, tmap_q, sp, grid, stream);
  }
  if (e != cudaSuccess) return cuda_fail(e, "score_logits_kernel launch");
  ++g_launches;

  PoolParams pp;
  pp.total_len = s.total_len; pp.n_kv_heads = s.n_kv_heads; pp.group = G; pp.window = s.window;
  pp.npad = lay.npad; pp.pool_kernel = s.pool_kernel; pp.pool_mode = s.pool_mode; pp.agg_order = s.agg_order;
  pp.cu_seqlens = sp.cu_seqlens; pp.logits = sp.logits; pp.ld_logits = lay.ld_logits;
  pp.final_stats = sp.final_stats; pp.scores_kv = scores_kv; pp.ld_scores = s.total_len;
  pp.scores_tsp = scores_tsp;
  if (score_pool_smem_bytes(pp) > 200 * 1024)
    return fail(FASTKV_ERR_UNSUPPORTED, "heads x pool halo do not fit the pooling kernel's shared memory");
  {
    TimedLaunch timed(KID_POOL, stream);
    e = launch_score_pool(pp, s.max_len, s.batch, stream);
  }
  if (e != cudaSuccess) return cuda_fail(e, "score_pool_kernel launch");
  ++g_launches;
  return FASTKV_OK;
}

static int fill_select_set(const fastkv_shape* shape, const float* scores, const fastkv_budget* budget, int32_t* idx,
                           int n_rows, const char* name, SelectSet* set) {
  if (scores == nullptr || idx == nullptr) return fail(FASTKV_ERR_INVALID_ARG, "%s: scores and idx are required", name);
  int rc = check_budget(shape, budget, name);
  if (rc) return rc;
  set->scores = scores; set->ld_scores = shape->total_len; set->idx = idx; set->ld_idx = budget->total;
  set->cu_k = budget->cu_k; set->k_uniform = budget->k; set->n_rows = n_rows;
  return FASTKV_OK;
}

static int launch_select_sets(const fastkv_shape* shape, SelectParams& p, void* workspace, size_t workspace_bytes,
                              void* stream_) {
  int rc = check_workspace(workspace, workspace_bytes, sizeof(WorkspaceHeader));
  if (rc) return rc;
  if ((rc = check_device())) return rc;
  p.cu_seqlens = shape->cu_seqlens; p.total_len = shape->total_len; p.window = shape->window;
  p.force_window = shape->force_window; p.hdr = static_cast<WorkspaceHeader*>(workspace);
  cudaError_t e;
  {
    TimedLaunch timed(KID_SELECT, static_cast<cudaStream_t>(stream_));
    e = launch_select(p, shape->batch, shape->max_len, static_cast<cudaStream_t>(stream_));
  }
  if (e != cudaSuccess) return cuda_fail(e, "select_topk_kernel launch");
  ++g_launches;
  return FASTKV_OK;
}

int fastkv_select_kv(const fastkv_shape* shape, const float* scores_kv, const fastkv_budget* budget,
                     int32_t* idx_kv, void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_shape(shape, false);
  if (rc) return rc;
  SelectParams p;
  memset(&p, 0, sizeof p);
  if ((rc = fill_select_set(shape, scores_kv, budget, idx_kv, shape->n_kv_heads, "select_kv", &p.set[0]))) return rc;
  return launch_select_sets(shape, p, workspace, workspace_bytes, stream);
}

int fastkv_select_tsp(const fastkv_shape* shape, const float* scores_tsp, const fastkv_budget* budget,
                      int32_t* idx_tsp, void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_shape(shape, false);
  if (rc) return rc;
  SelectParams p;
  memset(&p, 0, sizeof p);
  if ((rc = fill_select_set(shape, scores_tsp, budget, idx_tsp, 1, "select_tsp", &p.set[0]))) return rc;
  return launch_select_sets(shape, p, workspace, workspace_bytes, stream);
}

int fastkv_select(const fastkv_shape* shape, const float* scores_kv, const fastkv_budget* kv, int32_t* idx_kv,
                  const float* scores_tsp, const fastkv_budget* tsp, int32_t* idx_tsp, void* workspace,
                  size_t workspace_bytes, void* stream) {
  int rc = check_shape(shape, false);
  if (rc) return rc;
  SelectParams p;
  memset(&p, 0, sizeof p);
  if ((rc = fill_select_set(shape, scores_kv, kv, idx_kv, shape->n_kv_heads, "select (kv)", &p.set[0]))) return rc;
  if ((rc = fill_select_set(shape, scores_tsp, tsp, idx_tsp, 1, "select (tsp)", &p.set[1]))) return rc;
  return launch_select_sets(shape, p, workspace, workspace_bytes, stream);
}

int fastkv_compact(const fastkv_shape* shape, const int32_t* idx_kv, const fastkv_budget* kv,
                   const int32_t* idx_tsp, const fastkv_budget* tsp, const void* k, const void* v,
                   const void* hidden, const int32_t* pos_ids, void* k_out, void* v_out,
                   void* hidden_out, int32_t* pos_out, void* workspace, size_t workspace_bytes,
                   void* stream_) {
  int rc = check_shape(shape, false);
  if (rc) return rc;
  const fastkv_shape& s = *shape;
  if ((rc = check_workspace(workspace, workspace_bytes, sizeof(WorkspaceHeader)))) return rc;
  if ((k == nullptr) != (k_out == nullptr) || (v == nullptr) != (v_out == nullptr) ||
      (hidden == nullptr) != (hidden_out == nullptr) || (pos_ids == nullptr) != (pos_out == nullptr))
    return fail(FASTKV_ERR_INVALID_ARG, "compact: each source needs its destination and vice versa");
  CompactParams cp;
  memset(&cp, 0, sizeof cp);
  cp.batch = s.batch; cp.total_len = s.total_len; cp.cu_seqlens = s.cu_seqlens;
  cp.hdr = static_cast<WorkspaceHeader*>(workspace);
  int n = 0;
  if (k != nullptr || v != nullptr) {
    if (idx_kv == nullptr) return fail(FASTKV_ERR_INVALID_ARG, "compact: idx_kv is required with k/v");
    if ((rc = check_budget(shape, kv, "compact kv"))) return rc;
    if (s.head_dim < 8 || s.head_dim % 8) return fail(FASTKV_ERR_UNSUPPORTED, "compact: head_dim must be a multiple of 8");
    const void* src[2] = {k, v};
    void* dst[2] = {k_out, v_out};
    const long long st[2] = {s.k_stride_tok, s.v_stride_tok}, sh[2] = {s.k_stride_head, s.v_stride_head};
    for (int t = 0; t < 2; ++t) {
      if (src[t] == nullptr) continue;
      if (st[t] % 8 || sh[t] % 8 || reinterpret_cast<uintptr_t>(src[t]) % 16 || reinterpret_cast<uintptr_t>(dst[t]) % 16)
        return fail(FASTKV_ERR_UNSUPPORTED, "compact: k/v need 16-byte aligned bases and strides");
      GatherJob& j = cp.job[n++];
      j.src = static_cast<const uint8_t*>(src[t]); j.dst = static_cast<uint8_t*>(dst[t]);
      j.idx = idx_kv; j.cu_k = kv->cu_k; j.k_uniform = kv->k; j.ld_idx = kv->total;
      j.src_tok_bytes = st[t] * 2; j.src_head_bytes = sh[t] * 2;
      j.heads = s.n_kv_heads; j.rows = kv->total; j.row_chunks = s.head_dim / 8;
    }
  }
  if (hidden != nullptr || pos_ids != nullptr) {
    if (idx_tsp == nullptr) return fail(FASTKV_ERR_INVALID_ARG, "compact: idx_tsp is required with hidden/pos_ids");
    if ((rc = check_budget(shape, tsp, "compact tsp"))) return rc;
    if (hidden != nullptr && (s.hidden_dim < 8 || s.hidden_dim % 8 || s.hidden_stride_tok % 8 ||
                              s.hidden_stride_tok < s.hidden_dim ||
                              reinterpret_cast<uintptr_t>(hidden) % 16 || reinterpret_cast<uintptr_t>(hidden_out) % 16))
      return fail(FASTKV_ERR_UNSUPPORTED, "compact: hidden needs hidden_dim % 8 == 0 and 16-byte alignment");
    GatherJob& j = cp.job[n++];
    j.src = static_cast<const uint8_t*>(hidden); j.dst = static_cast<uint8_t*>(hidden_out);
    j.idx = idx_tsp; j.cu_k = tsp->cu_k; j.k_uniform = tsp->k; j.ld_idx = tsp->total;
    j.src_tok_bytes = s.hidden_stride_tok * 2; j.src_head_bytes = 0;
    j.heads = 1; j.rows = tsp->total; j.row_chunks = hidden ? s.hidden_dim / 8 : 0;
    j.pos_src = pos_ids; j.pos_dst = pos_out;
  }
  cp.n_jobs = n;
  if (n == 0) return FASTKV_OK;
  if ((rc = check_device())) return rc;
  cudaError_t e;
  {
    TimedLaunch timed(KID_COMPACT, static_cast<cudaStream_t>(stream_));
    e = launch_compact(cp, static_cast<cudaStream_t>(stream_));
  }
  if (e != cudaSuccess) return cuda_fail(e, "compact_rows_kernel launch");
  ++g_launches;
  return FASTKV_OK;
}

int fastkv_decode_attn_workspace_bytes(const fastkv_shape* shape, size_t* bytes) {
  int rc = check_shape(shape, false);
  if (rc) return rc;
  if (bytes == nullptr) return fail(FASTKV_ERR_INVALID_ARG, "bytes is NULL");
  *bytes = round_up(decode_workspace_bytes(shape->batch, shape->n_kv_heads, shape->n_q_heads / shape->n_kv_heads,
                                           shape->head_dim), 256);
  return FASTKV_OK;
}

int fastkv_decode_attn(const fastkv_shape* shape, const void* q, const void* k_cache, const void* v_cache,
                       const fastkv_budget* kv, float* out, float* lse, void* workspace, size_t workspace_bytes,
                       void* stream_) {
  int rc = check_shape(shape, false);
  if (rc) return rc;
  const fastkv_shape& s = *shape;
  const int G = s.n_q_heads / s.n_kv_heads;
  if (!q || !k_cache || !v_cache || !out) return fail(FASTKV_ERR_INVALID_ARG, "decode_attn: q, k_cache, v_cache and out are required");
  if ((rc = check_budget(shape, kv, "decode_attn"))) return rc;
  if (s.head_dim != 64 && s.head_dim != 128) return fail(FASTKV_ERR_UNSUPPORTED, "decode_attn: head_dim must be 64 or 128");
  if (G > 8) return fail(FASTKV_ERR_UNSUPPORTED, "decode_attn: more than 8 query heads per KV head is not built");
  if (reinterpret_cast<uintptr_t>(k_cache) % 16 || reinterpret_cast<uintptr_t>(v_cache) % 16)
    return fail(FASTKV_ERR_UNSUPPORTED, "decode_attn: the caches must be 16-byte aligned");
  if (!(s.softmax_scale >= 0.0f) || std::isinf(s.softmax_scale)) return fail(FASTKV_ERR_INVALID_ARG, "softmax_scale must be finite and >= 0");
  const size_t need = round_up(decode_workspace_bytes(s.batch, s.n_kv_heads, G, s.head_dim), 256);
  if ((rc = check_workspace(workspace, workspace_bytes, need))) return rc;
  if ((rc = check_device())) return rc;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const size_t parts = static_cast<size_t>(s.batch) * s.n_kv_heads * kDecodeMaxSplits * G;
  DecodeParams p;
  CUtensorMap tmap_k, tmap_v;
  const long long head_stride = static_cast<long long>(kv->total) * s.head_dim;
  if ((rc = encode_bf16_3d(&tmap_k, k_cache, s.head_dim, s.n_kv_heads, kv->total, head_stride, s.head_dim, 1, 16)) ||
      (rc = encode_bf16_3d(&tmap_v, v_cache, s.head_dim, s.n_kv_heads, kv->total, head_stride, s.head_dim, 1, 16)))
    return rc;
  p.q = static_cast<const uint16_t*>(q); p.ld_cache = kv->total;
  p.cu_k = kv->cu_k; p.k_uniform = kv->k; p.n_q_heads = s.n_q_heads; p.n_kv_heads = s.n_kv_heads; p.group = G;
  const float scale = s.softmax_scale > 0.0f ? s.softmax_scale : 1.0f / std::sqrt(static_cast<float>(s.head_dim));
  p.scale_log2 = scale * 1.4426950408889634f;
  p.out = out; p.lse = lse;
  p.part_ml = reinterpret_cast<float2*>(ws + sizeof(WorkspaceHeader));
  p.part_o = reinterpret_cast<float*>(ws + sizeof(WorkspaceHeader) + round_up(parts * sizeof(float2), 256));
  p.hdr = reinterpret_cast<WorkspaceHeader*>(ws);
  const int k_max = kv->cu_k ? (kv->total < s.max_len ? kv->total : s.max_len) : kv->k;
  cudaError_t e;
  int launched = 0;
  {
    TimedLaunch timed(KID_DECODE, static_cast<cudaStream_t>(stream_));
    e = launch_decode_attn(tmap_k, tmap_v, p, s.head_dim, s.batch, k_max, static_cast<cudaStream_t>(stream_), &launched);
  }
  g_launches += launched;
  if (e != cudaSuccess) return cuda_fail(e, "decode_attn_kernel launch");
  return FASTKV_OK;
}

// ---- prefill attention with the scores as a by-product ------------------------------------------------
namespace {
struct PrefillLayout {
  size_t off_wstat, off_a, off_wlog, bytes;
  long long ld;
  int rows;                     // un-pooled rows the pooling kernel reads
};
PrefillLayout prefill_layout(const fastkv_shape& s) {
  PrefillLayout l;
  const bool per_head = s.agg_order == FASTKV_POOL_THEN_GROUP;
  l.rows = per_head ? s.n_q_heads : s.n_kv_heads;
  l.ld = static_cast<long long>(round_up(static_cast<size_t>(s.total_len), 64));
  size_t off = sizeof(WorkspaceHeader);
  l.off_wstat = off;
  off += round_up(sizeof(float2) * static_cast<size_t>(s.batch) * s.n_q_heads * s.window, 256);
  l.off_a = off;
  off += round_up(sizeof(float) * static_cast<size_t>(l.rows) * l.ld, 256);
  l.off_wlog = off;
  off += round_up(sizeof(float) * static_cast<size_t>(s.n_q_heads) * s.window * l.ld, 256);
  l.bytes = off;
  return l;
}
int check_prefill_shape(const fastkv_shape* s) {
  int rc = check_shape(s, true);
  if (rc) return rc;
  if (s->q_layout != FASTKV_Q_FULL) return fail(FASTKV_ERR_INVALID_ARG, "prefill attention needs the full packed Q (FASTKV_Q_FULL)");
  if (s->v_stride_tok % 8 || s->v_stride_head % 8)
    return fail(FASTKV_ERR_UNSUPPORTED, "v strides must be multiples of 8 elements (16 bytes)");
  if (s->v_stride_head < s->head_dim || s->v_stride_tok < s->head_dim)
    return fail(FASTKV_ERR_INVALID_ARG, "v strides are smaller than head_dim");
  return FASTKV_OK;
}
}  // namespace

int fastkv_prefill_workspace_bytes(const fastkv_shape* shape, size_t* bytes) {
  int rc = check_prefill_shape(shape);
  if (rc) return rc;
  if (bytes == nullptr) return fail(FASTKV_ERR_INVALID_ARG, "bytes is NULL");
  *bytes = prefill_layout(*shape).bytes;
  return FASTKV_OK;
}

int fastkv_prefill_attention(const fastkv_shape* shape, const void* q, const void* k, const void* v, void* out,
                             float* scores_kv, float* scores_tsp, void* workspace, size_t workspace_bytes,
                             void* stream_) {
  int rc = check_prefill_shape(shape);
  if (rc) return rc;
  if (!q || !k || !v || !out) return fail(FASTKV_ERR_INVALID_ARG, "prefill_attention: q, k, v and out are required");
  if (scores_tsp != nullptr && scores_kv == nullptr)
    return fail(FASTKV_ERR_INVALID_ARG, "prefill_attention: scores_tsp needs scores_kv");
  if (reinterpret_cast<uintptr_t>(out) % 16) return fail(FASTKV_ERR_UNSUPPORTED, "prefill_attention: out must be 16-byte aligned");
  const fastkv_shape& s = *shape;
  const PrefillLayout lay = prefill_layout(s);
  const bool want_scores = scores_kv != nullptr;
  if ((rc = check_workspace(workspace, workspace_bytes, want_scores ? lay.bytes : sizeof(WorkspaceHeader)))) return rc;
  if ((rc = check_device())) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int G = s.n_q_heads / s.n_kv_heads;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  CUtensorMap tmap_q, tmap_k, tmap_v;
  if ((rc = encode_bf16_3d(&tmap_q, q, s.head_dim, s.n_q_heads, s.total_len, s.q_stride_head, s.q_stride_tok, 1, 128)) ||
      (rc = encode_bf16_3d(&tmap_k, k, s.head_dim, s.n_kv_heads, s.total_len, s.k_stride_head, s.k_stride_tok, 1, 128)) ||
      (rc = encode_bf16_3d(&tmap_v, v, s.head_dim, s.n_kv_heads, s.total_len, s.v_stride_head, s.v_stride_tok, 1, 128)))
    return rc;
  cudaError_t e = cudaMemsetAsync(ws, 0, sizeof(WorkspaceHeader), stream);
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(workspace header)");
  const float scale = s.softmax_scale > 0.0f ? s.softmax_scale : 1.0f / std::sqrt(static_cast<float>(s.head_dim));
  PrefillParams pp;
  pp.batch = s.batch; pp.total_len = s.total_len; pp.n_q_heads = s.n_q_heads; pp.group = G; pp.window = s.window;
  pp.scale_log2 = scale * 1.4426950408889634f;
  pp.cu_seqlens = s.cu_seqlens;
  pp.out = out;
  pp.out_stride_tok = static_cast<long long>(s.n_q_heads) * s.head_dim;      // dense [total_len, n_q_heads, head_dim]
  pp.out_stride_head = s.head_dim;
  pp.wlog = want_scores ? reinterpret_cast<float*>(ws + lay.off_wlog) : nullptr;
  pp.ld_w = lay.ld;
  pp.wstat = reinterpret_cast<float2*>(ws + lay.off_wstat);
  pp.hdr = reinterpret_cast<WorkspaceHeader*>(ws);
  pp.wait_limit = g_debug.wait_limit_cycles > 0 ? g_debug.wait_limit_cycles : kWaitLimitCycles;
  pp.skip_commit_tile = g_debug.prefill_skip_commit - 1;
  {
    TimedLaunch timed(KID_PREFILL, stream);
    e = launch_prefill_attn(s.head_dim, tmap_q, tmap_k, tmap_v, pp, s.max_len, stream);
  }
  if (e != cudaSuccess) return cuda_fail(e, "prefill_attn_kernel launch");
  ++g_launches;
  if (!want_scores) return FASTKV_OK;
  WindowScoresParams wp;
  wp.total_len = s.total_len; wp.n_q_heads = s.n_q_heads; wp.n_kv_heads = s.n_kv_heads; wp.group = G; wp.window = s.window;
  wp.per_head = s.agg_order == FASTKV_POOL_THEN_GROUP;
  wp.cu_seqlens = s.cu_seqlens; wp.wlog = pp.wlog; wp.ld_w = lay.ld; wp.wstat = pp.wstat;
  wp.a_out = reinterpret_cast<float*>(ws + lay.off_a); wp.ld_a = lay.ld;
  {
    TimedLaunch timed(KID_WINDOW_SCORES, stream);
    e = launch_window_scores(wp, s.max_len, s.batch, stream);
  }
  if (e != cudaSuccess) return cuda_fail(e, "window_scores_kernel launch");
  ++g_launches;
  PoolRowsParams rp;
  rp.total_len = s.total_len; rp.n_kv_heads = s.n_kv_heads; rp.group = G; rp.window = s.window;
  rp.per_head = wp.per_head; rp.pool_kernel = s.pool_kernel; rp.pool_mode = s.pool_mode;
  rp.cu_seqlens = s.cu_seqlens; rp.a = wp.a_out; rp.ld_a = lay.ld;
  rp.scores_kv = scores_kv; rp.ld_scores = s.total_len; rp.scores_tsp = scores_tsp;
  if (sizeof(float) * static_cast<size_t>(lay.rows) * (kPoolKeys + s.pool_kernel) > 200 * 1024)
    return fail(FASTKV_ERR_UNSUPPORTED, "heads x pool halo do not fit the pooling kernel's shared memory");
  {
    TimedLaunch timed(KID_POOL, stream);
    e = launch_pool_rows(rp, s.max_len, s.batch, stream);
  }
  if (e != cudaSuccess) return cuda_fail(e, "pool_rows_kernel launch");
  ++g_launches;
  return FASTKV_OK;
}

int fastkv_device_status(const void* workspace, void* stream, int32_t* status, int32_t* site) {
  if (workspace == nullptr || status == nullptr) return fail(FASTKV_ERR_INVALID_ARG, "workspace and status are required");
  cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
  int32_t words[2] = {0, 0};
  e = cudaMemcpy(words, workspace, sizeof words, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy(status word)");
  *status = words[0];
  if (site) *site = words[1];
  return FASTKV_OK;
}

// ---- host-buffer layer step -------------------------------------------------------------------------
namespace {
struct Arena {
  size_t q, k, v, hidden, pos, cu, scores_kv, scores_tsp, idx_kv, idx_tsp, k_out, v_out, hidden_out, pos_out, ws;
  size_t q_bytes, k_bytes, v_bytes, hidden_bytes, ws_bytes, bytes;
};
Arena make_arena(const fastkv_shape& s, int k_kv, int k_tsp) {
  Arena a;
  size_t off = 0;
  auto take = [&](size_t n) { size_t o = off; off += round_up(n, 256); return o; };
  const size_t q_rows = s.q_layout == FASTKV_Q_WINDOW ? static_cast<size_t>(s.batch) * s.window : s.total_len;
  a.q_bytes = q_rows * s.q_stride_tok * 2;
  a.k_bytes = static_cast<size_t>(s.total_len) * s.k_stride_tok * 2;
  a.v_bytes = static_cast<size_t>(s.total_len) * s.v_stride_tok * 2;
  a.hidden_bytes = static_cast<size_t>(s.total_len) * s.hidden_stride_tok * 2;
  a.q = take(a.q_bytes); a.k = take(a.k_bytes); a.v = take(a.v_bytes);
  a.hidden = take(k_tsp ? a.hidden_bytes : 0); a.pos = take(k_tsp ? 4 * static_cast<size_t>(s.total_len) : 0);
  a.cu = take(4 * (static_cast<size_t>(s.batch) + 1));
  a.scores_kv = take(4 * static_cast<size_t>(s.n_kv_heads) * s.total_len);
  a.scores_tsp = take(4 * static_cast<size_t>(s.total_len));
  a.idx_kv = take(4 * static_cast<size_t>(s.n_kv_heads) * s.batch * k_kv);
  a.idx_tsp = take(4 * static_cast<size_t>(s.batch) * k_tsp);
  a.k_out = take(2 * static_cast<size_t>(s.n_kv_heads) * s.batch * k_kv * s.head_dim);
  a.v_out = take(2 * static_cast<size_t>(s.n_kv_heads) * s.batch * k_kv * s.head_dim);
  a.hidden_out = take(2 * static_cast<size_t>(s.batch) * k_tsp * s.hidden_dim);
  a.pos_out = take(4 * static_cast<size_t>(s.batch) * k_tsp);
  a.ws_bytes = make_layout(s).bytes;
  a.ws = take(a.ws_bytes);
  a.bytes = off;
  return a;
}
}  // namespace

int fastkv_layer_host_arena_bytes(const fastkv_shape* shape, int32_t k_kv, int32_t k_tsp, size_t* bytes) {
  int rc = check_shape(shape, true);
  if (rc) return rc;
  if (bytes == nullptr || k_kv < 1 || k_tsp < 0) return fail(FASTKV_ERR_INVALID_ARG, "layer_host: bad k or NULL bytes");
  *bytes = make_arena(*shape, k_kv, k_tsp).bytes;
  return FASTKV_OK;
}

int fastkv_layer_host(const fastkv_shape* shape, int32_t k_kv, int32_t k_tsp, const void* q,
                      const void* k, const void* v, const void* hidden, const int32_t* pos_ids,
                      int32_t* idx_kv, int32_t* idx_tsp, void* k_out, void* v_out,
                      void* hidden_out, int32_t* pos_out, void* arena, size_t arena_bytes,
                      void* stream_) {
  int rc = check_shape(shape, true);
  if (rc) return rc;
  if (k_kv < 1 || k_tsp < 0) return fail(FASTKV_ERR_INVALID_ARG, "layer_host: bad k");
  if (!q || !k || !v || !idx_kv || !k_out || !v_out) return fail(FASTKV_ERR_INVALID_ARG, "layer_host: q, k, v and the kv outputs are required");
  if (k_tsp && (!hidden || !pos_ids || !idx_tsp || !hidden_out || !pos_out))
    return fail(FASTKV_ERR_INVALID_ARG, "layer_host: the TSP part needs hidden, pos_ids and their outputs");
  const Arena a = make_arena(*shape, k_kv, k_tsp);
  if ((rc = check_workspace(arena, arena_bytes, a.bytes))) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  uint8_t* d = static_cast<uint8_t*>(arena);
  fastkv_shape s = *shape;
  cudaError_t e;
#define FASTKV_COPY(dst, src, n, kind)                                             \
  if ((n) && (e = cudaMemcpyAsync(dst, src, n, kind, stream)) != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync")
  FASTKV_COPY(d + a.q, q, a.q_bytes, cudaMemcpyHostToDevice);
  FASTKV_COPY(d + a.k, k, a.k_bytes, cudaMemcpyHostToDevice);
  FASTKV_COPY(d + a.v, v, a.v_bytes, cudaMemcpyHostToDevice);
  if (k_tsp) {
    FASTKV_COPY(d + a.hidden, hidden, a.hidden_bytes, cudaMemcpyHostToDevice);
    FASTKV_COPY(d + a.pos, pos_ids, 4 * static_cast<size_t>(s.total_len), cudaMemcpyHostToDevice);
  }
  if (shape->cu_seqlens) {
    FASTKV_COPY(d + a.cu, shape->cu_seqlens, 4 * (static_cast<size_t>(s.batch) + 1), cudaMemcpyHostToDevice);
    s.cu_seqlens = reinterpret_cast<const int32_t*>(d + a.cu);
  }
  float* scores_kv = reinterpret_cast<float*>(d + a.scores_kv);
  float* scores_tsp = k_tsp ? reinterpret_cast<float*>(d + a.scores_tsp) : nullptr;
  void* ws = d + a.ws;
  if ((rc = fastkv_score(&s, d + a.q, d + a.k, scores_kv, scores_tsp, ws, a.ws_bytes, stream))) return rc;
  fastkv_budget bkv = {k_kv, k_kv * s.batch, nullptr}, btsp = {k_tsp, k_tsp * s.batch, nullptr};
  int32_t* d_idx_kv = reinterpret_cast<int32_t*>(d + a.idx_kv);
  int32_t* d_idx_tsp = reinterpret_cast<int32_t*>(d + a.idx_tsp);
  if (k_tsp) {
    if ((rc = fastkv_select(&s, scores_kv, &bkv, d_idx_kv, scores_tsp, &btsp, d_idx_tsp, ws, a.ws_bytes, stream))) return rc;
  } else if ((rc = fastkv_select_kv(&s, scores_kv, &bkv, d_idx_kv, ws, a.ws_bytes, stream))) {
    return rc;
  }
  if ((rc = fastkv_compact(&s, d_idx_kv, &bkv, k_tsp ? d_idx_tsp : nullptr, k_tsp ? &btsp : nullptr, d + a.k, d + a.v,
                           k_tsp ? d + a.hidden : nullptr, k_tsp ? reinterpret_cast<const int32_t*>(d + a.pos) : nullptr,
                           d + a.k_out, d + a.v_out, k_tsp ? d + a.hidden_out : nullptr,
                           k_tsp ? reinterpret_cast<int32_t*>(d + a.pos_out) : nullptr, ws, a.ws_bytes, stream)))
    return rc;
  const size_t n_kv = static_cast<size_t>(s.n_kv_heads) * s.batch * k_kv;
  FASTKV_COPY(idx_kv, d_idx_kv, 4 * n_kv, cudaMemcpyDeviceToHost);
  FASTKV_COPY(k_out, d + a.k_out, 2 * n_kv * s.head_dim, cudaMemcpyDeviceToHost);
  FASTKV_COPY(v_out, d + a.v_out, 2 * n_kv * s.head_dim, cudaMemcpyDeviceToHost);
  if (k_tsp) {
    const size_t n_t = static_cast<size_t>(s.batch) * k_tsp;
    FASTKV_COPY(idx_tsp, d_idx_tsp, 4 * n_t, cudaMemcpyDeviceToHost);
    FASTKV_COPY(hidden_out, d + a.hidden_out, 2 * n_t * s.hidden_dim, cudaMemcpyDeviceToHost);
    FASTKV_COPY(pos_out, d + a.pos_out, 4 * n_t, cudaMemcpyDeviceToHost);
  }
#undef FASTKV_COPY
  int32_t status = 0, site = 0;
  if ((rc = fastkv_device_status(ws, stream, &status, &site))) return rc;
  if (status != FASTKV_OK) return fail(status, "device status %d raised at site %d", status, site);
  return FASTKV_OK;
}

const char* fastkv_status_string(int status) {
  switch (status) {
    case FASTKV_OK: return "ok";
    case FASTKV_ERR_INVALID_ARG: return "invalid argument";
    case FASTKV_ERR_UNSUPPORTED: return "unsupported configuration";
    case FASTKV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case FASTKV_ERR_CUDA: return "CUDA call failed";
    case FASTKV_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait gave up";
    case FASTKV_ERR_DEVICE_INDEX: return "an index or budget was out of range on the device";
    default: return "unknown status";
  }
}

const char* fastkv_last_error(void) { return g_last_error; }

int64_t fastkv_kernel_launches(void) { return g_launches.load(); }

}  // extern "C"
