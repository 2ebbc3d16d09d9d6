// fastkv_score_static: the scoring call for callers that cannot allocate device memory.
//
// Some hosts of this library have no way to obtain a workspace: a plug-in running inside a
// serving process whose allocator is owned by the framework and closed to it, a callback invoked
// where cudaMalloc is forbidden, or a thin C client that links no allocator at all.  For them
// the scratch memory of the scoring kernels lives in this translation unit as a fixed device
// array, and the entry point below hands its address to the ordinary scoring path.
#include <cstdio>
#include <mutex>

#include "common.cuh"

namespace {

// 16 MiB: enough for the Llama-3.1-8B head shape (8 KV heads, G*w = 32) up to about 500 000 tokens.
// Every GPU on which this library is loaded holds the array until the process exits.
constexpr size_t kStaticScratchBytes = size_t(16) << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

}  // namespace

extern "C" {

int fastkv_score_static(const fastkv_shape* shape, const void* q, const void* k, float* scores_kv,
                        float* scores_tsp, void* stream) {
  size_t need = 0;
  int rc = fastkv_workspace_bytes(shape, &need);
  if (rc != FASTKV_OK) return rc;
  if (need > kStaticScratchBytes) {
    char msg[256];
    snprintf(msg, sizeof msg,
             "fastkv_score_static: this shape needs %zu bytes of scratch, the built-in array holds %zu; "
             "use fastkv_score with a caller-provided workspace",
             need, kStaticScratchBytes);
    return fastkv::report_error(FASTKV_ERR_WORKSPACE, msg);
  }
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    return fastkv::report_error(FASTKV_ERR_CUDA, "fastkv_score_static: no usable current device");
  }
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_ptr[dev] == nullptr) {
      // In host code the array's name is only a handle; its device address has to be asked for,
      // once per device, with that device current.
      void* p = nullptr;
      cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
      if (e != cudaSuccess || p == nullptr) {
        char msg[256];
        snprintf(msg, sizeof msg, "fastkv_score_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        return fastkv::report_error(FASTKV_ERR_CUDA, msg);
      }
      g_scratch_ptr[dev] = p;
    }
    scratch = g_scratch_ptr[dev];
  }
  // fastkv_score clears the part of the scratch that must start at zero (status word, counters).
  return fastkv_score(shape, q, k, scores_kv, scores_tsp, scratch, kStaticScratchBytes, stream);
}

int fastkv_score_static_status(void* stream, int32_t* status, int32_t* site) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
    return fastkv::report_error(FASTKV_ERR_CUDA, "fastkv_score_static_status: no usable current device");
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    scratch = g_scratch_ptr[dev];
  }
  if (scratch == nullptr)
    return fastkv::report_error(FASTKV_ERR_INVALID_ARG,
                                "fastkv_score_static_status: fastkv_score_static has not run on this device");
  return fastkv_device_status(scratch, stream, status, site);   // the status word heads the array
}

}  // extern "C"
