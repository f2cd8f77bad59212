// cosa_kap_select_static: Stage 1 for callers that may not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc when a request arrives: an inference
// server that handed the whole GPU to its own memory pool at start-up has nothing left for the
// driver to give, and a latency-critical serving loop cannot afford the device-wide
// synchronisation an allocation (or the matching free) implies.  The fast KAP path needs
// scratch memory between its kernels (screened scores, per-row best blocks, the redo list).
// Here that scratch is a fixed array in the library's own device image, so the call touches no
// allocator at all.  The price is a size limit and that every call on a device shares the array.
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t kStaticScratchBytes = 4u << 20;  // 4 MiB per device that loads the library

// Lives in device memory of every GPU that loads this library, until the process exits.
static __device__ __align__(256) unsigned char g_kap_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {nullptr};
std::mutex g_mu;

// Device address of the array on the current device.  In host code the array's name is only a
// handle for the runtime, never a pointer a kernel could use; the address comes from
// cudaGetSymbolAddress, asked once per device with that device current.
int static_scratch(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return COSA_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_kap_static_scratch);
    if (e != cudaSuccess || !ptr) return COSA_ERR_CUDA;
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return COSA_OK;
}

}  // namespace

extern "C" {

size_t cosa_kap_select_static_max_bytes(void) { return kStaticScratchBytes; }

int cosa_kap_select_static(const void* q, const void* k, const cosa_shape* shape, float budget, int32_t* out_order,
                           int32_t* out_count, void* stream, const cosa_options* opt) {
  cosa_options o;
  if (opt) o = *opt; else cosa_default_options(&o);
  o.workspace = nullptr;
  o.workspace_bytes = 0;
  if (!shape) return COSA_ERR_INVALID_ARG;
  const size_t need = cosa_workspace_bytes(0, shape, &o);
  if (need > kStaticScratchBytes) return COSA_ERR_WORKSPACE;  // problem too large for the built-in scratch
  void* scratch = nullptr;
  int rc = static_scratch(&scratch);
  if (rc != COSA_OK) return rc;
  o.workspace = scratch;                 // an explicit workspace: the call below never allocates
  o.workspace_bytes = kStaticScratchBytes;
  return cosa_kap_select_ex(q, k, shape, budget, out_order, out_count, stream, &o);
}

}  // extern "C"
