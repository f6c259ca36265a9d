// pisa_route_static: block routing for callers that cannot hand the library a workspace.
//
// Some callers of this library may not allocate device memory at all at the point where they need
// routing: code running inside a memory-pool-managed region where every byte is already assigned,
// plugin entry points of inference servers that forbid allocation after start-up, or a latency
// critical loop where cudaMalloc's implicit device synchronisation is not acceptable.  For them this
// file keeps the scratch that pisa_route needs in a file-scope device array that is part of the
// library image: it exists on every GPU that loads the library, from load until the process exits,
// and costs kStaticScratchBytes of device memory there whether or not the entry point is used.
#include <mutex>

#include "pisa_common.cuh"

namespace pisa {
// the routing of pisa_route on the caller's stream alone (no chunks on a second stream, hence no stream or
// event creation), and its scratch size
int route_unsplit(const pisa_params_t* p, const void* q, const void* k, const void* pyramid, int32_t* idx,
                  float* margin, void* ws, size_t ws_bytes, cudaStream_t s);
int route_unsplit_bytes(const pisa_params_t* p, size_t* bytes);
}  // namespace pisa

namespace {

constexpr size_t kStaticScratchBytes = 32u << 20;      // 32 MiB per GPU
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_route_scratch[kStaticScratchBytes];

// device address of g_route_scratch per device ordinal, filled on first use on that device
static void* g_scratch_addr[kMaxDevices] = {};
static std::mutex g_scratch_mutex;

// In host code the name g_route_scratch is only a handle for the runtime, not a device address;
// the address on the CURRENT device has to be asked for.
int scratch_for_current_device(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { pisa::record_cuda_error("cudaGetDevice", e); return PISA_ERR_CUDA; }
  if (dev < 0 || dev >= kMaxDevices) return PISA_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_route_scratch);
    if (e != cudaSuccess || ptr == nullptr) {
      pisa::record_cuda_error("cudaGetSymbolAddress(static routing scratch)", e);
      return PISA_ERR_CUDA;
    }
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return PISA_OK;
}

}  // namespace

extern "C" int pisa_route_static(const pisa_params_t* p, const void* q, const void* k, const void* pyramid,
                                 int32_t* idx, float* margin, void* stream) {
  size_t need = 0;
  int st = pisa::route_unsplit_bytes(p, &need);
  if (st != PISA_OK) return st;
  if (need > kStaticScratchBytes) return PISA_ERR_STATIC_SCRATCH_TOO_SMALL;
  void* scratch = nullptr;
  st = scratch_for_current_device(&scratch);
  if (st != PISA_OK) return st;
  // The routing runs as ONE sequence of launches on the caller's stream (pisa_route would cut a large
  // problem into chunks on a second, library-owned stream, whose creation allocates).  It clears the
  // status word and the list counters it needs at zero on the stream before its kernels read them;
  // everything else in the scratch is written before it is read.
  return pisa::route_unsplit(p, q, k, pyramid, idx, margin, scratch, need, (cudaStream_t)stream);
}

extern "C" size_t pisa_route_static_capacity(void) { return kStaticScratchBytes; }
