// vsa2_route_noalloc: the router + selection step for callers that must not allocate device memory.
//
// Some callers cannot call cudaMalloc (or any allocating routine) at the point where they need a block map:
// code that runs inside a region where allocation is forbidden or would deadlock (an allocator lock is held,
// a latency-critical loop that was sized up front, a plug-in whose host hands it no allocator), or a process
// whose memory budget was fixed at start-up.  vsa2_route needs a scratch workspace; this variant keeps that
// scratch in a file-scope device array of a fixed, modest size instead, so the caller passes inputs and
// outputs only.
#include <mutex>

#include "common.cuh"

#define VSA2_ROUTE_STATIC_BYTES VSA2_ROUTE_NOALLOC_MAX_BYTES   // 8 MiB, held by every GPU that has loaded the library's device code

// The scratch itself.  In host code this name is only a stand-in for the symbol, never a device address:
// the address is obtained once per device with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_route_scratch[VSA2_ROUTE_STATIC_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

// Device address of the scratch array on the CURRENT device (looked up on the first call per device).
int scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return VSA2_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return VSA2_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_route_scratch) != cudaSuccess || ptr == nullptr) return VSA2_ERR_CUDA;
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return VSA2_OK;
}
}  // namespace

extern "C" int vsa2_route_noalloc(const vsa2_params* p, const void* q, const void* k, const int32_t* budgets,
                                  const vsa2_map* map_out, int32_t* device_status, void* cuda_stream) {
  vsa2_sizes sz;
  int rc = vsa2_query_sizes(p, &sz);
  if (rc != VSA2_OK) return rc;
  if (sz.route_workspace_bytes > (size_t)VSA2_ROUTE_STATIC_BYTES) return VSA2_ERR_STATIC_SCRATCH;
  void* scratch = nullptr;
  if ((rc = scratch_address(&scratch)) != VSA2_OK) return rc;
  // vsa2_route clears the status block and the selection histograms itself and overwrites every other region
  // before reading it, so nothing of the previous call's contents is consumed.
  rc = vsa2_route(p, q, k, budgets, map_out, scratch, (size_t)VSA2_ROUTE_STATIC_BYTES, cuda_stream);
  if (rc != VSA2_OK) return rc;
  if (device_status != nullptr) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(device_status, scratch, sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
      return VSA2_ERR_CUDA;
  }
  return VSA2_OK;
}
