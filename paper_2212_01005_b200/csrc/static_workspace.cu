// ago_subgraph_run_static: the unfused modes without any caller-side or
// library-side allocation. The scratch for the tensors passed between launches
// lives in a fixed array that is part of the library image.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/ago.h"

struct ago_subgraph_s;

namespace ago {
ago_status_t run_unfused_in(ago_subgraph_s* h, const void* const* inputs, const void* const* weights,
                            void* const* outputs, void* ws, size_t ws_bytes, cudaStream_t stream);
ago_status_t report_failure(ago_status_t s, const char* msg);
}  // namespace ago

namespace {

// Every GPU that loads this library carries these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[AGO_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};  // device address of g_static_scratch, per device ordinal

}  // namespace

extern "C" ago_status_t ago_subgraph_run_static(ago_subgraph_t h, const void* const* inputs,
                                                const void* const* weights, void* const* outputs,
                                                void* cuda_stream) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return ago::report_failure(AGO_ERR_CUDA, cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return ago::report_failure(AGO_ERR_CUDA, "device ordinal out of range");
  void* ws = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
      // In host code the array's name is only a handle for the runtime, not an
      // address a kernel may use: ask for the address on the current device, once.
      void* p = nullptr;
      e = cudaGetSymbolAddress(&p, g_static_scratch);
      if (e != cudaSuccess || !p)
        return ago::report_failure(AGO_ERR_CUDA, e != cudaSuccess ? cudaGetErrorString(e) : "no address for the scratch array");
      g_scratch_addr[dev] = p;
    }
    ws = g_scratch_addr[dev];
  }
  return ago::run_unfused_in(reinterpret_cast<ago_subgraph_s*>(h), inputs, weights, outputs, ws,
                             (size_t)AGO_STATIC_SCRATCH_BYTES, static_cast<cudaStream_t>(cuda_stream));
}
