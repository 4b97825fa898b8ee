// Host side of the fused kernels: per-handle state, plan-time tile choice and
// the run-time dispatch onto the kernel of the matched family.
#pragma once
#include <cuda_runtime.h>

#include <string>

#include "plan.h"

namespace ago {

struct FusedState {
  int tile_rows = 0;       // downstream tile extent along the tiled dimension
  int grid = 0;            // CTAs
  int smem_bytes = 0;      // dynamic shared memory per CTA
  int variant = 0;         // kernel variant within the family (feed-forward chain: 1 = thread-block cluster, 3 = cluster of two CTA pairs)
  unsigned workspace_epoch = 0;   // bumped by every ago_subgraph_set_workspace: whatever a kernel family remembers about
                                  // the workspace contents (e.g. "already zeroed") is void after a new attach
  void* impl = nullptr;                  // kernel-family host state (parameters, tensor-map cache)
  void (*impl_free)(void*) = nullptr;
  ~FusedState() { if (impl && impl_free) impl_free(impl); }
};

// Opt-in to the full 227 KB of dynamic shared memory for `func`, once per device (thread-safe).
cudaError_t ensure_max_dynamic_smem(const void* func, int* done_flags);

// SMs of the current device (cudaDevAttrMultiProcessorCount, cached per device). Planning is host-only and may run
// where no device is present: then the count of the part this library is written for (B200: 148).
constexpr int kDefaultSMs = 148;
int device_sm_count();

// Kernel families (each in its own file).
ago_status_t mbv2_plan(Plan* plan, FusedState* st, std::string* err);
ago_status_t attention_plan(Plan* plan, FusedState* st, std::string* err);
ago_status_t attention_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                           void* output, unsigned int* status_word, cudaStream_t stream, std::string* err);
ago_status_t ffn_plan(Plan* plan, FusedState* st, std::string* err);
ago_status_t ffn_pair_plan(Plan* plan, FusedState* st, std::string* err);
ago_status_t ffn_pair_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                          void* output, void* workspace, unsigned int* status_word, cudaStream_t stream, std::string* err);
size_t ffn_pair_workspace_bytes(const Plan& plan);
ago_status_t ffn_cluster_plan(Plan* plan, FusedState* st, std::string* err);   // AGO_ERR_UNSUPPORTED: no cluster split for this shape
ago_status_t ffn_cluster_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                             void* output, void* workspace, unsigned int* status_word, cudaStream_t stream, std::string* err);
size_t ffn_cluster_workspace_bytes(const Plan& plan);   // 0 unless row blocks are split over clusters
size_t ffn_workspace_bytes(const Plan& plan);
ago_status_t ffn_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                     void* output, void* workspace, unsigned int* status_word, cudaStream_t stream, std::string* err);
ago_status_t conv3x3_plan(Plan* plan, FusedState* st, std::string* err);
ago_status_t conv3x3_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                         void* output, unsigned int* status_word, cudaStream_t stream, std::string* err);
ago_status_t pwpw_plan(Plan* plan, FusedState* st, std::string* err);
ago_status_t pwpw_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                      void* output, unsigned int* status_word, cudaStream_t stream, std::string* err);
ago_status_t dwdw_plan(Plan* plan, FusedState* st, std::string* err);
ago_status_t dwdw_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                      void* output, unsigned int* status_word, cudaStream_t stream, std::string* err);
ago_status_t mbv2_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                      void* output, unsigned int* status_word, cudaStream_t stream, std::string* err);

// Launch configuration of a fused kernel: programmatic stream serialization allowed, so the grid may be
// scheduled while the previous grid of the stream drains (the kernels call griddepcontrol.wait before
// touching device memory). Use with cudaLaunchKernelEx(&cfg.config, kernel, args...).
struct FusedLaunch {
  cudaLaunchConfig_t config;
  cudaLaunchAttribute attr[1];
  FusedLaunch(dim3 grid, int threads, size_t smem_bytes, cudaStream_t stream) {
    config = cudaLaunchConfig_t{};
    config.gridDim = grid;
    config.blockDim = dim3((unsigned)threads, 1, 1);
    config.dynamicSmemBytes = smem_bytes;
    config.stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    config.attrs = attr;
    config.numAttrs = 1;
  }
};

// Chooses tiles and shared-memory budget for plan->fused_kernel; fills
// plan->tile_rows / smem_bytes. Host only.
ago_status_t fused_plan(Plan* plan, FusedState* st, std::string* err);

// Scratch the fused kernel needs in device memory (0 for most families).
size_t fused_workspace_bytes(const Plan& plan);

// Enqueue the fused kernel.
ago_status_t fused_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                       void* output, void* workspace, unsigned int* status_word, cudaStream_t stream,
                       std::string* err);

}  // namespace ago
