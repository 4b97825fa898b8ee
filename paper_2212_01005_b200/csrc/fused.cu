// Dispatch of the fused kernel families.
#include "fused.h"

namespace ago {

ago_status_t fused_plan(Plan* plan, FusedState* st, std::string* err) {
  switch (plan->fused_kernel) {
    case AGO_KERNEL_DEPTHWISE:
      return AGO_OK;
    default:
      *err = "fused mode: no kernel is built for this family yet";
      return AGO_ERR_UNSUPPORTED;
  }
}

size_t fused_workspace_bytes(const Plan&) { return 0; }

ago_status_t fused_run(const Plan& plan, FusedState*, const void* const*, const void* const*, void*, void*,
                       unsigned int*, cudaStream_t, std::string* err) {
  *err = "fused mode: no kernel is built for this family yet";
  return AGO_ERR_UNSUPPORTED;
}

}  // namespace ago
