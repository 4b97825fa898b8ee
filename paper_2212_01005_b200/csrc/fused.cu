// Dispatch of the fused kernel families.
#include "fused.h"

#include <mutex>

namespace ago {

cudaError_t ensure_max_dynamic_smem(const void* func, int* done_flags) {
  static std::mutex guard;   // the per-kernel flag arrays are shared by every handle and thread
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(guard);
  if (done_flags[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess) done_flags[dev] = 1;
  return e;
}

int device_sm_count() {
  static std::mutex guard;
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();   // planning on a host without a device is legal: clear the sticky "no device" error
    return kDefaultSMs;
  }
  std::lock_guard<std::mutex> lock(guard);
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
      cudaGetLastError();
      return kDefaultSMs;
    }
    cached[dev] = n;
  }
  return cached[dev];
}

ago_status_t fused_plan(Plan* plan, FusedState* st, std::string* err) {
  switch (plan->fused_kernel) {
    case AGO_KERNEL_DEPTHWISE:
      return AGO_OK;
    case AGO_KERNEL_MBV2_BLOCK:
    case AGO_KERNEL_PW_DW:
    case AGO_KERNEL_DW_PW:
      return mbv2_plan(plan, st, err);
    case AGO_KERNEL_DW_DW:
      return dwdw_plan(plan, st, err);
    case AGO_KERNEL_PW_PW:
    case AGO_KERNEL_GEMM_PERMUTE_GEMM:
      return pwpw_plan(plan, st, err);
    case AGO_KERNEL_ATTENTION:
      return attention_plan(plan, st, err);
    case AGO_KERNEL_FFN: {
      // many rows: the cluster of two CTA pairs (256 rows per weight tile); else the cluster kernel where the shape
      // splits over 2..4 CTAs; else the kernel that tiles the reduction
      ago_status_t s = ffn_pair_plan(plan, st, err);
      if (s == AGO_ERR_UNSUPPORTED) s = ffn_cluster_plan(plan, st, err);
      return s == AGO_ERR_UNSUPPORTED ? ffn_plan(plan, st, err) : s;
    }
    case AGO_KERNEL_CONV3X3_PAIR:
      return conv3x3_plan(plan, st, err);
    default:
      *err = "fused mode: no kernel is built for this family yet";
      return AGO_ERR_UNSUPPORTED;
  }
}

size_t fused_workspace_bytes(const Plan& plan) {
  if (plan.fused_kernel != AGO_KERNEL_FFN) return 0;
  if (plan.fused_variant == 3) return ffn_pair_workspace_bytes(plan);
  return plan.fused_variant == 0 ? ffn_workspace_bytes(plan) : ffn_cluster_workspace_bytes(plan);
}

ago_status_t fused_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                       void* output, void* workspace, unsigned int* status_word, cudaStream_t stream,
                       std::string* err) {
  switch (plan.fused_kernel) {
    case AGO_KERNEL_MBV2_BLOCK:
    case AGO_KERNEL_PW_DW:
    case AGO_KERNEL_DW_PW:
      return mbv2_run(plan, st, inputs, weights, output, status_word, stream, err);
    case AGO_KERNEL_DW_DW:
      return dwdw_run(plan, st, inputs, weights, output, status_word, stream, err);
    case AGO_KERNEL_PW_PW:
    case AGO_KERNEL_GEMM_PERMUTE_GEMM:
      return pwpw_run(plan, st, inputs, weights, output, status_word, stream, err);
    case AGO_KERNEL_ATTENTION:
      return attention_run(plan, st, inputs, weights, output, status_word, stream, err);
    case AGO_KERNEL_FFN:
      if (st->variant == 3) return ffn_pair_run(plan, st, inputs, weights, output, workspace, status_word, stream, err);
      if (st->variant == 1) return ffn_cluster_run(plan, st, inputs, weights, output, workspace, status_word, stream, err);
      return ffn_run(plan, st, inputs, weights, output, workspace, status_word, stream, err);
    case AGO_KERNEL_CONV3X3_PAIR:
      return conv3x3_run(plan, st, inputs, weights, output, status_word, stream, err);
    default:
      *err = "fused mode: no kernel is built for this family yet";
      return AGO_ERR_UNSUPPORTED;
  }
}

}  // namespace ago
