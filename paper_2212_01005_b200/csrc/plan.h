// Internal host-side plan of a subgraph: validated operators with inferred
// shapes, the grouping into mini-subgraphs (one complex operator plus its
// trailing simple operators, Section III-A), the category of every
// complex -> complex link (Section III-B) and the kernel chosen for fused mode.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

#include "../../include/ago.h"

namespace ago {

struct Shape {
  int rank = 0;
  int64_t d[AGO_MAX_RANK] = {0, 0, 0, 0};
  int64_t numel() const {
    int64_t n = 1;
    for (int i = 0; i < rank; ++i) n *= d[i];
    return n;
  }
  int64_t last() const { return d[rank - 1]; }
  bool operator==(const Shape& o) const {
    if (rank != o.rank) return false;
    for (int i = 0; i < rank; ++i)
      if (d[i] != o.d[i]) return false;
    return true;
  }
};

struct OpInfo {
  ago_op_t op;
  Shape in, out;
  int weight = -1;  // index into weights[] for CONV2D / GEMM / BIAS_ADD
  bool complex_op() const { return op.kind <= AGO_OP_BATCHED_PV; }
  bool depthwise() const { return op.kind == AGO_OP_CONV2D && op.p[5] > 1; }
  bool pointwise() const {
    return op.kind == AGO_OP_CONV2D && op.p[5] == 1 && op.p[1] == 1 && op.p[2] == 1 && op.p[3] == 1 && op.p[4] == 0;
  }
};

// One kernel launch of an unfused mode: ops [first, last] of the chain.
struct Stage {
  int first = 0, last = 0;
  int complex_index = -1;  // index of the complex op (== first) or -1 for a simple-only stage
  bool softmax = false;    // a SOFTMAX_ROWS launch
  bool transpose = false;  // a TRANSPOSE launch
};

// Element-wise operator program executed in a kernel epilogue (conventional
// fusion) or by the stand-alone element-wise kernel (per-op mode).
enum EpiCode : int { EPI_BIAS = 0, EPI_RELU, EPI_RELU6, EPI_GELU, EPI_SCALE, EPI_ADD };
constexpr int kMaxEpi = 8;
struct EpiProgram {
  int n = 0;
  int code[kMaxEpi];
  const void* ptr[kMaxEpi];  // EPI_BIAS: float32 vector; EPI_ADD: tensor of the output's dtype and shape
  float f[kMaxEpi];
};

struct Plan {
  int mode = AGO_MODE_FUSED;
  int dtype = AGO_BF16;
  int num_inputs = 0;
  Shape inputs[AGO_MAX_INPUTS];
  std::vector<OpInfo> ops;
  std::vector<Stage> stages;          // launches of this handle's unfused mode
  std::vector<int64_t> weight_bytes;  // per weights[] entry
  std::vector<int> link_category;     // per complex -> complex pair
  Shape output;
  int fused_kernel = AGO_KERNEL_NONE;
  int fused_variant = 0;              // kernel variant within the family, chosen at plan time
  int64_t flops_tensor = 0, flops_cuda = 0, sfu_ops = 0, io_bytes = 0, intermediate_bytes = 0;
  int64_t max_intermediate_bytes = 0;  // largest tensor passed between launches
  int tile_rows = 0;
  int smem_bytes = 0;
  int64_t workspace_traffic_bytes = 0;   // fused kernel: bytes it moves through its device-memory workspace per run
  int num_launches = 1;
};

inline int64_t elem_bytes(int dtype) { return dtype == AGO_FP32 ? 4 : 2; }

// Builds the plan; returns AGO_OK or an error with `err` filled.
ago_status_t build_plan(const ago_subgraph_desc_t* desc, Plan* plan, std::string* err);

}  // namespace ago
