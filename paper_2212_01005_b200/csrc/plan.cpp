// Host-side planner: validates the operator list, infers shapes, groups the
// chain into mini-subgraphs, classifies complex -> complex links and matches
// the chain against the fused kernel families.
#include "plan.h"

#include <cstdio>
#include <cstring>
#include <utility>

namespace ago {

namespace {

std::string fmt(const char* f, long long a = 0, long long b = 0, long long c = 0) {
  char buf[256];
  std::snprintf(buf, sizeof(buf), f, a, b, c);
  return buf;
}

int64_t out_extent(int64_t H, int64_t R, int64_t stride, int64_t pad) {
  int64_t span = H + 2 * pad - R;
  return span < 0 ? 0 : span / stride + 1;
}

bool is_simple_elementwise(int kind) {
  return kind == AGO_OP_BIAS_ADD || kind == AGO_OP_RELU || kind == AGO_OP_RELU6 || kind == AGO_OP_GELU_TANH ||
         kind == AGO_OP_SCALE || kind == AGO_OP_ADD_INPUT || kind == AGO_OP_RESHAPE;   // a reshape is a view
}

// Category of the link whose downstream operator is `down` (Section III-B):
// depthwise reuses its input only along H2, W2; pointwise convolution and
// matrix multiplication only along O2; anything else along O2, H2 and W2.
int classify_link(const OpInfo& down) {
  if (down.depthwise()) return AGO_LINK_DOWNSTREAM_DEPTHWISE;
  if (down.pointwise() || down.op.kind == AGO_OP_GEMM || down.op.kind == AGO_OP_BATCHED_PV ||
      down.op.kind == AGO_OP_BATCHED_QKT)
    return AGO_LINK_DOWNSTREAM_POINTWISE;
  return AGO_LINK_GENERAL;
}

bool kinds_are(const std::vector<OpInfo>& ops, std::initializer_list<int> kinds) {
  if (ops.size() != kinds.size()) return false;
  size_t i = 0;
  for (int k : kinds)
    if (ops[i++].op.kind != k) return false;
  return true;
}

bool conv3x3_s1p1(const OpInfo& o) {
  return o.op.kind == AGO_OP_CONV2D && o.op.p[5] == 1 && o.op.p[1] == 3 && o.op.p[2] == 3 && o.op.p[3] == 1 &&
         o.op.p[4] == 1;
}

int match_fused_family(const Plan& p) {
  const auto& ops = p.ops;
  // depthwise-only mini-subgraph: one depthwise conv followed by element-wise ops
  if (!ops.empty() && ops[0].depthwise()) {
    bool ok = true;
    for (size_t i = 1; i < ops.size(); ++i) ok = ok && is_simple_elementwise(ops[i].op.kind);
    if (ok) return AGO_KERNEL_DEPTHWISE;
  }
  if (p.dtype != AGO_BF16) return AGO_KERNEL_NONE;
  // 1x1 conv + bias + ReLU6 -> depthwise 3x3 (pad 1, stride 1|2) + bias + ReLU6 -> 1x1 conv + bias [-> + input 0]
  {
    const int base[] = {AGO_OP_CONV2D, AGO_OP_BIAS_ADD, AGO_OP_RELU6, AGO_OP_CONV2D,
                        AGO_OP_BIAS_ADD, AGO_OP_RELU6, AGO_OP_CONV2D, AGO_OP_BIAS_ADD};
    if (ops.size() == 8 || ops.size() == 9) {
      bool ok = true;
      for (int i = 0; i < 8; ++i) ok = ok && ops[i].op.kind == base[i];
      if (ok && ops.size() == 9) ok = ops[8].op.kind == AGO_OP_ADD_INPUT && ops[8].op.p[0] == 0;
      if (ok) {
        const OpInfo& dw = ops[3];
        ok = ops[0].pointwise() && ops[6].pointwise() && dw.depthwise() && dw.op.p[1] == 3 && dw.op.p[2] == 3 &&
             dw.op.p[4] == 1 && (dw.op.p[3] == 1 || dw.op.p[3] == 2);
      }
      if (ok) return AGO_KERNEL_MBV2_BLOCK;
    }
  }
  // the two-complex-operator pairs of the micro-benchmark (Section VI-B), each convolution with bias (+ ReLU6)
  {
    auto dw3x3 = [](const OpInfo& o) {
      return o.depthwise() && o.op.p[1] == 3 && o.op.p[2] == 3 && o.op.p[4] == 1 && (o.op.p[3] == 1 || o.op.p[3] == 2);
    };
    if (kinds_are(ops, {AGO_OP_CONV2D, AGO_OP_BIAS_ADD, AGO_OP_RELU6, AGO_OP_CONV2D, AGO_OP_BIAS_ADD, AGO_OP_RELU6})) {
      if (ops[0].pointwise() && dw3x3(ops[3])) return AGO_KERNEL_PW_DW;
      if (dw3x3(ops[0]) && dw3x3(ops[3]) && ops[0].op.p[3] == 1 && ops[3].op.p[3] == 1) return AGO_KERNEL_DW_DW;
    }
    if (kinds_are(ops, {AGO_OP_CONV2D, AGO_OP_BIAS_ADD, AGO_OP_RELU6, AGO_OP_CONV2D, AGO_OP_BIAS_ADD}) && dw3x3(ops[0]) &&
        ops[3].pointwise())
      return AGO_KERNEL_DW_PW;
    // conv, bias, [ReLU6], conv, bias, [ReLU6] with two pointwise convolutions
    if (ops.size() >= 4 && ops.size() <= 6 && ops[0].pointwise() && ops[1].op.kind == AGO_OP_BIAS_ADD) {
      size_t i = 2;
      if (ops[i].op.kind == AGO_OP_RELU6) ++i;
      if (i + 1 < ops.size() && ops[i].pointwise() && ops[i + 1].op.kind == AGO_OP_BIAS_ADD &&
          (i + 2 == ops.size() || (i + 3 == ops.size() && ops[i + 2].op.kind == AGO_OP_RELU6)))
        return AGO_KERNEL_PW_PW;
    }
  }
  // GEMM -> [M, N1] viewed as [G, A, B, N1] -> + input -> swap (A, B) -> [M, N1] -> GEMM: between the two products
  // the rows are only permuted
  if (kinds_are(ops, {AGO_OP_GEMM, AGO_OP_RESHAPE, AGO_OP_ADD_INPUT, AGO_OP_RESHAPE, AGO_OP_TRANSPOSE, AGO_OP_RESHAPE,
                      AGO_OP_GEMM, AGO_OP_RESHAPE}) &&
      ops[0].in.rank == 2 && ops[3].out.rank == 4 && ops[4].op.p[0] + ops[4].op.p[1] == 3 && ops[5].out.rank == 2 &&
      ops[2].op.p[0] == 1)
    return AGO_KERNEL_GEMM_PERMUTE_GEMM;
  if (kinds_are(ops, {AGO_OP_GEMM, AGO_OP_BIAS_ADD, AGO_OP_GELU_TANH, AGO_OP_GEMM, AGO_OP_BIAS_ADD}))
    return AGO_KERNEL_FFN;
  if (kinds_are(ops, {AGO_OP_CONV2D, AGO_OP_BIAS_ADD, AGO_OP_RELU, AGO_OP_CONV2D, AGO_OP_BIAS_ADD,
                      AGO_OP_ADD_INPUT, AGO_OP_RELU}) &&
      conv3x3_s1p1(ops[0]) && conv3x3_s1p1(ops[3]) && ops[5].op.p[0] == 0)
    return AGO_KERNEL_CONV3X3_PAIR;
  if (kinds_are(ops, {AGO_OP_BATCHED_QKT, AGO_OP_SCALE, AGO_OP_SOFTMAX_ROWS, AGO_OP_BATCHED_PV}) &&
      ops[0].op.p[0] == 1 && ops[3].op.p[0] == 2)
    return AGO_KERNEL_ATTENTION;
  return AGO_KERNEL_NONE;
}

}  // namespace

ago_status_t build_plan(const ago_subgraph_desc_t* desc, Plan* plan, std::string* err) {
  if (!desc) { *err = "desc is NULL"; return AGO_ERR_INVALID_ARG; }
  if (desc->struct_size != sizeof(ago_subgraph_desc_t)) {
    *err = fmt("desc.struct_size is %lld, this library expects %lld", desc->struct_size, (long long)sizeof(ago_subgraph_desc_t));
    return AGO_ERR_INVALID_ARG;
  }
  if (desc->mode < AGO_MODE_FUSED || desc->mode > AGO_MODE_PER_OP) { *err = "unknown mode"; return AGO_ERR_INVALID_ARG; }
  if (desc->num_inputs < 1 || desc->num_inputs > AGO_MAX_INPUTS) { *err = "num_inputs must be 1..4"; return AGO_ERR_INVALID_ARG; }
  if (desc->num_ops < 1 || desc->num_ops > AGO_MAX_OPS || !desc->ops) { *err = "num_ops must be 1..32 and ops non-NULL"; return AGO_ERR_INVALID_ARG; }
  Plan& p = *plan;
  p.mode = desc->mode;
  p.num_inputs = desc->num_inputs;
  p.dtype = desc->input_dtype[0];
  if (p.dtype != AGO_BF16 && p.dtype != AGO_FP32) { *err = "unknown input dtype"; return AGO_ERR_INVALID_ARG; }
  if (desc->output_dtype != p.dtype) { *err = "output dtype must equal the input dtype"; return AGO_ERR_INVALID_ARG; }
  const int64_t vec = 16 / elem_bytes(p.dtype);
  for (int i = 0; i < desc->num_inputs; ++i) {
    if (desc->input_dtype[i] != p.dtype) { *err = "all inputs must share one dtype"; return AGO_ERR_INVALID_ARG; }
    int r = desc->input_rank[i];
    if (r < 2 || r > AGO_MAX_RANK) { *err = fmt("input %lld: rank must be 2..4", i); return AGO_ERR_SHAPE; }
    p.inputs[i].rank = r;
    for (int k = 0; k < r; ++k) {
      if (desc->input_shape[i][k] <= 0) { *err = fmt("input %lld: dimension %lld is not positive", i, k); return AGO_ERR_SHAPE; }
      p.inputs[i].d[k] = desc->input_shape[i][k];
    }
    if (p.inputs[i].last() % vec != 0) {
      *err = fmt("input %lld: innermost extent %lld is not a multiple of %lld (16-byte rows)", i, p.inputs[i].last(), vec);
      return AGO_ERR_SHAPE;
    }
  }

  Shape cur = p.inputs[0];
  int nw = 0;
  for (int i = 0; i < desc->num_ops; ++i) {
    OpInfo oi;
    oi.op = desc->ops[i];
    oi.in = cur;
    const int32_t* q = oi.op.p;
    switch (oi.op.kind) {
      case AGO_OP_CONV2D: {
        if (cur.rank != 4) { *err = fmt("op %lld (CONV2D): input must be NHWC rank 4", i); return AGO_ERR_SHAPE; }
        int64_t O = q[0], R = q[1], S = q[2], st = q[3], pad = q[4], g = q[5];
        int64_t C = cur.d[3];
        if (O <= 0 || R <= 0 || S <= 0 || st <= 0 || pad < 0) { *err = fmt("op %lld (CONV2D): bad O/R/S/stride/pad", i); return AGO_ERR_SHAPE; }
        if (!(g == 1 || (g == C && O == C))) { *err = fmt("op %lld (CONV2D): groups must be 1, or C with O == C (depthwise)", i); return AGO_ERR_SHAPE; }
        if (O % vec != 0) { *err = fmt("op %lld (CONV2D): O = %lld is not a multiple of %lld", i, O, vec); return AGO_ERR_SHAPE; }
        int64_t Ho = out_extent(cur.d[1], R, st, pad), Wo = out_extent(cur.d[2], S, st, pad);
        if (Ho <= 0 || Wo <= 0) { *err = fmt("op %lld (CONV2D): empty output", i); return AGO_ERR_SHAPE; }
        oi.weight = nw++;
        p.weight_bytes.push_back((g == 1 ? O * R * S * C : R * S * C) * elem_bytes(p.dtype));
        cur.d[1] = Ho; cur.d[2] = Wo; cur.d[3] = O;
        int64_t macs = cur.d[0] * Ho * Wo * O * R * S * (g == 1 ? C : 1);
        if (g == 1) p.flops_tensor += 2 * macs; else p.flops_cuda += 2 * macs;
        break;
      }
      case AGO_OP_GEMM: {
        int64_t N = q[0], K = cur.last();
        if (N <= 0 || N % vec != 0) { *err = fmt("op %lld (GEMM): N = %lld must be a positive multiple of %lld", i, N, vec); return AGO_ERR_SHAPE; }
        oi.weight = nw++;
        p.weight_bytes.push_back(K * N * elem_bytes(p.dtype));
        p.flops_tensor += 2 * (cur.numel() / K) * K * N;
        cur.d[cur.rank - 1] = N;
        break;
      }
      case AGO_OP_BATCHED_QKT: {
        int idx = q[0]; int64_t heads = q[1], hd = q[2];
        if (cur.rank != 3) { *err = fmt("op %lld (BATCHED_QKT): input must be [B,S,E]", i); return AGO_ERR_SHAPE; }
        if (idx < 0 || idx >= p.num_inputs || !(p.inputs[idx] == cur)) { *err = fmt("op %lld (BATCHED_QKT): K input index/shape mismatch", i); return AGO_ERR_SHAPE; }
        if (heads <= 0 || hd <= 0 || heads * hd != cur.d[2] || hd % vec != 0) { *err = fmt("op %lld (BATCHED_QKT): heads*head_dim must equal E", i); return AGO_ERR_SHAPE; }
        if (cur.d[1] % vec != 0) { *err = fmt("op %lld (BATCHED_QKT): S must be a multiple of %lld", i, vec); return AGO_ERR_SHAPE; }
        int64_t B = cur.d[0], S = cur.d[1];
        p.flops_tensor += 2 * B * heads * S * S * hd;
        cur.rank = 4; cur.d[0] = B; cur.d[1] = heads; cur.d[2] = S; cur.d[3] = S;
        break;
      }
      case AGO_OP_BATCHED_PV: {
        int idx = q[0]; int64_t heads = q[1], hd = q[2];
        if (cur.rank != 4 || cur.d[2] != cur.d[3] || cur.d[1] != heads) { *err = fmt("op %lld (BATCHED_PV): input must be [B,heads,S,S]", i); return AGO_ERR_SHAPE; }
        if (idx < 0 || idx >= p.num_inputs || p.inputs[idx].rank != 3 || p.inputs[idx].d[0] != cur.d[0] ||
            p.inputs[idx].d[1] != cur.d[2] || p.inputs[idx].d[2] != heads * hd || hd <= 0 || hd % vec != 0) {
          *err = fmt("op %lld (BATCHED_PV): V input index/shape mismatch", i); return AGO_ERR_SHAPE;
        }
        int64_t B = cur.d[0], S = cur.d[2];
        p.flops_tensor += 2 * B * heads * S * S * hd;
        cur.rank = 3; cur.d[0] = B; cur.d[1] = S; cur.d[2] = heads * hd; cur.d[3] = 0;
        break;
      }
      case AGO_OP_RESHAPE: {
        const int r = q[0];
        if (r < 2 || r > AGO_MAX_RANK) { *err = fmt("op %lld (RESHAPE): rank must be 2..4", i); return AGO_ERR_SHAPE; }
        Shape nsh; nsh.rank = r;
        for (int k = 0; k < r; ++k) nsh.d[k] = q[1 + k];
        for (int k = 0; k < r; ++k)
          if (nsh.d[k] <= 0) { *err = fmt("op %lld (RESHAPE): dimension %lld must be positive", i, k); return AGO_ERR_SHAPE; }
        if (nsh.numel() != cur.numel() || nsh.last() != cur.last()) {
          *err = fmt("op %lld (RESHAPE): the new shape must keep the element count and the last dimension", i);
          return AGO_ERR_SHAPE;
        }
        if (i == 0) { *err = "op 0 (RESHAPE): a reshape must follow an operator"; return AGO_ERR_UNSUPPORTED; }
        cur = nsh;
        break;
      }
      case AGO_OP_TRANSPOSE: {
        const int a = q[0], b = q[1];
        if (a < 0 || b < 0 || a == b || a >= cur.rank - 1 || b >= cur.rank - 1) {
          *err = fmt("op %lld (TRANSPOSE): two different axes below the last one are required", i);
          return AGO_ERR_SHAPE;
        }
        std::swap(cur.d[a], cur.d[b]);
        break;
      }
      case AGO_OP_BIAS_ADD:
        oi.weight = nw++;
        p.weight_bytes.push_back(cur.last() * 4);
        break;
      case AGO_OP_RELU: case AGO_OP_RELU6: case AGO_OP_SCALE:
        break;
      case AGO_OP_GELU_TANH: case AGO_OP_SOFTMAX_ROWS:
        p.sfu_ops += cur.numel();
        break;
      case AGO_OP_ADD_INPUT: {
        int idx = q[0];
        if (idx < 0 || idx >= p.num_inputs || !(p.inputs[idx] == cur)) { *err = fmt("op %lld (ADD_INPUT): input index/shape mismatch", i); return AGO_ERR_SHAPE; }
        break;
      }
      default:
        *err = fmt("op %lld: unknown operator kind %lld", i, oi.op.kind);
        return AGO_ERR_INVALID_ARG;
    }
    oi.out = cur;
    p.ops.push_back(oi);
  }
  p.output = cur;

  if (p.dtype == AGO_FP32) {
    for (auto& o : p.ops)
      if (o.complex_op() && !o.depthwise()) { *err = "FP32 I/O is supported for depthwise-only subgraphs"; return AGO_ERR_UNSUPPORTED; }
  }

  // Link categories between consecutive complex operators.
  int prev_complex = -1;
  for (size_t i = 0; i < p.ops.size(); ++i) {
    if (!p.ops[i].complex_op()) continue;
    if (prev_complex >= 0) p.link_category.push_back(classify_link(p.ops[i]));
    prev_complex = (int)i;
  }

  // Launch list of the unfused modes.
  if (p.mode == AGO_MODE_PER_OP) {
    for (int i = 0; i < (int)p.ops.size(); ++i) {
      if (p.ops[i].op.kind == AGO_OP_RESHAPE && !p.stages.empty()) { p.stages.back().last = i; continue; }   // a view
      Stage s; s.first = s.last = i;
      s.complex_index = p.ops[i].complex_op() ? i : -1;
      s.softmax = p.ops[i].op.kind == AGO_OP_SOFTMAX_ROWS;
      s.transpose = p.ops[i].op.kind == AGO_OP_TRANSPOSE;
      p.stages.push_back(s);
    }
  } else {
    // Mini-subgraphs: a complex operator plus the element-wise operators that
    // follow it (Section III-A). A row softmax needs whole rows, so it is a
    // launch of its own; a run of EPI programs longer than kMaxEpi is split.
    int i = 0, n = (int)p.ops.size();
    while (i < n) {
      Stage s; s.first = i;
      if (p.ops[i].op.kind == AGO_OP_SOFTMAX_ROWS || p.ops[i].op.kind == AGO_OP_TRANSPOSE) {
        s.softmax = p.ops[i].op.kind == AGO_OP_SOFTMAX_ROWS; s.transpose = !s.softmax;
        s.last = i; ++i;
        while (i < n && p.ops[i].op.kind == AGO_OP_RESHAPE) s.last = i++;   // views of its result
        p.stages.push_back(s);
        continue;
      }
      if (p.ops[i].complex_op()) s.complex_index = i;
      int j = i + 1, cnt = p.ops[i].complex_op() ? 0 : 1;
      while (j < n && is_simple_elementwise(p.ops[j].op.kind) && cnt < kMaxEpi) { ++j; ++cnt; }
      s.last = j - 1;
      p.stages.push_back(s);
      i = j;
    }
  }
  for (size_t s = 0; s + 1 < p.stages.size(); ++s) {
    int64_t b = p.ops[p.stages[s].last].out.numel() * elem_bytes(p.dtype);
    if (b > p.max_intermediate_bytes) p.max_intermediate_bytes = b;
  }
  // Intermediate traffic of the per-mini-subgraph mode (write + read), a mode-independent figure.
  {
    int n = (int)p.ops.size();
    for (int i = 0; i + 1 < n; ++i) {
      // launch boundaries of that mode; views on either side of a boundary do not move it
      int nx = i + 1;
      while (nx < n && p.ops[nx].op.kind == AGO_OP_RESHAPE) ++nx;
      if (nx >= n || p.ops[i].op.kind == AGO_OP_RESHAPE) continue;
      const int kn = p.ops[nx].op.kind, ki = p.ops[i].op.kind;
      bool boundary = p.ops[nx].complex_op() || kn == AGO_OP_SOFTMAX_ROWS || kn == AGO_OP_TRANSPOSE ||
                      ki == AGO_OP_SOFTMAX_ROWS || ki == AGO_OP_TRANSPOSE;
      if (boundary) p.intermediate_bytes += 2 * p.ops[i].out.numel() * elem_bytes(p.dtype);
    }
  }

  p.io_bytes = p.output.numel() * elem_bytes(p.dtype);
  for (int i = 0; i < p.num_inputs; ++i) p.io_bytes += p.inputs[i].numel() * elem_bytes(p.dtype);
  for (int64_t b : p.weight_bytes) p.io_bytes += b;

  p.fused_kernel = AGO_KERNEL_NONE;
  p.num_launches = (int)p.stages.size();
  if (p.mode == AGO_MODE_FUSED) {
    p.fused_kernel = match_fused_family(p);
    if (p.fused_kernel == AGO_KERNEL_NONE) {
      *err = "fused mode: the operator chain matches no fused kernel family (depthwise-only; 1x1 -> depthwise 3x3 -> 1x1 "
             "and its pairs; GEMM -> GELU -> GEMM; conv3x3 -> conv3x3 + input -> ReLU; QK^T -> scale -> softmax -> PV; "
             "GEMM -> + input -> row transpose -> GEMM)";
      return AGO_ERR_UNSUPPORTED;
    }
    p.num_launches = 1;
  }
  return AGO_OK;
}

}  // namespace ago
