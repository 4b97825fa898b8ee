// Fused pair of pointwise convolutions: 1x1 conv + bias [+ ReLU6] -> 1x1 conv + bias [+ ReLU6], one kernel
// (the "two pointwise convolutions" subgraph of the micro-benchmark, Section VI-B; in MobileNetV2-like networks
// the linear bottleneck of one block followed by the expansion of the next).
//
// Both operators are matrix multiplications over the pixel rows, so the link is the "downstream pointwise"
// category of Section III-B: the downstream tile keeps all its output channels and is tiled over rows, the upstream
// tile it needs is the same rows with all middle channels -- nothing is recomputed. Per CTA (128 pixel rows):
//   P1  asynchronous 16-byte copies: the X tile and both weight matrices -> K-major operands without swizzle
//       (planes of [row][8 channels], one plane per 8 reduction channels); rows past the tensor and the padding
//       of the channel counts to MMA granularity are zero-filled
//   P2  tcgen05.mma: mid[128 x C1] = X[128 x C0] * W1^T                         (TMEM, fp32)
//   P3  TMEM -> registers: + b1 [ReLU6], bf16 -> shared memory as the A operand of the second product
//   P4  tcgen05.mma: out[128 x C2] = mid[128 x C1] * W2^T                       (TMEM, same columns)
//   P5  TMEM -> registers: + b2 [ReLU6], bf16 -> staging tile (over the dead X tile) -> coalesced 16-byte stores;
//       the 128 output rows are one contiguous range of the NHWC tensor.
// Two CTAs share an SM (tensor memory: 256 columns each), so one CTA's copies overlap the other's epilogues.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>

#include "fused.h"
#include "tc_common.cuh"

namespace ago {

namespace {

using namespace tc;

constexpr int kThreads = 256;
constexpr int kBM = 128;

struct PwPwParams {
  const __nv_bfloat16* x;    // [M][C0]
  const __nv_bfloat16* w1;   // [C1][C0]
  const float* b1;
  const __nv_bfloat16* w2;   // [C2][C1]
  const float* b2;
  __nv_bfloat16* out;        // [M][C2]
  unsigned int* status;
  int M, C0, C1, C2;
  int C0p, C1p, C2p;         // padded to the MMA granularity (16)
  int act1, act2;            // ReLU6 after the first / second convolution
  uint32_t k0_recip, k0p_recip, k1p_recip, k2_recip;   // reciprocals of the 16-byte pieces per row: C0/8, C0p/8, C1p/8, C2/8
  int x_plane, a_plane, w1_plane, w2_plane, pitch;     // byte strides of the operand planes; row pitch of the staging tile
  int tmem_cols;
  int off_x, off_a, off_w1, off_w2, off_b, off_bar;
};

__device__ __forceinline__ float relu6f(float v) { return fminf(fmaxf(v, 0.0f), 6.0f); }

__global__ void __launch_bounds__(kThreads)
pwpw_fused_kernel(const PwPwParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  float* sB1 = reinterpret_cast<float*>(smem + p.off_b);
  float* sB2 = sB1 + p.C1p;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);   // [0] first product complete, [1] second
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 3);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int row0 = blockIdx.x * kBM;
  const int rows = min(kBM, p.M - row0);
  const uint32_t sx = smem_u32(smem + p.off_x), sa = smem_u32(smem + p.off_a);
  const uint32_t sw1 = smem_u32(smem + p.off_w1), sw2 = smem_u32(smem + p.off_w2);

  if (tid == 0) {
    *abort_flag = 0u;
    mbar_init(bars, 1);
    mbar_init(bars + 1, 1);
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  grid_dependency_wait();
  grid_launch_dependents();
  // ---- P1: operands -> planes. Consecutive threads take consecutive 16-byte pieces of a row in device memory. ----
  {
    const int k0 = p.C0 >> 3, k0p = p.C0p >> 3, k1 = p.C1 >> 3, k1p = p.C1p >> 3;
    const uint8_t* x0 = reinterpret_cast<const uint8_t*>(p.x) + (int64_t)row0 * p.C0 * 2;
    for (int i = tid; i < kBM * k0; i += kThreads) {
      const int r = (int)fast_div((uint32_t)i, (uint32_t)k0, p.k0_recip), k = i - r * k0;
      const bool in = r < rows;
      cp_async_16(sx + (uint32_t)(k * p.x_plane + r * 16), in ? x0 + (int64_t)r * p.C0 * 2 + k * 16 : reinterpret_cast<const uint8_t*>(p.x), in ? 16u : 0u);
    }
    if (k0p > k0)   // the half-empty last reduction step
      for (int r = tid; r < kBM; r += kThreads) *reinterpret_cast<uint4*>(smem + p.off_x + k0 * p.x_plane + r * 16) = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < p.C1p * k0p; i += kThreads) {
      const int r = (int)fast_div((uint32_t)i, (uint32_t)k0p, p.k0p_recip), k = i - r * k0p;
      const bool in = r < p.C1 && k < k0;
      cp_async_16(sw1 + (uint32_t)(k * p.w1_plane + r * 16), in ? reinterpret_cast<const uint8_t*>(p.w1) + ((int64_t)r * p.C0 + k * 8) * 2 : reinterpret_cast<const uint8_t*>(p.x), in ? 16u : 0u);
    }
    for (int i = tid; i < p.C2p * k1p; i += kThreads) {
      const int r = (int)fast_div((uint32_t)i, (uint32_t)k1p, p.k1p_recip), k = i - r * k1p;
      const bool in = r < p.C2 && k < k1;
      cp_async_16(sw2 + (uint32_t)(k * p.w2_plane + r * 16), in ? reinterpret_cast<const uint8_t*>(p.w2) + ((int64_t)r * p.C1 + k * 8) * 2 : reinterpret_cast<const uint8_t*>(p.x), in ? 16u : 0u);
    }
    cp_async_commit();
    for (int i = tid; i < p.C1p + p.C2p; i += kThreads)
      sB1[i] = i < p.C1p ? (i < p.C1 ? __ldg(p.b1 + i) : 0.0f) : (i - p.C1p < p.C2 ? __ldg(p.b2 + i - p.C1p) : 0.0f);
    cp_async_wait_all();
    fence_proxy_async_smem();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
  const int half = warp >> 2;             // warps 0-3 and 4-7 share the 16-column groups of an epilogue alternately
  const int r = (warp & 3) * 32 + lane;   // this thread's row of the tile = its tensor-memory lane

  // ---- P2: first product ----
  if (tid == 0) {
    const uint32_t idesc = make_idesc_bf16(128, (uint32_t)p.C1p);
    const uint64_t ad = make_smem_desc(sx, (uint32_t)p.x_plane, 128, SW_NONE);
    const uint64_t bd = make_smem_desc(sw1, (uint32_t)p.w1_plane, 128, SW_NONE);
    for (int ks = 0; ks < p.C0p / 16; ++ks)
      umma_bf16(tmem_base, ad + (uint64_t)((uint32_t)(2 * ks * p.x_plane) >> 4), bd + (uint64_t)((uint32_t)(2 * ks * p.w1_plane) >> 4), idesc, ks > 0);
    umma_commit(bars);
  }
  __syncwarp();
  mbar_wait(bars, 0, abort_flag, p.status, 0x601);
  tcgen05_fence_after_sync();
  // ---- P3: + b1 [ReLU6] -> A operand of the second product (thread = row: conflict-free 16-byte stores) ----
  for (int g = half; g < p.C1p / 16; g += 2) {
    uint32_t v[16];
    tmem_ld_x16(tmem_base + lane_base + g * 16, v);
    tmem_ld_wait();
    uint32_t w[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float y0 = __uint_as_float(v[2 * j]) + sB1[g * 16 + 2 * j], y1 = __uint_as_float(v[2 * j + 1]) + sB1[g * 16 + 2 * j + 1];
      if (p.act1) { y0 = relu6f(y0); y1 = relu6f(y1); }
      w[j] = pack_bf16x2(y0, y1);
    }
    *reinterpret_cast<uint4*>(smem + p.off_a + (2 * g) * p.a_plane + r * 16) = make_uint4(w[0], w[1], w[2], w[3]);
    *reinterpret_cast<uint4*>(smem + p.off_a + (2 * g + 1) * p.a_plane + r * 16) = make_uint4(w[4], w[5], w[6], w[7]);
  }
  fence_proxy_async_smem();
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  // ---- P4: second product, over the drained columns of the first ----
  if (tid == 0) {
    const uint32_t idesc = make_idesc_bf16(128, (uint32_t)p.C2p);
    const uint64_t ad = make_smem_desc(sa, (uint32_t)p.a_plane, 128, SW_NONE);
    const uint64_t bd = make_smem_desc(sw2, (uint32_t)p.w2_plane, 128, SW_NONE);
    for (int ks = 0; ks < p.C1p / 16; ++ks)
      umma_bf16(tmem_base, ad + (uint64_t)((uint32_t)(2 * ks * p.a_plane) >> 4), bd + (uint64_t)((uint32_t)(2 * ks * p.w2_plane) >> 4), idesc, ks > 0);
    umma_commit(bars + 1);
  }
  __syncwarp();
  mbar_wait(bars + 1, 0, abort_flag, p.status, 0x602);
  tcgen05_fence_after_sync();
  // ---- P5: + b2 [ReLU6] -> staging tile over the X tile (both products have read it) -> device memory ----
  uint8_t* stage = smem + p.off_x;
  for (int g = half; g < p.C2p / 16; g += 2) {
    uint32_t v[16];
    tmem_ld_x16(tmem_base + lane_base + g * 16, v);
    tmem_ld_wait();
    uint32_t w[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float y0 = __uint_as_float(v[2 * j]) + sB2[g * 16 + 2 * j], y1 = __uint_as_float(v[2 * j + 1]) + sB2[g * 16 + 2 * j + 1];
      if (p.act2) { y0 = relu6f(y0); y1 = relu6f(y1); }
      w[j] = pack_bf16x2(y0, y1);
    }
    uint8_t* dst = stage + r * p.pitch + g * 32;
    *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
    if (g * 16 + 8 < p.C2) *reinterpret_cast<uint4*>(dst + 16) = make_uint4(w[4], w[5], w[6], w[7]);
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  {
    const int k2 = p.C2 >> 3;
    uint4* o0 = reinterpret_cast<uint4*>(p.out + (int64_t)row0 * p.C2);   // the tile's rows are contiguous
    for (int i = tid; i < rows * k2; i += kThreads) {
      const int rr = (int)fast_div((uint32_t)i, (uint32_t)k2, p.k2_recip), k = i - rr * k2;
      o0[i] = *reinterpret_cast<const uint4*>(stage + rr * p.pitch + k * 16);
    }
  }
  if (warp == 1) tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
}

int round_up(int v, int m) { return (v + m - 1) / m * m; }

struct PwPwHost {
  PwPwParams prm;
  int smem_bytes = 0;
};

}  // namespace

ago_status_t pwpw_plan(Plan* plan, FusedState* st, std::string* err) {
  // conv, bias, [relu6], conv, bias, [relu6]
  const auto& ops = plan->ops;
  int i2 = 2;
  auto* host = new PwPwHost();
  PwPwParams& q = host->prm;
  q = PwPwParams{};
  if (ops[2].op.kind == AGO_OP_RELU6) { q.act1 = 1; i2 = 3; }
  q.act2 = (int)ops.size() > i2 + 2 ? 1 : 0;
  const OpInfo& a = ops[0];
  q.C0 = (int)a.in.d[3];
  q.M = (int)(a.in.numel() / q.C0);
  q.C1 = a.op.p[0];
  q.C2 = ops[i2].op.p[0];
  auto bad = [&](const char* m) { *err = std::string("fused pointwise pair: ") + m; delete host; return AGO_ERR_UNSUPPORTED; };
  if (q.C0 % 8 || q.C1 % 8 || q.C2 % 8) return bad("channel counts must be multiples of 8");
  q.C0p = round_up(q.C0, 16); q.C1p = round_up(q.C1, 16); q.C2p = round_up(q.C2, 16);
  if (q.C1p > 256 || q.C2p > 256) return bad("more than 256 middle or output channels is not supported");
  if (q.C0p > 1024) return bad("more than 1024 input channels is not supported");
  q.k0_recip = fast_div_recip(q.C0 / 8); q.k0p_recip = fast_div_recip(q.C0p / 8);
  q.k1p_recip = fast_div_recip(q.C1p / 8); q.k2_recip = fast_div_recip(q.C2 / 8);
  // planes are padded by one 16-byte entry so that the pieces of one row (consecutive planes) fall into different banks
  q.x_plane = kBM * 16 + 16;
  q.a_plane = kBM * 16;
  q.w1_plane = q.C1p * 16 + 16;
  q.w2_plane = q.C2p * 16 + 16;
  q.pitch = q.C2 * 2 + 16;
  q.tmem_cols = 32;
  while (q.tmem_cols < std::max(q.C1p, q.C2p)) q.tmem_cols *= 2;
  int off = 0;
  auto take = [&](int bytes) { int o = off; off = round_up(off + bytes, 128); return o; };
  q.off_x = take(std::max(q.C0p / 8 * q.x_plane, kBM * q.pitch));
  q.off_a = take(q.C1p / 8 * q.a_plane);
  q.off_w1 = take(q.C0p / 8 * q.w1_plane);
  q.off_w2 = take(q.C1p / 8 * q.w2_plane);
  q.off_b = take((q.C1p + q.C2p) * 4);
  q.off_bar = take(64);
  host->smem_bytes = off + 128;
  if (host->smem_bytes > 227 * 1024) return bad("the operands of one row tile do not fit shared memory");
  if ((long)kBM * (q.C0 / 8) > 65535 || (long)q.C1p * (q.C0p / 8) > 65535 || (long)q.C2p * (q.C1p / 8) > 65535)
    return bad("operand too large for the copy index arithmetic");
  st->impl = host;
  st->impl_free = [](void* p) { delete static_cast<PwPwHost*>(p); };
  st->tile_rows = kBM; st->grid = (q.M + kBM - 1) / kBM; st->smem_bytes = host->smem_bytes;
  plan->tile_rows = kBM; plan->smem_bytes = host->smem_bytes;
  return AGO_OK;
}

ago_status_t pwpw_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                      void* output, unsigned int* status_word, cudaStream_t stream, std::string* err) {
  (void)plan;
  PwPwHost* host = static_cast<PwPwHost*>(st->impl);
  PwPwParams q = host->prm;
  q.x = static_cast<const __nv_bfloat16*>(inputs[0]);
  q.w1 = static_cast<const __nv_bfloat16*>(weights[0]); q.b1 = static_cast<const float*>(weights[1]);
  q.w2 = static_cast<const __nv_bfloat16*>(weights[2]); q.b2 = static_cast<const float*>(weights[3]);
  q.out = static_cast<__nv_bfloat16*>(output);
  q.status = status_word;
  {
    static int smem_opt_in[64] = {};
    cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(pwpw_fused_kernel), smem_opt_in);
    if (e != cudaSuccess) { *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  }
  FusedLaunch launch(dim3((unsigned)((q.M + kBM - 1) / kBM)), kThreads, (size_t)host->smem_bytes, stream);
  cudaError_t e = cudaLaunchKernelEx(&launch.config, pwpw_fused_kernel, q);
  if (e != cudaSuccess) { *err = std::string("fused pointwise pair launch: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  return AGO_OK;
}

}  // namespace ago
