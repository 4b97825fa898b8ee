// Fused pair of pointwise convolutions: 1x1 conv + bias [+ ReLU6] -> 1x1 conv + bias [+ ReLU6], one kernel
// (the "two pointwise convolutions" subgraph of the micro-benchmark, Section VI-B; in MobileNetV2-like networks
// the linear bottleneck of one block followed by the expansion of the next).
//
// Both operators are matrix multiplications over the pixel rows, so the link is the "downstream pointwise"
// category of Section III-B: the downstream tile keeps all its output channels and is tiled over rows, the upstream
// tile it needs is the same rows with all middle channels -- nothing is recomputed. CTAs are persistent (two per SM,
// out of phase: one copies while the other computes) and walk over tiles of 128 pixel rows. Per tile:
//   P1  TMA: the X tile as K-major blocks of 64 channels (128-byte swizzle); rows past the tensor and channels past
//       C0 read as zero. Both weight matrices are fetched once per CTA into the same layout with plain loads.
//   P2  tcgen05.mma: mid[128 x C1] = X[128 x C0] * W1^T                         (TMEM, fp32)
//   P3  TMEM -> registers: + b1 [ReLU6], bf16 -> shared memory as the swizzled A operand of the second product
//   P4  tcgen05.mma: out[128 x C2] = mid[128 x C1] * W2^T                       (TMEM, same columns)
//   P5  TMEM -> registers: + b2 [ReLU6], bf16 -> staging tile (over the dead X tile) -> coalesced 16-byte stores;
//       the 128 output rows are one contiguous range of the NHWC tensor. The next X tile is requested as soon as
//       the staging tile has been read.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <unordered_map>

#include "fused.h"
#include "tc_common.cuh"
#include "tmap.h"

namespace ago {

namespace {

using namespace tc;

constexpr int kThreads = 256;
constexpr int kBM = 128, kBK = 64;
constexpr int kXBlock = kBM * kBK * 2;   // one K block of the X / mid tile: 16 KB

struct PwPwParams {
  const __nv_bfloat16* w1;   // [C1][C0]
  const __nv_bfloat16* w2;   // [C2][C1]
  const float* b1;
  const float* b2;
  __nv_bfloat16* out;        // [M][C2]
  unsigned int* status;
  int M, C0, C1, C2;
  int C0p, C1p, C2p;         // padded to the MMA granularity (16)
  int nkb0, nkb1;            // 64-channel K blocks of the first / second product
  int act1, act2;            // ReLU6 after the first / second convolution
  uint32_t k2_recip;         // reciprocal of the 16-byte pieces per output row (C2 / 8)
  uint32_t c0_recip, c1_recip;   // ... per padded weight row (C0p / 8, C1p / 8)
  int pitch;                 // row pitch of the staging tile
  int x_tx;                  // bytes one X tile brings in (TMA transaction count)
  int tmem_cols;
  int off_x, off_a, off_w1, off_w2, off_b, off_bar;
};

__device__ __forceinline__ float relu6f(float v) { return fminf(fmaxf(v, 0.0f), 6.0f); }

__global__ void __launch_bounds__(kThreads)
pwpw_fused_kernel(const __grid_constant__ CUtensorMap tmap_x, const PwPwParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sX = smem + p.off_x;
  uint8_t* sA = smem + p.off_a;
  uint8_t* sW1 = smem + p.off_w1;
  uint8_t* sW2 = smem + p.off_w2;
  float* sB1 = reinterpret_cast<float*>(smem + p.off_b);
  float* sB2 = sB1 + p.C1p;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
  uint64_t* bar_x = bars;        // X tile landed
  uint64_t* bar_m1 = bars + 2;   // first product complete
  uint64_t* bar_m2 = bars + 3;   // second product complete
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 5);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int k2 = p.C2 >> 3;
  const int ntiles = (p.M + kBM - 1) / kBM;

  if (tid == 0) {
    *abort_flag = 0u;
    for (int i = 0; i < 4; ++i) mbar_init(bars + i, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmap_x);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  auto load_x = [&](int tile) {   // one thread
    mbar_arrive_expect_tx(bar_x, (uint32_t)p.x_tx);
    for (int kb = 0; kb < p.nkb0; ++kb) tma_load_2d(sX + kb * kXBlock, &tmap_x, bar_x, kb * kBK, tile * kBM);
  };
  grid_dependency_wait();
  grid_launch_dependents();
  if (tid == 0 && (int)blockIdx.x < ntiles) load_x(blockIdx.x);
  // Weights: every CTA of the grid reads the same few kilobytes at the same time, so they are fetched with a few
  // wide coalesced requests per warp (16 bytes per thread, all loads of a batch in flight before its first store)
  // instead of one TMA request per matrix row, and written to the swizzled K-major blocks by hand; rows and
  // reduction channels added by the padding are zero.
  {
    constexpr int kBatch = 4;
    const int c0 = p.C0p >> 3, c1 = p.C1p >> 3;              // 16-byte chunks per padded row
    const int n1 = p.C1p * c0, nw = n1 + p.C2p * c1;
    for (int base = tid; base < nw; base += kBatch * kThreads) {
      uint4 v[kBatch];
      uint32_t dst[kBatch];
#pragma unroll
      for (int k = 0; k < kBatch; ++k) {
        const int i = base + k * kThreads;
        v[k] = make_uint4(0, 0, 0, 0);
        dst[k] = 0xffffffffu;
        if (i < nw) {
          const bool first = i < n1;
          const int j = first ? i : i - n1;
          const int cpr = first ? c0 : c1;
          const int row = (int)fast_div((uint32_t)j, (uint32_t)cpr, first ? p.c0_recip : p.c1_recip), ch = j - row * cpr;
          const int K = first ? p.C0 : p.C1, R = first ? p.C1 : p.C2, Rp = first ? p.C1p : p.C2p;
          dst[k] = (uint32_t)((first ? p.off_w1 : p.off_w2) + (ch >> 3) * Rp * 128) + swz_offset((uint32_t)row, (uint32_t)(ch & 7), 128);
          if (row < R && ch * 8 < K)
            v[k] = __ldg(reinterpret_cast<const uint4*>((first ? p.w1 : p.w2) + (int64_t)row * K + ch * 8));
        }
      }
#pragma unroll
      for (int k = 0; k < kBatch; ++k)
        if (dst[k] != 0xffffffffu) *reinterpret_cast<uint4*>(smem + dst[k]) = v[k];
    }
  }
  for (int i = tid; i < p.C1p + p.C2p; i += kThreads)
    sB1[i] = i < p.C1p ? (i < p.C1 ? __ldg(p.b1 + i) : 0.0f) : (i - p.C1p < p.C2 ? __ldg(p.b2 + i - p.C1p) : 0.0f);
  fence_proxy_async_smem();
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
  const int half = warp >> 2;             // warps 0-3 and 4-7 share the 16-column groups of an epilogue alternately
  const int r = (warp & 3) * 32 + lane;   // this thread's row of the tile = its tensor-memory lane
  const uint32_t idesc1 = make_idesc_bf16(128, (uint32_t)p.C1p), idesc2 = make_idesc_bf16(128, (uint32_t)p.C2p);

  for (int tile = blockIdx.x, it = 0; tile < ntiles; tile += gridDim.x, ++it) {
    const uint32_t par = (uint32_t)it & 1u;
    const int row0 = tile * kBM, rows = min(kBM, p.M - row0);
    // ---- P2: first product ----
    if (tid == 0) {
      mbar_wait(bar_x, par, abort_flag, p.status, 0x600);
      tcgen05_fence_after_sync();
      for (int kb = 0; kb < p.nkb0; ++kb) {
        const uint64_t ad = make_smem_desc(smem_u32(sX + kb * kXBlock), 0, 1024, SW_128B);
        const uint64_t bd = make_smem_desc(smem_u32(sW1 + kb * p.C1p * 128), 0, 1024, SW_128B);
        const int ksteps = min(4, (p.C0p - kb * kBK) / 16);
        for (int ks = 0; ks < ksteps; ++ks) umma_bf16(tmem_base, ad + 2u * ks, bd + 2u * ks, idesc1, (kb | ks) != 0);
      }
      umma_commit(bar_m1);
    }
    __syncwarp();
    mbar_wait(bar_m1, par, abort_flag, p.status, 0x601);
    tcgen05_fence_after_sync();
    // ---- P3: + b1 [ReLU6] -> swizzled A operand of the second product ----
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
      uint8_t* blk = sA + (g >> 2) * kXBlock;              // 64 channels per block = 4 groups = 8 chunks of 16 bytes
      const uint32_t ch = (uint32_t)(g & 3) * 2u;
      *reinterpret_cast<uint4*>(blk + swz_offset((uint32_t)r, ch, 128)) = make_uint4(w[0], w[1], w[2], w[3]);
      *reinterpret_cast<uint4*>(blk + swz_offset((uint32_t)r, ch + 1u, 128)) = make_uint4(w[4], w[5], w[6], w[7]);
    }
    fence_proxy_async_smem();
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    // ---- P4: second product, over the drained columns of the first ----
    if (tid == 0) {
      for (int kb = 0; kb < p.nkb1; ++kb) {
        const uint64_t ad = make_smem_desc(smem_u32(sA + kb * kXBlock), 0, 1024, SW_128B);
        const uint64_t bd = make_smem_desc(smem_u32(sW2 + kb * p.C2p * 128), 0, 1024, SW_128B);
        const int ksteps = min(4, (p.C1p - kb * kBK) / 16);
        for (int ks = 0; ks < ksteps; ++ks) umma_bf16(tmem_base, ad + 2u * ks, bd + 2u * ks, idesc2, (kb | ks) != 0);
      }
      umma_commit(bar_m2);
    }
    __syncwarp();
    mbar_wait(bar_m2, par, abort_flag, p.status, 0x602);
    tcgen05_fence_after_sync();
    // ---- P5: + b2 [ReLU6] -> staging tile over the X tile (the first product has read it) -> device memory ----
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
      uint8_t* dst = sX + r * p.pitch + g * 32;
      *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
      if (g * 16 + 8 < p.C2) *reinterpret_cast<uint4*>(dst + 16) = make_uint4(w[4], w[5], w[6], w[7]);
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    {
      uint4* o0 = reinterpret_cast<uint4*>(p.out + (int64_t)row0 * p.C2);   // the tile's rows are contiguous
      for (int i = tid; i < rows * k2; i += kThreads) {
        const int rr = (int)fast_div((uint32_t)i, (uint32_t)k2, p.k2_recip), k = i - rr * k2;
        o0[i] = *reinterpret_cast<const uint4*>(sX + rr * p.pitch + k * 16);
      }
    }
    __syncthreads();   // the staging tile has been read: its buffer takes the next X tile
    tcgen05_fence_after_sync();
    if (tid == 0 && tile + (int)gridDim.x < ntiles) {
      fence_proxy_async_smem();
      load_x(tile + gridDim.x);
    }
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
}

int round_up(int v, int m) { return (v + m - 1) / m * m; }

struct PwPwHost {
  PwPwParams prm;
  int smem_bytes = 0;
  int grid = 0;   // persistent CTAs: two per SM
  std::unordered_map<const void*, CUtensorMap> maps;   // X tensor maps by base address
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
  q.nkb0 = (q.C0 + kBK - 1) / kBK; q.nkb1 = (q.C1p + kBK - 1) / kBK;
  q.k2_recip = fast_div_recip(q.C2 / 8);
  q.c0_recip = fast_div_recip(q.C0p / 8); q.c1_recip = fast_div_recip(q.C1p / 8);
  q.pitch = q.C2 * 2 + 16;
  q.x_tx = q.nkb0 * kXBlock;
  q.tmem_cols = 32;
  while (q.tmem_cols < std::max(q.C1p, q.C2p)) q.tmem_cols *= 2;
  int off = 0;
  auto take = [&](int bytes) { int o = off; off = round_up(off + bytes, 1024); return o; };
  q.off_x = take(std::max(q.nkb0 * kXBlock, kBM * q.pitch));
  q.off_a = take(q.nkb1 * kXBlock);
  q.off_w1 = take(q.nkb0 * q.C1p * 128);
  q.off_w2 = take(q.nkb1 * q.C2p * 128);
  q.off_b = take((q.C1p + q.C2p) * 4);
  q.off_bar = take(64);
  host->smem_bytes = off + 1024;
  if (host->smem_bytes > 227 * 1024) return bad("the operands of one row tile do not fit shared memory");
  if ((long)kBM * (q.C2 / 8) > 65535 || (long)q.C1p * (q.C0p / 8) > 65535 || (long)q.C2p * (q.C1p / 8) > 65535)
    return bad("operands too large for the copy index arithmetic");
  host->grid = std::min((q.M + kBM - 1) / kBM, 2 * 148);
  st->impl = host;
  st->impl_free = [](void* p) { delete static_cast<PwPwHost*>(p); };
  st->tile_rows = kBM; st->grid = host->grid; st->smem_bytes = host->smem_bytes;
  plan->tile_rows = kBM; plan->smem_bytes = host->smem_bytes;
  return AGO_OK;
}

ago_status_t pwpw_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                      void* output, unsigned int* status_word, cudaStream_t stream, std::string* err) {
  (void)plan;
  PwPwHost* host = static_cast<PwPwHost*>(st->impl);
  PwPwParams q = host->prm;
  q.w1 = static_cast<const __nv_bfloat16*>(weights[0]); q.b1 = static_cast<const float*>(weights[1]);
  q.w2 = static_cast<const __nv_bfloat16*>(weights[2]); q.b2 = static_cast<const float*>(weights[3]);
  q.out = static_cast<__nv_bfloat16*>(output);
  q.status = status_word;
  // X [M][C0] as K-major tiles of 128 rows x 64 channels
  CUtensorMap mx;
  {
    auto it = host->maps.find(inputs[0]);
    if (it == host->maps.end()) {
      CUtensorMap m;
      const uint64_t dims[2] = {(uint64_t)q.C0, (uint64_t)q.M};
      const uint64_t strides[1] = {(uint64_t)q.C0 * 2};
      const uint32_t box[2] = {(uint32_t)kBK, (uint32_t)kBM};
      if (!encode_tmap_bf16(&m, inputs[0], 2, dims, strides, box, 128, err)) return AGO_ERR_CUDA;
      if (host->maps.size() > 4096) host->maps.clear();
      it = host->maps.emplace(inputs[0], m).first;
    }
    mx = it->second;
  }
  {
    static int smem_opt_in[64] = {};
    cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(pwpw_fused_kernel), smem_opt_in);
    if (e != cudaSuccess) { *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  }
  FusedLaunch launch(dim3((unsigned)host->grid), kThreads, (size_t)host->smem_bytes, stream);
  cudaError_t e = cudaLaunchKernelEx(&launch.config, pwpw_fused_kernel, mx, q);
  if (e != cudaSuccess) { *err = std::string("fused pointwise pair launch: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  return AGO_OK;
}

}  // namespace ago
