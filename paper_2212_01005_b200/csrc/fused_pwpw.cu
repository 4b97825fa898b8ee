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
//
// The same kernel serves the projection chain of a patch-unfolded attention block (Section VI-B: matrix
// multiplication, reshape, add, reshape, transpose, reshape, matrix multiplication, reshape): the reshapes are
// views, the add takes a second input tensor, and the transpose of two leading axes only permutes the rows between
// the products -- so the tile's output rows are stored at their permuted positions and no layout operator costs a
// pass over memory. There the weights are GEMM operands ([K][N], used as N-major B operands as they lie in memory)
// and the tensor to add arrives by TMA in the buffer of the second product's A operand, which the first epilogue
// updates in place.
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

constexpr int kThreads = 512;
constexpr int kColWarps = kThreads / 128;   // warps that share the 16-column groups of one tensor-memory lane quarter
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
  int BR;                    // rows per tile (<= 128): chosen so that the tiles split evenly over the resident CTAs
  int C0p, C1p, C2p;         // padded to the MMA granularity (16)
  int nkb0, nkb1;            // 64-channel K blocks of the first / second product
  int act1, act2;            // ReLU6 after the first / second convolution
  int w_nmajor;              // weights are [K][N] (GEMM operator) instead of [N][K] (1x1 convolution)
  int has_res;               // + a tensor [M][C1] after the first product
  int perm_a, perm_b;        // output row ((g * a + i) * b + j) is stored as row ((g * b + j) * a + i); 0: no permutation
  int w1_block, w2_block;    // byte distance between the 64-wide blocks of the weight tiles
  uint32_t k2_recip;         // reciprocal of the 16-byte pieces per output row (C2 / 8)
  uint32_t c0_recip, c1_recip;   // ... per padded row of W1 / W2 as they lie in memory
  int pitch;                 // row pitch of the staging tile
  int x_tx;                  // bytes one X tile (and its tile of the added tensor) brings in (TMA transaction count)
  int tmem_cols;
  int off_x, off_a, off_w1, off_w2, off_b, off_rows, off_bar;
};

__device__ __forceinline__ float relu6f(float v) { return fminf(fmaxf(v, 0.0f), 6.0f); }

__global__ void __launch_bounds__(kThreads)
pwpw_fused_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_r, const PwPwParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sX = smem + p.off_x;
  uint8_t* sA = smem + p.off_a;
  uint8_t* sW1 = smem + p.off_w1;
  uint8_t* sW2 = smem + p.off_w2;
  float* sB1 = reinterpret_cast<float*>(smem + p.off_b);
  float* sB2 = sB1 + p.C1p;
  int* sRows = reinterpret_cast<int*>(smem + p.off_rows);   // destination row of every row of the tile
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
  uint64_t* bar_x = bars;        // X tile landed
  uint64_t* bar_m1 = bars + 2;   // first product complete
  uint64_t* bar_m2 = bars + 3;   // second product complete
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 5);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int k2 = p.C2 >> 3;
  const int ntiles = (p.M + p.BR - 1) / p.BR;   // tiles of BR <= 128 rows: the MMAs still span 128 rows, the rest is ignored

  if (tid == 0) {
    *abort_flag = 0u;
    for (int i = 0; i < 4; ++i) mbar_init(bars + i, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmap_x);
    if (p.has_res) tma_prefetch_desc(&tmap_r);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  auto load_x = [&](int tile) {   // one thread
    mbar_arrive_expect_tx(bar_x, (uint32_t)p.x_tx);
    for (int kb = 0; kb < p.nkb0; ++kb) tma_load_2d(sX + kb * kXBlock, &tmap_x, bar_x, kb * kBK, tile * p.BR);
    if (p.has_res)   // the second product of the previous tile has read this buffer
      for (int kb = 0; kb < p.nkb1; ++kb) tma_load_2d(sA + kb * kXBlock, &tmap_r, bar_x, kb * kBK, tile * p.BR);
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
    // [N][K] weights: a piece is (row n, 16-byte chunk of k) -> K-major block k / 64, row n;
    // [K][N] weights: a piece is (row k, 16-byte chunk of n) -> N-major block n / 64, row k
    const int r1 = p.w_nmajor ? p.C0p : p.C1p, c1n = (p.w_nmajor ? p.C1p : p.C0p) >> 3;     // padded rows, chunks per row
    const int r2 = p.w_nmajor ? p.C1p : p.C2p, c2n = (p.w_nmajor ? p.C2p : p.C1p) >> 3;
    const int vr1 = p.w_nmajor ? p.C0 : p.C1, vc1 = p.w_nmajor ? p.C1 : p.C0;                // valid rows, valid row length
    const int vr2 = p.w_nmajor ? p.C1 : p.C2, vc2 = p.w_nmajor ? p.C2 : p.C1;
    const int n1 = r1 * c1n, nw = n1 + r2 * c2n;
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
          const int cpr = first ? c1n : c2n;
          const int row = (int)fast_div((uint32_t)j, (uint32_t)cpr, first ? p.c0_recip : p.c1_recip), ch = j - row * cpr;
          const int vr = first ? vr1 : vr2, vc = first ? vc1 : vc2;
          dst[k] = (uint32_t)((first ? p.off_w1 : p.off_w2) + (ch >> 3) * (first ? p.w1_block : p.w2_block)) +
                   swz_offset((uint32_t)row, (uint32_t)(ch & 7), 128);
          if (row < vr && ch * 8 < vc)
            v[k] = __ldg(reinterpret_cast<const uint4*>((first ? p.w1 : p.w2) + (int64_t)row * vc + ch * 8));
        }
      }
#pragma unroll
      for (int k = 0; k < kBatch; ++k)
        if (dst[k] != 0xffffffffu) *reinterpret_cast<uint4*>(smem + dst[k]) = v[k];
    }
  }
  for (int i = tid; i < p.C1p + p.C2p; i += kThreads)
    sB1[i] = i < p.C1p ? (i < p.C1 && p.b1 ? __ldg(p.b1 + i) : 0.0f) : (i - p.C1p < p.C2 && p.b2 ? __ldg(p.b2 + i - p.C1p) : 0.0f);
  fence_proxy_async_smem();
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
  const int half = warp >> 2;             // the warps of a lane quarter take the 16-column groups of an epilogue round-robin
  const int r = (warp & 3) * 32 + lane;   // this thread's row of the tile = its tensor-memory lane
  const uint32_t idesc1 = make_idesc_bf16(128, (uint32_t)p.C1p, 0, (uint32_t)p.w_nmajor);
  const uint32_t idesc2 = make_idesc_bf16(128, (uint32_t)p.C2p, 0, (uint32_t)p.w_nmajor);

  for (int tile = blockIdx.x, it = 0; tile < ntiles; tile += gridDim.x, ++it) {
    const uint32_t par = (uint32_t)it & 1u;
    const int row0 = tile * p.BR, rows = min(p.BR, p.M - row0);
    if (p.perm_a > 0 && tid < kBM) {   // read after two barriers below
      const int m = row0 + tid, ab = p.perm_a * p.perm_b;
      const int g = m / ab, rem = m - g * ab, i = rem / p.perm_b, j = rem - i * p.perm_b;
      sRows[tid] = (g * p.perm_b + j) * p.perm_a + i;
    }
    // ---- P2: first product (warp 0, converged; MMAs predicated on one elected lane, see tc_common.cuh) ----
    if (warp == 0) {
      const uint32_t elected = elect_one();
      mbar_wait(bar_x, par, abort_flag, p.status, 0x600);
      tcgen05_fence_after_sync();
      for (int kb = 0; kb < p.nkb0; ++kb) {
        const uint64_t ad = make_smem_desc(smem_u32(sX + kb * kXBlock), 0, 1024, SW_128B);
        // K-major B: one block per 64 reduction channels, 32 bytes per step; N-major B: 16 rows of 128 bytes per step,
        // the 64-column blocks w1_block apart (LBO)
        const uint64_t bd = p.w_nmajor ? make_smem_desc(smem_u32(sW1 + kb * 4 * 2048), (uint32_t)p.w1_block, 1024, SW_128B)
                                       : make_smem_desc(smem_u32(sW1 + kb * p.w1_block), 0, 1024, SW_128B);
        const uint32_t bstep = p.w_nmajor ? 2048u >> 4 : 2u;
        const int ksteps = min(4, (p.C0p - kb * kBK) / 16);
        for (int ks = 0; ks < ksteps; ++ks) umma_bf16_elected_acc(tmem_base, ad + 2u * ks, bd + bstep * ks, idesc1, elected, (kb | ks) != 0);
      }
      umma_commit_elected(bar_m1, elected);
    }
    __syncwarp();
    mbar_wait(bar_m1, par, abort_flag, p.status, 0x601);
    if (p.has_res) mbar_wait(bar_x, par, abort_flag, p.status, 0x604);   // every reader of the added tensor observes its arrival
    tcgen05_fence_after_sync();
    // ---- P3: + b1 [ReLU6] -> swizzled A operand of the second product ----
    for (int g = half; g < p.C1p / 16; g += kColWarps) {
      uint32_t v[16];
      tmem_ld_x16(tmem_base + lane_base + g * 16, v);
      tmem_ld_wait();
      uint8_t* blk = sA + (g >> 2) * kXBlock;              // 64 channels per block = 4 groups = 8 chunks of 16 bytes
      const uint32_t ch = (uint32_t)(g & 3) * 2u;
      uint4* d0 = reinterpret_cast<uint4*>(blk + swz_offset((uint32_t)r, ch, 128));
      uint4* d1 = reinterpret_cast<uint4*>(blk + swz_offset((uint32_t)r, ch + 1u, 128));
      uint32_t add[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};   // the tensor to add lies where the result goes
      if (p.has_res) {
        const uint4 a0 = *d0, a1 = *d1;
        add[0] = a0.x; add[1] = a0.y; add[2] = a0.z; add[3] = a0.w; add[4] = a1.x; add[5] = a1.y; add[6] = a1.z; add[7] = a1.w;
      }
      uint32_t w[8];
      float bv[16];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float4 t4 = *reinterpret_cast<const float4*>(sB1 + g * 16 + 4 * j);
        bv[4 * j] = t4.x; bv[4 * j + 1] = t4.y; bv[4 * j + 2] = t4.z; bv[4 * j + 3] = t4.w;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float y0 = __uint_as_float(v[2 * j]) + bv[2 * j] + bf16_lo(add[j]);
        float y1 = __uint_as_float(v[2 * j + 1]) + bv[2 * j + 1] + bf16_hi(add[j]);
        if (p.act1) { y0 = relu6f(y0); y1 = relu6f(y1); }
        w[j] = pack_bf16x2(y0, y1);
      }
      *d0 = make_uint4(w[0], w[1], w[2], w[3]);
      *d1 = make_uint4(w[4], w[5], w[6], w[7]);
    }
    fence_proxy_async_smem();
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    // ---- P4: second product, over the drained columns of the first ----
    if (warp == 0) {
      const uint32_t elected = elect_one();
      for (int kb = 0; kb < p.nkb1; ++kb) {
        const uint64_t ad = make_smem_desc(smem_u32(sA + kb * kXBlock), 0, 1024, SW_128B);
        const uint64_t bd = p.w_nmajor ? make_smem_desc(smem_u32(sW2 + kb * 4 * 2048), (uint32_t)p.w2_block, 1024, SW_128B)
                                       : make_smem_desc(smem_u32(sW2 + kb * p.w2_block), 0, 1024, SW_128B);
        const uint32_t bstep = p.w_nmajor ? 2048u >> 4 : 2u;
        const int ksteps = min(4, (p.C1p - kb * kBK) / 16);
        for (int ks = 0; ks < ksteps; ++ks) umma_bf16_elected_acc(tmem_base, ad + 2u * ks, bd + bstep * ks, idesc2, elected, (kb | ks) != 0);
      }
      umma_commit_elected(bar_m2, elected);
    }
    __syncwarp();
    mbar_wait(bar_m2, par, abort_flag, p.status, 0x602);
    tcgen05_fence_after_sync();
    // ---- P5: + b2 [ReLU6] -> staging tile over the X tile (the first product has read it) -> device memory ----
    for (int g = half; g < p.C2p / 16; g += kColWarps) {
      uint32_t v[16];
      tmem_ld_x16(tmem_base + lane_base + g * 16, v);
      tmem_ld_wait();
      uint32_t w[8];
      float bv[16];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float4 t4 = *reinterpret_cast<const float4*>(sB2 + g * 16 + 4 * j);
        bv[4 * j] = t4.x; bv[4 * j + 1] = t4.y; bv[4 * j + 2] = t4.z; bv[4 * j + 3] = t4.w;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float y0 = __uint_as_float(v[2 * j]) + bv[2 * j], y1 = __uint_as_float(v[2 * j + 1]) + bv[2 * j + 1];
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
      uint4* o0 = reinterpret_cast<uint4*>(p.out + (int64_t)row0 * p.C2);   // without a permutation the tile's rows are contiguous
      for (int i = tid; i < rows * k2; i += kThreads) {
        const int rr = (int)fast_div((uint32_t)i, (uint32_t)k2, p.k2_recip), k = i - rr * k2;
        const uint4 val = *reinterpret_cast<const uint4*>(sX + rr * p.pitch + k * 16);
        if (p.perm_a > 0) reinterpret_cast<uint4*>(p.out + (int64_t)sRows[rr] * p.C2)[k] = val;
        else o0[i] = val;
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
  bool chain = false;   // the GEMM -> + input -> row transpose -> GEMM chain instead of two 1x1 convolutions
  std::unordered_map<const void*, CUtensorMap> maps, maps_r;   // tensor maps of X / of the added tensor by base address
};

}  // namespace

ago_status_t pwpw_plan(Plan* plan, FusedState* st, std::string* err) {
  const auto& ops = plan->ops;
  auto* host = new PwPwHost();
  PwPwParams& q = host->prm;
  q = PwPwParams{};
  auto bad = [&](const char* m) { *err = std::string("fused pointwise pair: ") + m; delete host; return AGO_ERR_UNSUPPORTED; };
  const OpInfo& a = ops[0];
  q.C0 = (int)a.in.last();
  q.M = (int)(a.in.numel() / q.C0);
  q.C1 = a.op.p[0];
  if (plan->fused_kernel == AGO_KERNEL_GEMM_PERMUTE_GEMM) {
    // gemm, reshape, add_input, reshape [G, A, B, C1], transpose (A, B), reshape, gemm, reshape
    host->chain = true;
    q.w_nmajor = 1; q.has_res = 1;
    q.C2 = ops[6].op.p[0];
    q.perm_a = (int)ops[3].out.d[1]; q.perm_b = (int)ops[3].out.d[2];
    if (a.in.numel() >= (1ll << 31) || ops[7].out.numel() >= (1ll << 31)) return bad("tensors of 2^31 elements or more are not supported");
  } else {
    // conv, bias, [relu6], conv, bias, [relu6]
    int i2 = 2;
    if (ops[2].op.kind == AGO_OP_RELU6) { q.act1 = 1; i2 = 3; }
    q.act2 = (int)ops.size() > i2 + 2 ? 1 : 0;
    q.C2 = ops[i2].op.p[0];
  }
  if (q.C0 % 8 || q.C1 % 8 || q.C2 % 8) return bad("channel counts must be multiples of 8");
  q.C0p = round_up(q.C0, 16); q.C1p = round_up(q.C1, 16); q.C2p = round_up(q.C2, 16);
  if (q.C1p > 256 || q.C2p > 256) return bad("more than 256 middle or output channels is not supported");
  q.nkb0 = (q.C0 + kBK - 1) / kBK; q.nkb1 = (q.C1p + kBK - 1) / kBK;
  q.k2_recip = fast_div_recip(q.C2 / 8);
  const int w1_chunks = (q.w_nmajor ? q.C1p : q.C0p) / 8, w2_chunks = (q.w_nmajor ? q.C2p : q.C1p) / 8;
  const int w1_rows = q.w_nmajor ? q.C0p : q.C1p, w2_rows = q.w_nmajor ? q.C1p : q.C2p;
  q.c0_recip = fast_div_recip(w1_chunks); q.c1_recip = fast_div_recip(w2_chunks);
  q.w1_block = w1_rows * 128; q.w2_block = w2_rows * 128;
  const int w1_bytes = (w1_chunks + 7) / 8 * q.w1_block, w2_bytes = (w2_chunks + 7) / 8 * q.w2_block;
  q.pitch = q.C2 * 2 + 16;
  q.tmem_cols = 32;
  while (q.tmem_cols < std::max(q.C1p, q.C2p)) q.tmem_cols *= 2;
  int off = 0;
  auto take = [&](int bytes) { int o = off; off = round_up(off + bytes, 1024); return o; };
  q.off_x = take(std::max(q.nkb0 * kXBlock, kBM * q.pitch));
  q.off_a = take(q.nkb1 * kXBlock);
  q.off_w1 = take(w1_bytes);
  q.off_w2 = take(w2_bytes);
  q.off_b = take((q.C1p + q.C2p) * 4);
  q.off_rows = take(kBM * 4);
  q.off_bar = take(64);
  host->smem_bytes = off + 1024;
  if (host->smem_bytes > 227 * 1024) return bad("the operands of one row tile do not fit shared memory");
  if ((long)kBM * (q.C2 / 8) > 65535 || (long)w1_rows * w1_chunks > 65535 || (long)w2_rows * w2_chunks > 65535)
    return bad("operands too large for the copy index arithmetic");
  // Rows per tile: with k = rounds of 128-row tiles over the resident CTAs, the smallest tile height that still
  // needs k rounds -- the same number of rounds, less work in each
  const int per_sm = host->smem_bytes <= 113 * 1024 ? 2 : 1, slots = per_sm * device_sm_count();
  const long k = ((long)(q.M + kBM - 1) / kBM + slots - 1) / slots;
  q.BR = (int)std::min<long>(kBM, (q.M + k * slots - 1) / (k * slots));
  q.x_tx = (q.nkb0 + (q.has_res ? q.nkb1 : 0)) * q.BR * 128;
  host->grid = std::min((q.M + q.BR - 1) / q.BR, slots);
  st->impl = host;
  st->impl_free = [](void* p) { delete static_cast<PwPwHost*>(p); };
  st->tile_rows = q.BR; st->grid = host->grid; st->smem_bytes = host->smem_bytes;
  plan->tile_rows = q.BR; plan->smem_bytes = host->smem_bytes;
  return AGO_OK;
}

ago_status_t pwpw_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                      void* output, unsigned int* status_word, cudaStream_t stream, std::string* err) {
  (void)plan;
  PwPwHost* host = static_cast<PwPwHost*>(st->impl);
  PwPwParams q = host->prm;
  if (host->chain) {
    q.w1 = static_cast<const __nv_bfloat16*>(weights[0]); q.w2 = static_cast<const __nv_bfloat16*>(weights[1]);
    q.b1 = nullptr; q.b2 = nullptr;
  } else {
    q.w1 = static_cast<const __nv_bfloat16*>(weights[0]); q.b1 = static_cast<const float*>(weights[1]);
    q.w2 = static_cast<const __nv_bfloat16*>(weights[2]); q.b2 = static_cast<const float*>(weights[3]);
  }
  q.out = static_cast<__nv_bfloat16*>(output);
  q.status = status_word;
  // [M][C] bf16 matrices as K-major tiles of 128 rows x 64 channels
  auto get_map = [&](std::unordered_map<const void*, CUtensorMap>& cache, const void* base, int C, CUtensorMap* out) -> bool {
    auto it = cache.find(base);
    if (it == cache.end()) {
      CUtensorMap m;
      const uint64_t dims[2] = {(uint64_t)C, (uint64_t)q.M};
      const uint64_t strides[1] = {(uint64_t)C * 2};
      const uint32_t box[2] = {(uint32_t)kBK, (uint32_t)q.BR};
      if (!encode_tmap_bf16(&m, base, 2, dims, strides, box, 128, err)) return false;
      if (cache.size() > 4096) cache.clear();
      it = cache.emplace(base, m).first;
    }
    *out = it->second;
    return true;
  };
  CUtensorMap mx, mr;
  if (!get_map(host->maps, inputs[0], q.C0, &mx)) return AGO_ERR_CUDA;
  mr = mx;
  if (host->chain && !get_map(host->maps_r, inputs[1], q.C1, &mr)) return AGO_ERR_CUDA;
  {
    static int smem_opt_in[64] = {};
    cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(pwpw_fused_kernel), smem_opt_in);
    if (e != cudaSuccess) { *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  }
  FusedLaunch launch(dim3((unsigned)host->grid), kThreads, (size_t)host->smem_bytes, stream);
  cudaError_t e = cudaLaunchKernelEx(&launch.config, pwpw_fused_kernel, mx, mr, q);
  if (e != cudaSuccess) { *err = std::string("fused pointwise pair launch: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  return AGO_OK;
}

}  // namespace ago
