// Fused inverted-residual block: 1x1 conv + bias + ReLU6 -> depthwise 3x3
// (pad 1, stride 1|2) + bias + ReLU6 -> 1x1 conv + bias [+ input], one kernel.
//
// Tiling follows Section III-B. The pointwise -> depthwise link is the
// "downstream depthwise" category: the depthwise tile keeps its spatial extent
// and is tiled over channels (o1 = o2, here 16 channels per chunk). The
// depthwise -> pointwise link is the "downstream pointwise" category: the
// project tile keeps ALL output channels and is tiled over rows (a strip of R
// output rows of one image per CTA), so nothing is recomputed except the
// expand convolution on the strip's one-row halo.
//
// Per CTA (one image, R output rows, full width):
//   P1  TMA loads the NHWC input strip with halo (out-of-image -> 0, channels
//       padded to the MMA K granularity by the box) into a swizzled K-major tile.
//   for each 16-channel chunk c of the expanded tensor:
//     P2  tcgen05.mma: expand[pixels x 16] = X[pixels x Cin] * W1[c]^T   (TMEM, fp32)
//     P3  TMEM -> registers: + b1, ReLU6, zero outside the image (the depthwise
//         conv pads the post-activation tensor), bf16 -> shared memory
//     P4  CUDA cores: depthwise 3x3 + bd + ReLU6 over the resident chunk, result
//         written as the K-major A operand of the project GEMM
//     P5  tcgen05.mma: out[pixels x Cout] += DW[pixels x 16] * W3[:, c]^T  (TMEM)
//   P6  TMEM -> registers: + b3 (+ x), bf16, 16-byte stores.
// The expand MMA of chunk c+1 is issued before the CUDA-core work of chunk c.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdlib>
#include <unordered_map>

#include "fused.h"
#include "tc_common.cuh"
#include "tmap.h"

namespace ago {

namespace {

using namespace tc;

constexpr int kComputeWarps = 28;                  // expand epilogue, depthwise, project epilogue
constexpr int kComputeThreads = kComputeWarps * 32;
constexpr int kIssuers = 4;                        // one MMA-issuing warp per SM sub-partition
constexpr int kThreads = kComputeThreads + 32 * kIssuers;
constexpr int kChunk = 16;      // expanded channels per chunk = one MMA K step of the project GEMM
constexpr int kChunkRowBytes = 32;

struct Mbv2Params {
  const __nv_bfloat16* x;
  const __nv_bfloat16* w1;
  const float* b1;
  const __nv_bfloat16* wd;
  const float* bd;
  const __nv_bfloat16* w3;
  const float* b3;
  __nv_bfloat16* out;
  unsigned int* status;
  int N, H, W, Cin, Cexp, Cout, stride, Ho, Wo, residual;
  int R, strips, IH, IW, P_in, M1, M2;
  int Kp, row_bytes, swizzle;   // input / W1 tiles: padded K, bytes per row, tc::SwizzleMode
  int Coutp, NC;
  int tmem_cols, ecol0, pcol0;
  int e_plane, d_plane;         // byte distance between the two 8-channel planes of an E / D chunk
  // shared-memory byte offsets (from the 1024-aligned base)
  int off_x, off_w1, off_e, off_d, off_w3, off_wd, off_b1, off_bd, off_b3, off_bar;
};

__device__ __forceinline__ uint32_t relu6_pack(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  h = __hmin2(__hmax2(h, __floats2bfloat162_rn(0.0f, 0.0f)), __floats2bfloat162_rn(6.0f, 6.0f));
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ float2 bf16x2_to_f2(uint32_t w) { return make_float2(bf16_lo(w), bf16_hi(w)); }
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }

__device__ __forceinline__ uint32_t lds32(uint32_t saddr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(saddr));
  return v;
}
__device__ __forceinline__ void sts32(uint32_t saddr, uint32_t v) {
  asm volatile("st.shared.u32 [%0], %1;" ::"r"(saddr), "r"(v) : "memory");
}

// Depthwise 3x3 over the resident E chunk for one (channel pair, output column)
// and output rows [r0, r1): E and D chunks are two planes of [pixel][8 channels]
// (16 bytes per pixel), which is also the un-swizzled K-major operand layout.
// e_col / d_col are 32-bit shared-memory addresses.
template <int STRIDE>
__device__ __forceinline__ void depthwise_column(uint32_t e_col, uint32_t d_col, int r0, int r1, int IW, int Wo,
                                                 const float2 (&w)[9], float2 bias) {
  const uint32_t e_pitch = (uint32_t)IW * 16u, d_pitch = (uint32_t)Wo * 16u;
  if (STRIDE == 1) {
    // walk down the input rows once; each row feeds the three output rows it overlaps
    float2 a0 = bias, a1 = bias, a2 = bias;   // output rows i, i-1, i-2
    uint32_t src = e_col + (uint32_t)r0 * e_pitch;
    uint32_t dst = d_col + (uint32_t)r0 * d_pitch;
    // the first two input rows complete no output
#pragma unroll
    for (int pre = 0; pre < 2; ++pre) {
      const float2 x0 = bf16x2_to_f2(lds32(src)), x1 = bf16x2_to_f2(lds32(src + 16)), x2 = bf16x2_to_f2(lds32(src + 32));
      src += e_pitch;
      a0 = fma2(x0, w[0], a0); a0 = fma2(x1, w[1], a0); a0 = fma2(x2, w[2], a0);
      a1 = fma2(x0, w[3], a1); a1 = fma2(x1, w[4], a1); a1 = fma2(x2, w[5], a1);
      a2 = a1; a1 = a0; a0 = bias;
    }
    for (int i = r0; i < r1; ++i) {   // input row i + 2 completes output row i
      const float2 x0 = bf16x2_to_f2(lds32(src)), x1 = bf16x2_to_f2(lds32(src + 16)), x2 = bf16x2_to_f2(lds32(src + 32));
      src += e_pitch;
      a2 = fma2(x0, w[6], a2); a2 = fma2(x1, w[7], a2); a2 = fma2(x2, w[8], a2);
      sts32(dst, relu6_pack(a2.x, a2.y));
      dst += d_pitch;
      a1 = fma2(x0, w[3], a1); a1 = fma2(x1, w[4], a1); a1 = fma2(x2, w[5], a1);
      a0 = fma2(x0, w[0], a0); a0 = fma2(x1, w[1], a0); a0 = fma2(x2, w[2], a0);
      a2 = a1; a1 = a0; a0 = bias;
    }
  } else {
    for (int r = r0; r < r1; ++r) {
      float2 a = bias;
      const uint32_t src = e_col + (uint32_t)(r * STRIDE) * e_pitch;
#pragma unroll
      for (int kr = 0; kr < 3; ++kr)
#pragma unroll
        for (int ks = 0; ks < 3; ++ks)
          a = fma2(bf16x2_to_f2(lds32(src + (uint32_t)kr * e_pitch + (uint32_t)ks * 16u)), w[kr * 3 + ks], a);
      sts32(d_col + (uint32_t)r * d_pitch, relu6_pack(a.x, a.y));
    }
  }
}

__global__ void __launch_bounds__(kThreads, 1)
mbv2_fused_kernel(const __grid_constant__ CUtensorMap tmap_x, const Mbv2Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sX = smem + p.off_x;
  uint8_t* sW1 = smem + p.off_w1;
  uint8_t* sE = smem + p.off_e;
  uint8_t* sD = smem + p.off_d;
  uint8_t* sW3 = smem + p.off_w3;
  float* sWd = reinterpret_cast<float*>(smem + p.off_wd);
  float* sB1 = reinterpret_cast<float*>(smem + p.off_b1);
  float* sBd = reinterpret_cast<float*>(smem + p.off_bd);
  float* sB3 = reinterpret_cast<float*>(smem + p.off_b3);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
  uint64_t* bar_x = bars + 0;       // input strip landed (TMA)
  uint64_t* bar_w = bars + 1;       // weights staged by the compute warps
  uint64_t* bar_e = bars + 2;       // [2] expand accumulators of buffer b complete (MMA commit)
  uint64_t* bar_d = bars + 4;       // [2] project MMA has consumed D[b] (MMA commit)
  uint64_t* bar_tfree = bars + 6;   // [2] expand buffer b drained and E chunk written (compute -> issuer)
  uint64_t* bar_dready = bars + 8;  // [2] D[b] written (compute -> issuer)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 10);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 11);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n = blockIdx.x / p.strips, strip = blockIdx.x % p.strips;
  const int ho0 = strip * p.R;
  const int rows_valid = min(p.R, p.Ho - ho0);
  const int gh0 = ho0 * p.stride - 1;   // image row of tile row 0
  const int d_bytes = 2 * p.d_plane;

  if (tid == kComputeThreads) {
    // first issuer lane: barriers, then the input strip's TMA right away
    *abort_flag = 0u;
    mbar_init(bar_x, 1);
    mbar_init(bar_w, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_e + i, kIssuers);
      mbar_init(bar_d + i, kIssuers);
      mbar_init(bar_tfree + i, 1);
      mbar_init(bar_dready + i, 1);
    }
    fence_mbar_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmap_x);
    mbar_arrive_expect_tx(bar_x, (uint32_t)(p.P_in * p.row_bytes));
    tma_load_4d(sX, &tmap_x, bar_x, 0, -1, gh0, n);
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp >= kComputeWarps) {
    // ================= MMA issue warps: issuer i owns M tiles i, i+4, ... (one lane each) =================
    const int iw = warp - kComputeWarps;
    if (lane == 0) {
      const uint32_t idesc_e = make_idesc_bf16(128, kChunk);
      const uint32_t idesc_p = make_idesc_bf16(128, (uint32_t)p.Coutp);
      const uint32_t sbo_x = 8u * (uint32_t)p.row_bytes;
      const uint64_t xdesc0 = make_smem_desc(smem_u32(sX), 0, sbo_x, p.swizzle);
      const uint64_t w1desc0 = make_smem_desc(smem_u32(sW1), 0, sbo_x, p.swizzle);
      // D: un-swizzled K-major; the two 8-channel planes are the two K core-matrix columns
      const uint64_t ddesc0 = make_smem_desc(smem_u32(sD), (uint32_t)p.d_plane, 128, SW_NONE);
      const uint64_t w3desc0 = make_smem_desc(smem_u32(sW3), 0, 256, SW_32B);
      const int ksteps = p.Kp / 16;
      const uint32_t a_tile_step = (uint32_t)(128 * p.row_bytes) >> 4;

      auto issue_expand = [&](int c) {
        const int b = c & 1;
        const uint64_t bdesc = w1desc0 + (uint64_t)((c * kChunk * p.row_bytes) >> 4);
        for (int t = iw; t < p.M1; t += kIssuers) {
          const uint64_t adesc = xdesc0 + (uint64_t)t * a_tile_step;
          const uint32_t d_tmem = tmem_base + p.ecol0 + (b * p.M1 + t) * kChunk;
          umma_bf16(d_tmem, adesc, bdesc, idesc_e, 0);
          for (int ks = 1; ks < ksteps; ++ks) umma_bf16(d_tmem, adesc + 2u * ks, bdesc + 2u * ks, idesc_e, 1);
        }
        umma_commit(bar_e + b);
      };
      mbar_wait(bar_w, 0, abort_flag, p.status, 0x100);
      mbar_wait(bar_x, 0, abort_flag, p.status, 0x101);
      tcgen05_fence_after_sync();
      issue_expand(0);
      if (p.NC > 1) issue_expand(1);
      for (int c = 0; c < p.NC; ++c) {
        const int b = c & 1;
        const uint32_t ph = (uint32_t)(c >> 1) & 1u;
        if (c + 2 < p.NC) {
          mbar_wait(bar_tfree + b, ph, abort_flag, p.status, 0x105);
          tcgen05_fence_after_sync();
          issue_expand(c + 2);
        }
        mbar_wait(bar_dready + b, ph, abort_flag, p.status, 0x106);
        tcgen05_fence_after_sync();
        const uint64_t bdesc = w3desc0 + (uint64_t)((c * p.Coutp * kChunkRowBytes) >> 4);
        for (int t = iw; t < p.M2; t += kIssuers)
          umma_bf16(tmem_base + p.pcol0 + t * p.Coutp, ddesc0 + (uint64_t)((b * d_bytes + t * 128 * 16) >> 4), bdesc,
                    idesc_p, c > 0);
        umma_commit(bar_d + b);
      }
    }
    __syncwarp();
  } else {
    // ================================== compute warps ==================================
    const int ctid = tid;   // compute warps are warps 0 .. kComputeWarps-1
    // ---- stage weights and biases (generic proxy), in the operand layouts the MMAs read ----
    {
      const int chunks_per_row = p.row_bytes >> 4;
      for (int i = ctid; i < p.Cexp * chunks_per_row; i += kComputeThreads) {
        const int row = i / chunks_per_row, ch = i % chunks_per_row;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (ch * 8 < p.Cin) v = __ldg(reinterpret_cast<const uint4*>(p.w1 + (size_t)row * p.Cin + ch * 8));
        *reinterpret_cast<uint4*>(sW1 + swz_offset(row, ch, p.row_bytes)) = v;
      }
      for (int i = ctid; i < p.NC * p.Coutp * 2; i += kComputeThreads) {
        const int half = i & 1, row = (i >> 1) % p.Coutp, c = (i >> 1) / p.Coutp;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (row < p.Cout) v = __ldg(reinterpret_cast<const uint4*>(p.w3 + (size_t)row * p.Cexp + c * kChunk + half * 8));
        *reinterpret_cast<uint4*>(sW3 + c * p.Coutp * kChunkRowBytes + swz_offset(row, half, kChunkRowBytes)) = v;
      }
      for (int i = ctid; i < 9 * p.Cexp; i += kComputeThreads) sWd[i] = __bfloat162float(p.wd[i]);
      for (int i = ctid; i < p.Cexp; i += kComputeThreads) { sB1[i] = p.b1[i]; sBd[i] = p.bd[i]; }
      for (int i = ctid; i < p.Coutp; i += kComputeThreads) sB3[i] = i < p.Cout ? p.b3[i] : 0.0f;
    }
    fence_proxy_async_smem();
    named_barrier_sync(1, kComputeThreads);
    if (ctid == 0) mbar_arrive(bar_w);

    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    // Depthwise work split: thread = (channel pair, slot); a slot walks one output column of one row group.
    constexpr int kSlots = kComputeThreads / 8;
    const int cp = ctid & 7, slot = ctid >> 3;
    const int groups = max(1, min(rows_valid, kSlots / max(1, min(p.Wo, kSlots))));
    const int rows_per_group = (rows_valid + groups - 1) / groups;
    const int dw_items = p.Wo * groups;
    const int cp_off = (cp & 3) * 4;   // byte offset inside a 16-byte pixel entry
    // first depthwise item of this slot (most shapes have at most one per slot)
    const int item0_g = slot / p.Wo, item0_wo = slot - item0_g * p.Wo;
    // expand-epilogue rows of this thread: tile (warp>>2) + 7k; bit k of the masks: row exists / is an in-image pixel
    uint32_t e_exist = 0, e_inimg = 0;
    for (int t = warp >> 2, k = 0; t < p.M1; t += kComputeWarps / 4, ++k) {
      const int pix = t * 128 + (warp & 3) * 32 + lane;
      const int ih = pix / p.IW, iw = pix - ih * p.IW;
      const int gh = gh0 + ih;
      if (pix < p.P_in) {
        e_exist |= 1u << k;
        if (gh >= 0 && gh < p.H && iw >= 1 && iw <= p.W) e_inimg |= 1u << k;
      }
    }

    for (int c = 0; c < p.NC; ++c) {
      const int b = c & 1;
      mbar_wait(bar_e + b, (uint32_t)(c >> 1) & 1u, abort_flag, p.status, 0x102);
      tcgen05_fence_after_sync();

      // ---- P3: expand epilogue -> E chunk: + b1, ReLU6, zero outside the image, bf16 ----
      for (int t = warp >> 2, k = 0; t < p.M1; t += kComputeWarps / 4, ++k) {
        uint32_t acc[16];
        tmem_ld_x16(tmem_base + lane_base + p.ecol0 + (b * p.M1 + t) * kChunk, acc);
        tmem_ld_wait();
        const int pix = t * 128 + (warp & 3) * 32 + lane;
        if ((e_exist >> k) & 1u) {
          uint32_t w[8];
          if ((e_inimg >> k) & 1u) {
            const float4* bb = reinterpret_cast<const float4*>(sB1 + c * kChunk);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float4 bv = bb[j];
              w[2 * j] = relu6_pack(__uint_as_float(acc[4 * j]) + bv.x, __uint_as_float(acc[4 * j + 1]) + bv.y);
              w[2 * j + 1] = relu6_pack(__uint_as_float(acc[4 * j + 2]) + bv.z, __uint_as_float(acc[4 * j + 3]) + bv.w);
            }
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) w[j] = 0u;
          }
          *reinterpret_cast<uint4*>(sE + pix * 16) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(sE + p.e_plane + pix * 16) = make_uint4(w[4], w[5], w[6], w[7]);
        }
      }
      tcgen05_fence_before_sync();
      named_barrier_sync(1, kComputeThreads);
      if (ctid == 0) mbar_arrive(bar_tfree + b);

      // D[b] was read by the project MMA of chunk c-2
      if (c >= 2) mbar_wait(bar_d + b, (uint32_t)((c - 2) >> 1) & 1u, abort_flag, p.status, 0x103);

      // ---- P4: depthwise 3x3 + bias + ReLU6 on CUDA cores: E chunk -> D[b] (A operand of the project GEMM) ----
      {
        const int ch = c * kChunk + cp * 2;
        float2 wgt[9];
#pragma unroll
        for (int tap = 0; tap < 9; ++tap) wgt[tap] = *reinterpret_cast<const float2*>(sWd + tap * p.Cexp + ch);
        const float2 bias = *reinterpret_cast<const float2*>(sBd + ch);
        const uint32_t e_plane = smem_u32(sE) + (uint32_t)((cp >> 2) * p.e_plane + cp_off);
        const uint32_t d_plane = smem_u32(sD) + (uint32_t)(b * d_bytes + (cp >> 2) * p.d_plane + cp_off);
        for (int item = slot; item < dw_items; item += kSlots) {
          int g = item0_g, wo = item0_wo;
          if (item != slot) { g = item / p.Wo; wo = item - g * p.Wo; }
          const int r0 = g * rows_per_group, r1 = min(rows_valid, r0 + rows_per_group);
          if (p.stride == 1)
            depthwise_column<1>(e_plane + wo * 16, d_plane + wo * 16, r0, r1, p.IW, p.Wo, wgt, bias);
          else
            depthwise_column<2>(e_plane + wo * 32, d_plane + wo * 16, r0, r1, p.IW, p.Wo, wgt, bias);
        }
      }
      fence_proxy_async_smem();
      named_barrier_sync(1, kComputeThreads);
      if (ctid == 0) mbar_arrive(bar_dready + b);
    }

    // ---- P6: project epilogue: + b3 (+ residual), bf16, 16-byte stores ----
    {
      const int last = p.NC - 1;
      mbar_wait(bar_d + (last & 1), (uint32_t)(last >> 1) & 1u, abort_flag, p.status, 0x104);
      tcgen05_fence_after_sync();
      const int valid_pix = rows_valid * p.Wo;
      const size_t gpix0 = ((size_t)n * p.Ho + ho0) * p.Wo;
      for (int t = warp >> 2; t < p.M2; t += kComputeWarps / 4) {
        const int po = t * 128 + (warp & 3) * 32 + lane;
        for (int j0 = 0; j0 < p.Coutp; j0 += 16) {
          uint32_t acc[16];
          tmem_ld_x16(tmem_base + lane_base + p.pcol0 + t * p.Coutp + j0, acc);
          tmem_ld_wait();
          if (po < valid_pix) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const int j = j0 + h * 8;
              if (j < p.Cout) {
                float v[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) v[q] = __uint_as_float(acc[h * 8 + q]) + sB3[j + q];
                const size_t off = (gpix0 + po) * p.Cout + j;
                if (p.residual) {
                  const uint4 xr = __ldg(reinterpret_cast<const uint4*>(p.x + off));
                  v[0] += bf16_lo(xr.x); v[1] += bf16_hi(xr.x); v[2] += bf16_lo(xr.y); v[3] += bf16_hi(xr.y);
                  v[4] += bf16_lo(xr.z); v[5] += bf16_hi(xr.z); v[6] += bf16_lo(xr.w); v[7] += bf16_hi(xr.w);
                }
                *reinterpret_cast<uint4*>(p.out + off) =
                    make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
              }
            }
          }
        }
      }
    }
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
}

int round_up(int v, int m) { return (v + m - 1) / m * m; }

struct Mbv2Host {
  Mbv2Params prm;
  int smem_bytes = 0;
  std::unordered_map<const void*, CUtensorMap> maps;
};

bool layout(Mbv2Params& q, int R, int* smem_bytes) {
  q.R = R;
  q.strips = (q.Ho + R - 1) / R;
  q.IH = (R - 1) * q.stride + 3;
  q.IW = q.W + 2;
  q.P_in = q.IH * q.IW;
  q.M1 = (q.P_in + 127) / 128;
  q.M2 = (R * q.Wo + 127) / 128;
  if (q.IH > 256 || q.IW > 256 || q.M1 > 8) return false;
  const int cols = 2 * q.M1 * kChunk + q.M2 * q.Coutp;
  if (cols > 512) return false;
  q.tmem_cols = 32;
  while (q.tmem_cols < cols) q.tmem_cols *= 2;
  q.ecol0 = 0;
  q.pcol0 = 2 * q.M1 * kChunk;
  int off = 0;
  auto take = [&](int bytes) { int o = off; off = round_up(off + bytes, 1024); return o; };
  q.off_x = take(q.M1 * 128 * q.row_bytes);
  q.off_w1 = take(q.Cexp * q.row_bytes);
  // two 8-channel planes per chunk, offset by 64 mod 128 bytes so that a warp's
  // 2 x 64-byte accesses (4 pixels x 4 channel pairs per plane) never share a bank
  q.e_plane = round_up(q.P_in * 16, 128) + 64;
  q.d_plane = q.M2 * 128 * 16 + 64;
  q.off_e = take(2 * q.e_plane);
  q.off_d = take(2 * 2 * q.d_plane);
  q.off_w3 = take(q.NC * q.Coutp * kChunkRowBytes);
  q.off_wd = take(9 * q.Cexp * 4);
  q.off_b1 = take(q.Cexp * 4);
  q.off_bd = take(q.Cexp * 4);
  q.off_b3 = take(q.Coutp * 4);
  q.off_bar = take(128);
  *smem_bytes = off + 1024;  // slack for the 1024-byte alignment of the base
  return *smem_bytes <= 227 * 1024;
}

}  // namespace

ago_status_t mbv2_plan(Plan* plan, FusedState* st, std::string* err) {
  const OpInfo& e = plan->ops[0];
  const OpInfo& d = plan->ops[3];
  const OpInfo& pr = plan->ops[6];
  auto* host = new Mbv2Host();
  Mbv2Params& q = host->prm;
  q = Mbv2Params{};
  q.N = (int)e.in.d[0]; q.H = (int)e.in.d[1]; q.W = (int)e.in.d[2]; q.Cin = (int)e.in.d[3];
  q.Cexp = e.op.p[0]; q.Cout = pr.op.p[0]; q.stride = d.op.p[3];
  q.Ho = (int)d.out.d[1]; q.Wo = (int)d.out.d[2];
  q.residual = plan->ops.size() == 9 ? 1 : 0;
  auto bad = [&](const char* m) { *err = std::string("fused inverted-residual block: ") + m; delete host; return AGO_ERR_UNSUPPORTED; };
  if (q.Cin > 64) return bad("more than 64 input channels is not supported yet");
  if (q.Cexp % kChunk != 0) return bad("expanded channels must be a multiple of 16");
  if (q.Cout > 256) return bad("more than 256 output channels is not supported");
  if (q.residual && (q.stride != 1 || q.Cin != q.Cout)) return bad("residual needs stride 1 and Cin == Cout");
  q.Kp = q.Cin <= 16 ? 16 : (q.Cin <= 32 ? 32 : 64);
  q.row_bytes = q.Kp * 2;
  q.swizzle = q.Kp == 16 ? tc::SW_32B : (q.Kp == 32 ? tc::SW_64B : tc::SW_128B);
  q.Coutp = round_up(q.Cout, 16);
  q.NC = q.Cexp / kChunk;
  // Rows per CTA: fewest waves over the SMs, then least halo + tail work.
  int best_R = 0; double best_cost = 0; int best_smem = 0;
  const int sms = 148;
  for (int R = 1; R <= q.Ho; ++R) {
    Mbv2Params t = q; int smem = 0;
    if (!layout(t, R, &smem)) continue;
    const long ctas = (long)q.N * t.strips;
    const long waves = (ctas + sms - 1) / sms;
    const double cost = (double)waves * (t.M1 * 128.0 + 3.0 * t.M2 * 128.0 + 200.0);
    if (best_R == 0 || cost < best_cost) { best_R = R; best_cost = cost; best_smem = smem; }
  }
  if (best_R == 0) return bad("no row-strip tiling fits shared memory / tensor memory");
  layout(q, best_R, &best_smem);
  host->smem_bytes = best_smem;
  st->impl = host;
  st->impl_free = [](void* p) { delete static_cast<Mbv2Host*>(p); };
  st->tile_rows = best_R; st->grid = q.N * q.strips; st->smem_bytes = best_smem;
  plan->tile_rows = best_R; plan->smem_bytes = best_smem;
  return AGO_OK;
}

ago_status_t mbv2_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                      void* output, unsigned int* status_word, cudaStream_t stream, std::string* err) {
  Mbv2Host* host = static_cast<Mbv2Host*>(st->impl);
  Mbv2Params q = host->prm;
  q.x = static_cast<const __nv_bfloat16*>(inputs[0]);
  q.w1 = static_cast<const __nv_bfloat16*>(weights[0]); q.b1 = static_cast<const float*>(weights[1]);
  q.wd = static_cast<const __nv_bfloat16*>(weights[2]); q.bd = static_cast<const float*>(weights[3]);
  q.w3 = static_cast<const __nv_bfloat16*>(weights[4]); q.b3 = static_cast<const float*>(weights[5]);
  q.out = static_cast<__nv_bfloat16*>(output);
  q.status = status_word;
  auto it = host->maps.find(inputs[0]);
  if (it == host->maps.end()) {
    CUtensorMap m;
    const uint64_t dims[4] = {(uint64_t)q.Cin, (uint64_t)q.W, (uint64_t)q.H, (uint64_t)q.N};
    const uint64_t strides[3] = {(uint64_t)q.Cin * 2, (uint64_t)q.W * q.Cin * 2, (uint64_t)q.H * q.W * q.Cin * 2};
    const uint32_t box[4] = {(uint32_t)q.Kp, (uint32_t)q.IW, (uint32_t)q.IH, 1};
    if (!encode_tmap_bf16(&m, inputs[0], 4, dims, strides, box, q.row_bytes, err)) return AGO_ERR_CUDA;
    if (host->maps.size() > 4096) host->maps.clear();
    it = host->maps.emplace(inputs[0], m).first;
  }
  {
    static int smem_opt_in[64] = {};
    cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(mbv2_fused_kernel), smem_opt_in);
    if (e != cudaSuccess) { *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  }
  mbv2_fused_kernel<<<q.N * q.strips, kThreads, host->smem_bytes, stream>>>(it->second, q);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { *err = std::string("fused inverted-residual launch: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  return AGO_OK;
}

}  // namespace ago
