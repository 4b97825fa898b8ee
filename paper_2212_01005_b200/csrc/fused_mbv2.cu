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

#include <unordered_map>

#include "fused.h"
#include "tc_common.cuh"
#include "tmap.h"

namespace ago {

namespace {

using namespace tc;

constexpr int kThreads = 256;
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
  // shared-memory byte offsets (from the 1024-aligned base)
  int off_x, off_w1, off_e, off_d, off_w3, off_wd, off_b1, off_bd, off_b3, off_bar;
};

__device__ __forceinline__ float relu6f(float v) { return fminf(fmaxf(v, 0.0f), 6.0f); }

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
  uint64_t* bar_x = bars + 0;
  uint64_t* bar_e = bars + 1;  // [2]
  uint64_t* bar_d = bars + 3;  // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 5);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 6);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n = blockIdx.x / p.strips, strip = blockIdx.x % p.strips;
  const int ho0 = strip * p.R;
  const int rows_valid = min(p.R, p.Ho - ho0);
  const int gh0 = ho0 * p.stride - 1;   // image row of tile row 0
  const int d_bytes = p.M2 * 128 * kChunkRowBytes;

  if (tid == 0) {
    *abort_flag = 0u;
    mbar_init(bar_x, 1);
    mbar_init(bar_e + 0, 1);
    mbar_init(bar_e + 1, 1);
    mbar_init(bar_d + 0, 1);
    mbar_init(bar_d + 1, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmap_x);
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  __syncthreads();
  if (tid == 0) {
    mbar_arrive_expect_tx(bar_x, (uint32_t)(p.P_in * p.row_bytes));
    tma_load_4d(sX, &tmap_x, bar_x, 0, -1, gh0, n);
  }

  // ---- stage weights and biases (generic proxy), in the operand layouts the MMAs read ----
  {
    const int chunks_per_row = p.row_bytes >> 4;
    for (int i = tid; i < p.Cexp * chunks_per_row; i += kThreads) {
      const int row = i / chunks_per_row, ch = i % chunks_per_row;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (ch * 8 < p.Cin) v = __ldg(reinterpret_cast<const uint4*>(p.w1 + (size_t)row * p.Cin + ch * 8));
      *reinterpret_cast<uint4*>(sW1 + swz_offset(row, ch, p.row_bytes)) = v;
    }
    for (int i = tid; i < p.NC * p.Coutp * 2; i += kThreads) {
      const int half = i & 1, row = (i >> 1) % p.Coutp, c = (i >> 1) / p.Coutp;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (row < p.Cout) v = __ldg(reinterpret_cast<const uint4*>(p.w3 + (size_t)row * p.Cexp + c * kChunk + half * 8));
      *reinterpret_cast<uint4*>(sW3 + c * p.Coutp * kChunkRowBytes + swz_offset(row, half, kChunkRowBytes)) = v;
    }
    for (int i = tid; i < 9 * p.Cexp; i += kThreads) sWd[i] = __bfloat162float(p.wd[i]);
    for (int i = tid; i < p.Cexp; i += kThreads) { sB1[i] = p.b1[i]; sBd[i] = p.bd[i]; }
    for (int i = tid; i < p.Coutp; i += kThreads) sB3[i] = i < p.Cout ? p.b3[i] : 0.0f;
  }
  fence_proxy_async_smem();
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;

  // Which of this thread's expand-tile rows are real in-image pixels (bit k: tile (warp>>2) + 2k).
  uint32_t inimg_mask = 0;
  for (int t = warp >> 2, k = 0; t < p.M1; t += 2, ++k) {
    const int pix = t * 128 + (warp & 3) * 32 + lane;
    const int ih = pix / p.IW, iw = pix % p.IW;
    const int gh = gh0 + ih;
    if (pix < p.P_in && gh >= 0 && gh < p.H && iw >= 1 && iw <= p.W) inimg_mask |= 1u << k;
  }

  mbar_wait(bar_x, 0, abort_flag, p.status, 0x101);

  const uint32_t idesc_e = make_idesc_bf16(128, kChunk);
  const uint32_t idesc_p = make_idesc_bf16(128, (uint32_t)p.Coutp);
  const uint32_t sbo_x = 8u * (uint32_t)p.row_bytes;
  const uint32_t x_addr = smem_u32(sX), w1_addr = smem_u32(sW1), d_addr = smem_u32(sD), w3_addr = smem_u32(sW3);

  auto issue_expand = [&](int c) {
    const int b = c & 1;
    for (int t = 0; t < p.M1; ++t) {
      for (int ks = 0; ks < p.Kp / 16; ++ks) {
        const uint64_t ad = make_smem_desc(x_addr + t * 128 * p.row_bytes + ks * 32, 0, sbo_x, p.swizzle);
        const uint64_t bd = make_smem_desc(w1_addr + c * kChunk * p.row_bytes + ks * 32, 0, sbo_x, p.swizzle);
        umma_bf16(tmem_base + p.ecol0 + (b * p.M1 + t) * kChunk, ad, bd, idesc_e, ks > 0);
      }
    }
    umma_commit(bar_e + b);
  };

  if (tid == 0) issue_expand(0);

  for (int c = 0; c < p.NC; ++c) {
    const int b = c & 1;
    if (tid == 0 && c + 1 < p.NC) {
      tcgen05_fence_after_sync();
      issue_expand(c + 1);
    }
    mbar_wait(bar_e + b, (c >> 1) & 1, abort_flag, p.status, 0x102);
    tcgen05_fence_after_sync();

    // ---- P3: expand epilogue -> E chunk [pixel][16 ch] bf16, 32-byte rows, swizzled ----
    for (int t = warp >> 2, k = 0; t < p.M1; t += 2, ++k) {
      uint32_t acc[16];
      tmem_ld_x16(tmem_base + lane_base + p.ecol0 + (b * p.M1 + t) * kChunk, acc);
      tmem_ld_wait();
      const int pix = t * 128 + (warp & 3) * 32 + lane;
      if (pix < p.P_in) {
        uint32_t w[8];
        if ((inimg_mask >> k) & 1u) {
          const float4* bb = reinterpret_cast<const float4*>(sB1 + c * kChunk);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float4 bv = bb[j];
            w[2 * j] = pack_bf16x2(relu6f(__uint_as_float(acc[4 * j]) + bv.x), relu6f(__uint_as_float(acc[4 * j + 1]) + bv.y));
            w[2 * j + 1] = pack_bf16x2(relu6f(__uint_as_float(acc[4 * j + 2]) + bv.z), relu6f(__uint_as_float(acc[4 * j + 3]) + bv.w));
          }
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j) w[j] = 0u;
        }
        const uint32_t flip = (pix >> 2) & 1u;
        uint8_t* row = sE + pix * kChunkRowBytes;
        *reinterpret_cast<uint4*>(row + ((0u ^ flip) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4*>(row + ((1u ^ flip) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
      }
    }
    tcgen05_fence_before_sync();
    __syncthreads();

    // D[b] was read by the project MMA of chunk c-2
    if (c >= 2) mbar_wait(bar_d + b, ((c - 2) >> 1) & 1, abort_flag, p.status, 0x103);

    // ---- P4: depthwise 3x3 + bias + ReLU6 on CUDA cores: E chunk -> D[b] (A operand of the project GEMM) ----
    {
      uint8_t* dD = sD + b * d_bytes;
      const int cg = tid & 1;                      // which 8 of the chunk's 16 channels
      const int cbase = c * kChunk + cg * 8;
      float wgt[9][8];
#pragma unroll
      for (int tap = 0; tap < 9; ++tap) {
        const float4 a = *reinterpret_cast<const float4*>(sWd + tap * p.Cexp + cbase);
        const float4 bq = *reinterpret_cast<const float4*>(sWd + tap * p.Cexp + cbase + 4);
        wgt[tap][0] = a.x; wgt[tap][1] = a.y; wgt[tap][2] = a.z; wgt[tap][3] = a.w;
        wgt[tap][4] = bq.x; wgt[tap][5] = bq.y; wgt[tap][6] = bq.z; wgt[tap][7] = bq.w;
      }
      float bias[8];
      {
        const float4 a = *reinterpret_cast<const float4*>(sBd + cbase);
        const float4 bq = *reinterpret_cast<const float4*>(sBd + cbase + 4);
        bias[0] = a.x; bias[1] = a.y; bias[2] = a.z; bias[3] = a.w;
        bias[4] = bq.x; bias[5] = bq.y; bias[6] = bq.z; bias[7] = bq.w;
      }
      const int nitems = 2 * p.Wo * rows_valid;
      for (int item = tid; item < nitems; item += kThreads) {
        const int rest = item >> 1;
        const int wo = rest % p.Wo, r = rest / p.Wo;
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = bias[j];
#pragma unroll
        for (int kr = 0; kr < 3; ++kr) {
#pragma unroll
          for (int ks = 0; ks < 3; ++ks) {
            const int pe = (r * p.stride + kr) * p.IW + wo * p.stride + ks;
            const uint4 v = *reinterpret_cast<const uint4*>(sE + pe * kChunkRowBytes + ((cg ^ ((pe >> 2) & 1)) << 4));
            const float* wv = wgt[kr * 3 + ks];
            acc[0] = fmaf(bf16_lo(v.x), wv[0], acc[0]); acc[1] = fmaf(bf16_hi(v.x), wv[1], acc[1]);
            acc[2] = fmaf(bf16_lo(v.y), wv[2], acc[2]); acc[3] = fmaf(bf16_hi(v.y), wv[3], acc[3]);
            acc[4] = fmaf(bf16_lo(v.z), wv[4], acc[4]); acc[5] = fmaf(bf16_hi(v.z), wv[5], acc[5]);
            acc[6] = fmaf(bf16_lo(v.w), wv[6], acc[6]); acc[7] = fmaf(bf16_hi(v.w), wv[7], acc[7]);
          }
        }
        const int po = r * p.Wo + wo;
        const uint4 o = make_uint4(pack_bf16x2(relu6f(acc[0]), relu6f(acc[1])), pack_bf16x2(relu6f(acc[2]), relu6f(acc[3])),
                                   pack_bf16x2(relu6f(acc[4]), relu6f(acc[5])), pack_bf16x2(relu6f(acc[6]), relu6f(acc[7])));
        *reinterpret_cast<uint4*>(dD + po * kChunkRowBytes + ((cg ^ ((po >> 2) & 1)) << 4)) = o;
      }
    }
    fence_proxy_async_smem();
    __syncthreads();

    // ---- P5: project GEMM accumulates this chunk ----
    if (tid == 0) {
      tcgen05_fence_after_sync();
      for (int t = 0; t < p.M2; ++t) {
        const uint64_t ad = make_smem_desc(d_addr + b * d_bytes + t * 128 * kChunkRowBytes, 0, 256, SW_32B);
        const uint64_t bd = make_smem_desc(w3_addr + c * p.Coutp * kChunkRowBytes, 0, 256, SW_32B);
        umma_bf16(tmem_base + p.pcol0 + t * p.Coutp, ad, bd, idesc_p, c > 0);
      }
      umma_commit(bar_d + b);
    }
  }

  // ---- P6: project epilogue: + b3 (+ residual), bf16, 16-byte stores ----
  {
    const int last = p.NC - 1;
    mbar_wait(bar_d + (last & 1), (last >> 1) & 1, abort_flag, p.status, 0x104);
    tcgen05_fence_after_sync();
    const int valid_pix = rows_valid * p.Wo;
    const size_t gpix0 = ((size_t)n * p.Ho + ho0) * p.Wo;
    for (int t = warp >> 2; t < p.M2; t += 2) {
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
  q.off_e = take(q.P_in * kChunkRowBytes);
  q.off_d = take(2 * q.M2 * 128 * kChunkRowBytes);
  q.off_w3 = take(q.NC * q.Coutp * kChunkRowBytes);
  q.off_wd = take(9 * q.Cexp * 4);
  q.off_b1 = take(q.Cexp * 4);
  q.off_bd = take(q.Cexp * 4);
  q.off_b3 = take(q.Coutp * 4);
  q.off_bar = take(64);
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
