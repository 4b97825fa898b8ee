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
//   P1  the compute warps copy the NHWC input strip (with its row halo; rows
//       outside the image -> 0, channels padded to the MMA K granularity), W1
//       and W3 into swizzled K-major tiles with coalesced 16-byte loads -- all
//       loads of a thread are issued before its first store, so the prologue
//       is one round trip to device memory. (A pixel is Cin * 2 bytes there,
//       e.g. 48: one TMA box row per pixel was several times slower.)
//   for each 16-channel chunk c of the expanded tensor:
//     P2  tcgen05.mma: expand[pixels x 16] = X[pixels x Cin] * W1[c]^T   (TMEM, fp32)
//     P3  TMEM -> registers: + b1, ReLU6, zero outside the image (the depthwise
//         conv pads the post-activation tensor), bf16 -> shared memory; the
//         padding columns of the E chunk are written once
//     P4  CUDA cores: depthwise 3x3 + bd + ReLU6 over the resident chunk with
//         mixed-precision FMAs (bf16 activations and weights as stored, fp32
//         accumulate), result written as the K-major A operand of the project GEMM
//     P5  tcgen05.mma: out[pixels x Cout] += DW[pixels x 16] * W3[:, c]^T  (TMEM)
//   P6  TMEM -> registers: + b3 (+ x), bf16, 16-byte stores.
// The expand MMA of chunk c+1 is issued before the CUDA-core work of chunk c.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstdlib>

#include "dw_common.cuh"
#include "fused.h"
#include "tc_common.cuh"

namespace ago {

namespace {

using namespace tc;
using namespace dw;

constexpr int kWarps = 32;                         // every warp computes; MMAs are issued inline by some of them
constexpr int kThreads = kWarps * 32;
// The warps form NG groups (2 or 4) that own the chunks c = g, g + NG, ...: two groups of 16 warps for strips whose
// chunk is real work (their phases overlap), four groups of 8 warps for small strips, where a chunk is a chain of
// latencies (MMA hand-off, tensor-memory round trip, two barriers) and more chains in flight is all that helps.
constexpr int kTilesPerWarp = 2;                   // expand-epilogue tiles per warp: at most 8 tiles over the 4 warps of a lane quarter
constexpr int kExpandIssuers = 2;                  // the last two warps of a group issue its expand GEMMs
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
  int groups;                   // warp groups: 2 or 4 (the kernel template's NG)
  int fold_b1;                  // the expand bias rides in two spare reduction channels of the expand GEMM (Cin < Kp)
  int R, strips, IH, IW, P_x, P_in, M1, M2;   // P_x = IH * W pixels in the input tile, P_in = IH * IW in an E chunk
  int Kp, row_bytes, swizzle;   // input / W1 tiles: padded K, bytes per row, tc::SwizzleMode
  int Coutp, NC;
  // 2^32 / d + 1 for the run-time divisors of the index arithmetic: x / d == __umulhi(x, recip) for x, d < 65536
  uint32_t coutp_recip, w_recip, strips_recip, per_row_recip, cexp8_recip;   // cexp8: Cexp / 8 (>= 2)
  int per_row, nseg, step_r, step_c, col_slots;   // depthwise item geometry (see the kernel), fixed per shape
  int tmem_cols, ecol0, pcol0;
  int e_plane, d_plane;         // byte distance between the two 8-channel planes of an E / D chunk
  // shared-memory byte offsets (from the 1024-aligned base)
  int off_x, off_w1, off_e, off_d, off_w3, off_wd, off_b1, off_bd, off_b3, off_bar;
};

// 16-byte shared-memory accesses by 32-bit shared address (immediate byte offset for the load).
template <int OFF>
__device__ __forceinline__ float4 lds128f(uint32_t saddr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4+%5];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(saddr), "n"(OFF));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t saddr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(saddr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// FOLD: the expand bias rides in the expand GEMM (see the prologue). EXPAND / PROJECT select the pairs of the
// block: <true, true> the whole block, <true, false> pointwise -> depthwise
// (the depthwise result of every chunk goes to device memory), <false, true> depthwise -> pointwise (every chunk of
// the input is copied into the E buffers instead of being computed).
template <bool EXPAND, bool PROJECT, bool FOLD, int NG>
__global__ void __launch_bounds__(kThreads, 1)
mbv2_fused_kernel(const Mbv2Params p) {
  constexpr int kGroupWarps = kWarps / NG;
  constexpr int kGroupThreads = kGroupWarps * 32;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sX = smem + p.off_x;
  uint8_t* sW1 = smem + p.off_w1;
  uint8_t* sE = smem + p.off_e;
  uint8_t* sD = smem + p.off_d;
  uint8_t* sW3 = smem + p.off_w3;
  const uint8_t* sWd = smem + p.off_wd;                   // [chunk][9 taps][16 channels] bf16
  float* sB1 = reinterpret_cast<float*>(smem + p.off_b1);
  float* sBd = reinterpret_cast<float*>(smem + p.off_bd);
  float* sB3 = reinterpret_cast<float*>(smem + p.off_b3);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
  uint64_t* bar_e = bars;           // [NG] expand accumulators of group g complete (MMA commit)
  uint64_t* bar_d = bars + 8;       // [NG] project MMA has consumed D[g] (MMA commit)
  uint64_t* bar_first = bars + 16;  // project GEMM of chunk 0 complete (it overwrites the output accumulators: the other groups issue after it)
  uint64_t* bar_done = bars + 17;   // every project MMA complete (the groups do not follow each other's bar_d phases)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 18);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 19);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n = (int)fast_div(blockIdx.x, (uint32_t)p.strips, p.strips_recip), strip = (int)blockIdx.x - n * p.strips;
  const int ho0 = strip * p.R;
  const int rows_valid = min(p.R, p.Ho - ho0);
  const int gh0 = ho0 * p.stride - 1;   // image row of tile row 0
  const int d_bytes = 2 * p.d_plane;

  if (tid == kThreads - 1) {
    *abort_flag = 0u;
    for (int i = 0; i < NG; ++i) {
      mbar_init(bar_e + i, kExpandIssuers);
      mbar_init(bar_d + i, (uint32_t)p.M2);
    }
    mbar_init(bar_first, (uint32_t)p.M2);
    mbar_init(bar_done, (uint32_t)(p.M2 * min(p.NC, NG)));
    fence_mbar_init();
    fence_proxy_async_smem();
  }
    // ---- P1: stage the input strip, the weights and the biases. Every 16-byte chunk is one slot; a thread first
    // issues the loads of all its slots, then stores them, so that the whole prologue costs one round trip to
    // device memory. (Pixels are Cin * 2 bytes apart there: coalesced plain loads of the contiguous strip serve
    // that better than one TMA box row per pixel.) X and W1 rows go to their swizzled K-major tiles, zero beyond
    // Cin; W3 to one [Coutp x 16 channels] slice per chunk; depthwise weights and biases are copied as they are.
    constexpr int kBX = 4, kBW = 2;   // slots per thread in the first (batched) pass: input strip / everything else
    const int cs = p.Kp == 16 ? 1 : (p.Kp == 32 ? 2 : 3);   // log2(16-byte chunks per tile row)
    const uint32_t nX = EXPAND ? (uint32_t)p.P_x << cs : 0u, nW1 = EXPAND ? (uint32_t)p.Cexp << cs : 0u;
    const uint32_t nW3 = PROJECT ? (uint32_t)(p.NC * p.Coutp * 2) : 0u;
    const uint32_t nWd = 9u * p.Cexp / 8u, nB = (uint32_t)p.Cexp / 4u, nB1 = EXPAND ? nB : 0u, nB3 = PROJECT ? (uint32_t)p.Cout / 4u : 0u;
    const uint32_t nW = nW1 + nW3 + nWd + nB1 + nB + nB3;
    // tile pixel `pix` is image pixel gh0 * W + pix of image n (strips are full-width rows): in the image for pix in [pix_lo, pix_hi)
    const int pix_lo = max(0, -gh0 * p.W), pix_hi = min(p.P_x, (p.H - gh0) * p.W);
    const uint8_t* x0 = reinterpret_cast<const uint8_t*>(p.x) + ((size_t)n * p.H + gh0) * p.W * p.Cin * 2;   // not dereferenced outside the image
    const uint32_t cmask = (1u << cs) - 1u, cin_chunks = (uint32_t)p.Cin >> 3, cin_bytes = (uint32_t)p.Cin * 2u;
    const uint32_t swz_mask = ((uint32_t)p.row_bytes >> 4) - 1u;
    // X and W1: row-major [row][Cin] -> swizzled rows of Kp channels; chunk i of a tile lies at byte 16 i, its 16-byte
    // column XORed with the row's swizzle phase (address bits 7..). Returns the shared-memory offset; src = null: zeros.
    auto x_slot = [&](uint32_t i, const uint8_t*& src) -> uint32_t {
      const uint32_t row = i >> cs, ch = i & cmask;
      src = (ch < cin_chunks && (int)row >= pix_lo && (int)row < pix_hi) ? x0 + row * cin_bytes + ch * 16u : nullptr;
      if (FOLD && ch == cin_chunks) src = reinterpret_cast<const uint8_t*>(uintptr_t(1));   // two channels of 1.0 (tag 1)
      return p.off_x + ((i << 4) ^ (((i >> 3) & swz_mask) << 4));
    };
    auto w_slot = [&](uint32_t i, const uint8_t*& src) -> uint32_t {
      if (i < nW1) {
        const uint32_t row = i >> cs, ch = i & cmask;
        src = ch < cin_chunks ? reinterpret_cast<const uint8_t*>(p.w1) + row * cin_bytes + ch * 16u : nullptr;
        if (FOLD && ch == cin_chunks) src = reinterpret_cast<const uint8_t*>(reinterpret_cast<uintptr_t>(p.b1 + row) | 2u);   // the bias (tag 2)
        return p.off_w1 + ((i << 4) ^ (((i >> 3) & swz_mask) << 4));
      }
      if ((i -= nW1) < nW3) {
        const uint32_t half = i & 1u, c = __umulhi(i >> 1, p.coutp_recip), row = (i >> 1) - c * p.Coutp;
        src = row < (uint32_t)p.Cout ? reinterpret_cast<const uint8_t*>(p.w3) + (row * p.Cexp + c * kChunk + half * 8u) * 2u : nullptr;
        return p.off_w3 + c * p.Coutp * kChunkRowBytes + swz_offset(row, half, kChunkRowBytes);
      }
      if ((i -= nW3) < nWd) {   // [tap][Cexp] in device memory -> [chunk][tap][16 channels]: a thread's nine taps lie 32 bytes apart
        const uint32_t tap = __umulhi(i, p.cexp8_recip), c8 = i - tap * ((uint32_t)p.Cexp >> 3);
        src = reinterpret_cast<const uint8_t*>(p.wd) + i * 16u;
        return p.off_wd + (c8 >> 1) * (9u * kChunkRowBytes) + tap * kChunkRowBytes + (c8 & 1u) * 16u;
      }
      if ((i -= nWd) < nB1) { src = reinterpret_cast<const uint8_t*>(p.b1) + i * 16u; return p.off_b1 + i * 16u; }
      if ((i -= nB1) < nB) { src = reinterpret_cast<const uint8_t*>(p.bd) + i * 16u; return p.off_bd + i * 16u; }
      i -= nB;
      src = reinterpret_cast<const uint8_t*>(p.b3) + i * 16u;
      return p.off_b3 + i * 16u;
    };
    // A slot's source: a 16-byte aligned address (or null: zeros); tag 1: the two channels of ones that multiply the
    // folded bias; tag 2: the address of one fp32 bias, split into bf16 high and low parts (their sum carries 16
    // mantissa bits, and 1.0 * part is exact in the fp32 accumulator).
    auto load_or_zero = [](const uint8_t* src) {
      const uintptr_t a = reinterpret_cast<uintptr_t>(src);
      if (!FOLD || (a & 3u) == 0u) return src ? __ldg(reinterpret_cast<const uint4*>(src)) : make_uint4(0, 0, 0, 0);
      if ((a & 3u) == 1u) return make_uint4(0x3F803F80u, 0, 0, 0);
      const float b = __ldg(reinterpret_cast<const float*>(a & ~uintptr_t(3)));
      const __nv_bfloat16 hi = __float2bfloat16_rn(b);
      const __nv_bfloat16 lo = __float2bfloat16_rn(b - __bfloat162float(hi));
      return make_uint4((uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(lo) << 16), 0, 0, 0);
    };
    // ---- per-thread work mapping: needs no device memory, so it runs before the wait for the previous grid of the
    // stream (with back-to-back launches it overlaps that grid's tail) ----
    const int g = warp / kGroupWarps;
    const int gwarp0 = g * kGroupWarps;           // first warp of the group
    const int gt = tid - gwarp0 * 32;             // thread index in the group
    const uint32_t gbar = 1u + (uint32_t)g;       // named barrier of the group
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const int gw = warp - gwarp0;                 // warp index in the group
    const int xi = gw - (kGroupWarps - kExpandIssuers);   // >= 0: this warp issues expand tiles xi, xi + 2, ...
    // Depthwise work split: thread = (channel pair, slot). Stride 1: an item is a block of 2 output rows x 7 output
    // columns (56 columns x 14 rows x 8 pairs = one item per thread of a group). Stride 2: an item is one output column
    // of one row group.
    constexpr int kSlots = kGroupThreads / 8;
    const int cp = gt & 7, slot = gt >> 3;
    const int cp_off = (cp & 3) * 4;   // byte offset inside a 16-byte pixel entry
    const uint32_t e_pitch = (uint32_t)p.IW * 16u, d_pitch = (uint32_t)p.Wo * 16u;
    const int per_row = p.per_row;                                         // items per output row (stride 1: column segments) / per row group
    int groups = 1, rows_per_group = rows_valid;                           // stride 2: row groups
    if (p.stride != 1) {
      groups = max(1, min(rows_valid, p.col_slots));
      rows_per_group = (rows_valid + groups - 1) / groups;
    }
    const int dw_items = per_row * (p.stride == 1 ? (rows_valid + 1) / 2 : groups);   // stride 1: blocks of two rows
    const int item0_r = (int)fast_div((uint32_t)slot, (uint32_t)per_row, p.per_row_recip), item0_c = slot - item0_r * per_row;   // the thread's first item
    const int step_r = p.step_r, step_c = p.step_c;                        // item += kSlots in (row, column) form
    const int e_bytes = 2 * p.e_plane;
    // Expand-epilogue tiles of this warp: the group's warps of one tensor-memory lane quarter (warp & 3) share the M1
    // tiles round-robin, at most kTilesPerWarp each. e_pix[k]: pixel index in an E plane (the tile has no padding
    // columns, the E chunk does), -1: no such pixel; bit k of e_inimg: the row lies inside the image (the rest is the
    // zero padding of the intermediate tensor).
    const int q_first = (((warp & 3) - gwarp0) & 3);                // group-relative index of the quarter's first warp
    const int q_mates = (kGroupWarps - q_first + 3) >> 2;           // warps of this quarter in the group (3 or 4)
    const int q_rank = (warp - gwarp0 - q_first) >> 2;              // this warp's rank among them
    constexpr uint32_t kNone = 0xffffffffu;
    uint32_t e_off[kTilesPerWarp];   // shared-memory address of the thread's pixel in plane 0 of the group's E buffer
    uint32_t e_inimg = 0;
#pragma unroll
    for (int k = 0; k < kTilesPerWarp; ++k) {
      const int t = q_rank + k * q_mates;
      const int pix = t * 128 + (warp & 3) * 32 + lane;
      const int ih = (int)fast_div((uint32_t)pix, (uint32_t)p.W, p.w_recip), iw = pix - ih * p.W;
      const int gh = gh0 + ih;
      e_off[k] = kNone;
      if (t < p.M1 && pix < p.P_x) {
        e_off[k] = smem_u32(sE) + (uint32_t)(g * e_bytes + (ih * p.IW + iw + 1) * 16);
        if (gh >= 0 && gh < p.H) e_inimg |= 1u << k;
      }
    }

    uint4 vx[kBX], vw[kBW];
    uint32_t dx[kBX], dw[kBW];
    // Without the expand GEMM a chunk is 16 channels of the input strip, copied asynchronously into one of the
    // group's two E buffers two chunks ahead: 16-byte pieces (pixel, 8-channel plane), rows outside the image
    // zero-filled. The piece geometry is the same for every chunk.
    constexpr int kPieces = 4;                      // P_x * 2 pieces <= 8 tiles * 128 * 2 over the group's threads
    uint32_t ld_src[kPieces], ld_dst[kPieces], ld_ok = 0u, ld_in = 0u;
    const uint8_t* xin = reinterpret_cast<const uint8_t*>(p.x) + ((int64_t)n * p.H + gh0) * p.W * p.Cexp * 2;   // row gh0 may lie outside
    if (!EXPAND) {
#pragma unroll
      for (int k = 0; k < kPieces; ++k) {
        const int i = gt + k * kGroupThreads;
        ld_src[k] = 0u; ld_dst[k] = 0u;
        if (i < p.P_x * 2) {
          const int pix = i >> 1, plane = i & 1;
          const int ih = (int)fast_div((uint32_t)pix, (uint32_t)p.W, p.w_recip), iw = pix - ih * p.W;
          ld_ok |= 1u << k;
          ld_dst[k] = (uint32_t)(plane * p.e_plane + (ih * p.IW + iw + 1) * 16);
          if (gh0 + ih >= 0 && gh0 + ih < p.H) { ld_in |= 1u << k; ld_src[k] = (uint32_t)(pix * p.Cexp * 2 + plane * 16); }
        }
      }
    }
    auto load_chunk = [&](int c, int b) {   // chunk c -> E buffer (g, b); always one commit group
      if (c < p.NC) {
        const uint32_t e0 = smem_u32(sE) + (uint32_t)((g * 2 + b) * e_bytes);   // two buffers per group
#pragma unroll
        for (int k = 0; k < kPieces; ++k) {
          if ((ld_ok >> k) & 1u) {
            const bool in = (ld_in >> k) & 1u;
            cp_async_16(e0 + ld_dst[k], in ? xin + ld_src[k] + c * kChunkRowBytes : reinterpret_cast<const uint8_t*>(p.x), in ? 16u : 0u);
          }
        }
      }
      cp_async_commit();
    };
    grid_dependency_wait();      // first access to device memory below
    grid_launch_dependents();
    if (!EXPAND) { load_chunk(g, 0); load_chunk(g + NG, 1); }   // the first two chunks travel while the weights are staged
#pragma unroll
    for (int k = 0; k < kBX; ++k) {
      const uint32_t i = (uint32_t)(tid + k * kThreads);
      const uint8_t* src = nullptr;
      dx[k] = 0xffffffffu;
      if (i < nX) dx[k] = x_slot(i, src);
      vx[k] = load_or_zero(src);
    }
#pragma unroll
    for (int k = 0; k < kBW; ++k) {
      const uint32_t i = (uint32_t)(tid + k * kThreads);
      const uint8_t* src = nullptr;
      dw[k] = 0xffffffffu;
      if (i < nW) dw[k] = w_slot(i, src);
      vw[k] = load_or_zero(src);
    }
    if (warp == 0) {
      tmem_alloc(tmem_slot, (uint32_t)p.tmem_cols);
      tmem_relinquish();
    }
#pragma unroll
    for (int k = 0; k < kBX; ++k)
      if (dx[k] != 0xffffffffu) *reinterpret_cast<uint4*>(smem + dx[k]) = vx[k];
#pragma unroll
    for (int k = 0; k < kBW; ++k)
      if (dw[k] != 0xffffffffu) *reinterpret_cast<uint4*>(smem + dw[k]) = vw[k];
    // shapes with more slots than the batched pass covers
    for (uint32_t i = (uint32_t)(tid + kBX * kThreads); i < nX; i += kThreads) {
      const uint8_t* src;
      const uint32_t d = x_slot(i, src);
      *reinterpret_cast<uint4*>(smem + d) = load_or_zero(src);
    }
    for (uint32_t i = (uint32_t)(tid + kBW * kThreads); i < nW; i += kThreads) {
      const uint8_t* src;
      const uint32_t d = w_slot(i, src);
      *reinterpret_cast<uint4*>(smem + d) = load_or_zero(src);
    }
    // the zero padding columns of the two E chunk buffers (written once: every chunk reuses them)
    constexpr int kEPlanes = (EXPAND ? NG : 2 * NG) * 2;   // one E buffer per group (two when the chunks are copied in), two planes each
    for (int i = tid; i < p.IH * 2 * kEPlanes; i += kThreads) {
      const int ih = i / (2 * kEPlanes), side = (i / kEPlanes) & 1, plane = i % kEPlanes;
      *reinterpret_cast<uint4*>(sE + plane * p.e_plane + (ih * p.IW + side * (p.IW - 1)) * 16) = make_uint4(0, 0, 0, 0);
    }
    fence_proxy_async_smem();
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

    // The warps form two groups of 16; group g owns the chunks c = g, g + 2, ... (expand buffer, E buffer and D
    // buffer g). A group alternates expand epilogue and depthwise stage with a group-wide barrier after each; the two
    // groups are out of phase, so one group's barrier and tensor-memory latencies hide behind the other's arithmetic.
    // MMAs are issued inline, right after the barrier that makes their operands ready: the expand GEMM of chunk c + 2
    // by the group's last two warps (at 56 x 56 they have no depthwise item), the project GEMM of chunk c by M2 warps,
    // one tile each -- a parked issuer warp would share its scheduler with busy warps and issue an MMA every few
    // hundred cycles, and the project GEMM is urgent: it must be through before the depthwise stage of chunk c + 2
    // may overwrite its operand.
    // Descriptors as (low, high) words: start address and LBO live in the low word, so an operand advances with one
    // 32-bit add (shared-memory addresses >> 4 stay below the 14-bit field limit).
    uint32_t e_tm[kTilesPerWarp];   // tensor-memory address of this warp's k-th expand tile (buffer g)
#pragma unroll
    for (int k = 0; k < kTilesPerWarp; ++k) {
      const int t = q_rank + k * q_mates;
      e_tm[k] = t < p.M1 ? tmem_base + lane_base + p.ecol0 + (g * p.M1 + t) * kChunk : kNone;
    }
    const uint32_t sbo_x = 8u * (uint32_t)p.row_bytes;
    const uint64_t xdesc0 = make_smem_desc(smem_u32(sX), 0, sbo_x, p.swizzle);
    const uint64_t w1desc0 = make_smem_desc(smem_u32(sW1), 0, sbo_x, p.swizzle);
    // D: un-swizzled K-major; the two 8-channel planes are the two K core-matrix columns
    const uint64_t ddesc0 = make_smem_desc(smem_u32(sD), (uint32_t)p.d_plane, 128, SW_NONE);
    const uint64_t w3desc0 = make_smem_desc(smem_u32(sW3), 0, 256, SW_32B);
    // MMAs are issued by whole, converged warps: the MMA itself is predicated on one elected lane, its descriptors are
    // ready 64-bit values (see tc_common.cuh: several times the issue rate of a lane-0 branch next to busy warps).
    const uint32_t elected = elect_one();
    // Expand issue state of the group's last two warps: tiles xi, xi + 2, ... of the group's chunks -> buffer g.
    const uint32_t idesc_e = make_idesc_bf16(128, kChunk);
    const uint64_t exp_a_step = (uint64_t)((uint32_t)(kExpandIssuers * 128 * p.row_bytes) >> 4);
    const uint64_t exp_a0 = xdesc0 + (uint64_t)((uint32_t)(max(xi, 0) * 128 * p.row_bytes) >> 4);
    const uint32_t exp_d_tmem0 = tmem_base + p.ecol0 + (g * p.M1 + max(xi, 0)) * kChunk;
    const uint64_t exp_b_step = (uint64_t)((uint32_t)(NG * kChunk * p.row_bytes) >> 4);   // the group's next chunk is c + NG
    uint64_t exp_b = w1desc0 + (uint64_t)((uint32_t)(g * kChunk * p.row_bytes) >> 4);
    const int ksteps = p.Kp / 16;
    const int exp_tiles = xi >= 0 ? (p.M1 - xi + kExpandIssuers - 1) / kExpandIssuers : 0;   // tiles this warp issues per chunk
    auto issue_expand = [&]() {   // whole warp; advances to the group's next chunk. Straight-line per reduction length.
      uint64_t a = exp_a0;
      uint32_t d_tmem = exp_d_tmem0;
      const uint64_t b = exp_b;
      if (ksteps == 2) {
#pragma unroll 1
        for (int t = 0; t < exp_tiles; ++t, a += exp_a_step, d_tmem += kExpandIssuers * kChunk) {
          umma_bf16_elected<false>(d_tmem, a, b, idesc_e, elected);
          umma_bf16_elected<true>(d_tmem, a + 2u, b + 2u, idesc_e, elected);
        }
      } else if (ksteps == 4) {
#pragma unroll 1
        for (int t = 0; t < exp_tiles; ++t, a += exp_a_step, d_tmem += kExpandIssuers * kChunk) {
          umma_bf16_elected<false>(d_tmem, a, b, idesc_e, elected);
          umma_bf16_elected<true>(d_tmem, a + 2u, b + 2u, idesc_e, elected);
          umma_bf16_elected<true>(d_tmem, a + 4u, b + 4u, idesc_e, elected);
          umma_bf16_elected<true>(d_tmem, a + 6u, b + 6u, idesc_e, elected);
        }
      } else {
#pragma unroll 1
        for (int t = 0; t < exp_tiles; ++t, a += exp_a_step, d_tmem += kExpandIssuers * kChunk)
          umma_bf16_elected<false>(d_tmem, a, b, idesc_e, elected);
      }
      umma_commit_elected(bar_e + g, elected);
      exp_b += exp_b_step;
    };
    // Project issue state of warp gw < M2 (tile gw), kept in three registers: a warp that runs a serial instruction
    // chain next to warps with dense arithmetic gets an issue slot only every few tens of cycles, so the path from
    // the barrier to the MMA is one add, the MMA and the commit.
    const uint32_t idesc_p = make_idesc_bf16(128, (uint32_t)p.Coutp);
    const uint64_t proj_a = ddesc0 + (uint64_t)((uint32_t)(g * d_bytes + gw * 128 * 16) >> 4);
    const uint32_t proj_d_tmem = tmem_base + p.pcol0 + gw * p.Coutp;
    const uint64_t proj_b_step = (uint64_t)((uint32_t)(NG * p.Coutp * kChunkRowBytes) >> 4);     // the group's next chunk is c + NG
    uint64_t proj_b = w3desc0 + (uint64_t)((uint32_t)(g * p.Coutp * kChunkRowBytes) >> 4);
    if (EXPAND && xi >= 0 && g < p.NC) {
      // group 1 issues its first expand GEMM once group 0's is through the tensor pipe: group 0 has the longer chain
      // of chunks, and its first epilogue would otherwise wait for both groups' MMAs
      // (with more than two groups the strips are small, the products short, and a chain of first products would cost
      // more than it saves; a waiter that falls two phases behind a barrier would also read the wrong parity)
      if (NG == 2 && g == 1) {
        if (lane == 0) mbar_wait(bar_e, 0, abort_flag, p.status, 0x107);
        __syncwarp();
      }
      issue_expand();
    }
    __syncwarp();
    // Waits on MMA completion are taken by ONE warp of the group, just before it arrives at the group barrier that
    // the others are parked at: a polling warp spends issue slots, sixteen of them a large share of the SM's.
    const bool waiter = gw == kGroupWarps - 1;
    if (EXPAND && g < p.NC) {
      if (waiter) mbar_wait(bar_e + g, 0, abort_flag, p.status, 0x102);   // the group's first expand GEMM
      named_barrier_sync(gbar, kGroupThreads);
    }
    // The thread's first depthwise item (for most shapes its only one) is the same for every chunk: offsets of its
    // first input / output pixel inside a plane and its extent (stride 1: columns, rows; stride 2: first and last row).
    const bool has_item = slot < dw_items;
    uint32_t it_e, it_d; int it_a, it_b;
    if (p.stride == 1) {
      const int wo = item0_c * kSegCols;
      it_e = (uint32_t)(2 * item0_r) * e_pitch + wo * 16; it_d = (uint32_t)(2 * item0_r) * d_pitch + wo * 16;
      it_a = min(kSegCols, p.Wo - wo); it_b = min(2, rows_valid - 2 * item0_r);
    } else {
      it_e = item0_c * 32; it_d = item0_c * 16;
      it_a = item0_r * rows_per_group; it_b = min(rows_valid, it_a + rows_per_group);
    }
    const uint32_t e_plane0 = smem_u32(sE) + (uint32_t)((EXPAND ? g : g * 2) * e_bytes + (cp >> 2) * p.e_plane + cp_off);
    const uint32_t d_plane = smem_u32(sD) + (uint32_t)(g * d_bytes + (cp >> 2) * p.d_plane + cp_off);
    // running shared-memory addresses of this thread's depthwise weights / bias and of the chunk's expand bias
    uint32_t wd_addr = smem_u32(sWd) + (uint32_t)(g * 9 * kChunkRowBytes + cp * 4);
    uint32_t bd_addr = smem_u32(sBd) + (uint32_t)((g * kChunk + cp * 2) * 4);
    uint32_t b1_addr = smem_u32(sB1) + (uint32_t)(g * kChunk * 4);
    for (int c = g, it = 0; c < p.NC; c += NG, ++it) {
      // ---- P3: expand epilogue of chunk c -> E[g]: + b1, ReLU6, zero outside the image, bf16 ----
      if (!EXPAND) cp_async_wait_but_one();   // this thread's pieces of chunk c have landed
      if (EXPAND) {
      tcgen05_fence_after_sync();
#pragma unroll
      for (int k = 0; k < kTilesPerWarp; ++k) {
        if (e_tm[k] == kNone) break;   // warp-uniform
        uint32_t acc[16];
        tmem_ld_x16(e_tm[k], acc);
        tmem_ld_wait();
        if (e_off[k] != kNone) {
          uint32_t w[8];
          if (FOLD && ((e_inimg >> k) & 1u)) {   // the bias came out of the expand GEMM
#pragma unroll
            for (int j = 0; j < 8; ++j) w[j] = relu6_pack(__uint_as_float(acc[2 * j]), __uint_as_float(acc[2 * j + 1]));
          } else if ((e_inimg >> k) & 1u) {
            const float4 b0 = lds128f<0>(b1_addr), b1v = lds128f<16>(b1_addr), b2 = lds128f<32>(b1_addr), b3v = lds128f<48>(b1_addr);
            w[0] = relu6_pack(__uint_as_float(acc[0]) + b0.x, __uint_as_float(acc[1]) + b0.y);
            w[1] = relu6_pack(__uint_as_float(acc[2]) + b0.z, __uint_as_float(acc[3]) + b0.w);
            w[2] = relu6_pack(__uint_as_float(acc[4]) + b1v.x, __uint_as_float(acc[5]) + b1v.y);
            w[3] = relu6_pack(__uint_as_float(acc[6]) + b1v.z, __uint_as_float(acc[7]) + b1v.w);
            w[4] = relu6_pack(__uint_as_float(acc[8]) + b2.x, __uint_as_float(acc[9]) + b2.y);
            w[5] = relu6_pack(__uint_as_float(acc[10]) + b2.z, __uint_as_float(acc[11]) + b2.w);
            w[6] = relu6_pack(__uint_as_float(acc[12]) + b3v.x, __uint_as_float(acc[13]) + b3v.y);
            w[7] = relu6_pack(__uint_as_float(acc[14]) + b3v.z, __uint_as_float(acc[15]) + b3v.w);
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) w[j] = 0u;
          }
          sts128(e_off[k], w[0], w[1], w[2], w[3]);
          sts128(e_off[k] + (uint32_t)p.e_plane, w[4], w[5], w[6], w[7]);
        }
      }
      b1_addr += (uint32_t)NG * kChunk * 4u;
      tcgen05_fence_before_sync();
      }
      // D[g] was read by the project GEMM of chunk c - 2
      if (PROJECT && waiter && it >= 1) mbar_wait(bar_d + g, (uint32_t)(it - 1) & 1u, abort_flag, p.status, 0x103);
      named_barrier_sync(gbar, kGroupThreads);
      if (EXPAND && xi >= 0 && c + NG < p.NC) {   // expand buffer g is drained: the expand GEMM of the group's next chunk
        tcgen05_fence_after_sync();
        issue_expand();
      }

      // ---- P4: depthwise 3x3 + bias + ReLU6 on CUDA cores: E[g] -> D[g] (A operand of the project GEMM) ----
      {
        uint32_t wgt[9];   // packed bf16 pairs
        wgt[0] = lds32<0>(wd_addr); wgt[1] = lds32<32>(wd_addr); wgt[2] = lds32<64>(wd_addr);
        wgt[3] = lds32<96>(wd_addr); wgt[4] = lds32<128>(wd_addr); wgt[5] = lds32<160>(wd_addr);
        wgt[6] = lds32<192>(wd_addr); wgt[7] = lds32<224>(wd_addr); wgt[8] = lds32<256>(wd_addr);
        const float2 bias = make_float2(__uint_as_float(lds32<0>(bd_addr)), __uint_as_float(lds32<4>(bd_addr)));
        wd_addr += (uint32_t)NG * 9u * kChunkRowBytes; bd_addr += (uint32_t)NG * kChunk * 4u;   // the group's next chunk is c + NG
        const uint32_t e_plane = e_plane0 + (EXPAND ? 0u : (uint32_t)((it & 1) * e_bytes));
        if (has_item) {   // the thread's first item: geometry fixed before the chunk loop
          if (p.stride == 1) depthwise_block(e_plane + it_e, d_plane + it_d, e_pitch, d_pitch, it_a, it_b, wgt, bias);
          else if (it_a < it_b) depthwise_column_s2(e_plane + it_e, d_plane + it_d, it_a, it_b, p.IW, p.Wo, wgt, bias);
        }
        if (dw_items > kSlots) {   // shapes with more items than slots
          int r = item0_r + step_r, col = item0_c + step_c;
          if (col >= per_row) { col -= per_row; ++r; }
          for (int item = slot + kSlots; item < dw_items; item += kSlots) {
            if (p.stride == 1) {
              const int wo = col * kSegCols;
              depthwise_block(e_plane + (uint32_t)(2 * r) * e_pitch + wo * 16, d_plane + (uint32_t)(2 * r) * d_pitch + wo * 16, e_pitch,
                              d_pitch, min(kSegCols, p.Wo - wo), min(2, rows_valid - 2 * r), wgt, bias);
            } else {
              const int r0 = r * rows_per_group, r1 = min(rows_valid, r0 + rows_per_group);
              if (r0 < r1) depthwise_column_s2(e_plane + col * 32, d_plane + col * 16, r0, r1, p.IW, p.Wo, wgt, bias);
            }
            r += step_r; col += step_c;
            if (col >= per_row) { col -= per_row; ++r; }
          }
        }
      }
      fence_proxy_async_smem();
      // the expand GEMM of the group's next chunk (issued after the previous barrier) is complete
      if (EXPAND && waiter && c + NG < p.NC) mbar_wait(bar_e + g, (uint32_t)(it + 1) & 1u, abort_flag, p.status, 0x102);
      named_barrier_sync(gbar, kGroupThreads);
      if (!EXPAND) load_chunk(c + 2 * NG, it & 1);   // the E buffer of chunk c is free
      if (!PROJECT) {
        // the depthwise result of the chunk is the output: 16-byte pieces (pixel, plane) of D[g] to device memory
        const int pieces = rows_valid * p.Wo * 2;
        __nv_bfloat16* o0 = p.out + ((size_t)n * p.Ho + ho0) * p.Wo * p.Cexp + c * kChunk;
        for (int i = gt; i < pieces; i += kGroupThreads) {
          const int pix = i >> 1, plane = i & 1;
          *reinterpret_cast<uint4*>(o0 + (size_t)pix * p.Cexp + plane * 8) =
              *reinterpret_cast<const uint4*>(sD + g * d_bytes + plane * p.d_plane + pix * 16);
        }
      }
      if (PROJECT && gw < p.M2) {   // D[g] is complete: the project GEMM of chunk c, one tile per warp
        // chunk 0 overwrites the accumulators: everything else is issued after it
        if (c >= 1 && c < NG) {
          if (lane == 0) mbar_wait(bar_first, 0, abort_flag, p.status, 0x106);
          __syncwarp();
        }
        tcgen05_fence_after_sync();
        umma_bf16_elected_acc(proj_d_tmem, proj_a, proj_b, idesc_p, elected, c > 0 ? 1u : 0u);
        umma_commit_elected(bar_d + g, elected);
        if (c == 0) umma_commit_elected(bar_first, elected);
        if (c + NG >= p.NC && !skip_signal_for_test(p.status, 0x104)) umma_commit_elected(bar_done, elected);
      }
      proj_b += proj_b_step;
    }

    // ---- P6: project epilogue: + b3 (+ residual), bf16, 16-byte stores ----
    if (PROJECT) {
      if (warp == kWarps - 1) mbar_wait(bar_done, 0, abort_flag, p.status, 0x104);
      __syncthreads();
      tcgen05_fence_after_sync();
      const int valid_pix = rows_valid * p.Wo;
      const size_t gpix0 = ((size_t)n * p.Ho + ho0) * p.Wo;
      for (int t = warp >> 2; t < p.M2; t += kWarps / 4) {
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
                if (EXPAND && p.residual) {
                  // stride 1, Cin == Cout: output pixel po is pixel po + W of the input tile (one halo row above)
                  const uint4 xr = *reinterpret_cast<const uint4*>(sX + swz_offset(po + p.W, j >> 3, p.row_bytes));
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
  bool expand = true, project = true;
};

bool layout(Mbv2Params& q, int R, bool expand, bool project, int* smem_bytes) {
  const int NG = q.groups, group_threads = kThreads / NG;
  q.R = R;
  q.strips = (q.Ho + R - 1) / R;
  q.strips_recip = fast_div_recip(q.strips);
  q.IH = (R - 1) * q.stride + 3;
  q.IW = q.W + 2;
  q.P_in = q.IH * q.IW;
  q.P_x = q.IH * q.W;
  q.M1 = (q.P_x + 127) / 128;
  q.M2 = (R * q.Wo + 127) / 128;
  if (q.IH > 256 || q.IW > 256 || q.M1 > 8) return false;
  // per group: at most kTilesPerWarp expand tiles per warp of a lane quarter, one project tile per warp, and (when the
  // chunks are copied in) four 16-byte pieces per thread
  if (q.M1 > kTilesPerWarp * (kWarps / NG / 4) || q.M2 > kWarps / NG || (!expand && q.P_x * 2 > 4 * group_threads)) return false;
  const int cols = (expand ? NG * q.M1 * kChunk : 0) + (project ? q.M2 * q.Coutp : 0);
  if (cols > 512) return false;
  q.tmem_cols = 32;
  while (q.tmem_cols < cols) q.tmem_cols *= 2;
  q.ecol0 = 0;
  q.pcol0 = expand ? NG * q.M1 * kChunk : 0;
  int off = 0;
  auto take = [&](int bytes) { int o = off; off = round_up(off + bytes, 1024); return o; };
  q.off_x = take(expand ? q.M1 * 128 * q.row_bytes : 0);
  q.off_w1 = take(expand ? q.Cexp * q.row_bytes : 0);
  // two 8-channel planes per chunk, offset by 64 mod 128 bytes so that a warp's
  // 2 x 64-byte accesses (4 pixels x 4 channel pairs per plane) never share a bank
  q.e_plane = round_up(q.P_in * 16, 128) + 64;
  q.d_plane = q.M2 * 128 * 16 + 64;
  q.off_e = take((expand ? NG : 2 * NG) * 2 * q.e_plane);   // one chunk buffer per group, two when the chunks are copied in
  q.off_d = take(NG * 2 * q.d_plane);
  q.off_w3 = take(project ? q.NC * q.Coutp * kChunkRowBytes : 0);
  q.off_wd = take(9 * q.Cexp * 2);
  q.off_b1 = take(expand ? q.Cexp * 4 : 0);
  q.off_bd = take(q.Cexp * 4);
  q.off_b3 = take(project ? q.Coutp * 4 : 0);
  q.off_bar = take(256);
  *smem_bytes = off + 1024;  // slack for the 1024-byte alignment of the base
  return *smem_bytes <= 227 * 1024;
}

}  // namespace

ago_status_t mbv2_plan(Plan* plan, FusedState* st, std::string* err) {
  // operator indices of the three convolutions in the chain (-1: the pair has none)
  const bool expand = plan->fused_kernel != AGO_KERNEL_DW_PW, project = plan->fused_kernel != AGO_KERNEL_PW_DW;
  const int i_dw = expand ? 3 : 0, i_pr = expand ? 6 : 3;
  const OpInfo& first = plan->ops[0];
  const OpInfo& d = plan->ops[i_dw];
  auto* host = new Mbv2Host();
  host->expand = expand; host->project = project;
  Mbv2Params& q = host->prm;
  q = Mbv2Params{};
  q.N = (int)first.in.d[0]; q.H = (int)first.in.d[1]; q.W = (int)first.in.d[2];
  q.Cexp = (int)d.in.d[3];
  q.Cin = expand ? (int)first.in.d[3] : 16;
  q.Cout = project ? plan->ops[i_pr].op.p[0] : 16;
  q.stride = d.op.p[3];
  q.Ho = (int)d.out.d[1]; q.Wo = (int)d.out.d[2];
  q.residual = plan->fused_kernel == AGO_KERNEL_MBV2_BLOCK && plan->ops.size() == 9 ? 1 : 0;
  auto bad = [&](const char* m) { *err = std::string("fused inverted-residual block: ") + m; delete host; return AGO_ERR_UNSUPPORTED; };
  if (q.Cin > 64) return bad("more than 64 input channels is not supported yet");
  if (q.Cexp % kChunk != 0) return bad("expanded channels must be a multiple of 16");
  if (q.Cout > 256) return bad("more than 256 output channels is not supported");
  if (q.residual && (q.stride != 1 || q.Cin != q.Cout)) return bad("residual needs stride 1 and Cin == Cout");
  q.Kp = q.Cin <= 16 ? 16 : (q.Cin <= 32 ? 32 : 64);
  q.row_bytes = q.Kp * 2;
  q.swizzle = q.Kp == 16 ? tc::SW_32B : (q.Kp == 32 ? tc::SW_64B : tc::SW_128B);
  q.Coutp = round_up(q.Cout, 16);
  q.fold_b1 = expand && q.Cin % 8 == 0 && q.Cin < q.Kp ? 1 : 0;
  q.NC = q.Cexp / kChunk;
  auto recip = [](int d) { return tc::fast_div_recip(d); };
  q.coutp_recip = recip(q.Coutp);
  q.w_recip = recip(q.W);
  q.cexp8_recip = recip(q.Cexp / 8);
  q.nseg = (q.Wo + kSegCols - 1) / kSegCols;
  q.per_row = q.stride == 1 ? q.nseg : q.Wo;
  q.per_row_recip = recip(q.per_row);
  auto set_groups = [&](Mbv2Params& t, int ng) {   // depthwise item geometry of a group of 32 / ng warps
    const int slots = kThreads / ng / 8;
    t.groups = ng;
    t.step_r = slots / t.per_row; t.step_c = slots - t.step_r * t.per_row;
    t.col_slots = slots / std::max(1, std::min(t.Wo, slots));
  };
  // Warp groups and rows per CTA: the least estimated time = waves x (fixed part + chunk loop), where the chunk loop
  // is the larger of the strip's arithmetic (issue-bound: about 0.8 cycles per pixel-tile unit and chunk, measured
  // on 56 x 56 strips) and the chain of latencies of the chunks one group owns (about 2.9k cycles per chunk,
  // measured on 28 x 28 strips). Small strips therefore run with four groups, large ones with two.
  int best_R = 0, best_ng = 2; double best_cost = 0; int best_smem = 0;
  const int sms = device_sm_count();
  for (int ng = 2; ng <= 8; ng *= 2) {
    for (int R = 1; R <= q.Ho; ++R) {
      Mbv2Params t = q; int smem = 0;
      set_groups(t, ng);
      if (!layout(t, R, expand, project, &smem)) continue;
      const long ctas = (long)q.N * t.strips;
      const long waves = (ctas + sms - 1) / sms;
      const double work = 0.8 * q.NC * (t.M1 * 128.0 + 3.0 * t.M2 * 128.0);
      const double chain = 2900.0 * ((q.NC + ng - 1) / ng);
      const double cost = (double)waves * (6000.0 + std::max(work, chain) + 0.01 * work);
      if (best_R == 0 || cost < best_cost) { best_R = R; best_ng = ng; best_cost = cost; best_smem = smem; }
    }
  }
  if (best_R == 0) return bad("no row-strip tiling fits shared memory / tensor memory");
  set_groups(q, best_ng);
  layout(q, best_R, expand, project, &best_smem);
  if ((long)q.N * q.strips > 65535) return bad("more than 65535 row strips in the batch");
  host->smem_bytes = best_smem;
  st->impl = host;
  st->impl_free = [](void* p) { delete static_cast<Mbv2Host*>(p); };
  st->tile_rows = best_R; st->grid = q.N * q.strips; st->smem_bytes = best_smem;
  plan->tile_rows = best_R; plan->smem_bytes = best_smem;
  return AGO_OK;
}

namespace {

template <bool EXPAND, bool PROJECT, bool FOLD, int NG>
ago_status_t launch_groups(const Mbv2Params& q, int smem_bytes, cudaStream_t stream, std::string* err) {
  static int smem_opt_in[64] = {};
  cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(mbv2_fused_kernel<EXPAND, PROJECT, FOLD, NG>), smem_opt_in);
  if (e != cudaSuccess) { *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  FusedLaunch launch(dim3((unsigned)(q.N * q.strips)), kThreads, (size_t)smem_bytes, stream);
  e = cudaLaunchKernelEx(&launch.config, mbv2_fused_kernel<EXPAND, PROJECT, FOLD, NG>, q);
  if (e != cudaSuccess) { *err = std::string("fused inverted-residual launch: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  return AGO_OK;
}
template <bool EXPAND, bool PROJECT, bool FOLD>
ago_status_t launch_variant(const Mbv2Params& q, int smem_bytes, cudaStream_t stream, std::string* err) {
  if (q.groups == 8) return launch_groups<EXPAND, PROJECT, FOLD, 8>(q, smem_bytes, stream, err);
  return q.groups == 4 ? launch_groups<EXPAND, PROJECT, FOLD, 4>(q, smem_bytes, stream, err)
                       : launch_groups<EXPAND, PROJECT, FOLD, 2>(q, smem_bytes, stream, err);
}

}  // namespace

ago_status_t mbv2_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                      void* output, unsigned int* status_word, cudaStream_t stream, std::string* err) {
  Mbv2Host* host = static_cast<Mbv2Host*>(st->impl);
  Mbv2Params q = host->prm;
  q.x = static_cast<const __nv_bfloat16*>(inputs[0]);
  int w = 0;   // weights in chain order: (w1, b1) (wd, bd) (w3, b3), without the pair's missing convolution
  if (host->expand) { q.w1 = static_cast<const __nv_bfloat16*>(weights[w]); q.b1 = static_cast<const float*>(weights[w + 1]); w += 2; }
  q.wd = static_cast<const __nv_bfloat16*>(weights[w]); q.bd = static_cast<const float*>(weights[w + 1]); w += 2;
  if (host->project) { q.w3 = static_cast<const __nv_bfloat16*>(weights[w]); q.b3 = static_cast<const float*>(weights[w + 1]); }
  q.out = static_cast<__nv_bfloat16*>(output);
  q.status = status_word;
  if (!host->expand) return launch_variant<false, true, false>(q, host->smem_bytes, stream, err);
  if (!host->project)
    return q.fold_b1 ? launch_variant<true, false, true>(q, host->smem_bytes, stream, err)
                     : launch_variant<true, false, false>(q, host->smem_bytes, stream, err);
  return q.fold_b1 ? launch_variant<true, true, true>(q, host->smem_bytes, stream, err)
                   : launch_variant<true, true, false>(q, host->smem_bytes, stream, err);
}

}  // namespace ago
