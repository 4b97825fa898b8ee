// Fused residual block: conv3x3 + bias + ReLU -> conv3x3 + bias -> + input -> ReLU,
// one kernel; the first convolution's output never leaves the SM.
//
// This link is the "general" category of Section III-B: the downstream 3x3
// convolution reuses its input along O2, H2 and W2, so any spatial tile of it
// needs a halo of the upstream output and fusion recomputes that halo. A CTA
// owns a strip of R output rows of one image (full width, all channels): it
// computes R + 2 rows of the first convolution (2 of them recomputed by the
// neighbouring strips) from R + 4 input rows.
//
// Both convolutions are implicit GEMMs on tcgen05: the activation tile sits in
// shared memory as [pixel][channels] rows in the swizzled K-major operand layout
// (exactly what one TMA box load produces), with pixels linearised over the
// PADDED width, so the operand of filter tap (dr, dc) is the same matrix at a
// start address shifted by (dr * Wp + dc - 1) rows. The swizzle is a function of
// the absolute shared-memory address, so such row-shifted start addresses are
// valid operands (verified on the device against a known matrix). Weights stream
// through a TMA ring, one filter row (3 taps) per stage.
//
//   P1  TMA: input strip with halo -> swizzled [pixel][channel] rows, zero outside the image
//   P2  tcgen05.mma: 9 taps x (I / 16) K-steps per 128-pixel tile            (TMEM)
//   P3  TMEM -> registers: + b1, ReLU, zero outside the image (the second
//       convolution pads the post-activation tensor), bf16 -> swizzled rows in shared memory
//   P5  tcgen05.mma: second convolution over the resident rows               (TMEM)
//   P6  TMEM -> registers: + b2 + x, ReLU, bf16, 16-byte stores
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <mutex>
#include <unordered_map>

#include "fused.h"
#include "tc_common.cuh"
#include "tmap.h"

namespace ago {

namespace {

using namespace tc;

constexpr int kEpiWarps = 16;                // four per TMEM lane quarter: each takes a quarter of the channels (at least 16)
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kMmaWarps = 4;                 // one issuing lane each, alternating M tiles: a single thread issues an MMA every ~70 cycles, the tensor pipe takes one every ~50
constexpr int kThreads = kEpiThreads + 32 + 32 * kMmaWarps;   // + TMA warp + MMA warps
constexpr int kMaxWStages = 4;     // ring stages; each holds one filter row = 3 taps

struct ConvParams {
  const __nv_bfloat16* x;
  const float* b1;
  const float* b2;
  __nv_bfloat16* out;
  unsigned int* status;
  int N, H, W, C;          // C = input = middle = output channels
  int R, strips, IH, Wp, P1, M1, P2, M2;
  int a1, a2;              // tiles [0,a1) of conv1 / [0,a2) of conv2 form the first pipeline group
  int stage_ok;            // the first 16 KB of the input rows are free for output staging whenever an output epilogue runs
  // single-convolution variant (a stage of the unfused mode): out = [relu](conv(x) + b2 [+ res])
  const __nv_bfloat16* res; // residual tensor (the pair kernel adds its own input)
  int residual, relu;
  int w_row_bytes, w_swizzle, w_stage_bytes;
  int wstages;             // ring stages in use (2..kMaxWStages)
  int off_x, off_y, off_w, off_bias, off_bar;
  uint32_t wp_recip;        // 2^32 / Wp + 1: pixel index -> (row, column) of the padded strip without a division
};

// SINGLE = false: the fused pair. SINGLE = true: one convolution with its simple operators (second-convolution
// passes only, reading the input rows directly), the tensor-core stage kernel of the unfused mode.
template <bool SINGLE>
__global__ void __launch_bounds__(kThreads, 1)
conv3x3_pair_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w1,
                    const __grid_constant__ CUtensorMap tmap_w2, const ConvParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sX = smem + p.off_x;   // first pixel row (1024-aligned; slack lies before it)
  uint8_t* sY = smem + p.off_y;   // the intermediate rows reuse the input rows' memory, two pixels lower
  uint8_t* sW = smem + p.off_w;
  float* sBias = reinterpret_cast<float*>(smem + p.off_bias);   // b1[C], b2[C]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
  uint64_t* bar_x = bars;                      // input strip landed
  uint64_t* bar_full = bars + 1;                  // [kMaxWStages] filter row landed
  uint64_t* bar_empty = bars + 1 + kMaxWStages;   // [kMaxWStages] filter row consumed
  uint64_t* bar_acc1 = bars + 1 + 2 * kMaxWStages;   // [2] first convolution, tile group g complete
  uint64_t* bar_y = bar_acc1 + 2;                 // [2] intermediate rows of group g written
  uint64_t* bar_acc2 = bar_acc1 + 4;              // [2] second convolution, tile group g complete
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_acc1 + 6);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bar_acc1 + 7);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n = blockIdx.x / p.strips, strip = blockIdx.x % p.strips;
  const int h0 = strip * p.R;
  const int rows_valid = min(p.R, p.H - h0);
  const int ksteps = p.C / 16;

  grid_dependency_wait();      // the previous grid of the stream has completed; device memory may be touched
  grid_launch_dependents();
  if (tid == kEpiThreads) {
    *abort_flag = 0u;
    mbar_init(bar_x, 1);
    for (int i = 0; i < kMaxWStages; ++i) { mbar_init(bar_full + i, 1); mbar_init(bar_empty + i, kMmaWarps); }
    for (int i = 0; i < 6; ++i) mbar_init(bar_acc1 + i, (i == 2 || i == 3) ? 1 : kMmaWarps);   // bar_y is arrived by one epilogue thread
    fence_mbar_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmap_x);
    mbar_arrive_expect_tx(bar_x, (uint32_t)(p.IH * p.Wp * p.w_row_bytes));
    tma_load_4d(sX, &tmap_x, bar_x, 0, -1, SINGLE ? h0 - 1 : h0 - 2, n);
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  if (tid < 2 * p.C) sBias[tid] = SINGLE ? (tid >= p.C && p.b2 ? p.b2[tid - p.C] : 0.0f) : (tid < p.C ? p.b1[tid] : p.b2[tid - p.C]);
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // The four MMA passes: (convolution, tile group) = (1,A) (1,B) (2,A) (2,B); each streams the 9 taps.
  const int pass_lo[4] = {0, SINGLE ? 0 : p.a1, 0, p.a2};
  const int pass_hi[4] = {SINGLE ? 0 : p.a1, SINGLE ? 0 : p.M1, p.a2, p.M2};

  if (warp == kEpiWarps) {
    // ================================ TMA producer: weight taps ================================
    if (lane == 0) {
      tma_prefetch_desc(&tmap_w1); tma_prefetch_desc(&tmap_w2);
      int i = 0;
      for (int ps = 0; ps < 4; ++ps) {
        if (pass_lo[ps] >= pass_hi[ps]) continue;      // empty group: the MMA warp skips it too
        for (int frow = 0; frow < 3; ++frow, ++i) {
          const int s = i % p.wstages;
          if (i >= p.wstages) mbar_wait(bar_empty + s, (uint32_t)((i / p.wstages) - 1) & 1u, abort_flag, p.status, 0x401);
          mbar_arrive_expect_tx(bar_full + s, (uint32_t)(3 * p.C * p.w_row_bytes));
          for (int t3 = 0; t3 < 3; ++t3)
            tma_load_3d(sW + (s * 3 + t3) * p.w_stage_bytes, ps < 2 ? &tmap_w1 : &tmap_w2, bar_full + s, 0, frow * 3 + t3, 0);
        }
      }
    }
    __syncwarp();
  } else if (warp > kEpiWarps) {
    // ================================ MMA issuers ================================
    const int iw = warp - kEpiWarps - 1;   // issuer iw takes tiles lo + iw, lo + iw + kMmaWarps, ...
    // Each issuing warp runs its loop converged; MMAs and commits are predicated on one elected lane and take ready
    // 64-bit descriptors (several times the issue rate of a lane-0 branch next to busy warps, see tc_common.cuh).
    {
      const uint32_t elected = elect_one();
      const uint32_t idesc = make_idesc_bf16(128, (uint32_t)p.C);
      const uint64_t wdesc0 = make_smem_desc(smem_u32(sW), 0, 8u * p.w_row_bytes, p.w_swizzle);
      mbar_wait(bar_x, 0, abort_flag, p.status, 0x402);
      int i = 0;
      for (int ps = 0; ps < 4; ++ps) {
        const int conv = ps >> 1, grp = ps & 1;
        uint64_t* done = (conv == 0 ? bar_acc1 : bar_acc2) + grp;
        if (conv == 1 && !SINGLE) mbar_wait(bar_y + grp, 0, abort_flag, p.status, 0x403);   // the intermediate rows this group reads are written
        if (pass_lo[ps] >= pass_hi[ps]) { umma_commit_elected(done, elected); continue; }
        // A: swizzled [pixel][channel] rows; K step = 32 bytes inside a row, 8-row groups are 8 rows apart (SBO).
        // Descriptor arithmetic is hoisted: one add per tile, constant strides per K step.
        const uint32_t rowu = (uint32_t)p.w_row_bytes >> 4;   // one pixel row in 16-byte units
        const uint64_t adesc0 = make_smem_desc(smem_u32(conv == 0 ? sX : sY), 0, 8u * p.w_row_bytes, p.w_swizzle);
        const int lo = pass_lo[ps], hi = pass_hi[ps];
        const uint64_t a_tile_step = (uint64_t)(kMmaWarps * 128 * rowu);
        tcgen05_fence_after_sync();
        for (int tap = 0; tap < 9; ++tap) {
          const int s = i % p.wstages;
          if (tap % 3 == 0) {
            mbar_wait(bar_full + s, (uint32_t)(i / p.wstages) & 1u, abort_flag, p.status, 0x404);
            tcgen05_fence_after_sync();
          }
          const int shift = (tap / 3) * p.Wp + (tap % 3) - 1;     // pixels = 16-byte units
          const uint64_t bdesc = wdesc0 + (uint64_t)((uint32_t)((s * 3 + tap % 3) * p.w_stage_bytes) >> 4);
          // (lo + iw) * 128 + shift may be negative for the first tile's first taps: the add wraps in the address field
          // exactly as the 32-bit add on the descriptor's low word did
          uint64_t a = (adesc0 & 0xffffffff00000000ull) |
                       (uint64_t)((uint32_t)adesc0 + (uint32_t)((lo + iw) * 128 + shift) * rowu);
          uint32_t d_tmem = tmem_base + (lo + iw) * p.C;
          if (ksteps == 4) {
            for (int mt = lo + iw; mt < hi; mt += kMmaWarps, a += a_tile_step, d_tmem += kMmaWarps * p.C) {
              umma_bf16_elected_acc(d_tmem, a, bdesc, idesc, elected, tap != 0);
              umma_bf16_elected<true>(d_tmem, a + 2u, bdesc + 2u, idesc, elected);
              umma_bf16_elected<true>(d_tmem, a + 4u, bdesc + 4u, idesc, elected);
              umma_bf16_elected<true>(d_tmem, a + 6u, bdesc + 6u, idesc, elected);
            }
          } else {
            for (int mt = lo + iw; mt < hi; mt += kMmaWarps, a += a_tile_step, d_tmem += kMmaWarps * p.C)
              for (int ks = 0; ks < ksteps; ++ks)
                umma_bf16_elected_acc(d_tmem, a + 2u * ks, bdesc + 2u * ks, idesc, elected, (ks | tap) != 0);
          }
          if (tap % 3 == 2) { umma_commit_elected(bar_empty + s, elected); ++i; }
        }
        umma_commit_elected(done, elected);
      }
    }
    __syncwarp();
  } else {
    // ================ epilogue warps: thread = (pixel row of a tile, half of the channels) ================
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const int row = (warp & 3) * 32 + lane;
    const int ncol = max(16, p.C / (kEpiWarps / 4));
    const int col0 = (warp >> 2) * ncol;
    const bool has_cols = col0 < p.C;

    // P3: intermediate = ReLU(acc + b1) inside the image, 0 outside -> swizzled rows; group A, then group B
    const uint32_t y_addr = smem_u32(sY);
    const uint32_t swz_mask = ((uint32_t)p.w_row_bytes >> 4) - 1u;
    // a thread's columns are fixed (ncol == 16 for 16, 32 and 64 channels): its biases stay in registers
    float bias1[16], bias2[16];
#pragma unroll
    for (int j = 0; j < 16; j += 4) {
      const float4 u = has_cols ? *reinterpret_cast<const float4*>(sBias + col0 + j) : make_float4(0.f, 0.f, 0.f, 0.f);
      const float4 w = has_cols ? *reinterpret_cast<const float4*>(sBias + p.C + col0 + j) : make_float4(0.f, 0.f, 0.f, 0.f);
      bias1[j] = u.x; bias1[j + 1] = u.y; bias1[j + 2] = u.z; bias1[j + 3] = u.w;
      bias2[j] = w.x; bias2[j + 1] = w.y; bias2[j + 2] = w.z; bias2[j + 3] = w.w;
    }
    for (int grp = 0; grp < (SINGLE ? 0 : 2); ++grp) {
      mbar_wait(bar_acc1 + grp, 0, abort_flag, p.status, 0x405);
      tcgen05_fence_after_sync();
      const int lo1 = grp ? p.a1 : 0, hi1 = grp ? p.M1 : p.a1;   // the group's tiles of the first convolution
      for (int mt = lo1; mt < hi1 && has_cols; ++mt) {
        const int m = mt * 128 + row;
        const int a = (int)fast_div((uint32_t)m, (uint32_t)p.Wp, p.wp_recip), b = m - a * p.Wp;
        const int gh = h0 - 1 + a;
        const bool inside = m < p.P1 && gh >= 0 && gh < p.H && b >= 1 && b <= p.W;
        for (int c0 = col0; c0 < col0 + ncol; c0 += 16) {
          uint32_t v[16];
          tmem_ld_x16(tmem_base + lane_base + mt * p.C + c0, v);
          tmem_ld_wait();
          uint32_t w[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float y0 = fmaxf(__uint_as_float(v[2 * j]) + bias1[2 * j], 0.0f);
            const float y1 = fmaxf(__uint_as_float(v[2 * j + 1]) + bias1[2 * j + 1], 0.0f);
            w[j] = inside ? pack_bf16x2(y0, y1) : 0u;
          }
          if (m < p.P1 + p.Wp) {   // a little past the tile so that shifted reads of valid rows never see stale data
            // 16-byte chunk index XOR address bits [7, ..): the swizzle the MMA and TMA apply to absolute addresses
            uint32_t a0 = y_addr + (uint32_t)m * p.w_row_bytes + (uint32_t)c0 * 2u;
            uint32_t a1 = a0 + 16u;
            a0 ^= ((a0 >> 7) & swz_mask) << 4;
            a1 ^= ((a1 >> 7) & swz_mask) << 4;
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a0), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a1), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
          }
        }
      }
      fence_proxy_async_smem();
      tcgen05_fence_before_sync();
      named_barrier_sync(1, kEpiThreads);
      if (tid == 0) mbar_arrive(bar_y + grp);
    }

    // P6: out = ReLU(acc + b2 + x); the residual is fetched before waiting for the accumulators. A thread owns one
    // pixel row of a tile, and pixels are C * 2 bytes apart in device memory: stored straight from the registers, a
    // warp's 16-byte stores would hit 32 different lines each. Instead the warp transposes its [32 pixels x ncol]
    // block through a private 2 KB staging area (the start of the input rows, no longer read by then), so that
    // consecutive lanes store consecutive 16-byte chunks of a pixel.
    const bool stage = p.stage_ok != 0;
    const uint32_t stg = smem_u32(sX) + (uint32_t)warp * 2048u;
    const int chl = ncol == 32 ? 2 : 1;                  // log2(16-byte chunks per staged row)
    const uint32_t rb = (uint32_t)ncol * 2u;             // bytes per staged row
    const uint32_t swz_w = ((uint32_t)lane >> (3 - chl)) & ((1u << chl) - 1u);   // chunk XOR of this lane's row
    for (int grp = 0; grp < 2; ++grp) {
      const int lo2 = grp ? p.a2 : 0, hi2 = grp ? p.M2 : p.a2;   // the group's tiles of the second convolution
      for (int mt = lo2; mt < hi2 || mt == lo2; ++mt) {
        const bool tile_ok = mt < hi2;
        const int m = mt * 128 + row;
        const int r = (int)fast_div((uint32_t)m, (uint32_t)p.Wp, p.wp_recip), cc = m - r * p.Wp;
        const bool valid = tile_ok && has_cols && r < rows_valid && cc >= 1 && cc <= p.W;
        const size_t pix = ((size_t)n * p.H + h0 + r) * p.W + (cc - 1);
        const bool do_res = SINGLE ? p.residual != 0 : true, do_relu = SINGLE ? p.relu != 0 : true;
        uint4 xr[4];
        if (SINGLE) {
#pragma unroll
          for (int j = 0; j < 4; ++j) xr[j] = make_uint4(0u, 0u, 0u, 0u);
        }
        if (valid && do_res) {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (j * 8 < ncol) xr[j] = __ldg(reinterpret_cast<const uint4*>((SINGLE ? p.res : p.x) + pix * p.C + col0 + j * 8));
        }
        if (mt == lo2) {
          mbar_wait(bar_acc2 + grp, 0, abort_flag, p.status, 0x406);
          tcgen05_fence_after_sync();
        }
        if (!tile_ok) break;
        if (has_cols) {
          for (int c0 = col0, jj = 0; c0 < col0 + ncol; c0 += 16, jj += 2) {
            uint32_t v[16];
            tmem_ld_x16(tmem_base + lane_base + mt * p.C + c0, v);
            tmem_ld_wait();
            if (valid) {
              const uint32_t xs[8] = {xr[jj].x, xr[jj].y, xr[jj].z, xr[jj].w, xr[jj + 1].x, xr[jj + 1].y, xr[jj + 1].z, xr[jj + 1].w};
              uint32_t w[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                float y0 = __uint_as_float(v[2 * j]) + bias2[2 * j] + bf16_lo(xs[j]);      // xs is zero without a residual
                float y1 = __uint_as_float(v[2 * j + 1]) + bias2[2 * j + 1] + bf16_hi(xs[j]);
                if (do_relu) { y0 = fmaxf(y0, 0.0f); y1 = fmaxf(y1, 0.0f); }
                w[j] = pack_bf16x2(y0, y1);
              }
              if (stage) {
                const uint32_t k0 = (uint32_t)(c0 - col0) >> 3;
                const uint32_t a0 = stg + (uint32_t)lane * rb + ((k0 ^ swz_w) << 4), a1 = stg + (uint32_t)lane * rb + (((k0 + 1u) ^ swz_w) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a0), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a1), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
              } else {
                *reinterpret_cast<uint4*>(p.out + pix * p.C + c0) = make_uint4(w[0], w[1], w[2], w[3]);
                *reinterpret_cast<uint4*>(p.out + pix * p.C + c0 + 8) = make_uint4(w[4], w[5], w[6], w[7]);
              }
            }
          }
          if (stage) {
            __syncwarp();
            const uint32_t vmask = __ballot_sync(0xffffffffu, valid);
            const unsigned long long goff = ((unsigned long long)pix * p.C + col0) * 2ull;   // byte offset of this lane's row
            for (int it = 0; it < (1 << chl); ++it) {
              const int pl = it * (32 >> chl) + (lane >> chl);
              const uint32_t ch = (uint32_t)lane & ((1u << chl) - 1u);
              const uint32_t lo = __shfl_sync(0xffffffffu, (uint32_t)goff, pl), hi = __shfl_sync(0xffffffffu, (uint32_t)(goff >> 32), pl);
              const uint32_t sw = ((uint32_t)pl >> (3 - chl)) & ((1u << chl) - 1u);
              uint4 val;
              asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w) : "r"(stg + (uint32_t)pl * rb + ((ch ^ sw) << 4)));
              if ((vmask >> pl) & 1u)
                *reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(p.out) + (((unsigned long long)hi << 32) | lo) + ch * 16u) = val;
            }
            __syncwarp();
          }
        }
      }
    }
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, 512);
}

struct ConvHost {
  ConvParams prm;
  int smem_bytes = 0;
  struct Key { const void* p; int which; bool operator==(const Key& o) const { return p == o.p && which == o.which; } };
  struct KeyHash { size_t operator()(const Key& k) const { return std::hash<const void*>()(k.p) ^ (size_t)k.which * 0x9e3779b97f4a7c15ull; } };
  std::unordered_map<Key, CUtensorMap, KeyHash> maps;
};

int round_up_i(int v, int m) { return (v + m - 1) / m * m; }

bool conv_layout(ConvParams& q, int R, int* smem_bytes) {
  q.R = R;
  q.strips = (q.H + R - 1) / R;
  q.IH = R + 4;
  q.Wp = q.W + 2;
  q.wp_recip = tc::fast_div_recip(q.Wp);
  q.P1 = (R + 2) * q.Wp; q.M1 = (q.P1 + 127) / 128;
  q.P2 = R * q.Wp; q.M2 = (q.P2 + 127) / 128;
  if (q.IH > 256 || q.Wp > 256 || q.M1 * q.C > 512) return false;
  // The intermediate rows alias the input rows, shifted down by two pixels: while the second tile
  // group of the first convolution still reads input pixels >= a1*128 - 1, the first group's epilogue
  // writes intermediate pixels < a1*128, i.e. input slots < a1*128 - 2.
  int off = 1024;   // slack before the rows: shifted operand rows start up to three pixels early
  q.off_x = off;
  q.off_y = off - 2 * q.w_row_bytes;
  const int reach_px = std::max(std::max(q.M1 * 128 + 2 * q.Wp + 2, q.P1 + q.Wp + 2), q.IH * q.Wp);
  const int x_reach = reach_px * q.w_row_bytes;
  off = round_up_i(off + x_reach, 1024);
  q.off_w = off;
  q.wstages = kMaxWStages;
  while (q.wstages > 2 && off + q.wstages * 3 * q.w_stage_bytes + 2048 + 1024 > 227 * 1024) --q.wstages;
  off += q.wstages * 3 * q.w_stage_bytes;
  q.off_bias = off;
  off += 1024;
  q.off_bar = off;
  off += 256;
  // pipeline groups: the second convolution's first group may only read intermediate rows the first
  // group of the first convolution produces
  q.a1 = (q.M1 + 1) / 2;   // even groups: a pass of only three tiles keeps the tensor pipe less busy than one of four or five
  if (q.a1 < 1) q.a1 = 1;
  q.a2 = (q.a1 * 128 - 2 * q.Wp - 1) / 128;
  if (q.a2 < 0) q.a2 = 0;
  if (q.a2 > q.M2) q.a2 = q.M2;
  if (q.a1 >= q.M1) { q.a1 = q.M1; }
  // Output staging uses the first 16 KB of the input rows. While the second group of the second convolution is
  // still being computed it reads intermediate pixels >= a2 * 128 - Wp - 1, which lie two pixel slots lower.
  const bool overlap = q.a2 > 0 && q.a2 < q.M2;   // an output epilogue runs next to MMAs that still read the rows
  const long free_bytes = overlap ? (long)(q.a2 * 128 - q.Wp - 3) * q.w_row_bytes : (long)x_reach;
  q.stage_ok = free_bytes >= kEpiWarps * 2048 ? 1 : 0;
  *smem_bytes = off + 1024;
  return *smem_bytes <= 227 * 1024;
}

}  // namespace

ago_status_t conv3x3_plan(Plan* plan, FusedState* st, std::string* err) {
  const OpInfo& c1 = plan->ops[0];
  auto* host = new ConvHost();
  ConvParams& q = host->prm;
  q = ConvParams{};
  q.N = (int)c1.in.d[0]; q.H = (int)c1.in.d[1]; q.W = (int)c1.in.d[2]; q.C = (int)c1.in.d[3];
  auto bad = [&](const char* m) { *err = std::string("fused conv3x3 pair: ") + m; delete host; return AGO_ERR_UNSUPPORTED; };
  if (c1.op.p[0] != q.C || plan->ops[3].op.p[0] != q.C) return bad("input, middle and output channel counts must be equal");
  if (q.C != 16 && q.C != 32 && q.C != 64) return bad("channel count must be 16, 32 or 64");
  q.w_row_bytes = q.C * 2;
  q.w_swizzle = q.C == 16 ? tc::SW_32B : (q.C == 32 ? tc::SW_64B : tc::SW_128B);
  q.w_stage_bytes = round_up_i(q.C * q.w_row_bytes, 1024);
  int best_R = 0, best_smem = 0; double best_cost = 0;
  for (int R = 1; R <= q.H; ++R) {
    ConvParams t = q; int smem = 0;
    if (!conv_layout(t, R, &smem)) continue;
    const long ctas = (long)q.N * t.strips;
    const long sms = device_sm_count(), waves = (ctas + sms - 1) / sms;
    const double cost = (double)waves * (t.M1 + t.M2 + 1.0);
    if (best_R == 0 || cost < best_cost) { best_R = R; best_cost = cost; best_smem = smem; }
  }
  if (best_R == 0) return bad("no row-strip tiling fits shared memory / tensor memory");
  conv_layout(q, best_R, &best_smem);
  host->smem_bytes = best_smem;
  st->impl = host;
  st->impl_free = [](void* p) { delete static_cast<ConvHost*>(p); };
  st->tile_rows = best_R; st->grid = q.N * q.strips; st->smem_bytes = best_smem;
  plan->tile_rows = best_R; plan->smem_bytes = best_smem;
  return AGO_OK;
}

ago_status_t conv3x3_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                         void* output, unsigned int* status_word, cudaStream_t stream, std::string* err) {
  ConvHost* host = static_cast<ConvHost*>(st->impl);
  ConvParams q = host->prm;
  q.x = static_cast<const __nv_bfloat16*>(inputs[0]);
  q.b1 = static_cast<const float*>(weights[1]);
  q.b2 = static_cast<const float*>(weights[3]);
  q.out = static_cast<__nv_bfloat16*>(output);
  q.status = status_word;
  q.res = q.x; q.residual = 1; q.relu = 1;
  auto get_map = [&](const void* base, int which, CUtensorMap* out) -> bool {
    ConvHost::Key key{base, which};
    auto it = host->maps.find(key);
    if (it == host->maps.end()) {
      CUtensorMap m;
      if (which == 0) {
        const uint64_t dims[4] = {(uint64_t)q.C, (uint64_t)q.W, (uint64_t)q.H, (uint64_t)q.N};
        const uint64_t strides[3] = {(uint64_t)q.C * 2, (uint64_t)q.W * q.C * 2, (uint64_t)q.H * q.W * q.C * 2};
        const uint32_t box[4] = {(uint32_t)q.C, (uint32_t)q.Wp, (uint32_t)q.IH, 1};
        if (!encode_tmap_bf16(&m, base, 4, dims, strides, box, q.w_row_bytes, err)) return false;
      } else {
        const uint64_t dims[3] = {(uint64_t)q.C, 9, (uint64_t)q.C};
        const uint64_t strides[2] = {(uint64_t)q.C * 2, (uint64_t)9 * q.C * 2};
        const uint32_t box[3] = {(uint32_t)q.C, 1, (uint32_t)q.C};
        if (!encode_tmap_bf16(&m, base, 3, dims, strides, box, q.w_row_bytes, err)) return false;
      }
      if (host->maps.size() > 4096) host->maps.clear();
      it = host->maps.emplace(key, m).first;
    }
    *out = it->second;
    return true;
  };
  CUtensorMap mx, mw1, mw2;
  if (!get_map(inputs[0], 0, &mx) || !get_map(weights[0], 1, &mw1) || !get_map(weights[2], 2, &mw2)) return AGO_ERR_CUDA;
  {
    static int smem_opt_in[64] = {};
    cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(conv3x3_pair_kernel<false>), smem_opt_in);
    if (e != cudaSuccess) { *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  }
  FusedLaunch launch(dim3((unsigned)(q.N * q.strips)), kThreads, (size_t)host->smem_bytes, stream);
  cudaError_t e = cudaLaunchKernelEx(&launch.config, conv3x3_pair_kernel<false>, mx, mw1, mw2, q);
  if (e != cudaSuccess) { *err = std::string("fused conv3x3 pair launch: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  return AGO_OK;
}

// ---- one convolution on the same kernel: the tensor-core stage of the unfused modes ------------------

namespace {

bool conv_layout_single(ConvParams& q, int R, int* smem_bytes) {
  q.R = R;
  q.strips = (q.H + R - 1) / R;
  q.IH = R + 2;
  q.Wp = q.W + 2;
  q.wp_recip = tc::fast_div_recip(q.Wp);
  q.P1 = 0; q.M1 = 0;
  q.P2 = R * q.Wp; q.M2 = (q.P2 + 127) / 128;
  if (q.IH > 256 || q.Wp > 256 || q.M2 * q.C > 512) return false;
  int off = 1024;
  q.off_x = off;
  q.off_y = off;            // the convolution reads the input rows themselves
  const int reach_px = std::max(q.M2 * 128 + 2 * q.Wp + 2, q.IH * q.Wp);
  const int x_reach = reach_px * q.w_row_bytes;
  off = round_up_i(off + x_reach, 1024);
  q.off_w = off;
  q.wstages = kMaxWStages;
  while (q.wstages > 2 && off + q.wstages * 3 * q.w_stage_bytes + 2048 + 1024 > 227 * 1024) --q.wstages;
  off += q.wstages * 3 * q.w_stage_bytes;
  q.off_bias = off;
  off += 1024;
  q.off_bar = off;
  off += 256;
  q.a1 = 0;
  q.a2 = (q.M2 + 1) / 2;
  const bool overlap = q.a2 > 0 && q.a2 < q.M2;
  const long free_bytes = overlap ? (long)(q.a2 * 128 - q.Wp - 1) * q.w_row_bytes : (long)x_reach;
  q.stage_ok = free_bytes >= kEpiWarps * 2048 ? 1 : 0;
  *smem_bytes = off + 1024;
  return *smem_bytes <= 227 * 1024;
}

struct SingleKey {
  const void *x, *w; int N, H, W, C;
  bool operator==(const SingleKey& o) const { return x == o.x && w == o.w && N == o.N && H == o.H && W == o.W && C == o.C; }
};
struct SingleKeyHash {
  size_t operator()(const SingleKey& k) const {
    return std::hash<const void*>()(k.x) ^ (std::hash<const void*>()(k.w) * 31u) ^ ((size_t)k.N << 40) ^ ((size_t)k.H << 24) ^ ((size_t)k.W << 8) ^ (size_t)k.C;
  }
};
struct SingleEntry { ConvParams prm; int smem_bytes; CUtensorMap mx, mw; };
std::mutex g_single_mutex;
std::unordered_map<SingleKey, SingleEntry, SingleKeyHash> g_single;

}  // namespace

bool conv3x3_tc_supported(int H, int W, int Cin, int Cout, int R, int S, int stride, int pad) {
  if (R != 3 || S != 3 || stride != 1 || pad != 1 || Cin != Cout) return false;
  if (Cin != 16 && Cin != 32 && Cin != 64) return false;
  return H >= 1 && W + 2 <= 256;
}

cudaError_t launch_conv3x3_tc(const void* x, const void* w, const float* bias, const void* res, void* out, int N, int H,
                              int W, int C, int relu, unsigned int* status, cudaStream_t stream) {
  SingleEntry entry;
  {
    std::lock_guard<std::mutex> lock(g_single_mutex);
    const SingleKey key{x, w, N, H, W, C};
    auto it = g_single.find(key);
    if (it == g_single.end()) {
      SingleEntry e{};
      ConvParams& q = e.prm;
      q.N = N; q.H = H; q.W = W; q.C = C;
      q.w_row_bytes = C * 2;
      q.w_swizzle = C == 16 ? tc::SW_32B : (C == 32 ? tc::SW_64B : tc::SW_128B);
      q.w_stage_bytes = round_up_i(C * q.w_row_bytes, 1024);
      int best_R = 0, best_smem = 0; double best_cost = 0;
      for (int R = 1; R <= H; ++R) {
        ConvParams t = q; int smem = 0;
        if (!conv_layout_single(t, R, &smem)) continue;
        const long sms = device_sm_count(), waves = ((long)N * t.strips + sms - 1) / sms;
        const double cost = (double)waves * (t.M2 + 1.0);
        if (best_R == 0 || cost < best_cost) { best_R = R; best_cost = cost; best_smem = smem; }
      }
      if (best_R == 0) return cudaErrorInvalidConfiguration;
      conv_layout_single(q, best_R, &best_smem);
      e.smem_bytes = best_smem;
      std::string err;
      const uint64_t xd[4] = {(uint64_t)C, (uint64_t)W, (uint64_t)H, (uint64_t)N};
      const uint64_t xs[3] = {(uint64_t)C * 2, (uint64_t)W * C * 2, (uint64_t)H * W * C * 2};
      const uint32_t xb[4] = {(uint32_t)C, (uint32_t)q.Wp, (uint32_t)q.IH, 1};
      if (!encode_tmap_bf16(&e.mx, x, 4, xd, xs, xb, q.w_row_bytes, &err)) return cudaErrorInvalidValue;
      const uint64_t wd[3] = {(uint64_t)C, 9, (uint64_t)C};
      const uint64_t ws[2] = {(uint64_t)C * 2, (uint64_t)9 * C * 2};
      const uint32_t wb[3] = {(uint32_t)C, 1, (uint32_t)C};
      if (!encode_tmap_bf16(&e.mw, w, 3, wd, ws, wb, q.w_row_bytes, &err)) return cudaErrorInvalidValue;
      if (g_single.size() > 4096) g_single.clear();
      it = g_single.emplace(key, e).first;
    }
    entry = it->second;
  }
  ConvParams q = entry.prm;
  q.x = static_cast<const __nv_bfloat16*>(x);
  q.b1 = nullptr; q.b2 = bias;
  q.res = static_cast<const __nv_bfloat16*>(res); q.residual = res != nullptr; q.relu = relu;
  q.out = static_cast<__nv_bfloat16*>(out);
  q.status = status;
  {
    static int smem_opt_in[64] = {};
    cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(conv3x3_pair_kernel<true>), smem_opt_in);
    if (e != cudaSuccess) return e;
  }
  conv3x3_pair_kernel<true><<<q.N * q.strips, kThreads, entry.smem_bytes, stream>>>(entry.mx, entry.mw, entry.mw, q);
  return cudaGetLastError();
}

}  // namespace ago
