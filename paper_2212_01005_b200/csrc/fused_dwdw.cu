// Fused pair of depthwise convolutions: depthwise 3x3 (pad 1, stride 1) + bias + ReLU6, twice, one kernel
// (the "two depthwise convolutions" subgraph of the micro-benchmark, Section VI-B).
//
// Both operators have no reduction over channels, so the pair is tiled over channels without any recomputation
// (Section III-B, downstream depthwise); the spatial tile of the upstream operator grows by the one-pixel halo of
// the downstream window, which is the only redundant work: a CTA that produces R output rows computes R + 2 rows
// of the intermediate tensor from R + 4 input rows.
//
// Per CTA (one image, R output rows, full width, 16 channels):
//   P1  asynchronous 16-byte copies bring the input rows into two planes of [pixel][8 channels] with a zero column
//       on either side; rows outside the image are zero-filled (padding of the first convolution)
//   P2  depthwise 1 on CUDA cores -> intermediate rows in the same layout; rows outside the image stay zero
//       (the second convolution pads the post-activation tensor, not the input)
//   P3  depthwise 2 -> output tile in shared memory
//   P4  16-byte stores of (pixel, plane) pieces to the NHWC output.
// Several CTAs share an SM, so one CTA's copies and stores overlap another's arithmetic.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>

#include "dw_common.cuh"
#include "fused.h"
#include "tc_common.cuh"

namespace ago {

namespace {

using namespace tc;
using namespace dw;

constexpr int kThreads = 512;
constexpr int kSlots = kThreads / 8;   // thread = (channel pair, slot); 8 pairs = the chunk's 16 channels
constexpr int kChunk = 16;

struct DwDwParams {
  const __nv_bfloat16* x;
  const __nv_bfloat16* w1;   // [3][3][C]
  const float* b1;
  const __nv_bfloat16* w2;
  const float* b2;
  __nv_bfloat16* out;
  int N, H, W, C;
  int R, strips, NC, IW;      // output rows per CTA, strips per image, channel chunks, W + 2
  int nseg;                   // 7-column segments per row
  int step_r, step_c;         // kThreads / 2 pixels as (rows, columns) of the image width
  uint32_t w_recip, nseg_recip;
  int x_plane, m_plane, d_plane;   // byte distance between the two 8-channel planes of each buffer
  int off_x, off_m, off_d;
};

__global__ void __launch_bounds__(kThreads)
dwdw_fused_kernel(const DwDwParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  const int tid = threadIdx.x;
  const int c = blockIdx.x, strip = blockIdx.y, n = blockIdx.z;
  const int ho0 = strip * p.R;
  const int rows_valid = min(p.R, p.H - ho0);
  const int gx0 = ho0 - 2;                       // image row of input-tile row 0; intermediate row j is image row ho0 - 1 + j
  const int XH = rows_valid + 4, MH = rows_valid + 2;
  const int cp = tid & 7, slot = tid >> 3;
  const int cp_off = (cp & 3) * 4;
  const uint32_t pitch = (uint32_t)p.IW * 16u, d_pitch = (uint32_t)p.W * 16u;
  const uint32_t sx = smem_u32(smem + p.off_x), sm = smem_u32(smem + p.off_m), sd = smem_u32(smem + p.off_d);

  grid_dependency_wait();
  grid_launch_dependents();
  // ---- P1: input rows -> two planes, one commit group ----
  {
    const uint8_t* xin = reinterpret_cast<const uint8_t*>(p.x) + ((int64_t)n * p.H + gx0) * p.W * p.C * 2 + c * kChunk * 2;
    const int pieces = XH * p.W * 2;
    // piece i = (pixel i / 2, plane i % 2); a thread's pieces are kThreads / 2 pixels apart: row and column advance
    // by fixed steps (one wrap at most), so the division is done once
    int pix = tid >> 1;
    const int plane = tid & 1;
    int ih = (int)fast_div((uint32_t)pix, (uint32_t)p.W, p.w_recip), iw = pix - ih * p.W;
    const uint8_t* src = xin + (int64_t)pix * p.C * 2 + plane * 16;
    uint32_t dst = sx + (uint32_t)(plane * p.x_plane + (ih * p.IW + iw + 1) * 16);
    const int64_t src_step = (int64_t)(kThreads / 2) * p.C * 2;
    const uint32_t dst_step = (uint32_t)((p.step_r * p.IW + p.step_c) * 16);
    for (int i = tid; i < pieces; i += kThreads) {
      const bool in = gx0 + ih >= 0 && gx0 + ih < p.H;
      cp_async_16(dst, in ? src : reinterpret_cast<const uint8_t*>(p.x), in ? 16u : 0u);
      src += src_step; dst += dst_step; ih += p.step_r; iw += p.step_c;
      if (iw >= p.W) { iw -= p.W; ++ih; dst += 2u * 16u; }   // the next row starts two padding columns later
    }
    cp_async_commit();
  }
  // weights and biases of this thread's channel pair (both convolutions)
  const int ch = c * kChunk + cp * 2;
  uint32_t wg1[9], wg2[9];
#pragma unroll
  for (int tap = 0; tap < 9; ++tap) {
    wg1[tap] = __ldg(reinterpret_cast<const uint32_t*>(p.w1 + tap * p.C + ch));
    wg2[tap] = __ldg(reinterpret_cast<const uint32_t*>(p.w2 + tap * p.C + ch));
  }
  const float2 bias1 = __ldg(reinterpret_cast<const float2*>(p.b1 + ch));
  const float2 bias2 = __ldg(reinterpret_cast<const float2*>(p.b2 + ch));
  // zero padding: the side columns of the input tile and of the intermediate tile, and the intermediate rows that
  // lie outside the image
  const int j_lo = max(0, 1 - ho0), j_hi = min(MH, p.H - ho0 + 1);   // intermediate rows [j_lo, j_hi) are in the image
  for (int i = tid; i < (XH + 1) * 4; i += kThreads) {
    const int ih = i >> 2, side = (i >> 1) & 1, plane = i & 1;
    *reinterpret_cast<uint4*>(smem + p.off_x + plane * p.x_plane + (ih * p.IW + side * (p.IW - 1)) * 16) = make_uint4(0, 0, 0, 0);
  }
  for (int i = tid; i < MH * 4; i += kThreads) {
    const int ih = i >> 2, side = (i >> 1) & 1, plane = i & 1;
    *reinterpret_cast<uint4*>(smem + p.off_m + plane * p.m_plane + (ih * p.IW + side * (p.IW - 1)) * 16) = make_uint4(0, 0, 0, 0);
  }
  {
    const int nz = j_lo + (MH - j_hi), per_row = p.IW * 2;   // rows outside the image: [0, j_lo) and [j_hi, MH)
    for (int i = tid; i < nz * per_row; i += kThreads) {
      const int z = i / per_row, k = i - z * per_row;
      const int j = z < j_lo ? z : j_hi + (z - j_lo);
      *reinterpret_cast<uint4*>(smem + p.off_m + (k & 1) * p.m_plane + (j * p.IW + (k >> 1)) * 16) = make_uint4(0, 0, 0, 0);
    }
  }
  cp_async_wait_all();
  __syncthreads();

  // ---- P2: depthwise 1 over the intermediate rows [j_lo, j_hi): blocks of 2 rows x 7 columns ----
  {
    const uint32_t src = sx + (uint32_t)((cp >> 2) * p.x_plane + cp_off);
    const uint32_t dst = sm + (uint32_t)((cp >> 2) * p.m_plane + cp_off) + 16u;   // column 0 of the tile is padding
    const int items = p.nseg * ((j_hi - j_lo + 1) >> 1);
    for (int item = slot; item < items; item += kSlots) {
      const int r = (int)fast_div((uint32_t)item, (uint32_t)p.nseg, p.nseg_recip), seg = item - r * p.nseg;
      const int j = j_lo + 2 * r, wo = seg * kSegCols;
      depthwise_block(src + (uint32_t)j * pitch + wo * 16, dst + (uint32_t)j * pitch + wo * 16, pitch, pitch,
                      min(kSegCols, p.W - wo), min(2, j_hi - j), wg1, bias1);
    }
  }
  __syncthreads();
  // ---- P3: depthwise 2 over the output rows ----
  {
    const uint32_t src = sm + (uint32_t)((cp >> 2) * p.m_plane + cp_off);
    const uint32_t dst = sd + (uint32_t)((cp >> 2) * p.d_plane + cp_off);
    const int items = p.nseg * ((rows_valid + 1) >> 1);
    for (int item = slot; item < items; item += kSlots) {
      const int r = (int)fast_div((uint32_t)item, (uint32_t)p.nseg, p.nseg_recip), seg = item - r * p.nseg;
      const int wo = seg * kSegCols;
      depthwise_block(src + (uint32_t)(2 * r) * pitch + wo * 16, dst + (uint32_t)(2 * r) * d_pitch + wo * 16, pitch, d_pitch,
                      min(kSegCols, p.W - wo), min(2, rows_valid - 2 * r), wg2, bias2);
    }
  }
  __syncthreads();
  // ---- P4: output tile -> device memory ----
  {
    __nv_bfloat16* o0 = p.out + ((size_t)n * p.H + ho0) * p.W * p.C + c * kChunk;
    const int pieces = rows_valid * p.W * 2;
    const int plane = tid & 1;
    __nv_bfloat16* dst = o0 + (size_t)(tid >> 1) * p.C + plane * 8;
    const uint8_t* src = smem + p.off_d + plane * p.d_plane + (tid >> 1) * 16;
    const size_t dst_step = (size_t)(kThreads / 2) * p.C;
    for (int i = tid; i < pieces; i += kThreads, dst += dst_step, src += (kThreads / 2) * 16)
      *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
  }
}

int round_up(int v, int m) { return (v + m - 1) / m * m; }

struct DwDwHost {
  DwDwParams prm;
  int smem_bytes = 0;
};

// Shared memory of a CTA with R output rows. The ragged blocks of the depthwise stages read up to one row and a few
// pixels past the rows they store: every buffer carries that slack.
int layout(DwDwParams& q, int R) {
  q.R = R;
  q.strips = (q.H + R - 1) / R;
  const int slack = (q.IW + 16) * 16;
  q.x_plane = round_up((R + 4) * q.IW * 16 + slack, 128) + 64;   // planes offset by 64 mod 128 bytes: conflict-free pairs
  q.m_plane = round_up((R + 2) * q.IW * 16 + slack, 128) + 64;
  q.d_plane = round_up(R * q.W * 16, 128) + 64;
  int off = 0;
  auto take = [&](int bytes) { int o = off; off = round_up(off + bytes, 128); return o; };
  q.off_x = take(2 * q.x_plane);
  q.off_m = take(2 * q.m_plane);
  q.off_d = take(2 * q.d_plane);
  return off + 128;
}

}  // namespace

ago_status_t dwdw_plan(Plan* plan, FusedState* st, std::string* err) {
  const OpInfo& a = plan->ops[0];
  auto* host = new DwDwHost();
  DwDwParams& q = host->prm;
  q = DwDwParams{};
  q.N = (int)a.in.d[0]; q.H = (int)a.in.d[1]; q.W = (int)a.in.d[2]; q.C = (int)a.in.d[3];
  auto bad = [&](const char* m) { *err = std::string("fused depthwise pair: ") + m; delete host; return AGO_ERR_UNSUPPORTED; };
  if (q.C % kChunk != 0) return bad("channels must be a multiple of 16");
  if (q.N > 65535 || q.W > 4096) return bad("batch or width too large");
  q.NC = q.C / kChunk;
  q.IW = q.W + 2;
  q.nseg = (q.W + kSegCols - 1) / kSegCols;
  q.w_recip = fast_div_recip(q.W);
  q.step_r = (kThreads / 2) / q.W; q.step_c = (kThreads / 2) % q.W;
  q.nseg_recip = fast_div_recip(q.nseg);
  // Rows per CTA: the halo (4 input rows, 2 intermediate rows) is amortised over R rows, while at least two CTAs
  // should share an SM (one computes while the other copies) and the grid should cover the SMs a few times.
  int best_R = 0; double best_cost = 0;
  for (int R = 1; R <= q.H; ++R) {
    DwDwParams t = q;
    const int smem = layout(t, R);
    if (smem > 110 * 1024) break;
    const long ctas = (long)q.N * t.strips * q.NC;
    const int per_sm = std::min(4, (227 * 1024) / (smem + 1024));
    const long slots = (long)device_sm_count() * per_sm, waves = (ctas + slots - 1) / slots;
    // time of a wave ~ arithmetic of its CTAs on one SM: rows of depthwise 1 + rows of depthwise 2, in slot-sized steps
    const int s1 = (t.nseg * ((R + 3) / 2) + kSlots - 1) / kSlots, s2 = (t.nseg * ((R + 1) / 2) + kSlots - 1) / kSlots;
    const double cost = (double)waves * per_sm * (s1 + s2 + 0.5);
    if (best_R == 0 || cost < best_cost) { best_R = R; best_cost = cost; }
  }
  if (best_R == 0) return bad("no row-strip tiling fits shared memory");
  host->smem_bytes = layout(q, best_R);
  st->impl = host;
  st->impl_free = [](void* p) { delete static_cast<DwDwHost*>(p); };
  st->tile_rows = best_R; st->grid = q.N * q.strips * q.NC; st->smem_bytes = host->smem_bytes;
  plan->tile_rows = best_R; plan->smem_bytes = host->smem_bytes;
  return AGO_OK;
}

ago_status_t dwdw_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                      void* output, unsigned int* status_word, cudaStream_t stream, std::string* err) {
  (void)plan; (void)status_word;
  DwDwHost* host = static_cast<DwDwHost*>(st->impl);
  DwDwParams q = host->prm;
  q.x = static_cast<const __nv_bfloat16*>(inputs[0]);
  q.w1 = static_cast<const __nv_bfloat16*>(weights[0]); q.b1 = static_cast<const float*>(weights[1]);
  q.w2 = static_cast<const __nv_bfloat16*>(weights[2]); q.b2 = static_cast<const float*>(weights[3]);
  q.out = static_cast<__nv_bfloat16*>(output);
  {
    static int smem_opt_in[64] = {};
    cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(dwdw_fused_kernel), smem_opt_in);
    if (e != cudaSuccess) { *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  }
  FusedLaunch launch(dim3((unsigned)q.NC, (unsigned)q.strips, (unsigned)q.N), kThreads, (size_t)host->smem_bytes, stream);
  cudaError_t e = cudaLaunchKernelEx(&launch.config, dwdw_fused_kernel, q);
  if (e != cudaSuccess) { *err = std::string("fused depthwise pair launch: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  return AGO_OK;
}

}  // namespace ago
