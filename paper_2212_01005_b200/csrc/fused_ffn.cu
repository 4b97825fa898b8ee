// Fused feed-forward chain: Y = GELU(X W1 + b1) W2 + b2 in one kernel; the
// hidden activations H never leave the SM.
//
// Tile choice (Section III-B, "downstream pointwise / matmul" category): the
// second GEMM reuses H only along its output columns, so a CTA's downstream tile
// keeps ALL output columns and is tiled over rows (128 tokens). What is tiled in
// addition is the second GEMM's REDUCTION dimension (the hidden units): a CTA
// owns 128 rows x G tiles of 128 hidden units, computes those H tiles exactly once
// (no recomputation of the upstream operator), applies bias + GELU, keeps them
// in shared memory and adds its partial product H[:, tiles] * W2[tiles, :] to an
// fp32 accumulation buffer in device memory, one 128-column output slice at a
// time (all 768 fp32 output columns of a row block do not fit tensor memory).
// The reductions into that buffer are what bounds the kernel, hence G as large as
// shared memory and the grid allow. The last CTA of a row block adds b2, rounds
// to bf16, writes the output and re-zeroes the buffer.
//
//   P1  TMA ring (32 KB stages): X [128 x 64] and W1 [64 x 128] tiles, later W2 [128 x 128] tiles
//   P2  tcgen05.mma: Hacc[128 x 128] = X[128 x K] * W1[K, tile g]     (TMEM, two buffers)
//   P3  TMEM -> registers: + b1, GELU(tanh), bf16 -> shared memory tile g (K-major operand);
//       overlaps the first GEMM of tile g + 1
//   P5  tcgen05.mma: for each 128-column slice of the output: acc = sum_g H_g * W2[tile g, slice]
//   P6  TMEM -> registers -> red.global.add.v4.f32 into the accumulation buffer;
//       last CTA per row block: + b2, bf16, store.
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

constexpr int kBM = 128;        // rows per CTA
constexpr int kBH = 128;        // hidden units per tile
constexpr int kBK = 64;         // K elements per ring stage of the first GEMM
constexpr int kBN = 128;        // output columns per slice of the second GEMM
constexpr int kMaxStages = 4;
constexpr int kMaxG = 4;        // hidden tiles per CTA; G + ring stages = 7 blocks of 32 KB
constexpr int kStageBytes = 32 * 1024;
constexpr int kEpiWarps = 8;    // two per tensor-memory lane quarter: each takes 64 of a tile's 128 columns
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kThreads = kEpiThreads + 64;   // + TMA warp + MMA warp

struct FfnParams {
  const float* b1;
  const float* b2;
  __nv_bfloat16* out;
  float* acc;              // [M][N2] fp32, zero between launches
  unsigned int* counters;  // [row blocks], zero between launches
  unsigned int* status;
  int M, K, Hid, N2;
  int kblocks;             // K / 64
  int nslices;             // N2 / 128
  int G;                   // hidden tiles per CTA
  int hctas;               // CTAs per row block = Hid / 128 / G
  int stages;              // ring stages in use
};

__device__ __forceinline__ float gelu_tanh_fast(float v) {
  const float u = 0.7978845608028654f * (v + 0.044715f * v * v * v);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
  return 0.5f * v * (1.0f + t);
}

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
ffn_fused_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w1,
                 const __grid_constant__ CUtensorMap tmap_w2, const FfnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sRing = smem;                                  // p.stages x 32 KB
  uint8_t* sH = smem + p.stages * kStageBytes;            // G x (2 x [128 x 64] bf16, 128-byte-swizzled)
  uint64_t* bars = reinterpret_cast<uint64_t*>(sH + p.G * kStageBytes);
  uint64_t* bar_full = bars;                      // [kMaxStages]
  uint64_t* bar_empty = bars + kMaxStages;        // [kMaxStages]
  uint64_t* bar_hacc = bars + 2 * kMaxStages;     // [2] first GEMM of a tile complete (accumulator buffer b)
  uint64_t* bar_hfree = bar_hacc + 2;             // [2] accumulator buffer b drained
  uint64_t* bar_hsm = bar_hacc + 4;               // [kMaxG] H tile g written to shared memory
  uint64_t* bar_out = bar_hacc + 4 + kMaxG;       // [2] output-slice accumulators complete
  uint64_t* bar_free = bar_out + 2;               // [2] output-slice accumulators drained
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_free + 2);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bar_free + 3);
  uint32_t* last_flag = const_cast<uint32_t*>(abort_flag) + 1;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int hc = blockIdx.x, rb = blockIdx.y;   // group of G hidden tiles, row block
  const int row0 = rb * kBM;
  const int G = p.G, stages = p.stages;
  grid_dependency_wait();      // the previous grid of the stream has completed; device memory may be touched
  grid_launch_dependents();
  // tensor memory: columns [0, 256) two first-GEMM accumulators, [256, 512) two output-slice accumulators
  constexpr uint32_t kOutCol = 256;

  if (tid == kEpiThreads) {
    *abort_flag = 0u;
    for (int i = 0; i < kMaxStages; ++i) { mbar_init(bar_full + i, 1); mbar_init(bar_empty + i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar_hacc + i, 1); mbar_init(bar_hfree + i, 1); mbar_init(bar_out + i, 1); mbar_init(bar_free + i, 1); }
    for (int i = 0; i < kMaxG; ++i) mbar_init(bar_hsm + i, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const int loads1 = G * p.kblocks;                  // ring uses of the first GEMM: (tile g, k block)
  const int total_loads = loads1 + p.nslices * G;    // then (output slice, tile g)

  if (warp == kEpiWarps) {
    // ================================ TMA producer ================================
    if (lane == 0) {
      tma_prefetch_desc(&tmap_x);
      tma_prefetch_desc(&tmap_w1);
      tma_prefetch_desc(&tmap_w2);
      int s = 0, round = 0;
      for (int i = 0; i < total_loads; ++i) {
        if (round > 0) mbar_wait(bar_empty + s, (uint32_t)(round - 1) & 1u, abort_flag, p.status, 0x301);
        uint8_t* st = sRing + s * kStageBytes;
        mbar_arrive_expect_tx(bar_full + s, kStageBytes);
        if (i < loads1) {
          const int g = i / p.kblocks, kb = i - g * p.kblocks;
          const int hid0 = (hc * G + g) * kBH;
          tma_load_2d(st, &tmap_x, bar_full + s, kb * kBK, row0);                          // X [128 rows x 64 k]
          tma_load_2d(st + 16384, &tmap_w1, bar_full + s, hid0, kb * kBK);                 // W1 [64 k x 64 n]
          tma_load_2d(st + 16384 + 8192, &tmap_w1, bar_full + s, hid0 + 64, kb * kBK);
        } else {
          const int u = (i - loads1) / G, g = (i - loads1) - u * G;
          const int n0 = ((u + hc) % p.nslices) * kBN;   // slices in rotated order: neighbouring CTAs reduce into different columns
          const int hid0 = (hc * G + g) * kBH;
          tma_load_2d(st, &tmap_w2, bar_full + s, n0, hid0);                               // W2 [128 k x 64 n]
          tma_load_2d(st + 16384, &tmap_w2, bar_full + s, n0 + 64, hid0);
        }
        if (++s == stages) { s = 0; ++round; }
      }
    }
    __syncwarp();
  } else if (warp == kEpiWarps + 1) {
    // ================================ MMA issuer ================================
    // the whole warp, converged; MMAs and commits predicated on one elected lane (see tc_common.cuh)
    {
      const uint32_t elected = elect_one();
      const uint32_t idesc = make_idesc_bf16(128, 128, 0, 1);   // A K-major, B N-major (weights as they lie in HBM)
      int s = 0, round = 0;
      // first GEMM: Hacc[g & 1][128 x 128] = X * W1[:, tile g]
      for (int g = 0; g < G; ++g) {
        const int b = g & 1;
        if (g >= 2) {
          mbar_wait(bar_hfree + b, (uint32_t)((g - 2) >> 1) & 1u, abort_flag, p.status, 0x308);
          tcgen05_fence_after_sync();
        }
        for (int kb = 0; kb < p.kblocks; ++kb) {
          mbar_wait(bar_full + s, (uint32_t)round & 1u, abort_flag, p.status, 0x302);
          tcgen05_fence_after_sync();
          const uint32_t st = smem_u32(sRing + s * kStageBytes);
          const uint64_t ad = make_smem_desc(st, 0, 1024, SW_128B);
          const uint64_t bd = make_smem_desc(st + 16384, 8192, 1024, SW_128B);
#pragma unroll
          for (int ks = 0; ks < kBK / 16; ++ks)
            umma_bf16_elected_acc(tmem_base + b * kBH, ad + 2u * ks, bd + (uint64_t)((ks * 2048) >> 4), idesc, elected, (kb | ks) != 0);
          umma_commit_elected(bar_empty + s, elected);
          if (++s == stages) { s = 0; ++round; }
        }
        umma_commit_elected(bar_hacc + b, elected);
      }
      // second GEMM: acc[u & 1][128 x 128] = sum over the G tiles of H_g * W2[tile g, slice u]
      for (int u = 0; u < p.nslices; ++u) {
        const int ab = u & 1;
        if (u >= 2) {
          mbar_wait(bar_free + ab, (uint32_t)((u - 2) >> 1) & 1u, abort_flag, p.status, 0x305);
          tcgen05_fence_after_sync();
        }
        for (int g = 0; g < G; ++g) {
          if (u == 0) mbar_wait(bar_hsm + g, 0, abort_flag, p.status, 0x303);
          mbar_wait(bar_full + s, (uint32_t)round & 1u, abort_flag, p.status, 0x304);
          tcgen05_fence_after_sync();
          const uint64_t hdesc = make_smem_desc(smem_u32(sH + g * kStageBytes), 0, 1024, SW_128B);
          const uint64_t bd = make_smem_desc(smem_u32(sRing + s * kStageBytes), 16384, 1024, SW_128B);
#pragma unroll
          for (int ks = 0; ks < kBH / 16; ++ks)
            umma_bf16_elected_acc(tmem_base + kOutCol + ab * kBN, hdesc + (uint64_t)(((ks >> 2) * kBM * 128 + (ks & 3) * 32) >> 4),
                      bd + (uint64_t)((ks * 2048) >> 4), idesc, elected, (g | ks) != 0);
          umma_commit_elected(bar_empty + s, elected);
          if (++s == stages) { s = 0; ++round; }
        }
        umma_commit_elected(bar_out + ab, elected);
      }
    }
    __syncwarp();
  } else {
    // ================ epilogue warps: thread = (row, half of a tile's 128 columns) ================
    const int row = (warp & 3) * 32 + lane;
    const int half = warp >> 2;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const bool row_ok = row0 + row < p.M;

    // P3: H_g = GELU(Hacc + b1) -> bf16 -> shared memory; column half h is K block h of the tile
    for (int g = 0; g < G; ++g) {
      const int b = g & 1;
      mbar_wait(bar_hacc + b, (uint32_t)(g >> 1) & 1u, abort_flag, p.status, 0x306);
      tcgen05_fence_after_sync();
      uint8_t* tile = sH + g * kStageBytes + half * (kBM * 128);
      const float* bb = p.b1 + (size_t)(hc * G + g) * kBH + half * 64;
#pragma unroll
      for (int c0 = 0; c0 < 64; c0 += 32) {
        uint32_t v[32];
        tmem_ld_x32(tmem_base + lane_base + b * kBH + half * 64 + c0, v);
        tmem_ld_wait();
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 b0 = __ldg(reinterpret_cast<const float4*>(bb + c0 + q * 8));
          const float4 b1v = __ldg(reinterpret_cast<const float4*>(bb + c0 + q * 8 + 4));
          const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1v.x, b1v.y, b1v.z, b1v.w};
          uint32_t w[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int e = q * 8 + j * 2;
            w[j] = pack_bf16x2(gelu_tanh_fast(__uint_as_float(v[e]) + bv[2 * j]),
                               gelu_tanh_fast(__uint_as_float(v[e + 1]) + bv[2 * j + 1]));
          }
          *reinterpret_cast<uint4*>(tile + swz_offset(row, (c0 >> 3) + q, 128)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      fence_proxy_async_smem();
      tcgen05_fence_before_sync();
      named_barrier_sync(1, kEpiThreads);
      if (tid == 0) { mbar_arrive(bar_hsm + g); mbar_arrive(bar_hfree + b); }
    }

    // P6: drain every output slice into the fp32 accumulation buffer
    float* acc_row = p.acc + (size_t)(row0 + row) * p.N2 + half * 64;
    for (int u = 0; u < p.nslices; ++u) {
      const int ab = u & 1;
      const int slice = (u + hc) % p.nslices;   // same rotation as the producer's load order
      mbar_wait(bar_out + ab, (uint32_t)(u >> 1) & 1u, abort_flag, p.status, 0x307);
      tcgen05_fence_after_sync();
#pragma unroll
      for (int c0 = 0; c0 < 64; c0 += 32) {
        uint32_t v[32];
        tmem_ld_x32(tmem_base + lane_base + kOutCol + ab * kBN + half * 64 + c0, v);
        tmem_ld_wait();
        // 16-byte vector reductions: the L2 atomic units work per element, so fewer, wider
        // operations beat narrower coalesced ones (measured: 4-wide 1.4x faster than scalar)
        if (row_ok) {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            red_add_v4(acc_row + slice * kBN + c0 + j * 4, __uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                       __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
        }
      }
      tcgen05_fence_before_sync();
      named_barrier_sync(1, kEpiThreads);
      if (tid == 0) mbar_arrive(bar_free + ab);
    }

    // Last CTA of this row block: out = bf16(acc + b2); leave the buffer and the counter zeroed.
    __threadfence();
    named_barrier_sync(1, kEpiThreads);
    if (tid == 0) {
      const unsigned int prev = atomicAdd(p.counters + rb, 1u);
      *last_flag = (prev == (unsigned int)p.hctas - 1u) ? 1u : 0u;
    }
    named_barrier_sync(1, kEpiThreads);
    if (*last_flag) {
      __threadfence();
      // the epilogue threads sweep the row block's rows with coalesced 16-byte accesses, eight loads in flight per
      // thread (one CTA finalises a whole row block: the sweep is latency-bound otherwise)
      const int vec_per_row = p.N2 / 4;
      const int rows_here = min(kBM, p.M - row0);
      const int total = rows_here * vec_per_row;
      float4* acc0 = reinterpret_cast<float4*>(p.acc + (size_t)row0 * p.N2);      // the row block is contiguous
      uint2* out0 = reinterpret_cast<uint2*>(p.out + (size_t)row0 * p.N2);
      constexpr int kInFlight = 8;
      for (int base = tid; base < total; base += kInFlight * kEpiThreads) {
        float4 a[kInFlight];
#pragma unroll
        for (int k = 0; k < kInFlight; ++k) {
          const int idx = base + k * kEpiThreads;
          a[k] = idx < total ? __ldcg(acc0 + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int k = 0; k < kInFlight; ++k) {
          const int idx = base + k * kEpiThreads;
          if (idx < total) {
            const int c = (idx % vec_per_row) * 4;
            const float4 bb = __ldg(reinterpret_cast<const float4*>(p.b2 + c));
            acc0[idx] = make_float4(0.f, 0.f, 0.f, 0.f);
            out0[idx] = make_uint2(pack_bf16x2(a[k].x + bb.x, a[k].y + bb.y), pack_bf16x2(a[k].z + bb.z, a[k].w + bb.w));
          }
        }
      }
      if (tid == 0) p.counters[rb] = 0u;
    }
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, 512);
}

struct FfnHost {
  FfnParams prm;
  int smem_bytes = 0;
  size_t acc_bytes = 0, ws_bytes = 0;
  const void* clean_ws = nullptr;   // workspace known to be zeroed (kept so by the kernel itself) ...
  unsigned clean_epoch = 0;         // ... as of this attach (FusedState::workspace_epoch)
  struct Key { const void* p; int which; bool operator==(const Key& o) const { return p == o.p && which == o.which; } };
  struct KeyHash { size_t operator()(const Key& k) const { return std::hash<const void*>()(k.p) ^ (size_t)k.which * 0x9e3779b97f4a7c15ull; } };
  std::unordered_map<Key, CUtensorMap, KeyHash> maps;
};

}  // namespace

size_t ffn_workspace_bytes(const Plan& plan) {
  const int64_t M = plan.inputs[0].numel() / plan.inputs[0].last();
  const int64_t N2 = plan.output.last();
  const size_t acc = ((size_t)M * N2 * 4 + 255) & ~size_t(255);
  const size_t cnt = (((size_t)(M + kBM - 1) / kBM) * 4 + 255) & ~size_t(255);
  return acc + cnt;
}

ago_status_t ffn_plan(Plan* plan, FusedState* st, std::string* err) {
  auto* host = new FfnHost();
  FfnParams& q = host->prm;
  q = FfnParams{};
  q.K = (int)plan->inputs[0].last();
  q.M = (int)(plan->inputs[0].numel() / q.K);
  q.Hid = plan->ops[0].op.p[0];
  q.N2 = plan->ops[3].op.p[0];
  auto bad = [&](const char* m) { *err = std::string("fused feed-forward chain: ") + m; delete host; return AGO_ERR_UNSUPPORTED; };
  if (q.K % kBK != 0) return bad("input width must be a multiple of 64");
  if (q.Hid % kBH != 0) return bad("hidden width must be a multiple of 128");
  if (q.N2 % kBN != 0) return bad("output width must be a multiple of 128");
  q.kblocks = q.K / kBK; q.nslices = q.N2 / kBN;
  // Hidden tiles per CTA: as many as possible (each divides the reductions into the accumulation buffer), as long as
  // the grid still fills the SMs about twice; G tiles and the ring share seven 32 KB blocks of shared memory.
  const int htiles = q.Hid / kBH, row_blocks = (q.M + kBM - 1) / kBM;
  q.G = 1;
  for (int g = kMaxG; g >= 2; --g)
    if (htiles % g == 0 && (long)row_blocks * (htiles / g) >= 2 * device_sm_count()) { q.G = g; break; }
  q.hctas = htiles / q.G;
  q.stages = std::min(kMaxStages, 7 - q.G);
  host->smem_bytes = (q.stages + q.G) * kStageBytes + 256 + 1024;
  host->acc_bytes = ((size_t)q.M * q.N2 * 4 + 255) & ~size_t(255);
  host->ws_bytes = ffn_workspace_bytes(*plan);
  // every CTA of a row block adds its partial output rows into the fp32 buffer; the last one reads it back and zeroes it
  plan->workspace_traffic_bytes = (int64_t)(q.hctas + 2) * q.M * q.N2 * 4;
  st->impl = host;
  st->impl_free = [](void* p) { delete static_cast<FfnHost*>(p); };
  st->tile_rows = kBM; st->grid = q.hctas * ((q.M + kBM - 1) / kBM); st->smem_bytes = host->smem_bytes;
  plan->tile_rows = kBM; plan->smem_bytes = host->smem_bytes;
  return AGO_OK;
}

ago_status_t ffn_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                     void* output, void* workspace, unsigned int* status_word, cudaStream_t stream, std::string* err) {
  FfnHost* host = static_cast<FfnHost*>(st->impl);
  FfnParams q = host->prm;
  q.b1 = static_cast<const float*>(weights[1]);
  q.b2 = static_cast<const float*>(weights[3]);
  q.out = static_cast<__nv_bfloat16*>(output);
  q.acc = static_cast<float*>(workspace);
  q.counters = reinterpret_cast<unsigned int*>(static_cast<char*>(workspace) + host->acc_bytes);
  q.status = status_word;
  if (host->clean_ws != workspace || host->clean_epoch != st->workspace_epoch) {
    // a workspace is zeroed at the first run after each attach; after that every launch leaves it zeroed (the caller
    // must not touch it in between: see ago_subgraph_set_workspace)
    cudaError_t e = cudaMemsetAsync(workspace, 0, host->ws_bytes, stream);
    if (e != cudaSuccess) { *err = std::string("cudaMemsetAsync(workspace): ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
    host->clean_ws = workspace;
    host->clean_epoch = st->workspace_epoch;
  }
  auto get_map = [&](const void* base, int which, CUtensorMap* out) -> bool {
    FfnHost::Key key{base, which};
    auto it = host->maps.find(key);
    if (it == host->maps.end()) {
      CUtensorMap m;
      uint64_t dims[2]; uint64_t strides[1]; uint32_t box[2];
      if (which == 0) { dims[0] = q.K; dims[1] = q.M; strides[0] = (uint64_t)q.K * 2; box[0] = kBK; box[1] = kBM; }
      else if (which == 1) { dims[0] = q.Hid; dims[1] = q.K; strides[0] = (uint64_t)q.Hid * 2; box[0] = 64; box[1] = kBK; }
      else { dims[0] = q.N2; dims[1] = q.Hid; strides[0] = (uint64_t)q.N2 * 2; box[0] = 64; box[1] = kBH; }
      if (!encode_tmap_bf16(&m, base, 2, dims, strides, box, 128, err)) return false;
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
    cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(ffn_fused_kernel), smem_opt_in);
    if (e != cudaSuccess) { *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  }
  dim3 grid(q.hctas, (q.M + kBM - 1) / kBM);
  FusedLaunch launch(grid, kThreads, (size_t)host->smem_bytes, stream);
  cudaError_t e = cudaLaunchKernelEx(&launch.config, ffn_fused_kernel, mx, mw1, mw2, q);
  if (e != cudaSuccess) { *err = std::string("fused feed-forward launch: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  return AGO_OK;
}

}  // namespace ago
