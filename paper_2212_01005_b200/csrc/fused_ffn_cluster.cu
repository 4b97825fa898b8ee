// Fused feed-forward chain on a thread-block cluster: Y = GELU(X W1 + b1) W2 + b2; the hidden activations H never leave
// the SMs. With enough row blocks to fill the device nothing is reduced through device memory and the run is one kernel;
// with few row blocks (config 1: 512 rows) each row block's hidden tiles are split over J clusters, whose output shares
// meet in an fp32 buffer (J additions per element), and a second, small launch turns the buffer into the output.
//
// Tile choice (Section III-B, "downstream pointwise / matmul"): the second GEMM reuses H only along its output
// columns, so the downstream tile keeps ALL output columns of a block of 128 rows. Those (768 fp32 columns for
// BERT-base) do not fit the tensor memory of one SM next to the first GEMM's accumulator -- but they fit the tensor
// memory of a CLUSTER: CS CTAs (CS = 2..4) work on the same 128 rows, CTA r owns output columns
// [r N2/CS, (r+1) N2/CS) and computes every CS-th tile of 128 hidden units. A finished H tile (bias, GELU, bf16,
// 32 KB as a swizzled K-major operand) is copied to the same shared-memory slot of every peer with one bulk
// shared-to-shared copy per peer (distributed shared memory), so every H tile is computed once and multiplied
// into all N2 output columns without recomputation and without reductions outside the SM.
//
// Per CTA (rank r), T = hidden tiles / CS steps:
//   ring   TMA producer warp: 32 KB stages -- X [128 x 64] + W1 [64 x 128] for the first GEMM, W2 [64 x N2/CS]
//          for the second
//   MMA    one thread: G1(t+1): Hacc[(t+1) & 1] = X W1[:, tile (t+1) CS + r]; then for k = 0..CS-1
//          G2(k): out += H slot k * W2[tile t CS + k, own columns]; its completion is committed onto CTA k's
//          "slot consumed" barrier
//   epi    8 warps: Hacc[t & 1] -> + b1, GELU, bf16 -> own slot r (after every CTA has consumed its previous
//          content) -> announce locally, bulk-copy to the peers' slot r with completion on their "slot full" barrier
//   end    out (TMEM) -> + b2 -> bf16 -> device memory
// Every wait is bounded; a CTA leaves only after a cluster barrier, so no peer copies into an exited CTA.
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

constexpr int kBM = 128;        // rows per cluster
constexpr int kBH = 128;        // hidden units per tile
constexpr int kBK = 64;         // reduction elements per ring stage
constexpr int kMaxCS = 4;       // CTAs per cluster
constexpr int kBlocks = 7;      // 32 KB blocks of shared memory: CS slots for H tiles + ring stages
constexpr int kMaxStages = 5;
constexpr int kStageBytes = 32 * 1024;
constexpr int kEpiWarps = 8;    // two per tensor-memory lane quarter: each takes 64 of a tile's 128 columns
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kThreads = kEpiThreads + 64;   // + TMA warp + MMA warp
constexpr uint32_t kOutCol = 256;            // tensor memory: [0, 256) two first-GEMM accumulators, [256, 256 + NC) the output

struct FfnClusterParams {
  const float* b1;
  const float* b2;
  __nv_bfloat16* out;
  unsigned int* status;
  int M, K, Hid, N2;
  int CS, NC;              // CTAs per cluster, output columns per CTA (N2 / CS, a multiple of 64, <= 256)
  int T;                   // steps per row block = Hid / 128 / CS
  int J, Tp;               // a row block is split over J clusters, each with Tp = T / J of its steps (J = 1: no split)
  float* acc;              // J > 1: fp32 [M x N2] partial sums, zero between launches
  int kblocks;             // K / 64
  int stages;              // ring stages = 7 - CS (at most 5)
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
ffn_cluster_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w1,
                   const __grid_constant__ CUtensorMap tmap_w2, const FfnClusterParams p) {
  extern __shared__ uint8_t smem_raw[];
  // the same offset in every CTA of the cluster: peers address each other's slots and barriers by it
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int CS = p.CS, stages = p.stages;
  uint8_t* sRing = smem;                                   // stages x 32 KB
  uint8_t* sH = smem + stages * kStageBytes;               // CS slots x (2 x [128 x 64] bf16, 128-byte-swizzled)
  uint64_t* bars = reinterpret_cast<uint64_t*>(sH + CS * kStageBytes);
  uint64_t* bar_full = bars;                       // [kMaxStages] ring stage landed
  uint64_t* bar_empty = bars + kMaxStages;         // [kMaxStages] ring stage consumed
  uint64_t* bar_hacc = bars + 2 * kMaxStages;      // [2] first GEMM complete in accumulator b
  uint64_t* bar_hfree = bar_hacc + 2;              // [2] accumulator b drained
  uint64_t* bar_hfull = bar_hacc + 4;              // [kMaxCS] H tile present in slot k (from CTA k)
  uint64_t* bar_hdone = bar_hfull + kMaxCS;        // own slot consumed by every CTA of the cluster (count CS)
  uint64_t* bar_out = bar_hdone + 1;               // second GEMM of a row block complete
  uint64_t* bar_outfree = bar_out + 1;             // output accumulators drained: the next row block may overwrite them
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_outfree + 1);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bar_outfree + 2);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int r = (int)cluster_ctarank();
  const int T = p.Tp, J = p.J;
  // A unit of work is (row block, one of the J parts of its hidden tiles): T steps. A cluster walks over the units
  // blockIdx.y, + gridDim.y, ...: its steps form one sequence, so the first GEMM of the next unit overlaps the tail of
  // the current one. With J = 1 a unit is a whole row block and its output is final; with J > 1 (few row blocks: the
  // hidden dimension is what fills the SMs) the J clusters of a row block add their outputs in device memory.
  const int row_blocks = (p.M + kBM - 1) / kBM;
  const int units = row_blocks * J;
  const int my_units = ((int)blockIdx.y < units) ? (units - 1 - (int)blockIdx.y) / (int)gridDim.y + 1 : 0;
  const int steps = my_units * T;
  auto unit_of = [&](int step) { return (int)blockIdx.y + (step / T) * (int)gridDim.y; };
  auto row0_of = [&](int step) { return (unit_of(step) / J) * kBM; };
  auto tile0_of = [&](int step) { return ((unit_of(step) % J) * T + step % T) * CS; };   // first of the step's CS hidden tiles
  grid_dependency_wait();      // the previous grid of the stream has completed; device memory may be touched
  grid_launch_dependents();

  if (tid == kEpiThreads) {
    *abort_flag = 0u;
    for (int i = 0; i < kMaxStages; ++i) { mbar_init(bar_full + i, 1); mbar_init(bar_empty + i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar_hacc + i, 1); mbar_init(bar_hfree + i, 1); }
    for (int i = 0; i < kMaxCS; ++i) mbar_init(bar_hfull + i, 1);
    mbar_init(bar_hdone, (uint32_t)CS);
    mbar_init(bar_out, 1);
    mbar_init(bar_outfree, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  cluster_sync_all();          // every CTA's barriers exist before a peer signals them
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const int n0 = r * p.NC;     // first output column of this CTA

  if (warp == kEpiWarps) {
    // ================================ TMA producer ================================
    if (lane == 0) {
      tma_prefetch_desc(&tmap_x);
      tma_prefetch_desc(&tmap_w1);
      tma_prefetch_desc(&tmap_w2);
      int s = 0, round = 0;
      auto next_stage = [&]() -> uint8_t* {
        if (round > 0) mbar_wait(bar_empty + s, (uint32_t)(round - 1) & 1u, abort_flag, p.status, 0x701);
        mbar_arrive_expect_tx(bar_full + s, kStageBytes);
        return sRing + s * kStageBytes;
      };
      auto advance = [&]() { if (++s == stages) { s = 0; ++round; } };
      auto load_g1 = [&](int step) {       // first GEMM of this CTA's hidden tile of that step
        const int hid0 = (tile0_of(step) + r) * kBH, row0 = row0_of(step);
        for (int kb = 0; kb < p.kblocks; ++kb) {
          uint8_t* st = next_stage();
          tma_load_2d(st, &tmap_x, bar_full + s, kb * kBK, row0);                          // X [128 rows x 64 k]
          tma_load_2d(st + 16384, &tmap_w1, bar_full + s, hid0, kb * kBK);                 // W1 [64 k x 64 n] twice
          tma_load_2d(st + 16384 + 8192, &tmap_w1, bar_full + s, hid0 + 64, kb * kBK);
          advance();
        }
      };
      if (steps > 0) load_g1(0);
      for (int step = 0; step < steps; ++step) {
        if (step + 1 < steps) load_g1(step + 1);
        for (int i = 0; i < CS; ++i) {      // second GEMM over hidden tile t CS + k: two stages of 64 hidden units
          const int k = (int)((r + CS - i) % CS);   // in the order the MMA warp consumes the slots: own tile first
          const int hid0 = (tile0_of(step) + k) * kBH;
          for (int h = 0; h < 2; ++h) {
            uint8_t* st = next_stage();
            for (int nb = 0; nb < 4; ++nb)   // W2 [64 k x 64 n] per block; blocks past NC read as zero and are not multiplied
              tma_load_2d(st + nb * 8192, &tmap_w2, bar_full + s, nb * 64 < p.NC ? n0 + nb * 64 : p.N2, hid0 + h * 64);
            advance();
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == kEpiWarps + 1) {
    // ================================ MMA issuer ================================
    // the whole warp, converged; MMAs and commits predicated on one elected lane (see tc_common.cuh)
    {
      const uint32_t elected = elect_one();
      const uint32_t idesc1 = make_idesc_bf16(128, kBH, 0, 1);              // A K-major, B N-major (weights as they lie in memory)
      const uint32_t idesc2 = make_idesc_bf16(128, (uint32_t)p.NC, 0, 1);
      int s = 0, round = 0;
      auto advance = [&]() { if (++s == stages) { s = 0; ++round; } };
      auto g1 = [&](int step) {
        const int b = step & 1;
        if (step >= 2) {
          mbar_wait(bar_hfree + b, (uint32_t)((step - 2) >> 1) & 1u, abort_flag, p.status, 0x702);
          tcgen05_fence_after_sync();
        }
        for (int kb = 0; kb < p.kblocks; ++kb) {
          mbar_wait(bar_full + s, (uint32_t)round & 1u, abort_flag, p.status, 0x703);
          tcgen05_fence_after_sync();
          const uint32_t st = smem_u32(sRing + s * kStageBytes);
          const uint64_t ad = make_smem_desc(st, 0, 1024, SW_128B);
          const uint64_t bd = make_smem_desc(st + 16384, 8192, 1024, SW_128B);
#pragma unroll
          for (int ks = 0; ks < kBK / 16; ++ks)
            umma_bf16_elected_acc(tmem_base + b * kBH, ad + 2u * ks, bd + (uint64_t)((ks * 2048) >> 4), idesc1, elected, (kb | ks) != 0);
          umma_commit_elected(bar_empty + s, elected);
          advance();
        }
        umma_commit_elected(bar_hacc + b, elected);
      };
      if (steps > 0) g1(0);
      for (int step = 0; step < steps; ++step) {
        if (step + 1 < steps) g1(step + 1);
        const int t = step % T, bi = step / T;
        if (t == 0 && bi >= 1) {   // the output accumulators of the previous row block have been drained
          mbar_wait(bar_outfree, (uint32_t)(bi - 1) & 1u, abort_flag, p.status, 0x709);
          tcgen05_fence_after_sync();
        }
        // Slots in the order their tiles arrive: this CTA's own tile first (no copy), then the tiles of ranks r - 1,
        // r - 2, ... -- every producer sends to rank + 1 first, so rank r - q's tile is the q-th to land here.
        for (int i = 0; i < CS; ++i) {
          const int k = (int)((r + CS - i) % CS);
          mbar_wait(bar_hfull + k, (uint32_t)step & 1u, abort_flag, p.status, 0x704);   // H tile t CS + k is in slot k
          for (int h = 0; h < 2; ++h) {
            mbar_wait(bar_full + s, (uint32_t)round & 1u, abort_flag, p.status, 0x705);
            tcgen05_fence_after_sync();
            const uint64_t hd = make_smem_desc(smem_u32(sH + k * kStageBytes + h * (kBM * 128)), 0, 1024, SW_128B);
            const uint64_t bd = make_smem_desc(smem_u32(sRing + s * kStageBytes), 8192, 1024, SW_128B);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              umma_bf16_elected_acc(tmem_base + kOutCol, hd + 2u * ks, bd + (uint64_t)((ks * 2048) >> 4), idesc2, elected, (t | i | h | ks) != 0);
            umma_commit_elected(bar_empty + s, elected);
            advance();
          }
          // slot k of this CTA has been read: tell its producer (CTA k)
          umma_commit_cluster_elected(cluster_map(smem_u32(bar_hdone), (uint32_t)k), elected);
        }
        if (t == T - 1) umma_commit_elected(bar_out, elected);
      }
    }
    __syncwarp();
  } else {
    // ================ epilogue warps: thread = (row, half of a tile's 128 columns) ================
    const int row = (warp & 3) * 32 + lane;
    const int half = warp >> 2;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    uint8_t* slot = sH + r * kStageBytes;          // this CTA produces into slot r everywhere

    for (int step = 0; step < steps; ++step) {
      const int b = step & 1, t = step % T;
      mbar_wait(bar_hacc + b, (uint32_t)(step >> 1) & 1u, abort_flag, p.status, 0x706);
      tcgen05_fence_after_sync();
      // every CTA has multiplied the previous content of slot r (and the copies that delivered it are complete)
      if (step >= 1) mbar_wait(bar_hdone, (uint32_t)(step - 1) & 1u, abort_flag, p.status, 0x707);
      uint8_t* tile = slot + half * (kBM * 128);
      const float* bb = p.b1 + (size_t)(tile0_of(step) + r) * kBH + half * 64;
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
      fence_proxy_async_smem();      // the MMA and the bulk copies read the tile through the async proxy
      tcgen05_fence_before_sync();
      named_barrier_sync(1, kEpiThreads);
      if (tid == 0) {
        mbar_arrive(bar_hfree + b);
        mbar_arrive(bar_hfull + r);                                   // the local consumer
        const uint32_t src = smem_u32(slot), bar = smem_u32(bar_hfull + r);
        for (int q = 1; q < CS; ++q) {                                // the peers, starting with the next rank
          const uint32_t peer = (uint32_t)((r + q) % CS);
          const uint32_t rbar = cluster_map(bar, peer);
          mbar_remote_arrive_expect_tx(rbar, kStageBytes);
          bulk_copy_to_cluster(cluster_map(src, peer), src, kStageBytes, rbar);
        }
      }
      if (t == T - 1) {
        // ---- output of the row block: out (TMEM) -> + b2 -> bf16 -> device memory; thread = (row, half of the CTA's columns) ----
        const int bi = step / T, row0 = row0_of(step);
        const bool row_ok = row0 + row < p.M;
        mbar_wait(bar_out, (uint32_t)bi & 1u, abort_flag, p.status, 0x708);
        tcgen05_fence_after_sync();
        const int hc = p.NC >> 1;                                          // columns per half: 32, 64, 96 or 128
        if (J > 1) {
          // ---- split row block: add this cluster's share into the fp32 buffer; a second, small kernel turns the buffer
          // into the output (+ b2, bf16) with every SM of the device and leaves it zeroed. (A last-arriver sweep inside
          // this kernel -- one CTA per column slice reading 96 KB back -- took 8 us on the critical path.) ----
          float* arow = p.acc + (size_t)(row0 + row) * p.N2 + n0 + half * hc;
          for (int c0 = 0; c0 < hc; c0 += 32) {
            uint32_t v[32];
            tmem_ld_x32(tmem_base + lane_base + kOutCol + half * hc + c0, v);
            tmem_ld_wait();
            if (row_ok) {
#pragma unroll
              for (int q = 0; q < 8; ++q)
                red_add_v4(arow + c0 + q * 4, __uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                           __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
            }
          }
          tcgen05_fence_before_sync();
          named_barrier_sync(1, kEpiThreads);
          if (tid == 0) mbar_arrive(bar_outfree);
          continue;
        }
        __nv_bfloat16* orow = p.out + (size_t)(row0 + row) * p.N2 + n0 + half * hc;
        const float* b2 = p.b2 + n0 + half * hc;
        for (int c0 = 0; c0 < hc; c0 += 32) {
          uint32_t v[32];
          tmem_ld_x32(tmem_base + lane_base + kOutCol + half * hc + c0, v);
          tmem_ld_wait();
          if (row_ok) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const float4 b0 = __ldg(reinterpret_cast<const float4*>(b2 + c0 + q * 8));
              const float4 b1v = __ldg(reinterpret_cast<const float4*>(b2 + c0 + q * 8 + 4));
              *reinterpret_cast<uint4*>(orow + c0 + q * 8) =
                  make_uint4(pack_bf16x2(__uint_as_float(v[q * 8]) + b0.x, __uint_as_float(v[q * 8 + 1]) + b0.y),
                             pack_bf16x2(__uint_as_float(v[q * 8 + 2]) + b0.z, __uint_as_float(v[q * 8 + 3]) + b0.w),
                             pack_bf16x2(__uint_as_float(v[q * 8 + 4]) + b1v.x, __uint_as_float(v[q * 8 + 5]) + b1v.y),
                             pack_bf16x2(__uint_as_float(v[q * 8 + 6]) + b1v.z, __uint_as_float(v[q * 8 + 7]) + b1v.w));
            }
          }
        }
        tcgen05_fence_before_sync();
        named_barrier_sync(1, kEpiThreads);
        if (tid == 0) mbar_arrive(bar_outfree);
      }
    }
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  cluster_sync_all();          // no CTA leaves while a peer may still copy into it or signal its barriers
  if (warp == 0) tmem_dealloc(tmem_base, 512);
}

// Second launch of a split run: out = bf16(acc + b2), acc = 0. One float4 per thread and iteration, coalesced.
__global__ void __launch_bounds__(256) ffn_cluster_finalize_kernel(float* acc, const float* b2, __nv_bfloat16* out, long long total4, int n2) {
  grid_dependency_wait();      // the additions of the first launch are complete and visible
  grid_launch_dependents();
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total4; i += stride) {
    const float4 a = __ldcg(reinterpret_cast<const float4*>(acc) + i);
    const float4 bb = __ldg(reinterpret_cast<const float4*>(b2 + (int)((i * 4) % n2)));
    reinterpret_cast<float4*>(acc)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    reinterpret_cast<uint2*>(out)[i] = make_uint2(pack_bf16x2(a.x + bb.x, a.y + bb.y), pack_bf16x2(a.z + bb.z, a.w + bb.w));
  }
}

struct FfnClusterHost {
  FfnClusterParams prm;
  int smem_bytes = 0;
  int clusters = 0;   // clusters launched = min(units of work, clusters the device keeps resident); 0: not asked yet
  size_t acc_bytes = 0, ws_bytes = 0;   // split row blocks: fp32 partial sums
  const void* clean_ws = nullptr;   // workspace known to be zeroed (kept so by the kernel itself) ...
  unsigned clean_epoch = 0;         // ... as of this attach (FusedState::workspace_epoch)
  struct Key { const void* p; int which; bool operator==(const Key& o) const { return p == o.p && which == o.which; } };
  struct KeyHash { size_t operator()(const Key& k) const { return std::hash<const void*>()(k.p) ^ (size_t)k.which * 0x9e3779b97f4a7c15ull; } };
  std::unordered_map<Key, CUtensorMap, KeyHash> maps;
};

void fill_launch(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, const FfnClusterParams& q, int clusters, int smem_bytes,
                 cudaStream_t stream) {
  *cfg = cudaLaunchConfig_t{};
  cfg->gridDim = dim3((unsigned)q.CS, (unsigned)clusters, 1);
  cfg->blockDim = dim3(kThreads, 1, 1);
  cfg->dynamicSmemBytes = (size_t)smem_bytes;
  cfg->stream = stream;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)q.CS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg->attrs = attr;
  cfg->numAttrs = 2;
}

}  // namespace

// AGO_ERR_UNSUPPORTED (without touching *err) when the shape has no cluster split: the caller falls back to the
// kernel that tiles the second GEMM's reduction across independent CTAs.
ago_status_t ffn_cluster_plan(Plan* plan, FusedState* st, std::string* err) {
  (void)err;
  FfnClusterParams q{};
  q.K = (int)plan->inputs[0].last();
  q.M = (int)(plan->inputs[0].numel() / q.K);
  q.Hid = plan->ops[0].op.p[0];
  q.N2 = plan->ops[3].op.p[0];
  if (q.K % kBK != 0 || q.Hid % kBH != 0) return AGO_ERR_UNSUPPORTED;
  const int htiles = q.Hid / kBH;
  // Cluster size: among the sizes whose column share fits tensor memory, the one with the least estimated time =
  // rounds of resident clusters x steps per row block x ring stages per step. Resident clusters of 1-CTA-per-SM
  // kernels on a B200 (148 SMs in GPCs of unequal size), as cudaOccupancyMaxActiveClusters reports them: 74 / 45 / 33
  // for sizes 2 / 3 / 4; the launch asks the device again and sizes its grid by the answer.
  const int row_blocks_plan = (q.M + kBM - 1) / kBM;
  const int resident[kMaxCS + 1] = {0, 0, 74, 45, 33};
  q.CS = 0;
  long best = 0;
  for (int cs = 2; cs <= kMaxCS; ++cs) {
    if (q.N2 % cs != 0 || htiles % cs != 0) continue;
    const int nc = q.N2 / cs;
    if (nc % 64 != 0 || nc > 256) continue;
    const long rounds = (row_blocks_plan + resident[cs] - 1) / resident[cs];
    const long cost = rounds * (htiles / cs) * (q.K / kBK + 2 * cs);
    if (q.CS == 0 || cost < best) { q.CS = cs; q.NC = nc; best = cost; }
  }
  if (q.CS == 0) return AGO_ERR_UNSUPPORTED;
  q.T = htiles / q.CS;
  q.J = 1;
  if ((long)row_blocks_plan * q.CS < 120) {
    // Few row blocks: one cluster per block of 128 rows leaves most SMs idle, and the hidden dimension is what can fill
    // them. A row block is split over J clusters (J divides its T steps); their outputs meet in an fp32 buffer in device
    // memory, J additions per element instead of one per hidden tile. J = as many parts as still fit one round of
    // resident clusters, each with at least one step.
    for (int j = q.T; j >= 1; --j)
      if (q.T % j == 0 && (long)row_blocks_plan * j <= resident[q.CS]) { q.J = j; break; }
    if (q.J == 1 || q.N2 % 4 != 0 || (q.NC / 2) % 32 != 0) return AGO_ERR_UNSUPPORTED;   // nothing to split: the other kernel
  }
  q.Tp = q.T / q.J;
  q.kblocks = q.K / kBK;
  q.stages = std::min(kMaxStages, kBlocks - q.CS);
  auto* host = new FfnClusterHost();
  host->prm = q;
  host->smem_bytes = (q.stages + q.CS) * kStageBytes + 256 + 1024;
  st->impl = host;
  st->impl_free = [](void* p) { delete static_cast<FfnClusterHost*>(p); };
  st->variant = 1;
  st->tile_rows = kBM; st->grid = q.CS * q.J * ((q.M + kBM - 1) / kBM); st->smem_bytes = host->smem_bytes;
  plan->tile_rows = kBM; plan->smem_bytes = host->smem_bytes;
  plan->fused_variant = q.J > 1 ? 2 : 1;
  if (q.J > 1) {
    host->acc_bytes = ((size_t)q.M * q.N2 * 4 + 255) & ~size_t(255);
    host->ws_bytes = host->acc_bytes;
    // every cluster of a row block adds its share into the buffer; the second launch reads it back and zeroes it
    plan->workspace_traffic_bytes = (int64_t)(q.J + 2) * q.M * q.N2 * 4;
    plan->num_launches = 2;
  }
  return AGO_OK;
}

size_t ffn_cluster_workspace_bytes(const Plan& plan) {
  if (plan.fused_variant != 2) return 0;
  const int64_t M = plan.inputs[0].numel() / plan.inputs[0].last();
  const int64_t N2 = plan.output.last();
  return ((size_t)M * N2 * 4 + 255) & ~size_t(255);
}

ago_status_t ffn_cluster_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                             void* output, void* workspace, unsigned int* status_word, cudaStream_t stream, std::string* err) {
  (void)plan;
  FfnClusterHost* host = static_cast<FfnClusterHost*>(st->impl);
  FfnClusterParams q = host->prm;
  q.b1 = static_cast<const float*>(weights[1]);
  q.b2 = static_cast<const float*>(weights[3]);
  q.out = static_cast<__nv_bfloat16*>(output);
  q.status = status_word;
  if (q.J > 1) {
    if (!workspace) { *err = "fused feed-forward (cluster, split row blocks): no workspace attached"; return AGO_ERR_INVALID_ARG; }
    q.acc = static_cast<float*>(workspace);
    if (host->clean_ws != workspace || host->clean_epoch != st->workspace_epoch) {
      // a workspace is zeroed at the first run after each attach; after that every launch leaves it zeroed (the caller
      // must not touch it in between)
      cudaError_t e = cudaMemsetAsync(workspace, 0, host->ws_bytes, stream);
      if (e != cudaSuccess) { *err = std::string("cudaMemsetAsync(workspace): ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
      host->clean_ws = workspace;
      host->clean_epoch = st->workspace_epoch;
    }
  }
  auto get_map = [&](const void* base, int which, CUtensorMap* out) -> bool {
    FfnClusterHost::Key key{base, which};
    auto it = host->maps.find(key);
    if (it == host->maps.end()) {
      CUtensorMap m;
      uint64_t dims[2]; uint64_t strides[1]; uint32_t box[2];
      if (which == 0) { dims[0] = q.K; dims[1] = q.M; strides[0] = (uint64_t)q.K * 2; box[0] = kBK; box[1] = kBM; }
      else if (which == 1) { dims[0] = q.Hid; dims[1] = q.K; strides[0] = (uint64_t)q.Hid * 2; box[0] = 64; box[1] = kBK; }
      else { dims[0] = q.N2; dims[1] = q.Hid; strides[0] = (uint64_t)q.N2 * 2; box[0] = 64; box[1] = 64; }
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
    cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(ffn_cluster_kernel), smem_opt_in);
    if (e != cudaSuccess) { *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  }
  cudaLaunchConfig_t cfg; cudaLaunchAttribute attr[2];
  const int row_blocks = (q.M + kBM - 1) / kBM;
  if (host->clusters == 0) {
    // persistent clusters: as many as the device keeps resident at once (one CTA per SM, CS SMs of one GPC each)
    fill_launch(&cfg, attr, q, row_blocks * q.J, host->smem_bytes, stream);
    int resident = 0;
    cudaError_t e = cudaOccupancyMaxActiveClusters(&resident, ffn_cluster_kernel, &cfg);
    if (e != cudaSuccess || resident < 1) {
      *err = std::string("fused feed-forward (cluster): no cluster of this size is schedulable: ") + cudaGetErrorString(e);
      return AGO_ERR_CUDA;
    }
    host->clusters = std::min(row_blocks * q.J, resident);
  }
  fill_launch(&cfg, attr, q, host->clusters, host->smem_bytes, stream);
  cudaError_t e = cudaLaunchKernelEx(&cfg, ffn_cluster_kernel, mx, mw1, mw2, q);
  if (e != cudaSuccess) { *err = std::string("fused feed-forward (cluster) launch: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  if (q.J > 1) {
    const long long total4 = (long long)q.M * q.N2 / 4;
    const int blocks = (int)std::min<long long>((total4 + 255) / 256, 4LL * device_sm_count());
    FusedLaunch fin(dim3((unsigned)blocks), 256, 0, stream);
    e = cudaLaunchKernelEx(&fin.config, ffn_cluster_finalize_kernel, q.acc, q.b2, q.out, total4, q.N2);
    if (e != cudaSuccess) { *err = std::string("fused feed-forward (cluster) finalisation launch: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  }
  return AGO_OK;
}

}  // namespace ago
