// Fused feed-forward chain on a cluster of two CTA PAIRS: Y = GELU(X W1 + b1) W2 + b2, one kernel; the hidden
// activations H never leave the SMs, nothing is recomputed and nothing is reduced through device memory.
//
// Tile choice (Section III-B, "downstream pointwise / matmul": keep ALL output columns of a block of rows, tile the
// rows). A cluster of four CTAs works on 256 rows. Ranks (0, 1) and (2, 3) are pairs whose MMAs span both CTAs
// (tcgen05.mma.cta_group::2, M = 256: CTA h of a pair holds rows h * 128 .. of X, of H and of the accumulators, and
// one half of every B tile). Pair P owns the output columns [P * N2 / 2, (P + 1) * N2 / 2) -- 384 fp32 columns of
// tensor memory for BERT-base, next to one 128-column accumulator of the first GEMM -- and computes every second
// tile of 128 hidden units. A finished H tile (bias, GELU, bf16; 32 KB per CTA as a swizzled K-major operand) stays
// in the CTA that made it and is copied once, by a bulk shared-to-shared copy (distributed shared memory, no
// multicast), to the CTA of the other pair that holds the same rows; both pairs then multiply it into their own
// output columns.
//
// Why pairs: with unpaired CTAs every SM streams a whole 128-wide B tile per 128 rows (64 - 128 flop per byte that
// crosses L2 -> SM, and that link, about 9 TB/s in all, is what bounds the unpaired cluster kernel). A pair streams
// each B tile once for 256 rows: 131 flop per byte for the chain at BERT-base widths.
//
// Per CTA (pair P, half h; h == 0 leads its pair), steps g = (row block, own hidden tile):
//   TMA     one thread: 24 KB stages -- X [128 x 64] + W1 [64 x 64] (this CTA's half of the tile) for the first
//           GEMM, W2 [64 x N2 / 4] for the second. Both CTAs' loads complete on the leader's barrier.
//   MMA     one warp of the leader, converged, an elected lane issuing: G1(g + 1) into the H accumulator, then G2 over
//           the two H tiles of step g
//   epi     8 warps: H accumulator -> registers (accumulator handed back at once) -> + b1, GELU, bf16 -> own slot
//           -> local "slot full" + bulk copy to the other pair; at the end of a row block: out -> + b2 -> bf16 -> Y
//   helper  one thread: arms the barrier the other pair's copy completes on; in the non-leading CTA it also relays
//           "accumulator drained" to the leader, and a thread of the idle MMA warp relays "slots full" and
//           "output drained". (An arrival on another CTA's barrier is a release at cluster scope and costs about a
//           thousand cycles: it is kept off the threads that feed the tensor pipe.)
// Rounds: the clusters the device keeps resident (33 of four CTAs on a B200) walk over the blocks of 256 rows. The blocks of
// a last, partial round are split into J parts of S / J steps on J clusters; part j stores its fp32 output share in plane j
// of the workspace (plain stores) and a second, elementwise launch adds the planes, + b2, -> bf16.
// Every wait is bounded; a CTA leaves only after a cluster barrier.
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

constexpr int kFM = 128;          // rows per CTA (256 per pair and per cluster)
constexpr int kFH = 128;          // hidden units per tile
constexpr int kFK = 64;           // reduction elements per ring stage
constexpr int kFStages = 6;
constexpr int kFStageBytes = 24 * 1024;
constexpr int kFSlotBytes = 32 * 1024;      // one H tile of this CTA's rows: 2 x [128 x 64] bf16, 128-byte swizzled
constexpr int kFEpiWarps = 8;
constexpr int kFEpiThreads = kFEpiWarps * 32;
constexpr int kFThreads = kFEpiThreads + 96;   // + TMA warp + MMA warp + helper warp
constexpr uint32_t kFOutCol = 128;          // tensor memory: [0, 128) first-GEMM accumulator, [128, 128 + NC) the output
constexpr int kFSmemBytes = kFStages * kFStageBytes + 2 * kFSlotBytes + 512 + 1024;

struct FfnPairParams {
  const float* b1;
  const float* b2;
  __nv_bfloat16* out;
  unsigned int* status;
  int M, K, Hid, N2;
  int NC;                  // output columns per pair = N2 / 2: 128, 256 or 384
  int S;                   // steps per row block = Hid / 256
  int kblocks;             // K / 64
  int units;               // blocks of 256 rows
  // The blocks of the last, partial round of resident clusters are split: each of the blocks [units_whole, units) is
  // shared by J clusters, S / J steps each; part j stores its output share as fp32 in plane j of a buffer in device
  // memory (plain stores: no atomics, nothing to zero, the same bits on every run) and a second launch adds the planes.
  int units_whole, J;
  float* acc;              // [J][split_rows][N2] fp32
  int split_rows;          // rows of the split blocks that exist: M - units_whole * 256
};

__device__ __forceinline__ float gelu_tanh_pair(float v) {
  const float u = 0.7978845608028654f * (v + 0.044715f * v * v * v);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
  return 0.5f * v * (1.0f + t);
}

__global__ void __launch_bounds__(kFThreads, 1)
ffn_pair_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w1,
                const __grid_constant__ CUtensorMap tmap_w2, const FfnPairParams p) {
  extern __shared__ uint8_t smem_raw[];
  // the same offsets in every CTA of the cluster: pairs and peers address each other's tiles and barriers by them
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sRing = smem;
  uint8_t* sH = smem + kFStages * kFStageBytes;          // slot k: the H tile made by pair k (these rows)
  uint64_t* bars = reinterpret_cast<uint64_t*>(sH + 2 * kFSlotBytes);
  uint64_t* bar_full = bars;                    // [6] leader: ring stage landed in both CTAs
  uint64_t* bar_empty = bars + 6;               // [6] ring stage consumed
  uint64_t* bar_hacc = bars + 12;               // first GEMM of a step complete (this CTA's rows)
  uint64_t* bar_hfree = bars + 13;              // this CTA's epilogue has read the H accumulator
  uint64_t* bar_phfree = bars + 14;             // leader: the same, relayed from the other CTA of the pair
  uint64_t* bar_slot = bars + 15;               // [2] the H tile of pair k is in slot k of this CTA
  uint64_t* bar_pslots = bars + 17;             // leader: both slots of the other CTA of the pair are full (relayed)
  uint64_t* bar_hdone = bars + 18;              // the tile this CTA made has been multiplied by both pairs (count 2)
  uint64_t* bar_out = bars + 19;                // second GEMM of a row block complete
  uint64_t* bar_outfree = bars + 20;            // this CTA's epilogue has read the output accumulators
  uint64_t* bar_poutfree = bars + 21;           // leader: the same, relayed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 22);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 23);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const int P = (int)(rank >> 1), h = (int)(rank & 1u);
  const bool leader = h == 0;
  const uint32_t lead_rank = rank & ~1u, mate_rank = rank ^ 1u, twin_rank = rank ^ 2u;   // pair leader, other CTA of the pair, same rows in the other pair
  const int S = p.S;
  // Work items: the whole blocks [0, units_whole), then J parts of S / J steps for each of the other blocks. A cluster
  // walks over the items blockIdx.y, + gridDim.y, ... (whole blocks first); its steps form one sequence.
  const int G = (int)gridDim.y, cidx = (int)blockIdx.y, Sp = S / p.J;
  const int n_all = p.units_whole + (p.units - p.units_whole) * p.J;
  const int n_items = cidx < n_all ? (n_all - 1 - cidx) / G + 1 : 0;
  const int n_w = cidx < p.units_whole ? (p.units_whole - 1 - cidx) / G + 1 : 0;
  const int steps = n_w * S + (n_items - n_w) * Sp;
  struct Step { int item, unit, sb, part; bool first, last, split; };   // sb: index of the pair of hidden tiles inside the block
  auto step_of = [&](int g) {
    Step r;
    if (g < n_w * S) {
      r.item = g / S; r.sb = g - r.item * S; r.unit = cidx + r.item * G;
      r.first = r.sb == 0; r.last = r.sb == S - 1; r.split = false; r.part = 0;
    } else {
      const int g2 = g - n_w * S, k = g2 / Sp, sp = g2 - k * Sp, q = cidx + (n_w + k) * G - p.units_whole;
      r.item = n_w + k; r.unit = p.units_whole + q / p.J; r.part = q % p.J; r.sb = r.part * Sp + sp;
      r.first = sp == 0; r.last = sp == Sp - 1; r.split = true;
    }
    return r;
  };
  // output chunks of the pair's NC columns: one MMA each (N <= 256): 128 | 256 | 256 + 128
  const int cn0 = min(p.NC, 256), cn1 = p.NC - cn0;
  const uint32_t g2_tx = (uint32_t)(p.NC / 2) * kFK * 2u;            // W2 bytes per stage and CTA
  const uint32_t g1_tx = (uint32_t)(kFM * kFK * 2 + 64 * kFK * 2);   // X + W1 bytes per stage and CTA
  grid_dependency_wait();
  grid_launch_dependents();

  if (tid == kFEpiThreads) {
    *abort_flag = 0u;
    for (int i = 0; i < 6; ++i) { mbar_init(bar_full + i, 1); mbar_init(bar_empty + i, 1); }
    mbar_init(bar_hacc, 1); mbar_init(bar_hfree, 1); mbar_init(bar_phfree, 1);
    mbar_init(bar_slot, 1); mbar_init(bar_slot + 1, 1); mbar_init(bar_pslots, 1);
    mbar_init(bar_hdone, 2);
    mbar_init(bar_out, 1); mbar_init(bar_outfree, 1); mbar_init(bar_poutfree, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == kFEpiWarps + 1) {      // a pair-wide allocation is issued by a warp of either CTA
    tmem_alloc_pair(tmem_slot, 512);
    tmem_relinquish_pair();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == kFEpiWarps) {
    // ================================ TMA producer (every CTA) ================================
    if (lane == 0) {
      tma_prefetch_desc(&tmap_x);
      tma_prefetch_desc(&tmap_w1);
      tma_prefetch_desc(&tmap_w2);
      int s = 0, round = 0;
      auto next_stage = [&](uint32_t tx_per_cta, uint32_t* full) -> uint8_t* {
        if (round > 0) mbar_wait_poll(bar_empty + s, (uint32_t)(round - 1) & 1u, abort_flag, p.status, 0x801);
        *full = cluster_map(smem_u32(bar_full + s), lead_rank);
        if (leader) mbar_arrive_expect_tx(bar_full + s, 2u * tx_per_cta);   // the leader announces both CTAs' bytes
        return sRing + s * kFStageBytes;
      };
      auto advance = [&]() { if (++s == kFStages) { s = 0; ++round; } };
      auto load_g1 = [&](int g) {       // first GEMM of the pair's hidden tile of step g: this CTA's rows, its half of the tile
        const Step st_ = step_of(g);
        const int hid0 = (2 * st_.sb + P) * kFH + h * 64, row0 = st_.unit * 2 * kFM + h * kFM;
        for (int kb = 0; kb < p.kblocks; ++kb) {
          uint32_t full;
          uint8_t* st = next_stage(g1_tx, &full);
          tma_load_2d_pair(st, &tmap_x, full, kb * kFK, row0);                   // X [128 rows x 64 k]
          tma_load_2d_pair(st + 16384, &tmap_w1, full, hid0, kb * kFK);          // W1 [64 k x 64 hidden]
          advance();
        }
      };
      if (steps > 0) load_g1(0);
      for (int g = 0; g < steps; ++g) {
        if (g + 1 < steps) load_g1(g + 1);
        for (int k = 0; k < 2; ++k) {   // second GEMM over the H tile of pair k: two stages of 64 hidden units
          const int hid0 = (2 * step_of(g).sb + k) * kFH;
          for (int kk = 0; kk < 2; ++kk) {
            uint32_t full;
            uint8_t* st = next_stage(g2_tx, &full);
            // this CTA's half of every output chunk, as blocks of [64 k x 64 n]
            const int c_first = P * p.NC + h * (cn0 / 2);
            for (int nb = 0; nb < cn0 / 2; nb += 64)
              tma_load_2d_pair(st + (nb >> 6) * 8192, &tmap_w2, full, c_first + nb, hid0 + kk * 64);
            if (cn1 > 0) tma_load_2d_pair(st + (cn0 / 128) * 8192, &tmap_w2, full, P * p.NC + cn0 + h * (cn1 / 2), hid0 + kk * 64);
            advance();
          }
        }
      }
    }
    __syncwarp();
  }
  else if (warp == kFEpiWarps + 1) {
    if (leader) {
      // ================================ MMA issuer (pair leader): whole warp, elected lane issues ================================
      const uint32_t elected = elect_one();
      const uint32_t idesc1 = make_idesc_bf16(256, kFH, 0, 1);               // A K-major, B N-major (weights as they lie in memory)
      const uint32_t idesc2a = make_idesc_bf16(256, (uint32_t)cn0, 0, 1);
      const uint32_t idesc2b = make_idesc_bf16(256, (uint32_t)max(cn1, 16), 0, 1);
      int s = 0, round = 0;
      auto advance = [&]() { if (++s == kFStages) { s = 0; ++round; } };
      auto commit_pair_bar = [&](uint64_t* bar) {      // onto the same barrier of both CTAs of this pair
        const uint32_t e = smem_u32(bar);
        umma_commit_pair_elected(cluster_map(e, rank), elected);
        umma_commit_pair_elected(cluster_map(e, mate_rank), elected);
      };
      auto g1 = [&](int g) {
        if (g >= 1) {      // both CTAs have read the accumulator of step g - 1 out of tensor memory
          mbar_wait_poll(bar_hfree, (uint32_t)(g - 1) & 1u, abort_flag, p.status, 0x802);
          mbar_wait_poll(bar_phfree, (uint32_t)(g - 1) & 1u, abort_flag, p.status, 0x803);
          tcgen05_fence_after_sync();
        }
        for (int kb = 0; kb < p.kblocks; ++kb) {
          mbar_wait_poll(bar_full + s, (uint32_t)round & 1u, abort_flag, p.status, 0x804);
          tcgen05_fence_after_sync();
          const uint32_t st = smem_u32(sRing + s * kFStageBytes);
          const uint64_t ad = make_smem_desc(st, 0, 1024, SW_128B);
          const uint64_t bd = make_smem_desc(st + 16384, 8192, 1024, SW_128B);
#pragma unroll
          for (int ks = 0; ks < kFK / 16; ++ks)
            umma_bf16_pair_elected(tmem_base, ad + 2u * ks, bd + (uint64_t)((ks * 2048) >> 4), idesc1, elected, (kb | ks) != 0);
          commit_pair_bar(bar_empty + s);
          advance();
        }
        commit_pair_bar(bar_hacc);
      };
      if (steps > 0) g1(0);
      for (int g = 0; g < steps; ++g) {
        if (g + 1 < steps) g1(g + 1);
        const Step cur = step_of(g);
        const int bi = cur.item;
        if (cur.first && bi >= 1) {   // the output accumulators of the previous row block have been read in both CTAs
          mbar_wait_poll(bar_outfree, (uint32_t)(bi - 1) & 1u, abort_flag, p.status, 0x805);
          mbar_wait_poll(bar_poutfree, (uint32_t)(bi - 1) & 1u, abort_flag, p.status, 0x806);
          tcgen05_fence_after_sync();
        }
        mbar_wait_poll(bar_pslots, (uint32_t)g & 1u, abort_flag, p.status, 0x807);     // both tiles of step g are in the other CTA
        for (int k = 0; k < 2; ++k) {
          mbar_wait_poll(bar_slot + k, (uint32_t)g & 1u, abort_flag, p.status, 0x808);  // ... and tile k is here
          tcgen05_fence_after_sync();
          for (int kk = 0; kk < 2; ++kk) {
            mbar_wait_poll(bar_full + s, (uint32_t)round & 1u, abort_flag, p.status, 0x809);
            tcgen05_fence_after_sync();
            const uint32_t st = smem_u32(sRing + s * kFStageBytes);
            const uint64_t hd = make_smem_desc(smem_u32(sH + k * kFSlotBytes + kk * (kFM * 128)), 0, 1024, SW_128B);
            const uint64_t bd0 = make_smem_desc(st, 8192, 1024, SW_128B);
            const uint64_t bd1 = make_smem_desc(st + (uint32_t)(cn0 / 128) * 8192u, 8192, 1024, SW_128B);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint32_t acc = (uint32_t)(!cur.first || (k | kk | ks) != 0);
              umma_bf16_pair_elected(tmem_base + kFOutCol, hd + 2u * ks, bd0 + (uint64_t)((ks * 2048) >> 4), idesc2a, elected, acc);
              if (cn1 > 0) umma_bf16_pair_elected(tmem_base + kFOutCol + (uint32_t)cn0, hd + 2u * ks, bd1 + (uint64_t)((ks * 2048) >> 4), idesc2b, elected, acc);
            }
            commit_pair_bar(bar_empty + s);
            advance();
          }
          // slot k has been read in both CTAs of this pair: tell the CTAs that made the tile (pair k)
          const uint32_t e = smem_u32(bar_hdone);
          umma_commit_pair_elected(cluster_map(e, (uint32_t)(2 * k)), elected);
          umma_commit_pair_elected(cluster_map(e, (uint32_t)(2 * k + 1)), elected);
        }
        if (cur.last) commit_pair_bar(bar_out);
      }
    } else if (lane == 0) {
      // ============ relay (the CTA that does not lead): "both slots full", "output drained" -> leader ============
      const uint32_t lead_pslots = cluster_map(smem_u32(bar_pslots), lead_rank);
      const uint32_t lead_poutfree = cluster_map(smem_u32(bar_poutfree), lead_rank);
      for (int g = 0; g < steps; ++g) {
        mbar_wait(bar_slot, (uint32_t)g & 1u, abort_flag, p.status, 0x80a);
        mbar_wait(bar_slot + 1, (uint32_t)g & 1u, abort_flag, p.status, 0x80b);
        mbar_remote_arrive(lead_pslots);
        const Step cur = step_of(g);
        if (cur.first && cur.item >= 1) {
          mbar_wait(bar_outfree, (uint32_t)(cur.item - 1) & 1u, abort_flag, p.status, 0x80c);
          mbar_remote_arrive(lead_poutfree);
        }
      }
    }
    __syncwarp();
  } else if (warp == kFEpiWarps + 2) {
    // ============ helper: arms the barrier of the other pair's copy; relays "accumulator drained" ============
    if (lane == 0) {
      const uint32_t lead_phfree = cluster_map(smem_u32(bar_phfree), lead_rank);
      for (int g = 0; g < steps; ++g) {
        mbar_arrive_expect_tx(bar_slot + (1 - P), (uint32_t)kFSlotBytes);
        if (!leader) {
          mbar_wait(bar_hfree, (uint32_t)g & 1u, abort_flag, p.status, 0x80d);
          mbar_remote_arrive(lead_phfree);
        }
        mbar_wait(bar_slot + (1 - P), (uint32_t)g & 1u, abort_flag, p.status, 0x80e);   // complete before the next phase is armed
      }
    }
    __syncwarp();
  }
  else if (warp < kFEpiWarps) {
    // ================ epilogue warps: thread = (row, half of a tile's 128 hidden units / of the pair's output columns) ================
    const int row = (warp & 3) * 32 + lane;
    const int half = warp >> 2;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    uint8_t* slot = sH + P * kFSlotBytes;          // this pair's tiles live in slot P of every CTA
    const uint32_t twin_slot = cluster_map(smem_u32(slot), twin_rank);
    const uint32_t twin_bar = cluster_map(smem_u32(bar_slot + P), twin_rank);
    const int hc = p.NC >> 1;                      // output columns per thread: 64, 128 or 192

    auto drain_output = [&](int bi, int unit, bool split, int part) {
      // ---- output of work item bi: out (TMEM) -> + b2 -> bf16 -> device memory; the share of a part of a split block goes
      // to its plane of the fp32 buffer instead (a second, small kernel adds the planes and writes the output) ----
      const int row0 = unit * 2 * kFM + h * kFM;
      const bool row_ok = row0 + row < p.M;
      mbar_wait(bar_out, (uint32_t)bi & 1u, abort_flag, p.status, 0x80f);
      tcgen05_fence_after_sync();
      const int n0 = P * p.NC + half * hc;
      if (split) {
        float* arow = p.acc + ((size_t)part * p.split_rows + (size_t)(row0 + row - p.units_whole * 2 * kFM)) * p.N2 + n0;
        for (int c0 = 0; c0 < hc; c0 += 32) {
          uint32_t v[32];
          tmem_ld_x32(tmem_base + lane_base + kFOutCol + (uint32_t)(half * hc + c0), v);
          tmem_ld_wait();
          if (row_ok) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
              *reinterpret_cast<uint4*>(arow + c0 + q * 4) = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
          }
        }
        tcgen05_fence_before_sync();
        named_barrier_sync(1, kFEpiThreads);
        if (tid == 0) mbar_arrive(bar_outfree);
        return;
      }
      __nv_bfloat16* orow = p.out + (size_t)(row0 + row) * p.N2 + n0;
      const float* b2 = p.b2 + n0;
      for (int c0 = 0; c0 < hc; c0 += 32) {
        uint32_t v[32];
        tmem_ld_x32(tmem_base + lane_base + kFOutCol + (uint32_t)(half * hc + c0), v);
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
      named_barrier_sync(1, kFEpiThreads);
      if (tid == 0) mbar_arrive(bar_outfree);
    };

    int prev_item = 0, prev_unit = 0, prev_part = 0; bool prev_split = false;     // the item whose last step has been seen
    for (int g = 0; g < steps; ++g) {
      const Step cur = step_of(g);
      const int sb = cur.sb;
      mbar_wait(bar_hacc, (uint32_t)g & 1u, abort_flag, p.status, 0x810);
      tcgen05_fence_after_sync();
      // the whole share of this thread goes to registers first, so that the accumulator is free for the next first GEMM
      uint32_t v[64];
      tmem_ld_x32(tmem_base + lane_base + (uint32_t)(half * 64), v);
      tmem_ld_x32(tmem_base + lane_base + (uint32_t)(half * 64 + 32), v + 32);
      tmem_ld_wait();
      tcgen05_fence_before_sync();
      named_barrier_sync(1, kFEpiThreads);
      if (tid == 0) mbar_arrive(bar_hfree);
      // both pairs have multiplied the previous content of this slot (and the copy that delivered it is complete)
      if (g >= 1) mbar_wait(bar_hdone, (uint32_t)(g - 1) & 1u, abort_flag, p.status, 0x811);
      uint8_t* tile = slot + half * (kFM * 128);
      const float* bb = p.b1 + (size_t)(2 * sb + P) * kFH + half * 64;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const float4 b0 = __ldg(reinterpret_cast<const float4*>(bb + q * 8));
        const float4 b1v = __ldg(reinterpret_cast<const float4*>(bb + q * 8 + 4));
        const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1v.x, b1v.y, b1v.z, b1v.w};
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int e = q * 8 + j * 2;
          w[j] = pack_bf16x2(gelu_tanh_pair(__uint_as_float(v[e]) + bv[2 * j]), gelu_tanh_pair(__uint_as_float(v[e + 1]) + bv[2 * j + 1]));
        }
        *reinterpret_cast<uint4*>(tile + swz_offset((uint32_t)row, (uint32_t)q, 128)) = make_uint4(w[0], w[1], w[2], w[3]);
      }
      fence_proxy_async_smem();      // the MMA and the bulk copy read the tile through the async proxy
      named_barrier_sync(1, kFEpiThreads);
      if (tid == 0) {
        mbar_arrive(bar_slot + P);                                          // the tile is in this CTA
        bulk_copy_to_cluster(twin_slot, smem_u32(slot), kFSlotBytes, twin_bar);   // ... and on its way to the other pair
      }
      // the output of the previous row block is complete once the first GEMM of this block's first step is
      if (cur.first && cur.item >= 1) drain_output(prev_item, prev_unit, prev_split, prev_part);
      if (cur.last) { prev_item = cur.item; prev_unit = cur.unit; prev_split = cur.split; prev_part = cur.part; }
    }
    if (steps > 0) drain_output(prev_item, prev_unit, prev_split, prev_part);
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  cluster_sync_all();          // no CTA leaves while another may still copy into it, signal its barriers or multiply into its tensor memory
  if (warp == kFEpiWarps + 1) tmem_dealloc_pair(tmem_base, 512);
}

// Second launch of a run with split blocks: out = bf16(sum of the J planes + b2) over the rows of the split blocks.
__global__ void __launch_bounds__(256) ffn_pair_finalize_kernel(const float* acc, const float* b2, __nv_bfloat16* out, long long total4, int n2, int J) {
  grid_dependency_wait();      // the stores of the first launch are complete and visible
  grid_launch_dependents();
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total4; i += stride) {
    float4 a = __ldg(reinterpret_cast<const float4*>(b2 + (int)((i * 4) % n2)));
    for (int j = 0; j < J; ++j) {
      const float4 v = __ldcg(reinterpret_cast<const float4*>(acc) + (long long)j * total4 + i);
      a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
    }
    reinterpret_cast<uint2*>(out)[i] = make_uint2(pack_bf16x2(a.x, a.y), pack_bf16x2(a.z, a.w));
  }
}

// How the blocks of 256 rows are dealt to the resident clusters: the whole rounds as they are; the blocks of a last,
// partial round are split into the largest J (a divisor of the S steps) whose parts still fit one round.
void pair_split(int units, int S, int* units_whole, int* J) {
  const int resident = device_sm_count() >= 148 ? 33 : std::max(1, device_sm_count() / 4 - 4);   // clusters of 4 (1 CTA per SM): 33 on a B200
  *units_whole = units; *J = 1;
  const int full = units / resident, rest = units % resident;
  if (full < 1 || rest == 0) return;
  for (int j = S; j >= 2; --j)
    if (S % j == 0 && rest * j <= resident) { *units_whole = full * resident; *J = j; return; }
}

struct FfnPairHost {
  FfnPairParams prm;
  size_t ws_bytes = 0;
  int clusters = 0;   // clusters launched = min(row blocks, clusters the device keeps resident); 0: not asked yet
  struct Key { const void* p; int which; bool operator==(const Key& o) const { return p == o.p && which == o.which; } };
  struct KeyHash { size_t operator()(const Key& k) const { return std::hash<const void*>()(k.p) ^ (size_t)k.which * 0x9e3779b97f4a7c15ull; } };
  std::unordered_map<Key, CUtensorMap, KeyHash> maps;
};

void fill_pair_launch(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, int clusters, cudaStream_t stream) {
  *cfg = cudaLaunchConfig_t{};
  cfg->gridDim = dim3(4u, (unsigned)clusters, 1);
  cfg->blockDim = dim3(kFThreads, 1, 1);
  cfg->dynamicSmemBytes = (size_t)kFSmemBytes;
  cfg->stream = stream;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 4; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg->attrs = attr;
  cfg->numAttrs = 2;
}

}  // namespace

// AGO_ERR_UNSUPPORTED (without touching *err) when the shape does not split over two pairs: the caller falls back
// to the unpaired cluster kernel or to the kernel that tiles the second GEMM's reduction.
size_t ffn_pair_workspace_bytes(const Plan& plan) {
  const int64_t K = plan.inputs[0].last(), M = plan.inputs[0].numel() / K;
  const int64_t N2 = plan.output.last();
  const int units = (int)((M + 2 * kFM - 1) / (2 * kFM)), S = plan.ops[0].op.p[0] / (2 * kFH);
  int whole = units, J = 1;
  pair_split(units, S, &whole, &J);
  if (J == 1) return 0;
  return ((size_t)J * (size_t)(M - (int64_t)whole * 2 * kFM) * N2 * 4 + 255) & ~size_t(255);   // J planes over the rows of the split blocks
}

ago_status_t ffn_pair_plan(Plan* plan, FusedState* st, std::string* err) {
  (void)err;
  FfnPairParams q{};
  q.K = (int)plan->inputs[0].last();
  q.M = (int)(plan->inputs[0].numel() / q.K);
  q.Hid = plan->ops[0].op.p[0];
  q.N2 = plan->ops[3].op.p[0];
  if (q.K % kFK != 0 || q.Hid % (2 * kFH) != 0 || q.N2 % 256 != 0 || q.N2 > 768) return AGO_ERR_UNSUPPORTED;
  q.NC = q.N2 / 2;
  q.S = q.Hid / (2 * kFH);
  q.kblocks = q.K / kFK;
  q.units = (q.M + 2 * kFM - 1) / (2 * kFM);
  // worth it only when the clusters (four SMs each) fill most of the device
  if ((long)q.units * 4 < (long)device_sm_count() * 3 / 4) return AGO_ERR_UNSUPPORTED;
  auto* host = new FfnPairHost();
  host->prm = q;
  st->impl = host;
  st->impl_free = [](void* p) { delete static_cast<FfnPairHost*>(p); };
  pair_split(q.units, q.S, &q.units_whole, &q.J);
  q.split_rows = q.M - q.units_whole * 2 * kFM;
  host->prm = q;
  st->variant = 3;
  plan->fused_variant = 3;
  if (q.J > 1) {
    const int64_t rows = std::min<int64_t>((int64_t)(q.units - q.units_whole) * 2 * kFM, (int64_t)q.M - (int64_t)q.units_whole * 2 * kFM);
    host->ws_bytes = ffn_pair_workspace_bytes(*plan);
    // every part writes its plane, the second launch reads the planes back
    plan->workspace_traffic_bytes = (int64_t)(2 * q.J) * rows * q.N2 * 4;
    plan->num_launches = 2;
  }
  st->tile_rows = 2 * kFM; st->grid = 4 * q.units; st->smem_bytes = kFSmemBytes;
  plan->tile_rows = 2 * kFM; plan->smem_bytes = kFSmemBytes;
  return AGO_OK;
}

ago_status_t ffn_pair_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                          void* output, void* workspace, unsigned int* status_word, cudaStream_t stream, std::string* err) {
  (void)plan;
  FfnPairHost* host = static_cast<FfnPairHost*>(st->impl);
  FfnPairParams q = host->prm;
  q.b1 = static_cast<const float*>(weights[1]);
  q.b2 = static_cast<const float*>(weights[3]);
  q.out = static_cast<__nv_bfloat16*>(output);
  q.status = status_word;
  q.acc = nullptr;
  if (q.J > 1) {
    if (!workspace) { *err = "fused feed-forward (paired cluster, split last round): no workspace attached"; return AGO_ERR_INVALID_ARG; }
    q.acc = static_cast<float*>(workspace);   // every element of it is written before it is read: nothing to zero
  }
  auto get_map = [&](const void* base, int which, CUtensorMap* out) -> bool {
    FfnPairHost::Key key{base, which};
    auto it = host->maps.find(key);
    if (it == host->maps.end()) {
      CUtensorMap m;
      uint64_t dims[2]; uint64_t strides[1]; uint32_t box[2];
      if (which == 0) { dims[0] = q.K; dims[1] = q.M; strides[0] = (uint64_t)q.K * 2; box[0] = kFK; box[1] = kFM; }
      else if (which == 1) { dims[0] = q.Hid; dims[1] = q.K; strides[0] = (uint64_t)q.Hid * 2; box[0] = 64; box[1] = kFK; }
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
    cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(ffn_pair_kernel), smem_opt_in);
    if (e != cudaSuccess) { *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  }
  cudaLaunchConfig_t cfg; cudaLaunchAttribute attr[2];
  if (host->clusters == 0) {
    fill_pair_launch(&cfg, attr, q.units, stream);
    int resident = 0;
    cudaError_t e = cudaOccupancyMaxActiveClusters(&resident, ffn_pair_kernel, &cfg);
    if (e != cudaSuccess || resident < 1) {
      *err = std::string("fused feed-forward (paired cluster): no cluster of four is schedulable: ") + cudaGetErrorString(e);
      return AGO_ERR_CUDA;
    }
    host->clusters = std::min(q.units, resident);
  }
  fill_pair_launch(&cfg, attr, host->clusters, stream);
  cudaError_t e = cudaLaunchKernelEx(&cfg, ffn_pair_kernel, mx, mw1, mw2, q);
  if (e != cudaSuccess) { *err = std::string("fused feed-forward (paired cluster) launch: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  if (q.J > 1) {
    const long long row_first = (long long)q.units_whole * 2 * kFM;
    const long long total4 = ((long long)q.M - row_first) * q.N2 / 4;
    const int blocks = (int)std::min<long long>((total4 + 255) / 256, 4LL * device_sm_count());
    FusedLaunch fin(dim3((unsigned)blocks), 256, 0, stream);
    e = cudaLaunchKernelEx(&fin.config, ffn_pair_finalize_kernel, (const float*)q.acc, q.b2, q.out + row_first * q.N2, total4, q.N2, q.J);
    if (e != cudaSuccess) { *err = std::string("fused feed-forward (paired cluster) finalisation launch: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  }
  return AGO_OK;
}

}  // namespace ago
