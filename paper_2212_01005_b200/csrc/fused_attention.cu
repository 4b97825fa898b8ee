// Fused attention: S = Q K^T, * scale, row softmax, O = P V -- one kernel; scores and
// probabilities never leave the SM.
//
// Tile choice (Section III-B, "downstream pointwise / matmul" category): the downstream
// contraction P V reuses its input only along its output columns, so its tile keeps ALL of them
// (head_dim) and is tiled over rows (128 queries). The softmax in between is a simple operator
// over whole rows, so the upstream tile is 128 query rows x ALL keys of the head.
//
// The (batch, head, 128-row query tile) items are numbered in that order and dealt out in equal
// consecutive runs to one persistent CTA per SM. K and V of the current (batch, head) stay in shared
// memory while the CTA walks over its query tiles; when the run crosses into the next head, the new K
// is fetched as soon as the last score product of the old head has completed and the new V as soon as
// its last P V has, both behind the softmax of the tiles in flight.
//
// The keys are processed in two halves by two independent groups of 384 threads (3 per query row and half).
// Each half is a softmax of its own -- its own row maximum, row sum and output accumulator P_h V_h in tensor
// memory -- and the epilogue joins them: with m = max(m_0, m_1) and f_h = exp(m_h - m),
// O = (f_0 O_0 + f_1 O_1) / (f_0 sum_0 + f_1 sum_1), the exact softmax over all keys. Nothing but the epilogue
// orders the groups against each other, so they drift apart: while one group keeps the special-function
// unit busy with its exponentials, the other waits for scores, reads tensor memory or exchanges maxima,
// and the tensor core runs ahead on the next tile's scores.
//
//   P1  TMA: K, V [S x 64] once per head of the run, Q [128 x 64] per tile -> 128-byte-swizzled tiles
//   P2  tcgen05.mma: S_h[128 x S/2] = Q K_h^T                            (TMEM, fp32, two buffers)
//   P3/P4  per half 384 threads (3 per query row, <= 64 score columns each, read from tensor memory in chunks of 32:
//       once for the row maximum, exchanged through shared memory, once more for
//       p = exp2((s - m_h) * scale * log2 e) -> bf16 -> shared memory (K-major operand) and the row sum)
//   P5  tcgen05.mma: O_h[128 x 64] = P_h V_h        (V is the N-major B operand, as it lies in HBM)
//   P6  the group of half 1: TMEM -> registers, (f_0 O_0 + f_1 O_1) / sum, bf16 -> a swizzled tile in shared memory (the
//       probability buffer of half 1, idle by then) -> one TMA store per tile (a row of one head is 128 bytes of a
//       2 E-byte output row: stores from the row-per-lane accumulator layout would touch 32 lines per instruction)
//
// Issue order of the MMA thread: when half 0's probabilities arrive, the next tile's half-0 scores go first (that
// group has nothing else to do) and P_0 V second; when half 1's arrive, P_1 V goes first (the epilogue waits for
// it) and the next half-1 scores second.
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

constexpr int kD = 64;                 // head dimension (one 128-byte swizzle row)
constexpr int kBlockM = 128;           // query rows per tile
constexpr int kKeyBlock = 128;         // keys per TMA box
constexpr int kSubParts = 3;           // threads per query row and half (each owns <= 64 score columns: two chunks of 32)
constexpr int kGroupThreads = kBlockM * kSubParts;
constexpr int kComputeThreads = 2 * kGroupThreads;
constexpr int kThreads = kComputeThreads + 64;   // + TMA warp + MMA warp
constexpr int kHalfCols = 192;         // tensor-memory columns reserved per score half
constexpr uint32_t kOCol = 2 * kHalfCols;   // O_0 at kOCol, O_1 at kOCol + kD

struct AttnParams {
  __nv_bfloat16* out;
  unsigned int* status;
  int B, S, heads, E;
  int Spad;        // keys rounded up to 16
  int nkb;         // 128-key TMA boxes
  int tiles;       // query tiles per head
  int total;       // items = B * heads * tiles
  int hw0, hw1;    // keys in half 0 / half 1 (multiples of 16, hw0 >= hw1 > 0)
  int pw0, pw1;    // columns per thread in each half (multiples of 32, <= 64)
  float scale_log2e;
  int off_q, off_k, off_v, off_p, off_red, off_bar;
  int p_half_bytes;
};

// 2^x on the special-function unit (arguments here are <= 0; results below 2^-126 flush to 0).
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(kThreads, 1)
attention_fused_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                       const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_o,
                       const AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem + p.off_q;
  uint8_t* sK = smem + p.off_k;
  uint8_t* sV = smem + p.off_v;
  uint8_t* sP = smem + p.off_p;                                // two halves of p_half_bytes
  float* sMax = reinterpret_cast<float*>(smem + p.off_red);     // [half][tile parity][kSubParts][128]: partial row maxima
  float* sSum = sMax + 2 * 2 * kSubParts * kBlockM;             // the same for the partial row sums
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
  uint64_t* bar_k = bars + 0;
  uint64_t* bar_v = bars + 1;
  uint64_t* bar_q = bars + 2;       // Q tile landed
  uint64_t* bar_qfree = bars + 3;   // both score MMAs of the tile have read Q
  uint64_t* bar_s = bars + 4;       // [2] score half complete
  uint64_t* bar_p = bars + 6;       // [2] probabilities of the half written, score half drained
  uint64_t* bar_pfree = bars + 8;   // [2] P V of the half has read the probabilities
  uint64_t* bar_o0 = bars + 10;     // P V of half 0 complete
  uint64_t* bar_stage = bars + 11;  // output tile staged in shared memory
  uint64_t* bar_o1 = bars + 12;     // P V of half 1 complete
  uint64_t* bar_ofree = bars + 13;  // epilogue has read the output accumulators
  uint64_t* bar_vfree = bars + 14;  // the last P V of a head has read V
  uint64_t* bar_stfree = bars + 15; // the output store has read the staged tile
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 17);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // This CTA's run of items [g0, g0 + n); item g = ((b * heads + h) * tiles + t).
  const int g0 = (int)((long long)blockIdx.x * p.total / gridDim.x);
  const int n = (int)((long long)(blockIdx.x + 1) * p.total / gridDim.x) - g0;
  const int u0 = g0 / p.tiles, t0 = g0 - u0 * p.tiles;
  const int b0 = u0 / p.heads, h0 = u0 - b0 * p.heads;
  grid_dependency_wait();      // the previous grid of the stream has completed; device memory may be touched
  grid_launch_dependents();

  if (tid == kComputeThreads) {
    *abort_flag = 0u;
    for (int i = 0; i < 16; ++i) mbar_init(bars + i, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmap_q);
    tma_prefetch_desc(&tmap_k);
    tma_prefetch_desc(&tmap_v);
    tma_prefetch_desc(&tmap_o);
    mbar_arrive_expect_tx(bar_k, (uint32_t)(p.nkb * kKeyBlock * kD * 2));
    for (int kb = 0; kb < p.nkb; ++kb) tma_load_3d(sK + kb * kKeyBlock * kD * 2, &tmap_k, bar_k, h0 * kD, kb * kKeyBlock, b0);
    mbar_arrive_expect_tx(bar_q, (uint32_t)(kBlockM * kD * 2));
    tma_load_3d(sQ, &tmap_q, bar_q, h0 * kD, t0 * kBlockM, b0);
    mbar_arrive_expect_tx(bar_v, (uint32_t)(p.nkb * kKeyBlock * kD * 2));
    for (int kb = 0; kb < p.nkb; ++kb) tma_load_3d(sV + kb * kKeyBlock * kD * 2, &tmap_v, bar_v, h0 * kD, kb * kKeyBlock, b0);
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == kComputeThreads / 32) {
    // ============================ TMA producer: the remaining Q tiles, K and V of the following heads ============================
    if (lane == 0) {
      int t = t0, h = h0, b = b0;
      uint32_t heads_done = 0;
      for (int i = 1; i < n; ++i) {
        const bool new_head = ++t == p.tiles;
        if (new_head) { t = 0; if (++h == p.heads) { h = 0; ++b; } }
        mbar_wait(bar_qfree, (uint32_t)(i - 1) & 1u, abort_flag, p.status, 0x201);   // every score product of item i - 1 has completed
        if (new_head) {
          mbar_arrive_expect_tx(bar_k, (uint32_t)(p.nkb * kKeyBlock * kD * 2));
          for (int kb = 0; kb < p.nkb; ++kb) tma_load_3d(sK + kb * kKeyBlock * kD * 2, &tmap_k, bar_k, h * kD, kb * kKeyBlock, b);
        }
        mbar_arrive_expect_tx(bar_q, (uint32_t)(kBlockM * kD * 2));
        tma_load_3d(sQ, &tmap_q, bar_q, h * kD, t * kBlockM, b);
        if (new_head) {
          mbar_wait(bar_vfree, heads_done & 1u, abort_flag, p.status, 0x216);
          ++heads_done;
          mbar_arrive_expect_tx(bar_v, (uint32_t)(p.nkb * kKeyBlock * kD * 2));
          for (int kb = 0; kb < p.nkb; ++kb) tma_load_3d(sV + kb * kKeyBlock * kD * 2, &tmap_v, bar_v, h * kD, kb * kKeyBlock, b);
        }
      }
    }
    __syncwarp();
  } else if (warp == kComputeThreads / 32 + 1) {
    // ============================ MMA issue (one lane) ============================
    if (lane == 0) {
      const uint64_t qdesc = make_smem_desc(smem_u32(sQ), 0, 1024, SW_128B);
      const uint64_t kdesc = make_smem_desc(smem_u32(sK), 0, 1024, SW_128B);
      const uint64_t pdesc = make_smem_desc(smem_u32(sP), 0, 1024, SW_128B);
      const uint64_t vdesc = make_smem_desc(smem_u32(sV), 0, 1024, SW_128B);
      const uint32_t idesc_o = make_idesc_bf16(128, kD, 0, 1);    // V is N-major
      const uint32_t idesc_s[2] = {make_idesc_bf16(128, (uint32_t)p.hw0), make_idesc_bf16(128, (uint32_t)p.hw1)};
      const int hw[2] = {p.hw0, p.hw1};

      // Descriptors as (low, high) words: the start address lives in the low word, so every operand of the unrolled
      // issue loops is one 32-bit add away from its base.
      const uint32_t q_lo = (uint32_t)qdesc, q_hi = (uint32_t)(qdesc >> 32), k_lo = (uint32_t)kdesc, k_hi = (uint32_t)(kdesc >> 32);
      const uint32_t p_lo = (uint32_t)pdesc, p_hi = (uint32_t)(pdesc >> 32), v_lo = (uint32_t)vdesc, v_hi = (uint32_t)(vdesc >> 32);
      auto issue_scores = [&](int half) {
        const uint32_t b0 = k_lo + ((uint32_t)(half * p.hw0 * kD * 2) >> 4);
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks)
          umma_bf16_lohi(tmem_base + half * kHalfCols, q_lo + 2u * ks, q_hi, b0 + 2u * ks, k_hi, idesc_s[half], ks > 0);
        umma_commit(bar_s + half);
      };
      auto issue_pv = [&](int half) {
        const uint32_t a0 = p_lo + ((uint32_t)(half * p.p_half_bytes) >> 4);
        const uint32_t b0 = v_lo + ((uint32_t)(half * p.hw0 * kD * 2) >> 4);
        const int ksteps = hw[half] / 16;
#pragma unroll
        for (int ks = 0; ks < kHalfCols / 16; ++ks)
          if (ks < ksteps)
            umma_bf16_lohi(tmem_base + kOCol + half * kD, a0 + (uint32_t)(((ks >> 2) * kBlockM * 128 + (ks & 3) * 32) >> 4), p_hi,
                           b0 + (uint32_t)((ks * 16 * kD * 2) >> 4), v_hi, idesc_o, ks != 0);
      };

      mbar_wait(bar_k, 0, abort_flag, p.status, 0x202);
      mbar_wait(bar_q, 0, abort_flag, p.status, 0x203);
      tcgen05_fence_after_sync();
      issue_scores(0);
      issue_scores(1);
      umma_commit(bar_qfree);
      int t = t0;
      uint32_t head_ph = 0;      // parity of the K / V loads of the current head
      bool first_of_head = true;
      for (int i = 0; i < n; ++i) {
        const uint32_t ph = (uint32_t)i & 1u;
        const bool last_of_head = t + 1 == p.tiles;   // the next item of the run, if any, belongs to the next head
        // ---- half 0 ----
        mbar_wait(bar_p + 0, ph, abort_flag, p.status, 0x204);
        if (i + 1 < n) {
          mbar_wait(bar_q, ph ^ 1u, abort_flag, p.status, 0x207);
          if (last_of_head) mbar_wait(bar_k, head_ph ^ 1u, abort_flag, p.status, 0x202);
          tcgen05_fence_after_sync();
          issue_scores(0);                       // next tile's half 0 into the buffer just drained: its group is waiting for it
        }
        if (first_of_head) mbar_wait(bar_v, head_ph, abort_flag, p.status, 0x205);
        if (i > 0) mbar_wait(bar_ofree, ph ^ 1u, abort_flag, p.status, 0x206);
        tcgen05_fence_after_sync();
        issue_pv(0);
        umma_commit(bar_o0);
        umma_commit(bar_pfree + 0);
        // ---- half 1 ----
        mbar_wait(bar_p + 1, ph, abort_flag, p.status, 0x208);
        tcgen05_fence_after_sync();
        issue_pv(1);                             // first: the epilogue of this tile waits for it
        umma_commit(bar_o1);
        umma_commit(bar_pfree + 1);
        if (last_of_head) umma_commit(bar_vfree);
        if (i + 1 < n) {
          issue_scores(1);
          umma_commit(bar_qfree);
        }
        first_of_head = last_of_head;
        if (last_of_head) { t = 0; head_ph ^= 1u; } else ++t;
      }
    }
    __syncwarp();
  } else {
    // ============================ softmax / epilogue warps ============================
    const int row = (warp & 3) * 32 + lane;     // TMEM lane = query row of the tile
    const int part = warp >> 2;
    const int grp = part >= kSubParts ? 1 : 0;  // the half of the keys this thread's group owns
    const int sub = part - grp * kSubParts;     // which slice of the half
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const float c = p.scale_log2e;
    const int hw = grp ? p.hw1 : p.hw0;
    const int pw = grp ? p.pw1 : p.pw0;
    const int nch = pw >> 5;                    // chunks of 32 columns per thread
    const int key_base = grp * p.hw0;
    const uint32_t s_addr = tmem_base + lane_base + grp * kHalfCols;
    uint8_t* pbase = sP + grp * p.p_half_bytes;
    const uint32_t bar_id = 1u + (uint32_t)grp;
    const bool leader = sub == 0 && row == 0;
    float* gMax = sMax + grp * (2 * kSubParts * kBlockM);
    float* gSum = sSum + grp * (2 * kSubParts * kBlockM);

    uint32_t sv[32];
    // One chunk of (at most) 32 score columns of this thread's row: col0 within the half, ncols in {0, 16, 32};
    // fast = all 32 present and none of them padding: straight-line code, no predicates.
    auto load_chunk = [&](int col0, int ncols) {
      if (ncols > 16) tmem_ld_x32(s_addr + col0, sv); else tmem_ld_x16(s_addr + col0, sv);
      tmem_ld_wait();
    };
    auto chunk_max = [&](int col0, int ncols, bool fast) -> float {
      float m = -INFINITY;
      if (fast) {
        float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          m4[0] = fmaxf(m4[0], __uint_as_float(sv[j]));
          m4[1] = fmaxf(m4[1], __uint_as_float(sv[j + 1]));
          m4[2] = fmaxf(m4[2], __uint_as_float(sv[j + 2]));
          m4[3] = fmaxf(m4[3], __uint_as_float(sv[j + 3]));
        }
        m = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
      } else {
        const int key0 = key_base + col0;
#pragma unroll
        for (int j = 0; j < 32; ++j) if (j < ncols && key0 + j < p.S) m = fmaxf(m, __uint_as_float(sv[j]));
      }
      return m;
    };
    auto chunk_exp = [&](int col0, int ncols, bool fast, float mc) -> float {
      float sum = 0.0f;
      if (fast) {
        // 32 columns = four 16-byte chunks of this row inside one 64-key block (col0 is a multiple of 32)
        uint8_t* rowp = pbase + (col0 >> 6) * (kBlockM * 128) + row * 128;
        const uint32_t ch0 = (uint32_t)(col0 & 63) >> 3, sw = (uint32_t)row & 7u;
        float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          uint32_t w[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float e0 = ex2_approx(fmaf(__uint_as_float(sv[g * 8 + 2 * j]), c, -mc));
            const float e1 = ex2_approx(fmaf(__uint_as_float(sv[g * 8 + 2 * j + 1]), c, -mc));
            s4[j] += e0 + e1;
            w[j] = pack_bf16x2(e0, e1);
          }
          *reinterpret_cast<uint4*>(rowp + (((ch0 + g) ^ sw) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        sum = (s4[0] + s4[1]) + (s4[2] + s4[3]);
      } else {
        const int key0 = key_base + col0;
#pragma unroll
        for (int g = 0; g < 4; ++g) {            // 8 columns = one 16-byte chunk of a probability row
          if (g * 8 < ncols) {
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int e = g * 8 + 2 * j;
              float e0 = ex2_approx(fmaf(__uint_as_float(sv[e]), c, -mc));
              float e1 = ex2_approx(fmaf(__uint_as_float(sv[e + 1]), c, -mc));
              if (key0 + e >= p.S) e0 = 0.0f;
              if (key0 + e + 1 >= p.S) e1 = 0.0f;
              sum += e0 + e1;
              w[j] = pack_bf16x2(e0, e1);
            }
            const int cc = col0 + g * 8;
            *reinterpret_cast<uint4*>(pbase + (cc >> 6) * (kBlockM * 128) + swz_offset(row, (uint32_t)(cc & 63) >> 3, 128)) =
                make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
      return sum;
    };
    auto reduce3 = [&](const float* a, bool is_max) -> float {
      const float x = a[row], y = a[kBlockM + row], z = a[2 * kBlockM + row];
      return is_max ? fmaxf(x, fmaxf(y, z)) : x + y + z;
    };

    // Threads whose 64 columns are all present and real keys read them in four pieces of 16 through two register
    // buffers: the load of the next piece is in flight while the current one is consumed.
    const bool piped = pw == 64 && sub * pw + 64 <= hw && key_base + sub * pw + 64 <= p.S;
    const uint32_t c_addr = s_addr + (uint32_t)(sub * pw);
    auto max16 = [&](const uint32_t (&v)[16]) -> float {
      float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int j = 0; j < 16; j += 4) {
        m4[0] = fmaxf(m4[0], __uint_as_float(v[j]));
        m4[1] = fmaxf(m4[1], __uint_as_float(v[j + 1]));
        m4[2] = fmaxf(m4[2], __uint_as_float(v[j + 2]));
        m4[3] = fmaxf(m4[3], __uint_as_float(v[j + 3]));
      }
      return fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
    };
    // 16 columns (piece q of the thread's 64) -> two 16-byte chunks of the probability row; returns their sum
    auto exp16 = [&](const uint32_t (&v)[16], int q, float mc) -> float {
      const int col = sub * 64 + q * 16;
      uint8_t* rowp = pbase + (col >> 6) * (kBlockM * 128) + row * 128;
      const uint32_t ch0 = (uint32_t)(col & 63) >> 3, sw = (uint32_t)row & 7u;
      float s2[2] = {0.f, 0.f};
#pragma unroll
      for (int g = 0; g < 2; ++g) {
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float e0 = ex2_approx(fmaf(__uint_as_float(v[g * 8 + 2 * j]), c, -mc));
          const float e1 = ex2_approx(fmaf(__uint_as_float(v[g * 8 + 2 * j + 1]), c, -mc));
          s2[j & 1] += e0 + e1;
          w[j] = pack_bf16x2(e0, e1);
        }
        *reinterpret_cast<uint4*>(rowp + (((ch0 + g) ^ sw) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
      }
      return s2[0] + s2[1];
    };

    for (int t = 0; t < n; ++t) {               // t: position of the item in this CTA's run
      const uint32_t ph = (uint32_t)t & 1u;
      float* myMax = gMax + ph * (kSubParts * kBlockM);
      float* mySum = gSum + ph * (kSubParts * kBlockM);
      // ---------------- pass 1: row maximum of this half ----------------
      mbar_wait(bar_s + grp, ph, abort_flag, p.status, 0x210);
      tcgen05_fence_after_sync();
      float m = -INFINITY;
      if (piped) {
        uint32_t (&va)[16] = reinterpret_cast<uint32_t (&)[16]>(sv[0]);
        uint32_t (&vb)[16] = reinterpret_cast<uint32_t (&)[16]>(sv[16]);
        tmem_ld_x16(c_addr, va);
        tmem_ld_wait_on(va);
        tmem_ld_x16(c_addr + 16, vb);
        m = max16(va);
        tmem_ld_wait_on(vb);
        tmem_ld_x16(c_addr + 32, va);
        m = fmaxf(m, max16(vb));
        tmem_ld_wait_on(va);
        tmem_ld_x16(c_addr + 48, vb);
        m = fmaxf(m, max16(va));
        tmem_ld_wait_on(vb);
        m = fmaxf(m, max16(vb));
      } else {
        for (int ch = 0; ch < nch; ++ch) {
          const int col0 = sub * pw + ch * 32;
          const int ncols = max(0, min(hw, col0 + 32) - col0);
          if (ncols > 0) {
            load_chunk(col0, ncols);
            m = fmaxf(m, chunk_max(col0, ncols, ncols == 32 && key_base + col0 + 32 <= p.S));
          }
        }
      }
      myMax[sub * kBlockM + row] = m;
      if (leader && t > 0) {
        mbar_wait(bar_pfree + grp, ph ^ 1u, abort_flag, p.status, 0x211);       // P V of the previous tile has read this half's probabilities
        if (grp == 1) bulk_wait_group_read_all();       // and this thread's output store has read its staged tile (same buffer)
      }
      named_barrier_sync(bar_id, kGroupThreads);
      const float mh = reduce3(myMax, true);
      // ---------------- pass 2: probabilities and row sum ----------------
      float sum = 0.0f;
      if (piped) {
        const float mc = mh * c;
        uint32_t (&va)[16] = reinterpret_cast<uint32_t (&)[16]>(sv[0]);
        uint32_t (&vb)[16] = reinterpret_cast<uint32_t (&)[16]>(sv[16]);
        tmem_ld_x16(c_addr, va);
        tmem_ld_wait_on(va);
        tmem_ld_x16(c_addr + 16, vb);
        sum = exp16(va, 0, mc);
        tmem_ld_wait_on(vb);
        tmem_ld_x16(c_addr + 32, va);
        sum += exp16(vb, 1, mc);
        tmem_ld_wait_on(va);
        tmem_ld_x16(c_addr + 48, vb);
        sum += exp16(va, 2, mc);
        tmem_ld_wait_on(vb);
        sum += exp16(vb, 3, mc);
      } else {
        for (int ch = 0; ch < nch; ++ch) {
          const int col0 = sub * pw + ch * 32;
          const int ncols = max(0, min(hw, col0 + 32) - col0);
          if (ncols > 0) {
            load_chunk(col0, ncols);
            sum += chunk_exp(col0, ncols, ncols == 32 && key_base + col0 + 32 <= p.S, mh * c);
          }
        }
      }
      mySum[sub * kBlockM + row] = sum;
      fence_proxy_async_smem();
      tcgen05_fence_before_sync();
      named_barrier_sync(bar_id, kGroupThreads);
      if (leader) mbar_arrive(bar_p + grp);      // probabilities written, score half drained

      if (grp == 1) {
        // ---------------- epilogue of the tile: join the halves, normalise, stage, store ----------------
        // Half 0's product, maxima and sums are long complete (bar_o0 follows that group's barriers and its arrival on
        // bar_p[0]): the weights and the f_0 O_0 terms are computed while the tensor core still works on P_1 V.
        mbar_wait(bar_o0, ph, abort_flag, p.status, 0x214);
        tcgen05_fence_after_sync();
        uint32_t (&oa)[16] = reinterpret_cast<uint32_t (&)[16]>(sv[0]);
        uint32_t (&ob)[16] = reinterpret_cast<uint32_t (&)[16]>(sv[16]);
        const uint32_t o_addr = tmem_base + lane_base + kOCol + sub * 32;
        float f1 = 0.0f;
        if (sub < 2) {                           // 32 of the 64 output columns each
          tmem_ld_x16(o_addr, oa);
          tmem_ld_x16(o_addr + 16, ob);
          const float m0 = reduce3(sMax + ph * (kSubParts * kBlockM), true);
          const float s0 = reduce3(sSum + ph * (kSubParts * kBlockM), false);
          const float s1 = reduce3(mySum, false);
          const float mm = fmaxf(m0, mh);
          float f0 = ex2_approx((m0 - mm) * c);
          f1 = ex2_approx((mh - mm) * c);
          const float inv = 1.0f / (f0 * s0 + f1 * s1);
          f0 *= inv; f1 *= inv;
          tmem_ld_wait_on(oa);
          tmem_ld_wait_on(ob);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            oa[j] = __float_as_uint(__uint_as_float(oa[j]) * f0);
            ob[j] = __float_as_uint(__uint_as_float(ob[j]) * f0);
          }
        }
        mbar_wait(bar_o1, ph, abort_flag, p.status, 0x215);
        tcgen05_fence_after_sync();
        if (sub < 2) {
          uint8_t* stage = pbase;                // P V of half 1 has completed: its probabilities are dead
          uint32_t oc[16];
          tmem_ld_x16(o_addr + kD, oc);
          tmem_ld_wait_on(oc);
#pragma unroll
          for (int j = 0; j < 16; ++j) oa[j] = __float_as_uint(fmaf(__uint_as_float(oc[j]), f1, __uint_as_float(oa[j])));
          tmem_ld_x16(o_addr + kD + 16, oc);     // in flight while the first 16 columns are packed and staged
#pragma unroll
          for (int j = 0; j < 2; ++j)
            *reinterpret_cast<uint4*>(stage + swz_offset(row, (uint32_t)(sub * 4 + j), 128)) =
                make_uint4(pack_bf16x2(__uint_as_float(oa[8 * j]), __uint_as_float(oa[8 * j + 1])),
                           pack_bf16x2(__uint_as_float(oa[8 * j + 2]), __uint_as_float(oa[8 * j + 3])),
                           pack_bf16x2(__uint_as_float(oa[8 * j + 4]), __uint_as_float(oa[8 * j + 5])),
                           pack_bf16x2(__uint_as_float(oa[8 * j + 6]), __uint_as_float(oa[8 * j + 7])));
          tmem_ld_wait_on(oc);
#pragma unroll
          for (int j = 0; j < 16; ++j) ob[j] = __float_as_uint(fmaf(__uint_as_float(oc[j]), f1, __uint_as_float(ob[j])));
#pragma unroll
          for (int j = 0; j < 2; ++j)
            *reinterpret_cast<uint4*>(stage + swz_offset(row, (uint32_t)(sub * 4 + 2 + j), 128)) =
                make_uint4(pack_bf16x2(__uint_as_float(ob[8 * j]), __uint_as_float(ob[8 * j + 1])),
                           pack_bf16x2(__uint_as_float(ob[8 * j + 2]), __uint_as_float(ob[8 * j + 3])),
                           pack_bf16x2(__uint_as_float(ob[8 * j + 4]), __uint_as_float(ob[8 * j + 5])),
                           pack_bf16x2(__uint_as_float(ob[8 * j + 6]), __uint_as_float(ob[8 * j + 7])));
        }
        fence_proxy_async_smem();
        tcgen05_fence_before_sync();
        named_barrier_sync(bar_id, kGroupThreads);
        if (leader) {
          mbar_arrive(bar_ofree);
          const int u = (g0 + t) / p.tiles, tq = g0 + t - u * p.tiles, b = u / p.heads;
          tma_store_3d(&tmap_o, pbase, (u - b * p.heads) * kD, tq * kBlockM, b);   // rows past S are clipped
          bulk_commit_group();
        }
      }
    }
    if (leader && grp == 1) bulk_wait_group_all();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, 512);
}

struct AttnHost {
  AttnParams prm;
  int smem_bytes = 0;
  std::unordered_map<const void*, CUtensorMap> maps;   // keyed by base pointer (box shape is the same for Q, K, V)
};

int round16(int v) { return (v + 15) / 16 * 16; }

}  // namespace

ago_status_t attention_plan(Plan* plan, FusedState* st, std::string* err) {
  const OpInfo& qk = plan->ops[0];
  auto* host = new AttnHost();
  AttnParams& q = host->prm;
  q = AttnParams{};
  q.B = (int)qk.in.d[0]; q.S = (int)qk.in.d[1]; q.E = (int)qk.in.d[2];
  q.heads = qk.op.p[1];
  auto bad = [&](const char* m) { *err = std::string("fused attention: ") + m; delete host; return AGO_ERR_UNSUPPORTED; };
  if (qk.op.p[2] != kD) return bad("head_dim must be 64");
  if (q.S > 2 * kHalfCols) return bad("more than 384 keys do not fit the score block in tensor memory");
  if (q.S < 32) return bad("fewer than 32 keys");
  if (!(plan->ops[1].op.f > 0.0f)) return bad("the score scale must be positive (the row maximum is taken before scaling)");
  q.Spad = round16(q.S);
  q.nkb = (q.Spad + kKeyBlock - 1) / kKeyBlock;
  q.tiles = (q.S + kBlockM - 1) / kBlockM;
  if ((long long)q.B * q.heads * q.tiles > 0x7fffffffLL) return bad("too many query tiles");
  q.total = q.B * q.heads * q.tiles;
  q.hw0 = round16((q.Spad + 1) / 2);
  q.hw1 = q.Spad - q.hw0;
  q.pw0 = ((q.hw0 + kSubParts - 1) / kSubParts + 31) / 32 * 32;
  q.pw1 = ((q.hw1 + kSubParts - 1) / kSubParts + 31) / 32 * 32;
  q.scale_log2e = plan->ops[1].op.f * 1.4426950408889634f;
  int off = 0;
  auto take = [&](int bytes) { int o = off; off = (off + bytes + 1023) / 1024 * 1024; return o; };
  q.off_q = take(kBlockM * kD * 2);
  q.off_k = take(q.nkb * kKeyBlock * kD * 2);
  q.off_v = take(q.nkb * kKeyBlock * kD * 2);
  q.p_half_bytes = ((q.hw0 + 63) / 64) * kBlockM * 128;
  q.off_p = take(2 * q.p_half_bytes);
  q.off_red = take(2 * 2 * 2 * kSubParts * kBlockM * 4);
  q.off_bar = take(256);
  host->smem_bytes = off + 1024;
  if (host->smem_bytes > 227 * 1024) return bad("shared memory budget exceeded");
  st->impl = host;
  st->impl_free = [](void* p) { delete static_cast<AttnHost*>(p); };
  st->tile_rows = kBlockM; st->grid = std::min(q.total, device_sm_count()); st->smem_bytes = host->smem_bytes;
  plan->tile_rows = kBlockM; plan->smem_bytes = host->smem_bytes;
  return AGO_OK;
}

ago_status_t attention_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                           void* output, unsigned int* status_word, cudaStream_t stream, std::string* err) {
  AttnHost* host = static_cast<AttnHost*>(st->impl);
  AttnParams q = host->prm;
  q.out = static_cast<__nv_bfloat16*>(output);
  q.status = status_word;
  const CUtensorMap* maps[4];
  for (int i = 0; i < 4; ++i) {
    const void* base = i < 3 ? inputs[i] : output;
    auto it = host->maps.find(base);
    if (it == host->maps.end()) {
      CUtensorMap m;
      const uint64_t dims[3] = {(uint64_t)q.E, (uint64_t)q.S, (uint64_t)q.B};
      const uint64_t strides[2] = {(uint64_t)q.E * 2, (uint64_t)q.S * q.E * 2};
      const uint32_t box[3] = {(uint32_t)kD, (uint32_t)kKeyBlock, 1};
      if (!encode_tmap_bf16(&m, base, 3, dims, strides, box, 128, err)) return AGO_ERR_CUDA;
      if (host->maps.size() > 4096) {     // pointers already fetched stay valid: unordered_map keeps its nodes until erased
        host->maps.clear();
        i = -1;
        continue;
      }
      it = host->maps.emplace(base, m).first;
    }
    maps[i] = &it->second;
  }
  {
    static int smem_opt_in[64] = {};
    cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(attention_fused_kernel), smem_opt_in);
    if (e != cudaSuccess) { *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  }
  dim3 grid((unsigned)std::min(q.total, device_sm_count()));     // one persistent CTA per SM (the shared memory admits no second one)
  FusedLaunch launch(grid, kThreads, (size_t)host->smem_bytes, stream);
  cudaError_t e = cudaLaunchKernelEx(&launch.config, attention_fused_kernel, *maps[0], *maps[1], *maps[2], *maps[3], q);
  if (e != cudaSuccess) { *err = std::string("fused attention launch: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  return AGO_OK;
}

}  // namespace ago
