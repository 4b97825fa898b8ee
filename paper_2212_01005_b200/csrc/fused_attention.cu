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
// The keys are processed in two halves by two independent groups of 128 threads (one thread per query row and half:
// four warps per group, so every scheduler of the SM hosts one warp of each group and the MMA-issuing thread shares its
// scheduler with two busy warps, not seven).
// Each half is a softmax of its own -- its own row maximum, row sum and output accumulator P_h V_h in tensor
// memory -- and the epilogue joins them: with m_h the reference value of half h, m = max(m_0, m_1) and f_h = exp(m_h - m),
// O = (f_0 O_0 + f_1 O_1) / (f_0 sum_0 + f_1 sum_1), the exact softmax over all keys. A thread owns its whole row of the
// half, so neither pass exchanges anything with another thread; nothing but the epilogue orders the groups against
// each other, so they drift apart: while one group keeps the special-function unit busy with its exponentials, the
// other waits for scores or reads tensor memory, and the tensor core runs ahead on the next tile's scores.
//
//   P1  TMA: K, V [S x 64] once per head of the run, Q [128 x 64] per tile -> 128-byte-swizzled tiles
//   P2  tcgen05.mma: S_h[128 x S/2] = Q K_h^T                            (TMEM, fp32, two buffers)
//   P3/P4  per half 128 threads (a row each, read from tensor memory ONCE, in chunks of 32 columns through two register
//       buffers -- the next chunk is in flight while the current one is consumed:
//       p = exp2((s - m_h) * scale * log2 e) -> bf16 -> shared memory (K-major operand) and the row sum, with m_h the
//       maximum of the row's first 32 scores. Softmax does not depend on the reference value; the true row maximum
//       only keeps the exponentials in range: when the last chunk is in registers, the partial row sum (it bounds every
//       exponential so far) and the last chunk's maximum tell whether it did; if not, the warp keeps the score half,
//       takes the true row maximum from it and repeats the pass. Three exponentials in four run on the
//       special-function unit, the fourth as a cubic on the FMA pipe)
//   P5  tcgen05.mma: O_h[128 x 64] = P_h V_h        (V is the N-major B operand, as it lies in HBM)
//   P6  four epilogue warps (a query row per thread): TMEM -> registers as soon as a half's product is complete (its
//       accumulator is released at once), (f_0 O_0 + f_1 O_1) / sum, bf16 -> per warp, pieces of 16 columns x 32 rows
//       staged in shared memory -> one TMA store per piece (stores from the row-per-lane register layout would touch
//       32 lines per instruction and hold up the load/store unit that the probability stores need)
//
// Issue order of the MMA warp, per half: as soon as the group has the last chunk of its score half in registers (and the
// reference has proved good enough), the next tile's scores of that half, so that the group finds them ready when it has
// written its last probabilities; when the probabilities have arrived, P_h V in blocks of 64 keys, each block's
// completion releasing that block of the probability buffer for the next tile.
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
constexpr int kGroupThreads = kBlockM;          // one thread per query row and half of the keys
constexpr int kGroupWarps = kGroupThreads / 32;
constexpr int kSoftmaxThreads = 2 * kGroupThreads;
constexpr int kEpiWarp0 = kSoftmaxThreads / 32;  // four epilogue warps (a query row per thread) follow the softmax warps
constexpr int kTmaWarp = kEpiWarp0 + 4;
constexpr int kMmaWarp = kTmaWarp + 1;
constexpr int kThreads = (kMmaWarp + 1) * 32;    // 448
constexpr int kHalfCols = 192;         // tensor-memory columns reserved per score half
// A row's exponentials are taken relative to the maximum of its first 32 scores, not of all of them (any reference gives
// the same softmax; the true maximum only guarantees the range). A row sum at or above this limit, or not a number, sends
// the warp through the exact two-pass path.
constexpr float kSumLimit = 1099511627776.0f;   // 2^40: a partial row sum below it bounds every exponential so far
constexpr float kRefSlack = 40.0f;              // the reference may lie this many powers of two below the last chunk's maximum
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
  float scale_log2e;
  int off_q, off_k, off_v, off_p, off_stage, off_red, off_bar;
  int p_half_bytes;
};

// 2^x on the special-function unit (arguments here are <= 0; results below 2^-126 flush to 0).
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 2^x on the FMA pipe, for a share of the exponentials (the special-function unit delivers 16 results per cycle and SM,
// which bounds the probability pass): x is split with the magic-number addition into an integer n, which goes straight
// into the exponent field, and a fraction f in [-0.5, 0.5], on which a cubic (fitted to 2^f, relative error < 8e-5, well
// below the bf16 rounding of the result) is evaluated. Results below 2^-125 are clamped there instead of flushed to 0.
__device__ __forceinline__ float ex2_poly(float x) {
  x = fmaxf(x, -125.0f);
  const float t = x + 12582912.0f;              // 1.5 * 2^23: round(x) appears in the low mantissa bits
  const float f = x - (t - 12582912.0f);
  float q = fmaf(f, 0.05517092f, 0.24260956f);
  q = fmaf(q, f, 0.69326097f);
  q = fmaf(q, f, 0.9999282f);
  return __uint_as_float(__float_as_uint(q) + (__float_as_uint(t) << 23));
}

// Orders the compiler only: no use of these registers moves above this point, no later write to them above their last use.
__device__ __forceinline__ void reg_order16(uint32_t (&v)[16]) {
  asm volatile(""
               : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]), "+r"(v[8]),
                 "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15])
               :
               : "memory");
}

// Two probabilities -> a pair of bf16 (round to nearest even).
__device__ __forceinline__ uint32_t pack_p(float e0, float e1) { return pack_bf16x2(e0, e1); }

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
  uint8_t* sStage = smem + p.off_stage;                        // per epilogue warp two [32 rows x 32 bytes] output pieces
  float* sJoin = reinterpret_cast<float*>(smem + p.off_red);    // [tile parity][half][maximum, sum][128]: row statistics of the halves
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
  uint64_t* bar_k = bars + 0;
  uint64_t* bar_v = bars + 1;
  uint64_t* bar_q = bars + 2;       // Q tile landed
  uint64_t* bar_qfree = bars + 3;   // both score MMAs of the tile have read Q
  uint64_t* bar_s = bars + 4;       // [2] score half complete
  uint64_t* bar_p = bars + 6;       // [2] probabilities of the half written (one arrival per warp)
  uint64_t* bar_d = bars + 8;       // [2] score half drained: every row of it is in registers (one arrival per warp)
  uint64_t* bar_pfree = bars + 16;  // [2][3] P V of the half has read 64-key block j of the probabilities
  uint64_t* bar_o = bars + 10;      // [2] P V of the half complete
  uint64_t* bar_ofree = bars + 12;  // [2] the epilogue warps have read the half's output accumulator (one arrival per warp)
  uint64_t* bar_vfree = bars + 14;  // the last P V of a head has read V
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 22);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 23);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // This CTA's run of items [g0, g0 + n); item g = ((b * heads + h) * tiles + t).
  const int g0 = (int)((long long)blockIdx.x * p.total / gridDim.x);
  const int n = (int)((long long)(blockIdx.x + 1) * p.total / gridDim.x) - g0;
  const int u0 = g0 / p.tiles, t0 = g0 - u0 * p.tiles;
  const int b0 = u0 / p.heads, h0 = u0 - b0 * p.heads;
  grid_dependency_wait();      // the previous grid of the stream has completed; device memory may be touched
  grid_launch_dependents();

  if (tid == kTmaWarp * 32) {
    *abort_flag = 0u;
    for (int i = 0; i < 22; ++i) mbar_init(bars + i, ((i >= 6 && i <= 9) || i == 12 || i == 13) ? kGroupWarps : 1);
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

  if (warp == kTmaWarp) {
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
  } else if (warp == kMmaWarp) {
    // ============================ MMA issue ============================
    // The whole warp runs this role, converged: the MMAs and commits are predicated on one elected lane and take ready
    // 64-bit descriptors (next to busy warps that issues several times faster than a lane-0 branch, see tc_common.cuh).
    {
      const uint32_t elected = elect_one();
      const uint64_t qdesc = make_smem_desc(smem_u32(sQ), 0, 1024, SW_128B);
      const uint64_t kdesc = make_smem_desc(smem_u32(sK), 0, 1024, SW_128B);
      const uint64_t pdesc = make_smem_desc(smem_u32(sP), 0, 1024, SW_128B);
      const uint64_t vdesc = make_smem_desc(smem_u32(sV), 0, 1024, SW_128B);
      const uint32_t idesc_o = make_idesc_bf16(128, kD, 0, 1);    // V is N-major
      const uint32_t idesc_s[2] = {make_idesc_bf16(128, (uint32_t)p.hw0), make_idesc_bf16(128, (uint32_t)p.hw1)};
      const int hw[2] = {p.hw0, p.hw1};
      auto issue_scores = [&](int half) {
        const uint64_t b0 = kdesc + (uint64_t)((uint32_t)(half * p.hw0 * kD * 2) >> 4);
        const uint32_t d = tmem_base + half * kHalfCols;
        umma_bf16_elected<false>(d, qdesc, b0, idesc_s[half], elected);
#pragma unroll
        for (int ks = 1; ks < kD / 16; ++ks) umma_bf16_elected<true>(d, qdesc + 2u * ks, b0 + 2u * ks, idesc_s[half], elected);
        umma_commit_elected(bar_s + half, elected);
      };
      // P_h V in blocks of 64 keys (four K steps): each block's completion releases that block of the probability buffer
      auto issue_pv_block = [&](int half, int blk) {
        const uint64_t a0 = pdesc + (uint64_t)((uint32_t)(half * p.p_half_bytes + blk * kBlockM * 128) >> 4);
        const uint64_t b0 = vdesc + (uint64_t)((uint32_t)((half * p.hw0 + blk * 64) * kD * 2) >> 4);
        const uint32_t d = tmem_base + kOCol + half * kD;
        const int ksteps = hw[half] / 16 - blk * 4;      // K steps left from this block on
        if (ksteps <= 0) return;
        umma_bf16_elected_acc(d, a0, b0, idesc_o, elected, blk != 0);
#pragma unroll
        for (int ks = 1; ks < 4; ++ks)
          if (ks < ksteps) umma_bf16_elected<true>(d, a0 + (uint64_t)((ks * 32) >> 4), b0 + (uint64_t)((ks * 16 * kD * 2) >> 4), idesc_o, elected);
        umma_commit_elected(bar_pfree + half * 3 + blk, elected);
      };

      mbar_wait(bar_k, 0, abort_flag, p.status, 0x202);
      mbar_wait(bar_q, 0, abort_flag, p.status, 0x203);
      tcgen05_fence_after_sync();
      issue_scores(0);
      issue_scores(1);
      umma_commit_elected(bar_qfree, elected);
      int t = t0;
      uint32_t head_ph = 0;      // parity of the K / V loads of the current head
      bool first_of_head = true;
      for (int i = 0; i < n; ++i) {
        const uint32_t ph = (uint32_t)i & 1u;
        const bool last_of_head = t + 1 == p.tiles;   // the next item of the run, if any, belongs to the next head
        // Per half: score half drained (its last chunk is in the group's registers) -> the next tile's scores of the
        // half, so that the group finds them ready when it has written its last probabilities; probabilities written ->
        // P_h V, block by block (each block's completion releases that block of the probability buffer).
        // ---- half 0 ----
        if (i + 1 < n) {
          mbar_wait(bar_d + 0, ph, abort_flag, p.status, 0x20a);
          mbar_wait(bar_q, ph ^ 1u, abort_flag, p.status, 0x207);
          if (last_of_head) mbar_wait(bar_k, head_ph ^ 1u, abort_flag, p.status, 0x202);
          tcgen05_fence_after_sync();
          issue_scores(0);
        }
        mbar_wait(bar_p + 0, ph, abort_flag, p.status, 0x204);
        if (first_of_head) mbar_wait(bar_v, head_ph, abort_flag, p.status, 0x205);
        if (i > 0) mbar_wait(bar_ofree + 0, ph ^ 1u, abort_flag, p.status, 0x206);
        tcgen05_fence_after_sync();
        issue_pv_block(0, 0);
        issue_pv_block(0, 1);
        issue_pv_block(0, 2);
        umma_commit_elected(bar_o + 0, elected);
        // ---- half 1 ----
        if (i + 1 < n) {
          mbar_wait(bar_d + 1, ph, abort_flag, p.status, 0x20b);
          tcgen05_fence_after_sync();
          issue_scores(1);
          umma_commit_elected(bar_qfree, elected);
        }
        mbar_wait(bar_p + 1, ph, abort_flag, p.status, 0x208);
        if (i > 0) mbar_wait(bar_ofree + 1, ph ^ 1u, abort_flag, p.status, 0x209);
        tcgen05_fence_after_sync();
        issue_pv_block(1, 0);
        issue_pv_block(1, 1);
        issue_pv_block(1, 2);
        umma_commit_elected(bar_o + 1, elected);
        if (last_of_head) umma_commit_elected(bar_vfree, elected);
        first_of_head = last_of_head;
        if (last_of_head) { t = 0; head_ph ^= 1u; } else ++t;
      }
    }
    __syncwarp();
  } else if (warp < kEpiWarp0) {
    // ============================ softmax warps ============================
    const int grp = warp >> 2;                  // the half of the keys this thread's group owns (warps 0-3 / 4-7)
    const int row = (warp & 3) * 32 + lane;     // TMEM lane = query row of the tile
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const float c = p.scale_log2e;
    const int hw = grp ? p.hw1 : p.hw0;
    const int key_base = grp * p.hw0;
    const int kv = min(hw, p.S - key_base);     // real keys of the half (> hw - 16; the other columns are padding)
    const int nch = (hw + 31) >> 5;             // 32-column chunks that hold columns of the half
    const uint32_t s_addr = tmem_base + lane_base + grp * kHalfCols;
    uint8_t* pbase = sP + grp * p.p_half_bytes;
    uint8_t* prow = pbase + row * 128;          // this row in the first 64-key block of the probability operand
    const uint32_t sw = (uint32_t)row & 7u;

    uint32_t va[32], vb[32];
    // The outstanding load of a 32-register buffer has landed (one wait; the second statement only orders the compiler).
    auto wait32 = [](uint32_t (&v)[32]) {
      tmem_ld_wait_on(reinterpret_cast<uint32_t (&)[16]>(v[0]));
      reg_order16(reinterpret_cast<uint32_t (&)[16]>(v[16]));
    };
    auto max32 = [](const uint32_t (&v)[32]) -> float {
      float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        m4[0] = fmaxf(m4[0], fmaxf(__uint_as_float(v[j]), __uint_as_float(v[j + 1])));
        m4[1] = fmaxf(m4[1], fmaxf(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3])));
        m4[2] = fmaxf(m4[2], fmaxf(__uint_as_float(v[j + 4]), __uint_as_float(v[j + 5])));
        m4[3] = fmaxf(m4[3], fmaxf(__uint_as_float(v[j + 6]), __uint_as_float(v[j + 7])));
      }
      return fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
    };
    auto max_tail = [](const uint32_t (&v)[32], int nreal) -> float {
      float m = -INFINITY;
#pragma unroll
      for (int j = 0; j < 32; ++j) if (j < nreal) m = fmaxf(m, __uint_as_float(v[j]));
      return m;
    };
    // 32 columns of real keys -> four 16-byte chunks of the probability row; s4 collects the row sum. All 32 exponentials
    // are issued back to back, in place, before anything consumes one: the special-function unit takes a warp's
    // instruction every eight cycles, and only independent ones in flight keep it busy from a single warp.
    auto exp32 = [&](uint32_t (&v)[32], uint8_t* blk, uint32_t ch0, float mc, float (&s4)[4]) {
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const float x = fmaf(__uint_as_float(v[j]), c, -mc);
        v[j] = __float_as_uint((j & 3) == 3 ? ex2_poly(x) : ex2_approx(x));   // one in four on the FMA pipe
      }
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float e0 = __uint_as_float(v[g * 8 + 2 * j]), e1 = __uint_as_float(v[g * 8 + 2 * j + 1]);
          s4[j] += e0 + e1;
          w[j] = pack_p(e0, e1);
        }
        *reinterpret_cast<uint4*>(blk + (((ch0 + g) ^ sw) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    };
    // The last chunk of a half: ncols (16 or 32) columns belong to the half, the first nreal of them are keys; the
    // probabilities of the padding columns are zeros (their V rows are zeros too, but must not meet a NaN).
    auto exp_tail = [&](uint32_t (&v)[32], uint8_t* blk, uint32_t ch0, int ncols, int nreal, float mc, float (&s4)[4]) {
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        if (g * 8 < ncols) {
          uint32_t w[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int e = g * 8 + 2 * j;
            float e0 = ex2_approx(fmaf(__uint_as_float(v[e]), c, -mc));
            float e1 = ex2_approx(fmaf(__uint_as_float(v[e + 1]), c, -mc));
            if (e >= nreal) e0 = 0.0f;
            if (e + 1 >= nreal) e1 = 0.0f;
            s4[j] += e0 + e1;
            w[j] = pack_p(e0, e1);
          }
          *reinterpret_cast<uint4*>(blk + (((ch0 + g) ^ sw) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
    };

    for (int t = 0; t < n; ++t) {               // t: position of the item in this CTA's run
      const uint32_t ph = (uint32_t)t & 1u;
      float* xm = sJoin + (ph * 2 + grp) * (2 * kBlockM);   // this half's row maxima and sums of the tile, for the epilogue
      // ---------------- reference value: maximum of the first chunk ----------------
      mbar_wait(bar_s + grp, ph, abort_flag, p.status, 0x210);
      tcgen05_fence_after_sync();
      tmem_ld_x32(s_addr, va);
      wait32(va);
      if (nch > 1) tmem_ld_x32(s_addr + 32u, vb);
      float m = kv >= 32 ? max32(va) : max_tail(va, kv);
      float sum;
      // Once the last chunk of the row is in registers it is known whether the reference was good enough: the sum of the
      // exponentials so far bounds every one of them, and the last chunk's maximum is taken directly. If so for every
      // row of the warp, the score half is released to the next tile's score product at once; otherwise it is kept,
      // the true row maximum is taken from it, and the pass is repeated before the half is released.
      auto last_chunk_landed = [&](int attempt, float partial_sum, float last_max) -> bool {
        const bool exact = attempt == 0 && __any_sync(0xffffffffu, !(partial_sum < kSumLimit) || !((last_max - m) * c < kRefSlack));
        if (!exact) {
          tcgen05_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_d + grp);
        }
        return exact;
      };
      // The loops below are rolled on purpose: every softmax warp runs the same few hundred instructions per pair of
      // chunks, which stay in the instruction cache, instead of a private stretch of straight-line code per chunk.
#pragma unroll 1
      for (int attempt = 0;; ++attempt) {
        // ---------------- probabilities and row sum (chunk 0 is in va, chunk 1 on its way to vb) ----------------
        bool exact = false;
        if (nch == 1) exact = last_chunk_landed(attempt, 0.0f, m);
        const float mc = m * c;
        float s4[4] = {0.f, 0.f, 0.f, 0.f};
        uint8_t* blk = prow;
#pragma unroll 1
        for (int ch = 0; ch < nch; ch += 2, blk += kBlockM * 128) {
          if (t > 0 && attempt == 0) {           // P V of the previous tile has read this 64-key block of the buffer
            if (lane == 0) mbar_wait(bar_pfree + grp * 3 + (ch >> 1), ph ^ 1u, abort_flag, p.status, 0x211);
            __syncwarp();
          }
          if (kv - ch * 32 >= 32) exp32(va, blk, 0u, mc, s4); else exp_tail(va, blk, 0u, hw - ch * 32, kv - ch * 32, mc, s4);
          if (ch + 1 < nch) {
            wait32(vb);
            if (ch + 2 < nch) tmem_ld_x32(s_addr + (uint32_t)((ch + 2) * 32), va);
            else exact = last_chunk_landed(attempt, (s4[0] + s4[1]) + (s4[2] + s4[3]),
                                           kv - ch * 32 >= 64 ? max32(vb) : max_tail(vb, kv - ch * 32 - 32));
            if (kv - ch * 32 >= 64) exp32(vb, blk, 4u, mc, s4); else exp_tail(vb, blk, 4u, hw - ch * 32 - 32, kv - ch * 32 - 32, mc, s4);
            if (ch + 2 < nch) {
              wait32(va);
              if (ch + 3 < nch) tmem_ld_x32(s_addr + (uint32_t)((ch + 3) * 32), vb);
              else exact = last_chunk_landed(attempt, (s4[0] + s4[1]) + (s4[2] + s4[3]),
                                             kv - ch * 32 >= 96 ? max32(va) : max_tail(va, kv - ch * 32 - 64));
            }
          }
        }
        sum = (s4[0] + s4[1]) + (s4[2] + s4[3]);
        if (!exact) break;
        // ---------------- exact path: the row maximum over all chunks first ----------------
        m = -INFINITY;
#pragma unroll 1
        for (int ch = 0; ch < nch; ++ch) {
          tmem_ld_x32(s_addr + (uint32_t)(ch * 32), va);
          wait32(va);
          m = fmaxf(m, kv - ch * 32 >= 32 ? max32(va) : max_tail(va, kv - ch * 32));
        }
        tmem_ld_x32(s_addr, va);
        wait32(va);
        if (nch > 1) tmem_ld_x32(s_addr + 32u, vb);
      }
      xm[row] = m;
      xm[kBlockM + row] = sum;
      fence_proxy_async_smem();
      tcgen05_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_p + grp);   // this warp's 32 rows of probabilities written, its score rows drained
    }
  } else {
    // ============================ epilogue warps: join the halves, normalise, store ============================
    // A thread owns a query row of the tile: 64 output values.
    const int row = (warp & 3) * 32 + lane;     // TMEM lane = query row of the tile
    const uint32_t o_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + kOCol;
    const float c = p.scale_log2e;
    uint32_t oa[32], ob[32], oc[16];
    uint8_t* stage = sStage + (warp & 3) * 2048;
    auto wait32 = [](uint32_t (&v)[32]) {
      tmem_ld_wait_on(reinterpret_cast<uint32_t (&)[16]>(v[0]));
      reg_order16(reinterpret_cast<uint32_t (&)[16]>(v[16]));
    };
    int u = g0 / p.tiles, tq = g0 - u * p.tiles;
    for (int t = 0; t < n; ++t) {
      const uint32_t ph = (uint32_t)t & 1u;
      // Half 0's product is complete long before half 1's: it is read, and its accumulator released, at once.
      mbar_wait(bar_o + 0, ph, abort_flag, p.status, 0x214);
      tcgen05_fence_after_sync();
      tmem_ld_x32(o_addr, oa);
      tmem_ld_x32(o_addr + 32, ob);
      wait32(oa);
      reg_order16(reinterpret_cast<uint32_t (&)[16]>(ob[0]));
      reg_order16(reinterpret_cast<uint32_t (&)[16]>(ob[16]));
      tcgen05_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_ofree + 0);            // O_0 is in registers: the next tile's P_0 V may overwrite it
      const int b = u / p.heads;
      mbar_wait(bar_o + 1, ph, abort_flag, p.status, 0x215);
      tcgen05_fence_after_sync();
      // Both groups' row statistics of this tile were written before their arrivals on bar_p, which the products follow.
      const float* xm = sJoin + ph * (4 * kBlockM);
      const float m0 = xm[row], s0 = xm[kBlockM + row], m1 = xm[2 * kBlockM + row], s1 = xm[3 * kBlockM + row];
      const float mm = fmaxf(m0, m1);
      float f0 = ex2_approx((m0 - mm) * c);
      float f1 = ex2_approx((m1 - mm) * c);
      const float inv = 1.0f / (f0 * s0 + f1 * s1);
      f0 *= inv; f1 *= inv;
      // Four pieces of 16 output columns: 32 bytes of each of the warp's 32 rows, staged (32-byte swizzle: rows four apart
      // take the other 16-byte slot) and written by one TMA store per piece, which clips the rows past S. Stores from the
      // row-per-lane register layout would touch 32 lines per instruction and hold up the load/store unit for everyone.
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        tmem_ld_x16(o_addr + kD + (uint32_t)(q * 16), oc);
        if (lane == 0) bulk_wait_group_read_but_one();       // the store issued two pieces ago has read this buffer
        tmem_ld_wait_on(oc);
        if (q == 3) {
          tcgen05_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_ofree + 1);        // O_1 is in registers
        } else {
          __syncwarp();
        }
        const uint32_t* o0 = q < 2 ? oa + q * 16 : ob + (q - 2) * 16;
#pragma unroll
        for (int j = 0; j < 16; ++j) oc[j] = __float_as_uint(fmaf(__uint_as_float(oc[j]), f1, __uint_as_float(o0[j]) * f0));
        uint8_t* piece = stage + (q & 1) * 1024;
#pragma unroll
        for (int j = 0; j < 2; ++j)
          *reinterpret_cast<uint4*>(piece + lane * 32 + ((((uint32_t)j) ^ (((uint32_t)lane >> 2) & 1u)) << 4)) =
              make_uint4(pack_bf16x2(__uint_as_float(oc[8 * j]), __uint_as_float(oc[8 * j + 1])),
                         pack_bf16x2(__uint_as_float(oc[8 * j + 2]), __uint_as_float(oc[8 * j + 3])),
                         pack_bf16x2(__uint_as_float(oc[8 * j + 4]), __uint_as_float(oc[8 * j + 5])),
                         pack_bf16x2(__uint_as_float(oc[8 * j + 6]), __uint_as_float(oc[8 * j + 7])));
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_3d(&tmap_o, piece, (u - b * p.heads) * kD + q * 16, tq * kBlockM + (warp & 3) * 32, b);
          bulk_commit_group();
        }
      }
      if (++tq == p.tiles) { tq = 0; ++u; }
    }
    if (lane == 0) bulk_wait_group_all();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, 512);
}

struct AttnHost {
  AttnParams prm;
  int smem_bytes = 0;
  std::unordered_map<const void*, CUtensorMap> maps;   // keyed by base pointer (+1 for the output map)
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
  q.scale_log2e = plan->ops[1].op.f * 1.4426950408889634f;
  int off = 0;
  auto take = [&](int bytes) { int o = off; off = (off + bytes + 1023) / 1024 * 1024; return o; };
  q.off_q = take(kBlockM * kD * 2);
  q.off_k = take(q.nkb * kKeyBlock * kD * 2);
  q.off_v = take(q.nkb * kKeyBlock * kD * 2);
  q.p_half_bytes = ((q.hw0 + 63) / 64) * kBlockM * 128;
  q.off_p = take(2 * q.p_half_bytes);
  q.off_stage = take(4 * 2 * 1024);
  q.off_red = take(2 * 2 * 2 * kBlockM * 4);
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
    // keyed by pointer and role: the output map has another box and swizzle than the input maps
    const void* key = reinterpret_cast<const void*>(reinterpret_cast<uintptr_t>(base) | (i == 3 ? 1u : 0u));
    auto it = host->maps.find(key);
    if (it == host->maps.end()) {
      CUtensorMap m;
      const uint64_t dims[3] = {(uint64_t)q.E, (uint64_t)q.S, (uint64_t)q.B};
      const uint64_t strides[2] = {(uint64_t)q.E * 2, (uint64_t)q.S * q.E * 2};
      const uint32_t box[3] = {(uint32_t)kD, (uint32_t)kKeyBlock, 1};
      const uint32_t obox[3] = {16, 32, 1};        // an epilogue warp's piece: 16 columns of its 32 rows
      if (!encode_tmap_bf16(&m, base, 3, dims, strides, i < 3 ? box : obox, i < 3 ? 128 : 32, err)) return AGO_ERR_CUDA;
      if (host->maps.size() > 4096) {     // pointers already fetched stay valid: unordered_map keeps its nodes until erased
        host->maps.clear();
        i = -1;
        continue;
      }
      it = host->maps.emplace(key, m).first;
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
