// Tensor-core GEMM of the unfused modes for large products: C[M][N] = epilogue(A[M][K] * B) on PAIRED CTAs
// (one launch per complex operator with its simple operators in the epilogue: Section III-A, "conventional
// fusion within a mini-subgraph"). The small-tile kernel (kernel_gemm_tc.cu) fetches 8 KB of operands per
// 128 x 128 x 16 product, which is all the shared memory delivers in the product's 64 cycles; this kernel is the
// one whose main loop is bound by the tensor pipe instead:
//
//   * a cluster of two CTAs computes a 256 x 256 output tile with tcgen05.mma.cta_group::2: each CTA holds 128 rows
//     of A and HALF of the B tile (128 of its 256 columns) and fetches both with its own TMA loads -- no multicast --
//     so a 256 x 256 x 16 product (128 cycles of tensor pipe) reads 8 KB per SM;
//   * persistent pairs walk over the output tiles; two accumulators in tensor memory (2 x 256 columns) let the
//     epilogue of tile i overlap the products of tile i + 1;
//   * roles per CTA: one TMA thread, one MMA thread (it issues in the leader CTA only), eight epilogue warps
//     (bias / activation / scale in fp32 -> 128-byte-swizzled staging tile -> TMA store, clipped at the edges).
//
// Barriers (per ring stage s, per accumulator a):
//   full[s]   leader only, count 1: the leader's TMA thread announces the bytes of both CTAs, both CTAs' loads complete there
//   empty[s]  each CTA, count 1: the leader's MMA thread commits onto both after the stage's products
//   accf[a]   each CTA, count 1: accumulator a complete (committed onto both CTAs by the leader)
//   acce[a]   leader only, count 3: its two epilogue groups and the peer (relayed by the peer's idle MMA warp) have read accumulator a
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <mutex>
#include <unordered_map>

#include "fused.h"
#include "kernels.h"
#include "tc_common.cuh"
#include "tmap.h"

namespace ago {

namespace {

using namespace tc;

constexpr int kPM = 128;                 // rows per CTA (256 per pair)
constexpr int kPK = 64;                  // reduction elements per ring stage
constexpr int kPStages = 5;
constexpr int kPStageBytes = 32 * 1024;  // A [128 x 64] + this CTA's half of B [<= 128 x 64]
constexpr int kPStagingBytes = 16 * 1024;   // [128 rows x 128 bytes]; two per group of epilogue warps (double-buffered)
constexpr int kPEpiWarps = 8;            // (tensor-memory lane quarter) x (column half)
constexpr int kPEpiThreads = kPEpiWarps * 32;
constexpr int kPThreads = kPEpiThreads + 64;
constexpr int kPSmemBytes = kPStages * kPStageBytes + 4 * kPStagingBytes + 256 + 1024;

struct GemmPairParams {
  int M, N, K;
  int BN;                  // columns per tile: 128 or 256
  int b_kmajor;
  int c_fp32;              // output element: fp32 (else bf16)
  int kblocks, tiles_m, tiles_n, pairs;
  // the simple operators in canonical order: + bias, activation 1, * scale, + tensor, activation 2
  const float* bias;       // or null
  const void* add;         // or null: bf16 tensor [M][N] with the output's leading dimension
  int64_t ldc;
  int act1, act2;          // EPI_RELU | EPI_RELU6 | EPI_GELU | -1
  float scale;
  unsigned int* status;
};

__device__ __forceinline__ float pair_activate(float x, int act) {
  if (act == EPI_RELU) return fmaxf(x, 0.0f);
  if (act == EPI_RELU6) return fminf(fmaxf(x, 0.0f), 6.0f);
  if (act == EPI_GELU) {
    const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
    return 0.5f * x * (1.0f + t);
  }
  return x;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                 const __grid_constant__ CUtensorMap tmap_c, const GemmPairParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sRing = smem;
  uint8_t* sStage = smem + kPStages * kPStageBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(sStage + 4 * kPStagingBytes);
  uint64_t* bar_full = bars;                   // [kPStages]
  uint64_t* bar_empty = bars + kPStages;       // [kPStages]
  uint64_t* bar_accf = bars + 2 * kPStages;    // [2]
  uint64_t* bar_acce = bar_accf + 2;           // [2]
  uint64_t* bar_drain = bar_acce + 2;          // [2] peer only, count 2: both of its epilogue groups have read accumulator a
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_drain + 2);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bar_drain + 3);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();             // 0: leader
  const int pair = (int)blockIdx.x >> 1;
  const int tiles = p.tiles_m * p.tiles_n;
  const int half_n = p.BN >> 1;                        // B columns held by each CTA

  if (tid == kPEpiThreads) {
    *abort_flag = 0u;
    for (int i = 0; i < kPStages; ++i) { mbar_init(bar_full + i, 1); mbar_init(bar_empty + i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar_accf + i, 1); mbar_init(bar_acce + i, 3); mbar_init(bar_drain + i, 2); }
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == kPEpiWarps + 1) {      // the MMA warp of either CTA allocates (a pair-wide allocation is issued by both CTAs)
    tmem_alloc_pair(tmem_slot, 512);
    tmem_relinquish_pair();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  cluster_sync_all();                // the peer's barriers exist before anything signals them
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == kPEpiWarps) {
    // ================================ TMA producer (both CTAs) ================================
    if (lane == 0) {
      tma_prefetch_desc(&tmap_a);
      tma_prefetch_desc(&tmap_b);
      const uint32_t b_bytes = (uint32_t)half_n * kPK * 2u;
      const uint32_t stage_tx = (uint32_t)(kPM * kPK * 2) + b_bytes;
      int s = 0, round = 0;
      for (int t = pair; t < tiles; t += p.pairs) {
        const int tm = t % p.tiles_m, tn = t / p.tiles_m;
        const int row0 = tm * 2 * kPM + (int)rank * kPM;
        const int n0 = tn * p.BN + (int)rank * half_n;
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (round > 0) mbar_wait_poll(bar_empty + s, (uint32_t)(round - 1) & 1u, abort_flag, p.status, 0x601);
          uint8_t* st = sRing + s * kPStageBytes;
          const uint32_t full = cluster_map(smem_u32(bar_full + s), 0u);   // the leader's barrier
          // The leader announces both CTAs' bytes with a plain local arrival. (An arrival from the peer would have to be
          // a release at cluster scope, which costs about a thousand cycles per stage: measured 98 -> 55 us on a
          // 12288 x 768 x 3072 product.) The peer's bytes may land before the announcement -- the transaction count
          // goes negative meanwhile -- but never in an earlier phase: the peer refills a stage only after the commit
          // that follows the products of its previous content.
          if (rank == 0) mbar_arrive_expect_tx(bar_full + s, 2u * stage_tx);
          tma_load_2d_pair(st, &tmap_a, full, kb * kPK, row0);                        // A [128 rows x 64 k]
          if (p.b_kmajor) {
            tma_load_2d_pair(st + 16384, &tmap_b, full, kb * kPK, n0);                // B [half_n n x 64 k]
          } else {
            for (int nb = 0; nb < half_n; nb += 64)                                   // B [64 k x 64 n] blocks
              tma_load_2d_pair(st + 16384 + (nb >> 6) * 8192, &tmap_b, full, n0 + nb, kb * kPK);
          }
          if (++s == kPStages) { s = 0; ++round; }
        }
      }
    }
    __syncwarp();
  } else if (warp == kPEpiWarps + 1) {
    // ================================ MMA issuer (leader CTA only) ================================
    if (lane == 0 && rank != 0) {
      // The peer's MMA warp has no products to issue: it relays "accumulator drained" to the leader. (An arrival on
      // another CTA's barrier is a release at cluster scope, about a thousand cycles: kept off the epilogue warps.)
      const uint32_t acce_leader = cluster_map(smem_u32(bar_acce), 0u);
      int it = 0;
      for (int t = pair; t < tiles; t += p.pairs, ++it) {
        const int a = it & 1;
        mbar_wait(bar_drain + a, (uint32_t)(it >> 1) & 1u, abort_flag, p.status, 0x605);
        mbar_remote_arrive(acce_leader + (uint32_t)(a * 8));
      }
    }
    if (rank == 0) {
      // the whole warp runs the loop converged; MMAs and commits are predicated on one elected lane (tc_common.cuh)
      const uint32_t elected = elect_one();
      const uint32_t idesc = make_idesc_bf16(256, (uint32_t)p.BN, 0, p.b_kmajor ? 0 : 1);
      int s = 0, round = 0, it = 0;
      for (int t = pair; t < tiles; t += p.pairs, ++it) {
        const int a = it & 1;
        if (it >= 2) {      // both CTAs have read accumulator a (tile it - 2) out of tensor memory
          mbar_wait_poll(bar_acce + a, (uint32_t)((it >> 1) - 1) & 1u, abort_flag, p.status, 0x602);
          tcgen05_fence_after_sync();
        }
        const uint32_t d_tmem = tmem_base + (uint32_t)(a * 256);
        for (int kb = 0; kb < p.kblocks; ++kb) {
          mbar_wait_poll(bar_full + s, (uint32_t)round & 1u, abort_flag, p.status, 0x603);
          tcgen05_fence_after_sync();
          const uint32_t st = smem_u32(sRing + s * kPStageBytes);
          const uint64_t ad = make_smem_desc(st, 0, 1024, SW_128B);
          const uint64_t bd = p.b_kmajor ? make_smem_desc(st + 16384, 0, 1024, SW_128B) : make_smem_desc(st + 16384, 8192, 1024, SW_128B);
#pragma unroll
          for (int ks = 0; ks < kPK / 16; ++ks)
            umma_bf16_pair_elected(d_tmem, ad + 2u * ks, bd + (p.b_kmajor ? (uint64_t)(2u * ks) : (uint64_t)((ks * 2048) >> 4)), idesc, elected, (kb | ks) != 0);
          const uint32_t e = smem_u32(bar_empty + s);
          umma_commit_pair_elected(cluster_map(e, 0u), elected);
          umma_commit_pair_elected(cluster_map(e, 1u), elected);
          if (++s == kPStages) { s = 0; ++round; }
        }
        if (!skip_signal_for_test(p.status, 0x604)) {
          const uint32_t f = smem_u32(bar_accf + a);
          umma_commit_pair_elected(cluster_map(f, 0u), elected);
          umma_commit_pair_elected(cluster_map(f, 1u), elected);
        }
      }
    }
    __syncwarp();
  } else {
    // ================ epilogue warps (both CTAs): thread = (row, column half) ================
    const int q = warp & 3, h = warp >> 2;
    const int row = q * 32 + lane;
    const uint32_t lane_base = (uint32_t)(q * 32) << 16;
    const int ht = tid & 127;                       // thread index within the column half
    uint8_t* stage0 = sStage + h * 2 * kPStagingBytes;
    int sbuf = 0;                                   // staging buffer of the next block
    const int esz = p.c_fp32 ? 4 : 2;
    const int bc = 128 / esz;                       // columns per staged block (128 bytes per row)
    int it = 0;
    for (int t = pair; t < tiles; t += p.pairs, ++it) {
      const int a = it & 1;
      const int tm = t % p.tiles_m, tn = t / p.tiles_m;
      const int row0 = tm * 2 * kPM + (int)rank * kPM;
      const int col_t = tn * p.BN;                  // first column of the tile
      mbar_wait(bar_accf + a, (uint32_t)(it >> 1) & 1u, abort_flag, p.status, 0x604);
      tcgen05_fence_after_sync();
      const uint32_t t_acc = tmem_base + lane_base + (uint32_t)(a * 256);
      // the two groups of four warps take alternate blocks of 128 bytes of the tile's rows, so a narrow last tile
      // (N = 144: blocks of 64, 64 and 16 columns) still splits between them
      for (int c0 = h * bc; c0 < p.BN; c0 += 2 * bc) {
        const int col = col_t + c0;
        if (col >= p.N) break;                      // uniform over the group: nothing of this block is stored
        // the store that last used this staging buffer (two blocks ago) has read it; the previous block's may still be reading the other
        uint8_t* stage = stage0 + sbuf * kPStagingBytes;
        sbuf ^= 1;
        if (ht == 0) bulk_wait_group_read_but_one();
        named_barrier_sync(1 + h, 128);
#pragma unroll 1
        for (int j0 = 0; j0 < bc; j0 += 32) {
          uint32_t v[32];
          tmem_ld_x32(t_acc + (uint32_t)(c0 + j0), v);
          tmem_ld_wait();
          float y[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) y[j] = __uint_as_float(v[j]);
          if (p.bias) {
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              const int cj = min(col + j0 + j, p.N - 4);      // N is a multiple of 8: clamped columns are clipped by the store
              const float4 b = __ldg(reinterpret_cast<const float4*>(p.bias + cj));
              y[j] += b.x; y[j + 1] += b.y; y[j + 2] += b.z; y[j + 3] += b.w;
            }
          }
          if (p.act1 >= 0 || p.scale != 1.0f) {
#pragma unroll
            for (int j = 0; j < 32; ++j) y[j] = pair_activate(y[j], p.act1) * p.scale;
          }
          if (p.add && row0 + row < p.M) {   // + tensor: this thread's row, 16-byte pieces (N is a multiple of 8)
            const __nv_bfloat16* arow = reinterpret_cast<const __nv_bfloat16*>(p.add) + (int64_t)(row0 + row) * p.ldc + col + j0;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              if (col + j0 + 8 * k < p.N) {
                const uint4 t = __ldg(reinterpret_cast<const uint4*>(arow + 8 * k));
                y[8 * k] += bf16_lo(t.x); y[8 * k + 1] += bf16_hi(t.x); y[8 * k + 2] += bf16_lo(t.y); y[8 * k + 3] += bf16_hi(t.y);
                y[8 * k + 4] += bf16_lo(t.z); y[8 * k + 5] += bf16_hi(t.z); y[8 * k + 6] += bf16_lo(t.w); y[8 * k + 7] += bf16_hi(t.w);
              }
            }
          }
          if (p.act2 >= 0) {
#pragma unroll
            for (int j = 0; j < 32; ++j) y[j] = pair_activate(y[j], p.act2);
          }
          if (p.c_fp32) {        // 32 columns = the whole 128-byte row of the staged block
#pragma unroll
            for (int k = 0; k < 8; ++k)
              *reinterpret_cast<float4*>(stage + swz_offset((uint32_t)row, (uint32_t)k, 128)) = make_float4(y[4 * k], y[4 * k + 1], y[4 * k + 2], y[4 * k + 3]);
          } else {               // 32 columns = half of the row: chunks j0 / 8 ..
#pragma unroll
            for (int k = 0; k < 4; ++k)
              *reinterpret_cast<uint4*>(stage + swz_offset((uint32_t)row, (uint32_t)((j0 >> 3) + k), 128)) =
                  make_uint4(pack_bf16x2(y[8 * k], y[8 * k + 1]), pack_bf16x2(y[8 * k + 2], y[8 * k + 3]),
                             pack_bf16x2(y[8 * k + 4], y[8 * k + 5]), pack_bf16x2(y[8 * k + 6], y[8 * k + 7]));
          }
        }
        fence_proxy_async_smem();
        named_barrier_sync(1 + h, 128);
        if (ht == 0 && row0 < p.M) {
          tma_store_2d(&tmap_c, stage, p.c_fp32 ? col * 2 : col, row0);   // fp32 tensors are mapped as pairs of 16-bit elements
          bulk_commit_group();
        }
      }
      // this half's share of accumulator a is in registers / shared memory: hand it back to the MMA thread
      tcgen05_fence_before_sync();
      named_barrier_sync(1 + h, 128);
      if (ht == 0) mbar_arrive(rank == 0 ? bar_acce + a : bar_drain + a);   // the leader's MMA thread waits on bar_acce; the peer's goes through its relay
    }
    if (ht == 0) bulk_wait_group_all();             // the stores have left shared memory and are complete
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  cluster_sync_all();          // neither CTA leaves (or frees tensor memory) while the other may still signal it or multiply into it
  if (warp == kPEpiWarps + 1) tmem_dealloc_pair(tmem_base, 512);
}

struct PairMapKey {
  const void* p; int d0, d1, b0, b1; int64_t ld;
  bool operator==(const PairMapKey& o) const { return p == o.p && d0 == o.d0 && d1 == o.d1 && b0 == o.b0 && b1 == o.b1 && ld == o.ld; }
};
struct PairMapKeyHash {
  size_t operator()(const PairMapKey& k) const {
    return std::hash<const void*>()(k.p) ^ ((size_t)k.d0 * 1000003u) ^ ((size_t)k.d1 * 10007u) ^ ((size_t)k.b0 << 7) ^ (size_t)k.b1 ^ ((size_t)k.ld << 20);
  }
};
std::mutex g_pair_mutex;
std::unordered_map<PairMapKey, CUtensorMap, PairMapKeyHash> g_pair_maps;
int g_pair_resident[64] = {};   // pairs the device keeps resident at once (0: not asked yet)

// 16-bit elements [d1 rows][d0 columns], leading dimension ld (elements); box [b1][b0], 128-byte swizzle
bool pair_map(const void* base, int d0, int d1, int64_t ld, int b0, int b1, CUtensorMap* out) {
  std::lock_guard<std::mutex> lock(g_pair_mutex);
  const PairMapKey key{base, d0, d1, b0, b1, ld};
  auto it = g_pair_maps.find(key);
  if (it == g_pair_maps.end()) {
    CUtensorMap m;
    const uint64_t dims[2] = {(uint64_t)d0, (uint64_t)d1};
    const uint64_t strides[1] = {(uint64_t)ld * 2};
    const uint32_t box[2] = {(uint32_t)b0, (uint32_t)b1};
    std::string err;
    if (!encode_tmap_bf16(&m, base, 2, dims, strides, box, 128, &err)) return false;
    if (g_pair_maps.size() > 4096) g_pair_maps.clear();
    it = g_pair_maps.emplace(key, m).first;
  }
  *out = it->second;
  return true;
}

// (+ bias) (activation) (* scale) (+ tensor) (activation): the simple operators this kernel applies, in this order
bool pair_epilogue(const EpiProgram& e, GemmPairParams* p) {
  p->bias = nullptr; p->add = nullptr; p->act1 = -1; p->act2 = -1; p->scale = 1.0f;
  int stage = 0;
  for (int i = 0; i < e.n; ++i) {
    const int c = e.code[i];
    const bool act = c == EPI_RELU || c == EPI_RELU6 || c == EPI_GELU;
    if (c == EPI_BIAS && stage < 1) { p->bias = static_cast<const float*>(e.ptr[i]); stage = 1; }
    else if (act && stage < 2) { p->act1 = c; stage = 2; }
    else if (c == EPI_SCALE && stage < 3) { p->scale = e.f[i]; stage = 3; }
    else if (c == EPI_ADD && stage < 4) { p->add = e.ptr[i]; stage = 4; }
    else if (act && stage == 4) { p->act2 = c; stage = 5; }
    else return false;
  }
  return true;
}

}  // namespace

// Unbatched products with enough rows to fill the SM pairs (wide or narrow, long or short reductions: the narrow,
// short ones -- 1x1 convolutions of a few tens of channels -- are bound by the output stream, which the persistent
// pairs overlap with the next tile's loads and products); everything else stays on the small-tile kernel.
bool gemm_pair_supported(const GemmArgs& a) {
  GemmPairParams probe{};
  if (!pair_epilogue(a.epi, &probe)) return false;
  if (a.a_dtype != AGO_BF16 || a.batches > 1) return false;
  if (a.a_im2col && !(a.R == 1 && a.S == 1 && a.stride == 1 && a.pad == 0)) return false;
  if (a.K % 8 != 0 || a.N % 8 != 0 || a.ldb % 8 != 0 || a.ldc % 8 != 0) return false;
  if (!a.a_im2col && a.lda % 8 != 0) return false;
  if (probe.add && a.c_dtype != AGO_BF16) return false;   // the added tensor has the I/O dtype of a bf16 subgraph
  if (a.M < 512) return false;
  // worth it once the 256-row tiles fill most of the SM pairs
  const long tiles = (long)((a.M + 255) / 256) * ((a.N + 255) / 256);
  return tiles * 2 >= device_sm_count() / 2;
}

cudaError_t launch_gemm_pair(const GemmArgs& a, cudaStream_t stream) {
  GemmPairParams p{};
  pair_epilogue(a.epi, &p);
  p.M = a.M; p.N = a.N; p.K = a.K;
  p.BN = a.N > 128 ? 256 : 128;
  p.b_kmajor = a.b_kmajor;
  p.c_fp32 = a.c_dtype == AGO_FP32 ? 1 : 0;
  p.kblocks = (a.K + kPK - 1) / kPK;
  p.tiles_m = (a.M + 2 * kPM - 1) / (2 * kPM);
  p.tiles_n = (a.N + p.BN - 1) / p.BN;
  p.status = a.status;
  p.ldc = a.ldc;
  const int64_t lda = a.a_im2col ? a.K : a.lda;
  CUtensorMap ma, mb, mc;
  if (!pair_map(a.A, a.K, a.M, lda, kPK, kPM, &ma)) return cudaErrorInvalidValue;
  if (a.b_kmajor ? !pair_map(a.B, a.K, a.N, a.ldb, kPK, p.BN / 2, &mb) : !pair_map(a.B, a.N, a.K, a.ldb, 64, kPK, &mb)) return cudaErrorInvalidValue;
  // the output as 16-bit elements: an fp32 tensor has twice the columns; blocks of 128 bytes x 128 rows
  const int cmul = p.c_fp32 ? 2 : 1;
  if (!pair_map(a.C, a.N * cmul, a.M, a.ldc * cmul, 64, kPM, &mc)) return cudaErrorInvalidValue;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  {
    static int smem_opt_in[64] = {};
    e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(gemm_pair_kernel), smem_opt_in);
    if (e != cudaSuccess) return e;
  }
  int resident;
  {
    std::lock_guard<std::mutex> lock(g_pair_mutex);
    if (g_pair_resident[dev] == 0) {
      cudaLaunchConfig_t cfg = cudaLaunchConfig_t{};
      cudaLaunchAttribute attr[1];
      cfg.gridDim = dim3(2 * 512, 1, 1); cfg.blockDim = dim3(kPThreads, 1, 1); cfg.dynamicSmemBytes = kPSmemBytes;
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr; cfg.numAttrs = 1;
      int n = 0;
      e = cudaOccupancyMaxActiveClusters(&n, gemm_pair_kernel, &cfg);
      if (e != cudaSuccess) return e;
      if (n < 1) return cudaErrorInvalidConfiguration;
      g_pair_resident[dev] = n;
    }
    resident = g_pair_resident[dev];
  }
  p.pairs = std::min(resident, p.tiles_m * p.tiles_n);
  gemm_pair_kernel<<<dim3(2 * p.pairs), kPThreads, kPSmemBytes, stream>>>(ma, mb, mc, p);
  return cudaGetLastError();
}

}  // namespace ago
