// Tensor-core GEMM of the unfused modes: C[M][N] = epilogue(A[M][K] * B), one launch per complex
// operator with its simple operators applied in the epilogue (Section III-A, "Conventional fusion
// within a mini-subgraph"). It serves the 1x1 convolutions (B = [N][K], K-major) and the GEMM
// operator (B = [K][N], N-major) and the batched per-head products of attention whenever the operands
// are bf16; everything else stays on the generic CUDA-core kernel. The point of this kernel is an honest baseline for the fused kernels:
// the intermediate tensors still travel through device memory, but the contraction itself runs on
// tcgen05 like theirs.
//
//   TMA ring (4 stages of A [128 x 64] + B [128 x 64]) -> tcgen05.mma 128 x N_tile x 16 into TMEM
//   -> 128 epilogue threads (one row each): simple operators in fp32, bf16 / fp32 vector stores.
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

constexpr int kBM = 128, kBN = 128, kBK = 64;
constexpr int kMaxStages = 4;   // ring stages: 3 when the grid exceeds one CTA per SM (two CTAs then share an SM and one CTA's epilogue
                                // overlaps the other's products), else 4; never more than the K blocks
constexpr int kStageBytes = 32 * 1024;
constexpr int kEpiThreads = 128;
constexpr int kThreads = kEpiThreads + 64;   // + TMA warp + MMA warp

struct GemmTcParams {
  void* C;
  int M, N, K;
  int64_t ldc;
  int b_kmajor;
  int c_dtype, add_dtype;
  int kblocks, stages;
  int heads;               // blockIdx.z = batch * heads + head
  int64_t c_sb, c_sh;      // element offsets of a batch / head in C (and in the EPI_ADD operand)
  int bar_off;             // shared-memory offset of the barriers: after the ring and after the epilogue's staging tile
  // the simple operators in canonical order: + bias, activation 1, * scale, + tensor, activation 2
  const float* bias;       // or null
  const void* add;         // or null; same shape and leading dimension as C
  int act1, act2;          // EPI_RELU | EPI_RELU6 | EPI_GELU | -1
  float scale;             // 1 when absent
  unsigned int* status;    // records a bounded wait that gave up (or null)
};

__device__ __forceinline__ float activate(float x, int act) {
  if (act == EPI_RELU) return fmaxf(x, 0.0f);
  if (act == EPI_RELU6) return fminf(fmaxf(x, 0.0f), 6.0f);
  return x;
}

__device__ __forceinline__ float gelu_tanh_f(float v) {
  const float c = 0.7978845608028654f;
  return 0.5f * v * (1.0f + tanhf(c * (v + 0.044715f * v * v * v)));
}

__global__ void __launch_bounds__(kThreads)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const GemmTcParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sRing = smem;
  const int kStages = p.stages;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.bar_off);
  uint64_t* bar_full = bars;
  uint64_t* bar_empty = bars + kMaxStages;
  uint64_t* bar_acc = bars + 2 * kMaxStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_acc + 1);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bar_acc + 2);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int row0 = blockIdx.x * kBM, n0 = blockIdx.y * kBN;
  const int zb = blockIdx.z / p.heads, zh = blockIdx.z - zb * p.heads;
  const int ncols = min(kBN, (p.N - n0 + 15) & ~15);   // MMA N of this tile (multiple of 16)

  if (tid == kEpiThreads) {
    *abort_flag = 0u;
    for (int i = 0; i < kStages; ++i) { mbar_init(bar_full + i, 1); mbar_init(bar_empty + i, 1); }
    mbar_init(bar_acc, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, 128);
    tmem_relinquish();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == kEpiThreads / 32) {
    // ================================ TMA producer ================================
    if (lane == 0) {
      tma_prefetch_desc(&tmap_a);
      tma_prefetch_desc(&tmap_b);
      for (int i = 0; i < p.kblocks; ++i) {
        const int s = i % kStages;
        if (i >= kStages) mbar_wait(bar_empty + s, (uint32_t)((i / kStages) - 1) & 1u, abort_flag, p.status, 0x501);
        uint8_t* st = sRing + s * kStageBytes;
        mbar_arrive_expect_tx(bar_full + s, kStageBytes);
        tma_load_4d(st, &tmap_a, bar_full + s, i * kBK, row0, zh, zb);          // A [128 rows x 64 k]
        if (p.b_kmajor) {
          tma_load_4d(st + 16384, &tmap_b, bar_full + s, i * kBK, n0, zh, zb);  // B [128 n x 64 k]
        } else {
          tma_load_4d(st + 16384, &tmap_b, bar_full + s, n0, i * kBK, zh, zb);  // B [64 k x 64 n], twice
          tma_load_4d(st + 16384 + 8192, &tmap_b, bar_full + s, n0 + 64, i * kBK, zh, zb);
        }
      }
    }
    __syncwarp();
  } else if (warp == kEpiThreads / 32 + 1) {
    // ================================ MMA issuer ================================
    // the whole warp, converged; MMAs and commits predicated on one elected lane (see tc_common.cuh)
    {
      const uint32_t elected = elect_one();
      const uint32_t idesc = make_idesc_bf16(128, (uint32_t)ncols, 0, p.b_kmajor ? 0 : 1);
      for (int i = 0; i < p.kblocks; ++i) {
        const int s = i % kStages;
        mbar_wait(bar_full + s, (uint32_t)(i / kStages) & 1u, abort_flag, p.status, 0x502);
        tcgen05_fence_after_sync();
        const uint32_t st = smem_u32(sRing + s * kStageBytes);
        const uint64_t ad = make_smem_desc(st, 0, 1024, SW_128B);
        const uint64_t bd = p.b_kmajor ? make_smem_desc(st + 16384, 0, 1024, SW_128B) : make_smem_desc(st + 16384, 8192, 1024, SW_128B);
#pragma unroll
        for (int ks = 0; ks < kBK / 16; ++ks)
          umma_bf16_elected_acc(tmem_base, ad + 2u * ks, bd + (p.b_kmajor ? (uint64_t)(2u * ks) : (uint64_t)((ks * 2048) >> 4)), idesc, elected, (i | ks) != 0);
        umma_commit_elected(bar_empty + s, elected);
      }
      if (!skip_signal_for_test(p.status, 0x503)) umma_commit_elected(bar_acc, elected);
    }
    __syncwarp();
  } else {
    // ============ epilogue: thread = row -> staging tile in shared memory -> coalesced stores ============
    const int r = warp * 32 + lane;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    const int esz = p.c_dtype == AGO_FP32 ? 4 : 2;
    const int ncv = min(ncols, p.N - n0);                 // valid columns of this tile (a multiple of 8)
    const int pitch = ncols * esz + 16;                   // staged row pitch: 16-byte stores of a quarter-warp hit distinct banks
    uint8_t* stage = sRing;                               // the ring is idle once the accumulator is complete
    mbar_wait(bar_acc, 0, abort_flag, p.status, 0x503);
    tcgen05_fence_after_sync();
    const bool gelu1 = p.act1 == EPI_GELU, gelu2 = p.act2 == EPI_GELU;
    for (int c0 = 0; c0 < ncols; c0 += 16) {
      uint32_t v[16];
      tmem_ld_x16(tmem_base + lane_base + c0, v);
      tmem_ld_wait();
      if (c0 >= ncv) break;                               // warp-uniform
      float y[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) y[j] = __uint_as_float(v[j]);
      const int col = n0 + c0;
      const int nv = min(16, ncv - c0);                   // 8 or 16
      if (p.bias) {
#pragma unroll
        for (int j = 0; j < 16; j += 4) {
          if (j < nv) {
            const float4 b = __ldg(reinterpret_cast<const float4*>(p.bias + col + j));
            y[j] += b.x; y[j + 1] += b.y; y[j + 2] += b.z; y[j + 3] += b.w;
          }
        }
      }
#pragma unroll
      for (int j = 0; j < 16; ++j) y[j] = (gelu1 ? gelu_tanh_f(y[j]) : activate(y[j], p.act1)) * p.scale;
      if (p.add && row0 + r < p.M) {
        const int64_t idx = zb * p.c_sb + zh * p.c_sh + (int64_t)(row0 + r) * p.ldc + col;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (h * 8 < nv) {
            if (p.add_dtype == AGO_FP32) {
              const float4* a4 = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.add) + idx + h * 8);
              const float4 a0 = __ldg(a4), a1 = __ldg(a4 + 1);
              y[h * 8] += a0.x; y[h * 8 + 1] += a0.y; y[h * 8 + 2] += a0.z; y[h * 8 + 3] += a0.w;
              y[h * 8 + 4] += a1.x; y[h * 8 + 5] += a1.y; y[h * 8 + 6] += a1.z; y[h * 8 + 7] += a1.w;
            } else {
              const uint4 a = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.add) + idx + h * 8));
              y[h * 8] += bf16_lo(a.x); y[h * 8 + 1] += bf16_hi(a.x); y[h * 8 + 2] += bf16_lo(a.y); y[h * 8 + 3] += bf16_hi(a.y);
              y[h * 8 + 4] += bf16_lo(a.z); y[h * 8 + 5] += bf16_hi(a.z); y[h * 8 + 6] += bf16_lo(a.w); y[h * 8 + 7] += bf16_hi(a.w);
            }
          }
        }
      }
#pragma unroll
      for (int j = 0; j < 16; ++j) y[j] = gelu2 ? gelu_tanh_f(y[j]) : activate(y[j], p.act2);
      uint8_t* dst = stage + r * pitch + c0 * esz;
      if (p.c_dtype == AGO_FP32) {
#pragma unroll
        for (int j = 0; j < 16; j += 4) *reinterpret_cast<float4*>(dst + j * 4) = make_float4(y[j], y[j + 1], y[j + 2], y[j + 3]);
      } else {
        *reinterpret_cast<uint4*>(dst) = make_uint4(pack_bf16x2(y[0], y[1]), pack_bf16x2(y[2], y[3]), pack_bf16x2(y[4], y[5]), pack_bf16x2(y[6], y[7]));
        *reinterpret_cast<uint4*>(dst + 16) = make_uint4(pack_bf16x2(y[8], y[9]), pack_bf16x2(y[10], y[11]), pack_bf16x2(y[12], y[13]), pack_bf16x2(y[14], y[15]));
      }
    }
    named_barrier_sync(1, kEpiThreads);
    // consecutive threads store consecutive 16-byte chunks of a row
    const int chunks = ncv * esz / 16;
    const int rows_here = min(kBM, p.M - row0);
    uint8_t* cbase = reinterpret_cast<uint8_t*>(p.C) + (zb * p.c_sb + zh * p.c_sh + (int64_t)row0 * p.ldc + n0) * esz;
    for (int i = tid; i < rows_here * chunks; i += kEpiThreads) {
      const int rr = i / chunks, ch = i - rr * chunks;
      *reinterpret_cast<uint4*>(cbase + (int64_t)rr * p.ldc * esz + ch * 16) = *reinterpret_cast<const uint4*>(stage + rr * pitch + ch * 16);
    }
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, 128);
}

struct MapKey {
  const void* p; int d0, d1, d2, d3, b0, b1; int64_t ld, sh, sb;
  bool operator==(const MapKey& o) const {
    return p == o.p && d0 == o.d0 && d1 == o.d1 && d2 == o.d2 && d3 == o.d3 && b0 == o.b0 && b1 == o.b1 && ld == o.ld && sh == o.sh && sb == o.sb;
  }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    return std::hash<const void*>()(k.p) ^ ((size_t)k.d0 * 1000003u) ^ ((size_t)k.d1 * 10007u) ^ ((size_t)k.d2 * 131u) ^ ((size_t)k.d3 * 31u) ^
           ((size_t)k.b0 << 7) ^ (size_t)k.b1 ^ ((size_t)k.ld << 20) ^ ((size_t)k.sh << 3) ^ ((size_t)k.sb << 11);
  }
};
std::mutex g_map_mutex;
std::unordered_map<MapKey, CUtensorMap, MapKeyHash> g_maps;

// bf16 matrices [d1 rows][d0 columns] with leading dimension ld, d2 heads sh elements apart in each of d3 batches
// sb elements apart; box [b1][b0] of one matrix, 128-byte swizzle
bool get_map(const void* base, int d0, int d1, int d2, int d3, int64_t ld, int64_t sh, int64_t sb, int b0, int b1, CUtensorMap* out) {
  std::lock_guard<std::mutex> lock(g_map_mutex);
  const MapKey key{base, d0, d1, d2, d3, b0, b1, ld, sh, sb};
  auto it = g_maps.find(key);
  if (it == g_maps.end()) {
    CUtensorMap m;
    const uint64_t dims[4] = {(uint64_t)d0, (uint64_t)d1, (uint64_t)d2, (uint64_t)d3};
    const uint64_t strides[3] = {(uint64_t)ld * 2, (uint64_t)sh * 2, (uint64_t)sb * 2};
    const uint32_t box[4] = {(uint32_t)b0, (uint32_t)b1, 1, 1};
    std::string err;
    if (!encode_tmap_bf16(&m, base, 4, dims, strides, box, 128, &err)) return false;
    if (g_maps.size() > 4096) g_maps.clear();
    it = g_maps.emplace(key, m).first;
  }
  *out = it->second;
  return true;
}

}  // namespace

// The simple operators as (+ bias) (activation) (* scale) (+ tensor) (activation), each at most once and in this order.
static bool canonical_epilogue(const EpiProgram& e, GemmTcParams* p) {
  p->bias = nullptr; p->add = nullptr; p->act1 = -1; p->act2 = -1; p->scale = 1.0f;
  int stage = 0;   // 0: nothing yet, 1: bias, 2: act1, 3: scale, 4: add, 5: act2
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

bool gemm_tc_supported(const GemmArgs& a) {
  GemmTcParams probe{};
  if (!canonical_epilogue(a.epi, &probe)) return false;
  if (a.a_dtype != AGO_BF16) return false;
  if (a.a_im2col && !(a.R == 1 && a.S == 1 && a.stride == 1 && a.pad == 0)) return false;
  if (a.K % 8 != 0 || a.N % 8 != 0) return false;
  // 16-byte rows, heads and batches for TMA and for the vector stores
  const int heads = std::max(a.heads, 1);
  if (!a.a_im2col && a.lda % 8 != 0) return false;
  if (a.ldb % 8 != 0 || a.ldc % 8 != 0) return false;
  if (a.batches > 1 && (a.a_sb % 8 || a.a_sh % 8 || a.b_sb % 8 || a.b_sh % 8 || a.c_sb % 8 || a.c_sh % 8)) return false;
  if (a.batches > 65535 || a.batches % heads != 0) return false;
  return true;
}

cudaError_t launch_gemm_tc(const GemmArgs& a, int add_dtype, cudaStream_t stream) {
  CUtensorMap ma, mb;
  const int heads = a.batches > 1 ? std::max(a.heads, 1) : 1, nb = std::max(a.batches, 1) / heads;
  const int64_t lda = a.a_im2col ? a.K : a.lda;
  // unbatched operands: the outer two dimensions have extent 1, their strides only need to be legal
  const int64_t a_sh = a.batches > 1 ? a.a_sh : lda * a.M, a_sb = a.batches > 1 ? a.a_sb : lda * a.M;
  const int64_t b_rows = a.b_kmajor ? a.N : a.K;
  const int64_t b_sh = a.batches > 1 ? a.b_sh : a.ldb * b_rows, b_sb = a.batches > 1 ? a.b_sb : a.ldb * b_rows;
  if (!get_map(a.A, a.K, a.M, heads, nb, lda, a_sh, a_sb, kBK, kBM, &ma)) return cudaErrorInvalidValue;
  if (a.b_kmajor ? !get_map(a.B, a.K, a.N, heads, nb, a.ldb, b_sh, b_sb, kBK, kBN, &mb)
                 : !get_map(a.B, a.N, a.K, heads, nb, a.ldb, b_sh, b_sb, 64, kBK, &mb)) return cudaErrorInvalidValue;
  GemmTcParams p{};
  p.C = a.C; p.M = a.M; p.N = a.N; p.K = a.K; p.ldc = a.ldc; p.b_kmajor = a.b_kmajor;
  p.c_dtype = a.c_dtype; p.add_dtype = add_dtype;
  p.kblocks = (a.K + kBK - 1) / kBK;
  p.heads = heads; p.c_sb = a.batches > 1 ? a.c_sb : 0; p.c_sh = a.batches > 1 ? a.c_sh : 0;
  canonical_epilogue(a.epi, &p);
  p.status = a.status;
  const long ctas = (long)((a.M + kBM - 1) / kBM) * ((a.N + kBN - 1) / kBN) * heads * nb;
  p.stages = std::min(ctas > device_sm_count() ? 3 : kMaxStages, p.kblocks);
  // the epilogue stages the output tile (128 rows x (columns x element size + 16) bytes) over the idle ring
  const int tile_cols = std::min(kBN, (a.N + 15) & ~15);
  const int staging = kBM * (tile_cols * (a.c_dtype == AGO_FP32 ? 4 : 2) + 16);
  p.bar_off = (std::max(p.stages * kStageBytes, staging) + 1023) & ~1023;
  const int smem = p.bar_off + 256 + 1024;
  const int smem_max = kMaxStages * kStageBytes + 256 + 1024;
  static std::once_flag once[64];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64)
    std::call_once(once[dev], [&] { cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max); });
  dim3 grid((a.M + kBM - 1) / kBM, (a.N + kBN - 1) / kBN, heads * nb);
  gemm_tc_kernel<<<grid, kThreads, smem, stream>>>(ma, mb, p);
  return cudaGetLastError();
}

}  // namespace ago
