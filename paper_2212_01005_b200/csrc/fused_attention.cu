// Fused attention: S = Q K^T, * scale, row softmax, O = P V -- one kernel per
// (batch, head, block of 128 query rows); scores and probabilities never leave
// the SM.
//
// Tile choice (Section III-B, "downstream pointwise / matmul" category): the
// downstream contraction P V reuses its input only along its output columns, so
// its tile keeps ALL of them (head_dim) and is tiled over rows (128 queries).
// The softmax in between is a simple operator over whole rows, so the upstream
// tile is 128 query rows x ALL keys: the full score block sits in tensor memory
// (128 lanes x S fp32 columns) and the exact two-pass softmax needs no rescaling.
//
//   P1  TMA: Q [128 x 64], K [S x 64], V [S x 64] -> 128-byte-swizzled tiles
//   P2  tcgen05.mma: S[128 x S] = Q K^T                         (TMEM, fp32)
//   P3/P4  CUDA cores, one thread per (row, half of the keys): TMEM -> registers,
//       row max (shuffle-free: one row per thread, halves exchanged through
//       shared memory), p = exp2((s - max) * scale * log2 e), bf16 -> shared
//       memory in the K-major operand layout, row sum
//   P5  tcgen05.mma: O[128 x 64] = P V   (V is the N-major B operand, as it lies in HBM)
//   P6  TMEM -> registers, * 1 / rowsum, bf16, 16-byte stores
#include <cuda.h>
#include <cuda_bf16.h>

#include <unordered_map>

#include "fused.h"
#include "tc_common.cuh"
#include "tmap.h"

namespace ago {

namespace {

using namespace tc;

constexpr int kD = 64;                 // head dimension (one 128-byte swizzle row)
constexpr int kBlockM = 128;           // query rows per CTA
constexpr int kKeyBlock = 128;         // keys per TMA box / per score MMA
constexpr int kComputeThreads = 256;   // two threads per query row (each half of the keys)
constexpr int kThreads = kComputeThreads + 32;

struct AttnParams {
  __nv_bfloat16* out;
  unsigned int* status;
  int B, S, heads, E;
  int Spad;        // keys rounded up to 16
  int nkb;         // key blocks of 128
  int half;        // first column of the second thread group's half (multiple of 16)
  float scale_log2e;
  int off_q, off_k, off_v, off_p, off_red, off_bar;
};

__global__ void __launch_bounds__(kThreads, 1)
attention_fused_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                       const __grid_constant__ CUtensorMap tmap_v, const AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem + p.off_q;
  uint8_t* sK = smem + p.off_k;
  uint8_t* sV = smem + p.off_v;
  uint8_t* sP = smem + p.off_p;
  float* sRed = reinterpret_cast<float*>(smem + p.off_red);   // [2][128] max, then [2][128] sum
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
  uint64_t* bar_qk = bars + 0;   // Q and K landed
  uint64_t* bar_v = bars + 1;    // V landed
  uint64_t* bar_s = bars + 2;    // scores complete
  uint64_t* bar_p = bars + 3;    // probabilities written
  uint64_t* bar_o = bars + 4;    // output accumulators complete
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 5);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 6);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int q0 = blockIdx.x * kBlockM, h = blockIdx.y, b = blockIdx.z;

  if (tid == kComputeThreads) {
    *abort_flag = 0u;
    for (int i = 0; i < 5; ++i) mbar_init(bars + i, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmap_q);
    tma_prefetch_desc(&tmap_k);
    tma_prefetch_desc(&tmap_v);
    mbar_arrive_expect_tx(bar_qk, (uint32_t)((kBlockM + p.nkb * kKeyBlock) * kD * 2));
    tma_load_3d(sQ, &tmap_q, bar_qk, h * kD, q0, b);
    for (int kb = 0; kb < p.nkb; ++kb) tma_load_3d(sK + kb * kKeyBlock * kD * 2, &tmap_k, bar_qk, h * kD, kb * kKeyBlock, b);
    mbar_arrive_expect_tx(bar_v, (uint32_t)(p.nkb * kKeyBlock * kD * 2));
    for (int kb = 0; kb < p.nkb; ++kb) tma_load_3d(sV + kb * kKeyBlock * kD * 2, &tmap_v, bar_v, h * kD, kb * kKeyBlock, b);
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t ocol0 = 384;   // output accumulators after the score block

  if (warp == kComputeThreads / 32) {
    // ============================ MMA issue (one lane) ============================
    if (lane == 0) {
      const uint64_t qdesc = make_smem_desc(smem_u32(sQ), 0, 1024, SW_128B);
      const uint64_t kdesc = make_smem_desc(smem_u32(sK), 0, 1024, SW_128B);
      mbar_wait(bar_qk, 0, abort_flag, p.status, 0x201);
      tcgen05_fence_after_sync();
      for (int kb = 0; kb < p.nkb; ++kb) {
        const int n = min(kKeyBlock, p.Spad - kb * kKeyBlock);
        const uint32_t idesc = make_idesc_bf16(128, (uint32_t)n);
        const uint64_t bd = kdesc + (uint64_t)((kb * kKeyBlock * kD * 2) >> 4);
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) umma_bf16(tmem_base + kb * kKeyBlock, qdesc + 2u * ks, bd + 2u * ks, idesc, ks > 0);
      }
      umma_commit(bar_s);

      // O = P V: P is K-major (64-key blocks of 128-byte rows), V is N-major as stored ([key][d])
      const uint64_t pdesc = make_smem_desc(smem_u32(sP), 0, 1024, SW_128B);
      const uint64_t vdesc = make_smem_desc(smem_u32(sV), 0, 1024, SW_128B);
      const uint32_t idesc_o = make_idesc_bf16(128, kD, 0, 1);
      mbar_wait(bar_v, 0, abort_flag, p.status, 0x202);
      mbar_wait(bar_p, 0, abort_flag, p.status, 0x203);
      tcgen05_fence_after_sync();
      const int ksteps = p.Spad / 16;
      for (int ks = 0; ks < ksteps; ++ks) {
        const uint64_t ad = pdesc + (uint64_t)(((ks >> 2) * kBlockM * 128 + (ks & 3) * 32) >> 4);
        const uint64_t bd = vdesc + (uint64_t)((ks * 16 * kD * 2) >> 4);
        umma_bf16(tmem_base + ocol0, ad, bd, idesc_o, ks > 0);
      }
      umma_commit(bar_o);
    }
    __syncwarp();
  } else {
    // ============================ softmax + epilogue warps ============================
    const int row = (warp & 3) * 32 + lane;     // TMEM lane = query row of this tile
    const int grp = warp >> 2;                  // which half of the keys / of the output columns
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const int c_begin = grp == 0 ? 0 : p.half;
    const int c_end = grp == 0 ? p.half : p.Spad;

    mbar_wait(bar_s, 0, abort_flag, p.status, 0x204);
    tcgen05_fence_after_sync();

    // pass 1: row maximum of the raw scores over this thread's half
    float m = -INFINITY;
    for (int c0 = c_begin; c0 < c_end; c0 += 16) {
      uint32_t v[16];
      tmem_ld_x16(tmem_base + lane_base + c0, v);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if (c0 + j < p.S) m = fmaxf(m, __uint_as_float(v[j]));
    }
    sRed[grp * kBlockM + row] = m;
    named_barrier_sync(1, kComputeThreads);
    m = fmaxf(sRed[row], sRed[kBlockM + row]);

    // pass 2: p = exp2((s - m) * scale * log2 e), rounded to bf16, into the A-operand layout
    const float c = p.scale_log2e;
    const float mc = m * c;
    float sum = 0.0f;
    for (int c0 = c_begin; c0 < c_end; c0 += 16) {
      uint32_t v[16];
      tmem_ld_x16(tmem_base + lane_base + c0, v);
      tmem_ld_wait();
      uint32_t w[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float e0 = exp2f(fmaf(__uint_as_float(v[2 * j]), c, -mc));
        float e1 = exp2f(fmaf(__uint_as_float(v[2 * j + 1]), c, -mc));
        if (c0 + 2 * j >= p.S) e0 = 0.0f;
        if (c0 + 2 * j + 1 >= p.S) e1 = 0.0f;
        const __nv_bfloat162 hb = __floats2bfloat162_rn(e0, e1);
        w[j] = *reinterpret_cast<const uint32_t*>(&hb);
        sum += __low2float(hb) + __high2float(hb);
      }
      // columns c0..c0+15 = two 16-byte chunks of key block c0/64
      uint8_t* blk = sP + (c0 >> 6) * (kBlockM * 128);
      const uint32_t ch = (uint32_t)(c0 & 63) >> 3;
      *reinterpret_cast<uint4*>(blk + swz_offset(row, ch, 128)) = make_uint4(w[0], w[1], w[2], w[3]);
      *reinterpret_cast<uint4*>(blk + swz_offset(row, ch + 1, 128)) = make_uint4(w[4], w[5], w[6], w[7]);
    }
    sRed[2 * kBlockM + grp * kBlockM + row] = sum;
    fence_proxy_async_smem();
    tcgen05_fence_before_sync();
    named_barrier_sync(1, kComputeThreads);
    if (tid == 0) mbar_arrive(bar_p);
    const float inv = 1.0f / (sRed[2 * kBlockM + row] + sRed[3 * kBlockM + row]);

    // epilogue: this thread stores 32 of the row's 64 output columns
    mbar_wait(bar_o, 0, abort_flag, p.status, 0x205);
    tcgen05_fence_after_sync();
    uint32_t o[32];
    tmem_ld_x32(tmem_base + lane_base + ocol0 + grp * 32, o);
    tmem_ld_wait();
    if (q0 + row < p.S) {
      __nv_bfloat16* dst = p.out + ((size_t)b * p.S + q0 + row) * p.E + h * kD + grp * 32;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        *reinterpret_cast<uint4*>(dst + j * 8) =
            make_uint4(pack_bf16x2(__uint_as_float(o[8 * j]) * inv, __uint_as_float(o[8 * j + 1]) * inv),
                       pack_bf16x2(__uint_as_float(o[8 * j + 2]) * inv, __uint_as_float(o[8 * j + 3]) * inv),
                       pack_bf16x2(__uint_as_float(o[8 * j + 4]) * inv, __uint_as_float(o[8 * j + 5]) * inv),
                       pack_bf16x2(__uint_as_float(o[8 * j + 6]) * inv, __uint_as_float(o[8 * j + 7]) * inv));
      }
    }
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, 512);
}

struct AttnHost {
  AttnParams prm;
  int smem_bytes = 0;
  struct Maps { CUtensorMap q, k, v; };
  std::unordered_map<const void*, CUtensorMap> maps;   // keyed by base pointer (box shape is the same for Q, K, V)
};

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
  if (q.S > 384) return bad("more than 384 keys do not fit the score block in tensor memory");
  q.Spad = (q.S + 15) / 16 * 16;
  q.nkb = (q.Spad + kKeyBlock - 1) / kKeyBlock;
  q.half = ((q.Spad / 2) + 15) / 16 * 16;
  q.scale_log2e = plan->ops[1].op.f * 1.4426950408889634f;
  int off = 0;
  auto take = [&](int bytes) { int o = off; off = (off + bytes + 1023) / 1024 * 1024; return o; };
  q.off_q = take(kBlockM * kD * 2);
  q.off_k = take(q.nkb * kKeyBlock * kD * 2);
  q.off_v = take(q.nkb * kKeyBlock * kD * 2);
  q.off_p = take(((q.Spad + 63) / 64) * kBlockM * 128);
  q.off_red = take(4 * kBlockM * 4);
  q.off_bar = take(128);
  host->smem_bytes = off + 1024;
  st->impl = host;
  st->impl_free = [](void* p) { delete static_cast<AttnHost*>(p); };
  st->tile_rows = kBlockM; st->grid = ((q.S + kBlockM - 1) / kBlockM) * q.heads * q.B; st->smem_bytes = host->smem_bytes;
  plan->tile_rows = kBlockM; plan->smem_bytes = host->smem_bytes;
  return AGO_OK;
}

ago_status_t attention_run(const Plan& plan, FusedState* st, const void* const* inputs, const void* const* weights,
                           void* output, unsigned int* status_word, cudaStream_t stream, std::string* err) {
  AttnHost* host = static_cast<AttnHost*>(st->impl);
  AttnParams q = host->prm;
  q.out = static_cast<__nv_bfloat16*>(output);
  q.status = status_word;
  const CUtensorMap* maps[3];
  for (int i = 0; i < 3; ++i) {
    auto it = host->maps.find(inputs[i]);
    if (it == host->maps.end()) {
      CUtensorMap m;
      const uint64_t dims[3] = {(uint64_t)q.E, (uint64_t)q.S, (uint64_t)q.B};
      const uint64_t strides[2] = {(uint64_t)q.E * 2, (uint64_t)q.S * q.E * 2};
      const uint32_t box[3] = {(uint32_t)kD, (uint32_t)kKeyBlock, 1};
      if (!encode_tmap_bf16(&m, inputs[i], 3, dims, strides, box, 128, err)) return AGO_ERR_CUDA;
      if (host->maps.size() > 4096) host->maps.clear();
      it = host->maps.emplace(inputs[i], m).first;
    }
    maps[i] = &it->second;
  }
  {
    static int smem_opt_in[64] = {};
    cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(attention_fused_kernel), smem_opt_in);
    if (e != cudaSuccess) { *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  }
  dim3 grid((q.S + kBlockM - 1) / kBlockM, q.heads, q.B);
  attention_fused_kernel<<<grid, kThreads, host->smem_bytes, stream>>>(*maps[0], *maps[1], *maps[2], q);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { *err = std::string("fused attention launch: ") + cudaGetErrorString(e); return AGO_ERR_CUDA; }
  return AGO_OK;
}

}  // namespace ago
