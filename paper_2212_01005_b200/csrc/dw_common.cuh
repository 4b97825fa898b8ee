// Depthwise 3x3 building blocks of the fused kernels: CUDA-core arithmetic on bf16 channel pairs held in
// shared memory as planes of [pixel][8 channels] (16 bytes per pixel), mixed-precision FMAs (bf16 operands as
// stored, fp32 accumulate), bias and ReLU6 fused into the store (Section III-A: simple operators are applied right
// after the window sum).
#pragma once
#include <cstdint>

namespace ago {
namespace dw {

// bf16x2(min(max(lo, 0), 6), min(max(hi, 0), 6)): the conversion clamps at 0, one packed min caps at 6.
__device__ __forceinline__ uint32_t relu6_pack(float lo, float hi) {
  uint32_t r;
  asm("{\n\t.reg .b32 t;\n\tcvt.rn.relu.bf16x2.f32 t, %2, %1;\n\tmin.bf16x2 %0, t, %3;\n\t}"
      : "=r"(r) : "f"(lo), "f"(hi), "r"(0x40C040C0u));   // the packed 6.0 is an operand, so one register serves every call
  return r;
}

// Shared-memory word loads / stores with an immediate byte offset.
template <int OFF>
__device__ __forceinline__ uint32_t lds32(uint32_t saddr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(saddr), "n"(OFF));
  return v;
}
template <int OFF = 0>
__device__ __forceinline__ void sts32(uint32_t saddr, uint32_t v) {
  asm volatile("st.shared.u32 [%0+%1], %2;" ::"r"(saddr), "n"(OFF), "r"(v) : "memory");
}

// acc += x * w for a packed pair of bf16 channels: the mixed-precision FMA takes the bf16 operands
// as they are (exact product, fp32 accumulate) -- no unpacking of the activations or the weights.
__device__ __forceinline__ void fma_pair(float2& acc, uint32_t x, uint32_t w) {
  asm("{\n\t.reg .b16 xl, xh, wl, wh;\n\t"
      "mov.b32 {xl, xh}, %2;\n\tmov.b32 {wl, wh}, %3;\n\t"
      "fma.rn.f32.bf16 %0, xl, wl, %0;\n\tfma.rn.f32.bf16 %1, xh, wh, %1;\n\t}"
      : "+f"(acc.x), "+f"(acc.y) : "r"(x), "r"(w));
}

struct Row3 { uint32_t v0, v1, v2; };   // three horizontally adjacent pixels of one channel pair
template <int PIX_STEP>
__device__ __forceinline__ Row3 load_row3(uint32_t a) {
  Row3 r;
  r.v0 = lds32<0>(a); r.v1 = lds32<PIX_STEP>(a); r.v2 = lds32<2 * PIX_STEP>(a);
  return r;
}
__device__ __forceinline__ uint32_t depthwise_point(const Row3& a, const Row3& b, const Row3& c, const uint32_t (&w)[9],
                                                    float2 bias) {
  float2 acc = bias;
  fma_pair(acc, a.v0, w[0]); fma_pair(acc, a.v1, w[1]); fma_pair(acc, a.v2, w[2]);
  fma_pair(acc, b.v0, w[3]); fma_pair(acc, b.v1, w[4]); fma_pair(acc, b.v2, w[5]);
  fma_pair(acc, c.v0, w[6]); fma_pair(acc, c.v1, w[7]); fma_pair(acc, c.v2, w[8]);
  return relu6_pack(acc.x, acc.y);
}

// E and D chunks are two planes of [pixel][8 channels] (16 bytes per pixel), which is also the
// un-swizzled K-major operand layout; all addresses below are 32-bit shared-memory addresses.
//
// Stride-2 depthwise 3x3 for one (channel pair, output column) and output rows [r0, r1), r1 > r0:
// consecutive output rows share one input row, which stays packed in registers (the loop body is
// unrolled over the two roles of that row).
__device__ __forceinline__ void depthwise_column_s2(uint32_t e_col, uint32_t d_col, int r0, int r1, int IW, int Wo,
                                                    const uint32_t (&w)[9], float2 bias) {
  const uint32_t e_pitch = (uint32_t)IW * 16u, d_pitch = (uint32_t)Wo * 16u;
  uint32_t src = e_col + (uint32_t)(r0 * 2) * e_pitch;
  uint32_t dst = d_col + (uint32_t)r0 * d_pitch;
  int n = r1 - r0;
  Row3 a = load_row3<16>(src), b, c;
  src += e_pitch;
  while (true) {
    b = load_row3<16>(src); c = load_row3<16>(src + e_pitch); src += 2 * e_pitch;
    sts32(dst, depthwise_point(a, b, c, w, bias)); dst += d_pitch;
    if (--n == 0) break;
    b = load_row3<16>(src); a = load_row3<16>(src + e_pitch); src += 2 * e_pitch;
    sts32(dst, depthwise_point(c, b, a, w, bias)); dst += d_pitch;
    if (--n == 0) break;
  }
}

// Stride-1 depthwise 3x3 for one channel pair and a block of 2 output rows x 7 output columns, fully
// unrolled: three input columns (4 rows each) stay packed in registers and rotate by renaming, all
// shared-memory offsets are immediates; each loaded pixel feeds up to six outputs. e_row: address of
// the block's first input pixel in the row above the first output row; d_row: address of its first
// output pixel; ncol <= 7 columns and nrows <= 2 rows are stored (the loads of a ragged block run
// past the valid pixels, inside shared memory; those results are dropped).
constexpr int kSegCols = 7;
__device__ __forceinline__ void depthwise_block(uint32_t e_row, uint32_t d_row, uint32_t e_pitch, uint32_t d_pitch, int ncol,
                                                int nrows, const uint32_t (&w)[9], float2 bias) {
  const uint32_t e0 = e_row, e1 = e0 + e_pitch, e2 = e1 + e_pitch, e3 = e2 + e_pitch;
  const uint32_t d0 = d_row, d1 = d_row + d_pitch;
  uint32_t c0[4], c1[4], c2[4];
  c0[0] = lds32<0>(e0); c0[1] = lds32<0>(e1); c0[2] = lds32<0>(e2); c0[3] = lds32<0>(e3);
  c1[0] = lds32<16>(e0); c1[1] = lds32<16>(e1); c1[2] = lds32<16>(e2); c1[3] = lds32<16>(e3);
#define AGO_DW_STEP(J, A, B, C)                                                                       \
  {                                                                                                   \
    C[0] = lds32<(J + 2) * 16>(e0); C[1] = lds32<(J + 2) * 16>(e1);                                   \
    C[2] = lds32<(J + 2) * 16>(e2); C[3] = lds32<(J + 2) * 16>(e3);                                   \
    float2 acc0 = bias, acc1 = bias;                                                                  \
    fma_pair(acc0, A[0], w[0]); fma_pair(acc0, B[0], w[1]); fma_pair(acc0, C[0], w[2]);               \
    fma_pair(acc0, A[1], w[3]); fma_pair(acc0, B[1], w[4]); fma_pair(acc0, C[1], w[5]);               \
    fma_pair(acc1, A[1], w[0]); fma_pair(acc1, B[1], w[1]); fma_pair(acc1, C[1], w[2]);               \
    fma_pair(acc0, A[2], w[6]); fma_pair(acc0, B[2], w[7]); fma_pair(acc0, C[2], w[8]);               \
    fma_pair(acc1, A[2], w[3]); fma_pair(acc1, B[2], w[4]); fma_pair(acc1, C[2], w[5]);               \
    fma_pair(acc1, A[3], w[6]); fma_pair(acc1, B[3], w[7]); fma_pair(acc1, C[3], w[8]);               \
    if (FULL || J < ncol) {                                                                           \
      sts32<J * 16>(d0, relu6_pack(acc0.x, acc0.y));                                                  \
      if (FULL || nrows > 1) sts32<J * 16>(d1, relu6_pack(acc1.x, acc1.y));                           \
    }                                                                                                 \
  }
  if (ncol == kSegCols && nrows == 2) {
    constexpr bool FULL = true;
    AGO_DW_STEP(0, c0, c1, c2) AGO_DW_STEP(1, c1, c2, c0) AGO_DW_STEP(2, c2, c0, c1) AGO_DW_STEP(3, c0, c1, c2)
    AGO_DW_STEP(4, c1, c2, c0) AGO_DW_STEP(5, c2, c0, c1) AGO_DW_STEP(6, c0, c1, c2)
  } else {
    constexpr bool FULL = false;
    AGO_DW_STEP(0, c0, c1, c2) AGO_DW_STEP(1, c1, c2, c0) AGO_DW_STEP(2, c2, c0, c1) AGO_DW_STEP(3, c0, c1, c2)
    AGO_DW_STEP(4, c1, c2, c0) AGO_DW_STEP(5, c2, c0, c1) AGO_DW_STEP(6, c0, c1, c2)
  }
#undef AGO_DW_STEP
}

}  // namespace dw
}  // namespace ago
