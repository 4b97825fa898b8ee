// Generic CUDA-core kernels of the unfused modes: one launch per operator
// (Section III-A, "Loop nest of a mini-subgraph without fusion") or per
// mini-subgraph with the simple operators applied in the epilogue (Section
// III-A, "Conventional fusion within a mini-subgraph"). They accept any valid
// shape; intermediates between launches live in device memory.
#include <cuda_bf16.h>

#include "kernels.h"

namespace ago {

namespace {

__device__ __forceinline__ float gelu_tanh_f(float v) {
  const float c = 0.7978845608028654f;
  return 0.5f * v * (1.0f + tanhf(c * (v + 0.044715f * v * v * v)));
}

// Storage type is a run-time flag (AGO_BF16 | AGO_FP32), uniform over the grid.
__device__ __forceinline__ float ld(const void* p, int64_t i, int dtype) {
  return dtype == AGO_FP32 ? reinterpret_cast<const float*>(p)[i]
                           : __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[i]);
}
__device__ __forceinline__ void st(void* p, int64_t i, float v, int dtype) {
  if (dtype == AGO_FP32) reinterpret_cast<float*>(p)[i] = v;
  else reinterpret_cast<__nv_bfloat16*>(p)[i] = __float2bfloat16_rn(v);
}

// The simple operators, applied in program order to one element. `c` is the
// index along the last dimension, `idx` the element's linear index.
__device__ __forceinline__ float run_epilogue(const EpiProgram& e, float v, int c, int64_t idx, int add_dtype) {
  for (int i = 0; i < e.n; ++i) {
    switch (e.code[i]) {
      case EPI_BIAS: v += reinterpret_cast<const float*>(e.ptr[i])[c]; break;
      case EPI_RELU: v = fmaxf(v, 0.0f); break;
      case EPI_RELU6: v = fminf(fmaxf(v, 0.0f), 6.0f); break;
      case EPI_GELU: v = gelu_tanh_f(v); break;
      case EPI_SCALE: v *= e.f[i]; break;
      case EPI_ADD: v += ld(e.ptr[i], idx, add_dtype); break;
    }
  }
  return v;
}

constexpr int TM = 64, TN = 64, TK = 16;

__global__ void __launch_bounds__(256) gemm_generic_kernel(const GemmArgs a) {
  __shared__ float As[TK][TM + 4];
  __shared__ float Bs[TK][TN + 4];
  const int batch = blockIdx.z;
  const int bb = batch / a.heads, hh = batch % a.heads;
  const int64_t a_off = bb * a.a_sb + hh * a.a_sh;
  const __nv_bfloat16* B = reinterpret_cast<const __nv_bfloat16*>(a.B) + bb * a.b_sb + hh * a.b_sh;
  const int64_t c_off = bb * a.c_sb + hh * a.c_sh;
  const int m0 = blockIdx.x * TM, n0 = blockIdx.y * TN;
  const int tid = threadIdx.x;
  const int tx = tid % 16, ty = tid / 16;
  float acc[4][4] = {};

  for (int k0 = 0; k0 < a.K; k0 += TK) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int idx = tid + e * 256;
      const int row = idx / TK, kk = idx % TK;
      const int m = m0 + row, k = k0 + kk;
      float v = 0.0f;
      if (m < a.M && k < a.K) {
        if (!a.a_im2col) {
          v = ld(a.A, a_off + (int64_t)m * a.lda + k, a.a_dtype);
        } else {
          const int ci = k % a.Cin;
          const int rs = k / a.Cin;
          const int s = rs % a.S, r = rs / a.S;
          const int wo = m % a.Wo;
          const int t = m / a.Wo;
          const int ho = t % a.Ho, img = t / a.Ho;
          const int h = ho * a.stride + r - a.pad, w = wo * a.stride + s - a.pad;
          if (h >= 0 && h < a.H && w >= 0 && w < a.W)
            v = ld(a.A, a_off + (((int64_t)img * a.H + h) * a.W + w) * a.Cin + ci, a.a_dtype);
        }
      }
      // operands of a contraction are bf16 values: an fp32 intermediate is rounded as it is loaded
      if (a.a_dtype == AGO_FP32) v = __bfloat162float(__float2bfloat16_rn(v));
      As[kk][row] = v;
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int idx = tid + e * 256;
      int nn, kk;
      if (a.b_kmajor) { nn = idx / TK; kk = idx % TK; } else { kk = idx / TN; nn = idx % TN; }
      const int n = n0 + nn, k = k0 + kk;
      float v = 0.0f;
      if (n < a.N && k < a.K)
        v = __bfloat162float(a.b_kmajor ? B[(int64_t)n * a.ldb + k] : B[(int64_t)k * a.ldb + n]);
      Bs[kk][nn] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= a.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= a.N) continue;
      const int64_t idx = c_off + (int64_t)m * a.ldc + n;
      st(a.C, idx, run_epilogue(a.epi, acc[i][j], n, idx, AGO_BF16), a.c_dtype);
    }
  }
}

__global__ void __launch_bounds__(256) depthwise_generic_kernel(const DepthwiseArgs a, int64_t total) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int c = (int)(idx % a.C);
  int64_t t = idx / a.C;
  const int wo = (int)(t % a.Wo); t /= a.Wo;
  const int ho = (int)(t % a.Ho);
  const int64_t n = t / a.Ho;
  float acc = 0.0f;
  for (int r = 0; r < a.R; ++r) {
    const int h = ho * a.stride + r - a.pad;
    if (h < 0 || h >= a.H) continue;
    for (int s = 0; s < a.S; ++s) {
      const int w = wo * a.stride + s - a.pad;
      if (w < 0 || w >= a.W) continue;
      {
        float x = ld(a.in, ((n * a.H + h) * a.W + w) * a.C + c, a.in_dtype);
        if (a.in_dtype != a.dtype) x = __bfloat162float(__float2bfloat16_rn(x));
        acc = fmaf(x, ld(a.w, (r * a.S + s) * a.C + c, a.dtype), acc);
      }
    }
  }
  st(a.out, idx, run_epilogue(a.epi, acc, c, idx, a.dtype), a.out_dtype);
}

__global__ void __launch_bounds__(256) elementwise_kernel(const void* x, void* y, int64_t numel, int C, int dtype,
                                                          int x_dtype, int y_dtype, const EpiProgram epi) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= numel) return;
  st(y, idx, run_epilogue(epi, ld(x, idx, x_dtype), (int)(idx % C), idx, dtype), y_dtype);
}

// One warp per row: p_j = exp(s_j - max) / sum.
__global__ void __launch_bounds__(256) softmax_rows_kernel(const void* x, void* y, int64_t rows, int cols,
                                                           int x_dtype, int y_dtype) {
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
  if (row >= rows) return;
  const int lane = threadIdx.x % 32;
  const int64_t base = row * cols;
  float m = -INFINITY;
  for (int j = lane; j < cols; j += 32) m = fmaxf(m, ld(x, base + j, x_dtype));
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  float sum = 0.0f;
  for (int j = lane; j < cols; j += 32) sum += expf(ld(x, base + j, x_dtype) - m);
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const float inv = 1.0f / sum;
  for (int j = lane; j < cols; j += 32) st(y, base + j, expf(ld(x, base + j, x_dtype) - m) * inv, y_dtype);
}

// Swap of two leading axes: the last axis moves as whole rows. One thread per VEC elements of an output row
// (VEC = 16 bytes when both tensors share a storage type and the row length allows it, else 1).
struct TransposeArgs {
  int64_t od[4];   // output shape padded to rank 4 in front
  int64_t is[4];   // input stride (elements) of every OUTPUT axis
};
template <int VEC, typename T>
__global__ void __launch_bounds__(256) transpose_vec_kernel(const T* x, T* y, const TransposeArgs a, int64_t total_vec) {
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= total_vec) return;
  const int64_t cv = a.od[3] / VEC;
  const int64_t c = (gid % cv) * VEC;
  int64_t t = gid / cv;
  const int64_t i2 = t % a.od[2]; t /= a.od[2];
  const int64_t i1 = t % a.od[1];
  const int64_t i0 = t / a.od[1];
  const int64_t src = i0 * a.is[0] + i1 * a.is[1] + i2 * a.is[2] + c;
  if (VEC * sizeof(T) == 16) {
    *reinterpret_cast<uint4*>(y + gid * VEC) = __ldg(reinterpret_cast<const uint4*>(x + src));
  } else {
    y[gid] = x[src];
  }
}
__global__ void __launch_bounds__(256) transpose_any_kernel(const void* x, void* y, const TransposeArgs a, int64_t total,
                                                            int x_dtype, int y_dtype) {
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= total) return;
  const int64_t c = gid % a.od[3];
  int64_t t = gid / a.od[3];
  const int64_t i2 = t % a.od[2]; t /= a.od[2];
  const int64_t i1 = t % a.od[1];
  const int64_t i0 = t / a.od[1];
  st(y, gid, ld(x, i0 * a.is[0] + i1 * a.is[1] + i2 * a.is[2] + c, x_dtype), y_dtype);
}

}  // namespace

cudaError_t launch_transpose(const void* x, void* y, const int64_t* dims, int rank, int a, int b, int x_dtype, int y_dtype,
                             cudaStream_t stream) {
  if (rank < 3 || rank > 4 || a == b || a < 0 || b < 0 || a >= rank - 1 || b >= rank - 1) return cudaErrorInvalidValue;
  int64_t id[4] = {1, 1, 1, 1}, istr[4];
  const int pad = 4 - rank;
  for (int k = 0; k < rank; ++k) id[pad + k] = dims[k];
  istr[3] = 1;
  for (int k = 2; k >= 0; --k) istr[k] = istr[k + 1] * id[k + 1];
  int perm[4] = {0, 1, 2, 3};
  perm[pad + a] = pad + b; perm[pad + b] = pad + a;
  TransposeArgs t;
  for (int k = 0; k < 4; ++k) { t.od[k] = id[perm[k]]; t.is[k] = istr[perm[k]]; }
  const int64_t total = id[0] * id[1] * id[2] * id[3];
  const int esz = x_dtype == AGO_FP32 ? 4 : 2;
  const int vec = 16 / esz;
  if (x_dtype == y_dtype && id[3] % vec == 0) {
    const int64_t tv = total / vec;
    const unsigned blocks = (unsigned)((tv + 255) / 256);
    if (esz == 4)
      transpose_vec_kernel<4, float><<<blocks, 256, 0, stream>>>(static_cast<const float*>(x), static_cast<float*>(y), t, tv);
    else
      transpose_vec_kernel<8, __nv_bfloat16><<<blocks, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(x), static_cast<__nv_bfloat16*>(y), t, tv);
  } else {
    const unsigned blocks = (unsigned)((total + 255) / 256);
    transpose_any_kernel<<<blocks, 256, 0, stream>>>(x, y, t, total, x_dtype, y_dtype);
  }
  return cudaGetLastError();
}

cudaError_t launch_gemm_generic(const GemmArgs& a, cudaStream_t stream) {
  dim3 grid((a.M + TM - 1) / TM, (a.N + TN - 1) / TN, a.batches);
  gemm_generic_kernel<<<grid, 256, 0, stream>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_depthwise_generic(const DepthwiseArgs& a, cudaStream_t stream) {
  const int64_t total = (int64_t)a.N * a.Ho * a.Wo * a.C;
  const unsigned blocks = (unsigned)((total + 255) / 256);
  depthwise_generic_kernel<<<blocks, 256, 0, stream>>>(a, total);
  return cudaGetLastError();
}

cudaError_t launch_elementwise(const void* x, void* y, int64_t numel, int C, int dtype, int x_dtype, int y_dtype,
                               const EpiProgram& epi, cudaStream_t stream) {
  const unsigned blocks = (unsigned)((numel + 255) / 256);
  elementwise_kernel<<<blocks, 256, 0, stream>>>(x, y, numel, C, dtype, x_dtype, y_dtype, epi);
  return cudaGetLastError();
}

cudaError_t launch_softmax_rows(const void* x, void* y, int64_t rows, int cols, int x_dtype, int y_dtype,
                                cudaStream_t stream) {
  const unsigned blocks = (unsigned)((rows + 7) / 8);
  softmax_rows_kernel<<<blocks, 256, 0, stream>>>(x, y, rows, cols, x_dtype, y_dtype);
  return cudaGetLastError();
}

}  // namespace ago
