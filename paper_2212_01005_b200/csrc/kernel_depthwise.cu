// Depthwise-only mini-subgraph as one kernel: depthwise convolution (no
// reduction over channels, Section III-B) with its simple operators applied
// per element right after the window sum (conventional fusion, Section III-A).
// HBM-bound: every thread owns one 16-byte channel vector, so all loads and the
// store are 128-bit and coalesced along NHWC's channel dimension. 3x3 windows
// with pad 1 (every depthwise stage of the benchmark chains) slide down a block
// of output rows: the window's three input rows stay in registers, packed as
// they were loaded, so an output costs three new loads instead of nine (with one
// pixel per thread the halo was re-read through L2 3.4 times); the other window
// shapes take one output pixel per thread and leave the overlap to L1 / L2.
#include <cuda_bf16.h>

#include "kernels.h"

namespace ago {

namespace {

template <typename T> struct Vec;
template <> struct Vec<float> {
  static constexpr int N = 4;
  __device__ static void load(const void* p, int64_t i, float* v) {
    const float4 t = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p) + i));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
  __device__ static void store(void* p, int64_t i, const float* v) {
    *reinterpret_cast<float4*>(reinterpret_cast<float*>(p) + i) = make_float4(v[0], v[1], v[2], v[3]);
  }
};
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void load(const void* p, int64_t i, float* v) {
    const uint4 t = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p) + i));
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      v[2 * k] = __uint_as_float(w[k] << 16);
      v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
  }
  __device__ static void store(void* p, int64_t i, const float* v) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
      w[k] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p) + i) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};

__device__ __forceinline__ float gelu_tanh_f(float v) {
  const float c = 0.7978845608028654f;
  return 0.5f * v * (1.0f + tanhf(c * (v + 0.044715f * v * v * v)));
}

template <typename T>
__global__ void __launch_bounds__(256) depthwise_vec_kernel(const DepthwiseArgs a, int64_t total_vec) {
  constexpr int V = Vec<T>::N;
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= total_vec) return;
  const int cv = a.C / V;
  const int c0 = (int)(gid % cv) * V;
  int64_t t = gid / cv;
  const int wo = (int)(t % a.Wo); t /= a.Wo;
  const int ho = (int)(t % a.Ho);
  const int64_t n = t / a.Ho;
  float acc[V];
#pragma unroll
  for (int k = 0; k < V; ++k) acc[k] = 0.0f;
  for (int r = 0; r < a.R; ++r) {
    const int h = ho * a.stride + r - a.pad;
    if (h < 0 || h >= a.H) continue;
    for (int s = 0; s < a.S; ++s) {
      const int w = wo * a.stride + s - a.pad;
      if (w < 0 || w >= a.W) continue;
      float x[V], f[V];
      Vec<T>::load(a.in, ((n * a.H + h) * a.W + w) * a.C + c0, x);
      Vec<T>::load(a.w, (int64_t)(r * a.S + s) * a.C + c0, f);
#pragma unroll
      for (int k = 0; k < V; ++k) acc[k] = fmaf(x[k], f[k], acc[k]);
    }
  }
  const int64_t o = gid * V;
  for (int i = 0; i < a.epi.n; ++i) {
    switch (a.epi.code[i]) {
      case EPI_BIAS: {
        const float* b = reinterpret_cast<const float*>(a.epi.ptr[i]) + c0;
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] += __ldg(b + k);
        break;
      }
      case EPI_RELU:
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] = fmaxf(acc[k], 0.0f);
        break;
      case EPI_RELU6:
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] = fminf(fmaxf(acc[k], 0.0f), 6.0f);
        break;
      case EPI_GELU:
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] = gelu_tanh_f(acc[k]);
        break;
      case EPI_SCALE:
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] *= a.epi.f[i];
        break;
      case EPI_ADD: {
        float y[V];
        Vec<T>::load(a.epi.ptr[i], o, y);
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] += y[k];
        break;
      }
    }
  }
  Vec<T>::store(a.out, o, acc);
}

// The epilogue program on one channel vector (fp32), `o` = element offset of the vector in the output.
template <typename T>
__device__ __forceinline__ void apply_epilogue(const DepthwiseArgs& a, float* acc, int c0, int64_t o) {
  constexpr int V = Vec<T>::N;
  for (int i = 0; i < a.epi.n; ++i) {
    switch (a.epi.code[i]) {
      case EPI_BIAS: {
        const float* b = reinterpret_cast<const float*>(a.epi.ptr[i]) + c0;
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] += __ldg(b + k);
        break;
      }
      case EPI_RELU:
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] = fmaxf(acc[k], 0.0f);
        break;
      case EPI_RELU6:
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] = fminf(fmaxf(acc[k], 0.0f), 6.0f);
        break;
      case EPI_GELU:
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] = gelu_tanh_f(acc[k]);
        break;
      case EPI_SCALE:
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] *= a.epi.f[i];
        break;
      case EPI_ADD: {
        float y[V];
        Vec<T>::load(a.epi.ptr[i], o, y);
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] += y[k];
        break;
      }
    }
  }
}

// 16 bytes of one pixel as loaded (8 bf16 or 4 fp32), zero outside the image.
template <typename T>
__device__ __forceinline__ uint4 load_raw(const void* p, int64_t elem, bool inside) {
  if (!inside) return make_uint4(0, 0, 0, 0);
  return __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(p) + elem));
}
// acc += x * w over the channels of one 16-byte vector
__device__ __forceinline__ void fma_vec(float* acc, const uint4& x, const uint4& w, float) {
  const float* xf = reinterpret_cast<const float*>(&x);
  const float* wf = reinterpret_cast<const float*>(&w);
#pragma unroll
  for (int k = 0; k < 4; ++k) acc[k] = fmaf(xf[k], wf[k], acc[k]);
}
__device__ __forceinline__ void fma_vec(float* acc, const uint4& x, const uint4& w, __nv_bfloat16) {
  // mixed-precision FMAs: the bf16 operands as stored, exact product, fp32 accumulate
  const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int k = 0; k < 4; ++k)
    asm("{\n\t.reg .b16 xl, xh, wl, wh;\n\t"
        "mov.b32 {xl, xh}, %2;\n\tmov.b32 {wl, wh}, %3;\n\t"
        "fma.rn.f32.bf16 %0, xl, wl, %0;\n\tfma.rn.f32.bf16 %1, xh, wh, %1;\n\t}"
        : "+f"(acc[2 * k]), "+f"(acc[2 * k + 1]) : "r"(xs[k]), "r"(ws[k]));
}

constexpr int kRowBlock = 8;   // output rows per thread of the sliding-window kernel

// 3x3 window, pad 1, stride STRIDE: thread = (image, block of kRowBlock output rows, output column, channel vector).
template <typename T, int STRIDE>
__global__ void __launch_bounds__(256, 3) depthwise3x3_rows_kernel(const DepthwiseArgs a, int64_t total_items) {
  constexpr int V = Vec<T>::N;
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= total_items) return;
  const int cv = a.C / V;
  const int c0 = (int)(gid % cv) * V;
  int64_t t = gid / cv;
  const int wo = (int)(t % a.Wo); t /= a.Wo;
  const int hblocks = (a.Ho + kRowBlock - 1) / kRowBlock;
  const int ho0 = (int)(t % hblocks) * kRowBlock;
  const int64_t n = t / hblocks;
  const int rows = min(kRowBlock, a.Ho - ho0);
  // the nine weight vectors are fetched where they are used (they hit in L1): holding them would cost 36 registers,
  // and this kernel lives on the number of threads, i.e. of loads in flight, per SM
  const T* wp = reinterpret_cast<const T*>(a.w) + c0;
  auto wv = [&](int k) { return __ldg(reinterpret_cast<const uint4*>(wp + (int64_t)k * a.C)); };
  const int wi0 = wo * STRIDE - 1;
  const bool in0 = wi0 >= 0, in2 = wi0 + 2 < a.W;        // the middle column is always inside
  const T* img = reinterpret_cast<const T*>(a.in) + n * (int64_t)a.H * a.W * a.C + c0;
  auto load_row = [&](int h, uint4* r) {
    const bool hin = h >= 0 && h < a.H;
    const int64_t base = ((int64_t)h * a.W + wi0) * a.C;
    r[0] = load_raw<T>(img, base, hin && in0);
    r[1] = load_raw<T>(img, base + a.C, hin);
    r[2] = load_raw<T>(img, base + 2 * a.C, hin && in2);
  };
  uint4 r0[3], r1[3], r2[3];
  int h = ho0 * STRIDE - 1;
  load_row(h, r0);
  load_row(h + 1, r1);
#pragma unroll
  for (int j = 0; j < kRowBlock; ++j) {
    if (j < rows) {
      load_row(h + 2, r2);
      float acc[V];
#pragma unroll
      for (int k = 0; k < V; ++k) acc[k] = 0.0f;
#pragma unroll
      for (int s = 0; s < 3; ++s) {
        fma_vec(acc, r0[s], wv(s), T());
        fma_vec(acc, r1[s], wv(3 + s), T());
        fma_vec(acc, r2[s], wv(6 + s), T());
      }
      const int64_t o = (((n * a.Ho + ho0 + j) * a.Wo + wo) * (int64_t)a.C) + c0;
      apply_epilogue<T>(a, acc, c0, o);
      Vec<T>::store(a.out, o, acc);
      if (STRIDE == 1) {
#pragma unroll
        for (int s = 0; s < 3; ++s) { r0[s] = r1[s]; r1[s] = r2[s]; }
        h += 1;
      } else {
#pragma unroll
        for (int s = 0; s < 3; ++s) r0[s] = r2[s];
        h += 2;
        if (j + 1 < rows) load_row(h + 1, r1);
      }
    }
  }
}

}  // namespace

cudaError_t launch_depthwise_fused(const DepthwiseArgs& a, cudaStream_t stream) {
  const int V = a.dtype == AGO_FP32 ? 4 : 8;
  if (a.R == 3 && a.S == 3 && a.pad == 1 && (a.stride == 1 || a.stride == 2) && a.W >= 2) {
    const int64_t items = (int64_t)a.N * ((a.Ho + kRowBlock - 1) / kRowBlock) * a.Wo * (a.C / V);
    // small tensors keep one output pixel per thread: row blocks would leave most of the device without threads
    if (items >= 100000) {
    const unsigned blocks = (unsigned)((items + 255) / 256);
    if (a.dtype == AGO_FP32) {
      if (a.stride == 1) depthwise3x3_rows_kernel<float, 1><<<blocks, 256, 0, stream>>>(a, items);
      else depthwise3x3_rows_kernel<float, 2><<<blocks, 256, 0, stream>>>(a, items);
    } else {
      if (a.stride == 1) depthwise3x3_rows_kernel<__nv_bfloat16, 1><<<blocks, 256, 0, stream>>>(a, items);
      else depthwise3x3_rows_kernel<__nv_bfloat16, 2><<<blocks, 256, 0, stream>>>(a, items);
    }
    return cudaGetLastError();
    }
  }
  const int64_t total = (int64_t)a.N * a.Ho * a.Wo * (a.C / V);
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (a.dtype == AGO_FP32)
    depthwise_vec_kernel<float><<<blocks, 256, 0, stream>>>(a, total);
  else
    depthwise_vec_kernel<__nv_bfloat16><<<blocks, 256, 0, stream>>>(a, total);
  return cudaGetLastError();
}

}  // namespace ago
