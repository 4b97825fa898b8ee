// Depthwise-only mini-subgraph as one kernel: depthwise convolution (no
// reduction over channels, Section III-B) with its simple operators applied
// per element right after the window sum (conventional fusion, Section III-A).
// HBM-bound: every thread owns one 16-byte channel vector of one output pixel,
// so all loads and the store are 128-bit and coalesced along NHWC's channel
// dimension; the 3x3 neighbourhood overlap is served by L1/L2.
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

}  // namespace

cudaError_t launch_depthwise_fused(const DepthwiseArgs& a, cudaStream_t stream) {
  const int V = a.dtype == AGO_FP32 ? 4 : 8;
  const int64_t total = (int64_t)a.N * a.Ho * a.Wo * (a.C / V);
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (a.dtype == AGO_FP32)
    depthwise_vec_kernel<float><<<blocks, 256, 0, stream>>>(a, total);
  else
    depthwise_vec_kernel<__nv_bfloat16><<<blocks, 256, 0, stream>>>(a, total);
  return cudaGetLastError();
}

}  // namespace ago
