// Launch functions of the device kernels. Every function enqueues on `stream`
// and returns the cudaError_t of the launch; none synchronises.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "plan.h"

namespace ago {

// ---- generic kernels of the unfused modes (CUDA cores) ----------------------

// C[m][n] = sum_k A(m,k) * B(n,k), fp32 accumulate, bf16 in/out, epilogue program.
struct GemmArgs {
  const void* A; const void* B; void* C;
  int M, N, K;
  // A: row-major [M][K] with leading dimension lda, or an implicit im2col view of an NHWC tensor
  int a_im2col; int64_t lda;
  int H, W, Cin, R, S, stride, pad, Ho, Wo;
  // B: K-major ([N][K], ldb) or N-major ([K][N], ldb)
  int b_kmajor; int64_t ldb;
  int64_t ldc;
  // batch = blockIdx.z = b * heads + h
  int batches, heads;
  int64_t a_sb, a_sh, b_sb, b_sh, c_sb, c_sh;
  int a_dtype, c_dtype;  // AGO_BF16 | AGO_FP32 storage of A and C (B and EPI_ADD operands are bf16)
  EpiProgram epi;
  unsigned int* status;  // device word that records a bounded wait that gave up (tensor-core kernel), or null
};
cudaError_t launch_gemm_generic(const GemmArgs& a, cudaStream_t stream);

// The same contraction on tcgen05 for the shapes it serves (bf16 A, plain [M][K] view, K, N, leading dimensions and
// batch / head strides multiples of 8); `add_dtype` is the storage type of EPI_ADD operands (the subgraph's I/O dtype).
bool gemm_tc_supported(const GemmArgs& a);
cudaError_t launch_gemm_tc(const GemmArgs& a, int add_dtype, cudaStream_t stream);
// Large unbatched products on paired CTAs (256 x 256 tiles, persistent; epilogues without a tensor operand).
bool gemm_pair_supported(const GemmArgs& a);
cudaError_t launch_gemm_pair(const GemmArgs& a, cudaStream_t stream);

struct DepthwiseArgs {
  const void* in; const void* w; void* out;
  int N, H, W, C, R, S, stride, pad, Ho, Wo;
  int dtype;      // AGO_BF16 | AGO_FP32: the subgraph's I/O dtype = dtype of weights and EPI_ADD operands
  int in_dtype;   // storage of `in`  (an fp32 intermediate in per-op mode, else == dtype)
  int out_dtype;  // storage of `out`
  EpiProgram epi;
};
cudaError_t launch_depthwise_generic(const DepthwiseArgs& a, cudaStream_t stream);

// y = program(x) element-wise over a [rows][C] view.
// `dtype` is the subgraph's I/O dtype (EPI_ADD operands); x and y may be fp32 intermediates.
cudaError_t launch_elementwise(const void* x, void* y, int64_t numel, int C, int dtype, int x_dtype, int y_dtype,
                               const EpiProgram& epi, cudaStream_t stream);
// Row softmax over the last dimension, fp32 math.
cudaError_t launch_softmax_rows(const void* x, void* y, int64_t rows, int cols, int x_dtype, int y_dtype,
                                cudaStream_t stream);

// y = x with axes a and b (both below the last axis) swapped; x has shape dims[rank], rank <= 4.
cudaError_t launch_transpose(const void* x, void* y, const int64_t* dims, int rank, int a, int b, int x_dtype, int y_dtype,
                             cudaStream_t stream);

// 3x3 stride-1 pad-1 convolution with equal channel counts (16, 32 or 64) on tensor cores: the fused pair's kernel
// restricted to one convolution. out = [relu](conv(x, w) + bias [+ res]); bf16 NHWC / OHWI, bias and res may be null.
bool conv3x3_tc_supported(int H, int W, int Cin, int Cout, int R, int S, int stride, int pad);
cudaError_t launch_conv3x3_tc(const void* x, const void* w, const float* bias, const void* res, void* out, int N, int H,
                              int W, int C, int relu, unsigned int* status, cudaStream_t stream);

// ---- fused kernels -------------------------------------------------------------

// Depthwise-only mini-subgraph tuned kernel (vectorised over channels).
cudaError_t launch_depthwise_fused(const DepthwiseArgs& a, cudaStream_t stream);

}  // namespace ago
