/*
 * CPU oracle for the fused-subgraph executor. TEST INFRASTRUCTURE ONLY.
 *
 * Every operator of a subgraph is written out as the plain loop nest that
 * defines it and applied to a fully materialised tensor, one operator after
 * the other, exactly as the paper's "loop nest of a mini-subgraph without
 * fusion" does (Section III-A, Fig. "Loop nest of a mini-subgraph without
 * fusion"). All arithmetic is fp64. Nothing here is tiled, fused, blocked or
 * reordered; OpenMP is applied to the outermost independent loop only.
 *
 * This file shares no code with the CUDA path. Only tests, the smoke check
 * and the benchmark's cpu_baseline / reference arm may call it.
 *
 * Layouts (0-based, row-major, innermost last):
 *   activations  NHWC            in[n][h][w][c]
 *   conv weight  OHWI            w[o][r][s][i]
 *   depthwise    [R][S][C]       w[r][s][c]
 *   gemm weight  [K][N]          w[k][n]
 *   attention    Q,K,V,O         [B][S][H*D], head h at columns h*D..h*D+D-1
 *   scores / P   [B][H][S][S]
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int ago_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Output extent of a strided, zero-padded sliding window. For stride 1 and no
 * padding this is H - R + 1, i.e. H1 = H2 + (R2 - 1) of Section III-B. */
int64_t ago_oracle_out_extent(int64_t H, int64_t R, int64_t stride, int64_t pad) {
  int64_t span = H + 2 * pad - R;
  if (span < 0) return 0;
  return span / stride + 1;
}

/* 2-d convolution (cross-correlation, no kernel flip): the loop nest of
 * Section III-A, Fig. "Loop nest of a mini-subgraph without fusion", restated
 * for NHWC / OHWI with explicit stride and zero padding of this operator's
 * own input:
 *   out[n,ho,wo,o] = sum_{r,s,i} in[n, ho*st + r - p, wo*st + s - p, i] * w[o,r,s,i]
 * Positions outside the input contribute 0. */
void ago_oracle_conv2d(const double* in, int64_t N, int64_t H, int64_t W, int64_t I,
                       const double* w, int64_t O, int64_t R, int64_t S,
                       int64_t stride, int64_t pad, double* out) {
  const int64_t Ho = ago_oracle_out_extent(H, R, stride, pad);
  const int64_t Wo = ago_oracle_out_extent(W, S, stride, pad);
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t n = 0; n < N; ++n) {
    for (int64_t ho = 0; ho < Ho; ++ho) {
      for (int64_t wo = 0; wo < Wo; ++wo) {
        for (int64_t o = 0; o < O; ++o) {
          double acc = 0.0;
          for (int64_t r = 0; r < R; ++r) {
            const int64_t h = ho * stride + r - pad;
            if (h < 0 || h >= H) continue;
            for (int64_t s = 0; s < S; ++s) {
              const int64_t x = wo * stride + s - pad;
              if (x < 0 || x >= W) continue;
              const double* ip = in + ((n * H + h) * W + x) * I;
              const double* wp = w + ((o * R + r) * S + s) * I;
              for (int64_t i = 0; i < I; ++i) acc += ip[i] * wp[i];
            }
          }
          out[((n * Ho + ho) * Wo + wo) * O + o] = acc;
        }
      }
    }
  }
}

/* Depthwise convolution: no reduction over the input-channel dimension
 * (Section III-B, "Removing the Re-computation"); channel multiplier 1:
 *   out[n,ho,wo,c] = sum_{r,s} in[n, ho*st + r - p, wo*st + s - p, c] * w[r,s,c] */
void ago_oracle_depthwise(const double* in, int64_t N, int64_t H, int64_t W, int64_t C,
                          const double* w, int64_t R, int64_t S,
                          int64_t stride, int64_t pad, double* out) {
  const int64_t Ho = ago_oracle_out_extent(H, R, stride, pad);
  const int64_t Wo = ago_oracle_out_extent(W, S, stride, pad);
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t n = 0; n < N; ++n) {
    for (int64_t ho = 0; ho < Ho; ++ho) {
      for (int64_t wo = 0; wo < Wo; ++wo) {
        for (int64_t c = 0; c < C; ++c) {
          double acc = 0.0;
          for (int64_t r = 0; r < R; ++r) {
            const int64_t h = ho * stride + r - pad;
            if (h < 0 || h >= H) continue;
            for (int64_t s = 0; s < S; ++s) {
              const int64_t x = wo * stride + s - pad;
              if (x < 0 || x >= W) continue;
              acc += in[((n * H + h) * W + x) * C + c] * w[(r * S + s) * C + c];
            }
          }
          out[((n * Ho + ho) * Wo + wo) * C + c] = acc;
        }
      }
    }
  }
}

/* Matrix multiplication out[m,n] = sum_k a[m,k] * w[k,n]; mathematically a
 * pointwise convolution on the [N*H*W, I] view (Section III-B, last
 * paragraph). */
void ago_oracle_gemm(const double* a, int64_t M, int64_t K,
                     const double* w, int64_t Nn, double* out) {
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m) {
    for (int64_t n = 0; n < Nn; ++n) {
      double acc = 0.0;
      for (int64_t k = 0; k < K; ++k) acc += a[m * K + k] * w[k * Nn + n];
      out[m * Nn + n] = acc;
    }
  }
}

/* Bias addition broadcast over all but the last dimension:
 * Sum[...] = Conv[...] + Bias[o] (Section III-A, second loop of the figure). */
void ago_oracle_bias_add(const double* x, int64_t rows, int64_t C,
                         const double* b, double* out) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t c = 0; c < C; ++c) out[r * C + c] = x[r * C + c] + b[c];
}

/* ReLU[...] = max(Sum[...], 0) (Section III-A, third loop of the figure). */
void ago_oracle_relu(const double* x, int64_t n, double* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) out[i] = x[i] > 0.0 ? x[i] : 0.0;
}

/* ReLU6: min(max(x,0),6) -- the MobileNetV2 activation (textbook definition;
 * the paper names ReLU only). */
void ago_oracle_relu6(const double* x, int64_t n, double* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    double v = x[i] > 0.0 ? x[i] : 0.0;
    out[i] = v < 6.0 ? v : 6.0;
  }
}

/* GELU, tanh form: 0.5 x (1 + tanh( sqrt(2/pi) (x + 0.044715 x^3) )). */
void ago_oracle_gelu_tanh(const double* x, int64_t n, double* out) {
  const double c = 0.79788456080286535587989211986876; /* sqrt(2/pi) */
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    const double v = x[i];
    out[i] = 0.5 * v * (1.0 + tanh(c * (v + 0.044715 * v * v * v)));
  }
}

void ago_oracle_scale(const double* x, int64_t n, double f, double* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) out[i] = x[i] * f;
}

/* Element-wise addition of two tensors of the same shape (residual "add",
 * one of the simple operators of Section I). */
void ago_oracle_add(const double* x, const double* y, int64_t n, double* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) out[i] = x[i] + y[i];
}

/* Row softmax over the last dimension:
 * p_j = exp(s_j - m) / sum_j exp(s_j - m), m = max_j s_j. */
void ago_oracle_softmax_rows(const double* x, int64_t rows, int64_t cols, double* out) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    const double* xr = x + r * cols;
    double* orow = out + r * cols;
    double m = xr[0];
    for (int64_t j = 1; j < cols; ++j) if (xr[j] > m) m = xr[j];
    double sum = 0.0;
    for (int64_t j = 0; j < cols; ++j) { orow[j] = exp(xr[j] - m); sum += orow[j]; }
    for (int64_t j = 0; j < cols; ++j) orow[j] /= sum;
  }
}

/* Per (b,h): scores[b,h,i,j] = sum_d q[b,i,h*D+d] * k[b,j,h*D+d]. */
void ago_oracle_batched_qkt(const double* q, const double* k, int64_t B, int64_t S,
                            int64_t Hh, int64_t D, double* out) {
  const int64_t E = Hh * D;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t b = 0; b < B; ++b) {
    for (int64_t h = 0; h < Hh; ++h) {
      for (int64_t i = 0; i < S; ++i) {
        for (int64_t j = 0; j < S; ++j) {
          double acc = 0.0;
          for (int64_t d = 0; d < D; ++d)
            acc += q[(b * S + i) * E + h * D + d] * k[(b * S + j) * E + h * D + d];
          out[((b * Hh + h) * S + i) * S + j] = acc;
        }
      }
    }
  }
}

/* Per (b,h): o[b,i,h*D+d] = sum_j p[b,h,i,j] * v[b,j,h*D+d]. */
void ago_oracle_batched_pv(const double* p, const double* v, int64_t B, int64_t S,
                           int64_t Hh, int64_t D, double* out) {
  const int64_t E = Hh * D;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t b = 0; b < B; ++b) {
    for (int64_t h = 0; h < Hh; ++h) {
      for (int64_t i = 0; i < S; ++i) {
        for (int64_t d = 0; d < D; ++d) {
          double acc = 0.0;
          for (int64_t j = 0; j < S; ++j)
            acc += p[((b * Hh + h) * S + i) * S + j] * v[(b * S + j) * E + h * D + d];
          out[(b * S + i) * E + h * D + d] = acc;
        }
      }
    }
  }
}
