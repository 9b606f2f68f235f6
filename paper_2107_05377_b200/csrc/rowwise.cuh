// Row helpers shared by the row-wise kernels and by the LayerNorm step inside the fused layer-tail
// kernel: one warp owns one row of H = V * 256 values held in registers (lane-strided groups of 8),
// statistics in fp32 with the mean subtracted before the variance.
#pragma once

#include "mt_kernels.h"

namespace mt {
namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ void unpack8(const uint4& u, float (&f)[8]) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 v = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    w[i] = *reinterpret_cast<uint32_t*>(&v);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// Row statistics are defined over segments of 64 consecutive columns, so that every kernel that
// normalises rows - these row-wise kernels, and the GEMM epilogue that only ever sees 64 columns of a
// row per thread - computes them with the same additions in the same order and gets the same bits:
//   segment:  eight sums of 8 consecutive values (left to right), combined as a balanced tree;
//             mean_s = sum / 64;  M2_s = the same scheme over (x - mean_s)^2
//   row:      mean = (mean_0 + mean_1 + ...) / S;  M2 = sum_s (M2_s + 64 (mean_s - mean)^2), s ascending;
//             rstd = rsqrt(M2 / H + eps);  y = fma((x - mean) * rstd, gamma, beta)
// (the exact pooled-variance identity for equal segment sizes).
__device__ __forceinline__ float sum8_in_order(const float (&x)[8]) {
  float s = x[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) s += x[i];
  return s;
}
__device__ __forceinline__ float sumsq8_in_order(const float (&x)[8], float mean) {
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float d = x[i] - mean;
    q = fmaf(d, d, q);
  }
  return q;
}
// Merges S segment statistics given in ascending order.
template <int S>
__device__ __forceinline__ void merge_segments(const float (&seg_mean)[S], const float (&seg_m2)[S], float inv_h, float eps,
                                               float* mean_out, float* rstd_out) {
  float mean = 0.f;
#pragma unroll
  for (int i = 0; i < S; ++i) mean += seg_mean[i];
  // (an intrinsic, so that the compiler cannot contract this product into the subtractions below in one
  // kernel and not in another: 1 / S is not a power of two for S = 12)
  mean = __fmul_rn(mean, 1.0f / static_cast<float>(S));
  float m2 = 0.f;
#pragma unroll
  for (int i = 0; i < S; ++i) {
    const float d = seg_mean[i] - mean;
    m2 += fmaf(64.0f * d, d, seg_m2[i]);
  }
  *mean_out = mean;
  *rstd_out = rsqrtf(fmaf(m2, inv_h, eps));
}

// Normalises the row held in x[V][8] (lane-strided vectors: lane l holds columns (v * 32 + l) * 8 .. + 7,
// so the eight lanes l / 8 == j of vector v hold segment v * 4 + j) and writes it.
template <int V>
__device__ __forceinline__ void normalise_store(float (&x)[V][8], const bf16* gamma, const bf16* beta, bf16* out,
                                                float* out32, int lane, float eps) {
  constexpr int H = V * 256;
  constexpr int S = V * 4;
  float seg_mean[S], seg_m2[S];
#pragma unroll
  for (int v = 0; v < V; ++v) {
    float s = sum8_in_order(x[v]);
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float mean_s = s * (1.0f / 64.0f);
    float q = sumsq8_in_order(x[v], mean_s);
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      seg_mean[v * 4 + j] = __shfl_sync(0xffffffffu, mean_s, j * 8);
      seg_m2[v * 4 + j] = __shfl_sync(0xffffffffu, q, j * 8);
    }
  }
  float mean, rstd;
  merge_segments<S>(seg_mean, seg_m2, 1.0f / H, eps, &mean, &rstd);
#pragma unroll
  for (int v = 0; v < V; ++v) {
    const int col = (v * 32 + lane) * 8;
    float g[8], b[8], y[8];
    unpack8(__ldg(reinterpret_cast<const uint4*>(gamma + col)), g);
    unpack8(__ldg(reinterpret_cast<const uint4*>(beta + col)), b);
#pragma unroll
    for (int i = 0; i < 8; ++i) y[i] = fmaf(__fmul_rn(x[v][i] - mean, rstd), g[i], b[i]);
    *reinterpret_cast<uint4*>(out + col) = pack8(y);
    if (out32 != nullptr) {
      *reinterpret_cast<float4*>(out32 + col) = make_float4(y[0], y[1], y[2], y[3]);
      *reinterpret_cast<float4*>(out32 + col + 4) = make_float4(y[4], y[5], y[6], y[7]);
    }
  }
}

}  // namespace
}  // namespace mt
