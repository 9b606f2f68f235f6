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

// Normalises the row held in x[V][8] (lane-strided vectors) and writes it.
template <int V>
__device__ __forceinline__ void normalise_store(float (&x)[V][8], const bf16* gamma, const bf16* beta, bf16* out,
                                                float* out32, int lane, float eps) {
  constexpr int H = V * 256;
  float s = 0.f;
#pragma unroll
  for (int v = 0; v < V; ++v)
#pragma unroll
    for (int i = 0; i < 8; ++i) s += x[v][i];
  const float mean = warp_sum(s) * (1.0f / H);
  float q = 0.f;
#pragma unroll
  for (int v = 0; v < V; ++v)
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float d = x[v][i] - mean;
      q += d * d;
    }
  const float rstd = rsqrtf(warp_sum(q) * (1.0f / H) + eps);
#pragma unroll
  for (int v = 0; v < V; ++v) {
    const int col = (v * 32 + lane) * 8;
    float g[8], b[8], y[8];
    unpack8(__ldg(reinterpret_cast<const uint4*>(gamma + col)), g);
    unpack8(__ldg(reinterpret_cast<const uint4*>(beta + col)), b);
#pragma unroll
    for (int i = 0; i < 8; ++i) y[i] = (x[v][i] - mean) * rstd * g[i] + b[i];
    *reinterpret_cast<uint4*>(out + col) = pack8(y);
    if (out32 != nullptr) {
      *reinterpret_cast<float4*>(out32 + col) = make_float4(y[0], y[1], y[2], y[3]);
      *reinterpret_cast<float4*>(out32 + col + 4) = make_float4(y[4], y[5], y[6], y[7]);
    }
  }
}

}  // namespace
}  // namespace mt
