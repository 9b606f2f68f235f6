// The memory-bound steps of the path: embedding gather + LayerNorm, LayerNorm, pooler + head.
// One warp owns one row of H values, held entirely in registers (H/256 groups of 8 per lane,
// 16-byte accesses, fully coalesced), statistics in fp32 with the mean subtracted before the
// variance.  LayerNorm reads the fp32 pre-normalisation sum and writes the result twice: bf16 for
// the next GEMM's operand and fp32 for the next residual add.

#include "rowwise.cuh"

namespace mt {
namespace {

constexpr int kRowThreads = 256;  // 8 rows per CTA
constexpr int kMaxParts = 4;       // ranges of K a row can be put together from (LayerNormParams::n_parts)

// PARTS: the row is put together from the partial sums of a split projection (LayerNormParams::n_parts > 0); a
// separate instantiation, so that the plain kernel keeps its registers and occupancy.
template <int V, bool PARTS>
__global__ void __launch_bounds__(kRowThreads) layernorm_kernel(const LayerNormParams p) {
  constexpr int H = V * 256;
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (kRowThreads / 32) + (threadIdx.x >> 5);
  const int g = blockIdx.y;
  // (the count of rows in use was written by the forward's first kernel, never by the immediate predecessor: it
  // may be read before the dependency wait)
  const int rows_in_use = p.rows_valid != nullptr ? min(p.rows, *p.rows_valid) : p.rows;
  grid_dependency_wait();
  grid_launch_dependents();
  if (row >= rows_in_use) return;
  float x[V][8];
  if (PARTS) {
    // the row from the partial sums of a GEMM whose K was split: the ranges in order, then the bias, then
    // the residual - residual + ((part_0 + part_1 + ...) + bias)
    const float* part = p.part[g] + static_cast<size_t>(row) * H;
    const float* res = p.residual[g] + static_cast<size_t>(row) * H;
    const size_t pitch = static_cast<size_t>(p.part_pitch) * H;
    const int n_parts = p.n_parts;   // at most kMaxParts (checked by the launcher)
    // every load of the row is issued before the first addition: one round trip to L2, not one per range
    float4 pa[V][kMaxParts], pb[V][kMaxParts], ra[V], rb[V];
    uint4 bias8[V];
#pragma unroll
    for (int v = 0; v < V; ++v) {
      const int col = (v * 32 + lane) * 8;
#pragma unroll
      for (int s = 0; s < kMaxParts; ++s) {
        if (s < n_parts) {
          pa[v][s] = *reinterpret_cast<const float4*>(part + s * pitch + col);
          pb[v][s] = *reinterpret_cast<const float4*>(part + s * pitch + col + 4);
        }
      }
      ra[v] = *reinterpret_cast<const float4*>(res + col);
      rb[v] = *reinterpret_cast<const float4*>(res + col + 4);
      bias8[v] = __ldg(reinterpret_cast<const uint4*>(p.bias[g] + col));
    }
#pragma unroll
    for (int v = 0; v < V; ++v) {
      float acc[8] = {pa[v][0].x, pa[v][0].y, pa[v][0].z, pa[v][0].w, pb[v][0].x, pb[v][0].y, pb[v][0].z, pb[v][0].w};
#pragma unroll
      for (int s = 1; s < kMaxParts; ++s) {
        if (s < n_parts) {
          acc[0] += pa[v][s].x; acc[1] += pa[v][s].y; acc[2] += pa[v][s].z; acc[3] += pa[v][s].w;
          acc[4] += pb[v][s].x; acc[5] += pb[v][s].y; acc[6] += pb[v][s].z; acc[7] += pb[v][s].w;
        }
      }
      float bias[8];
      unpack8(bias8[v], bias);
      const float r[8] = {ra[v].x, ra[v].y, ra[v].z, ra[v].w, rb[v].x, rb[v].y, rb[v].z, rb[v].w};
#pragma unroll
      for (int i = 0; i < 8; ++i) x[v][i] = r[i] + (acc[i] + bias[i]);
    }
  } else {
    const float* xin = p.x[g] + static_cast<size_t>(row) * H;
#pragma unroll
    for (int v = 0; v < V; ++v) {
      const float4 a = *reinterpret_cast<const float4*>(xin + (v * 32 + lane) * 8);
      const float4 b = *reinterpret_cast<const float4*>(xin + (v * 32 + lane) * 8 + 4);
      x[v][0] = a.x; x[v][1] = a.y; x[v][2] = a.z; x[v][3] = a.w;
      x[v][4] = b.x; x[v][5] = b.y; x[v][6] = b.z; x[v][7] = b.w;
    }
  }
  float* y32 = p.y32[g] != nullptr ? p.y32[g] + static_cast<size_t>(row) * H : nullptr;
  normalise_store<V>(x, p.gamma[g], p.beta[g], p.y[g] + static_cast<size_t>(row) * H, y32, lane, p.eps);
}

template <int V>
__global__ void __launch_bounds__(kRowThreads) embed_kernel(const EmbedParams p) {
  constexpr int H = V * 256;
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (kRowThreads / 32) + (threadIdx.x >> 5);
  grid_dependency_wait();
  grid_launch_dependents();
  if (row >= p.batch * p.seq) return;
  const int b = row / p.seq;
  const int pos = row - b * p.seq;
  int tok = p.token_ids[row];
  int seg = p.segment_ids[row];
  uint32_t flags = 0;
  if (tok < 0 || tok >= p.vocab) { flags |= kFlagBadToken; tok = tok < 0 ? 0 : p.vocab - 1; }
  if (seg < 0 || seg >= p.type_vocab) { flags |= kFlagBadSegment; seg = seg < 0 ? 0 : p.type_vocab - 1; }
  if (pos == 0) {
    const int len = p.lengths[b];
    if (len < 1 || len > p.seq) flags |= kFlagBadLength;
  }
  if (flags != 0 && lane == 0 && p.status != nullptr) atomicOr(p.status, flags);
  int out_row = row;
  if (p.row_start != nullptr) {
    int len = p.lengths[b];
    len = len < 1 ? 1 : (len > p.seq ? p.seq : len);
    if (p.packed && pos >= len) return;  // packed layout: padded positions do not exist
    out_row = p.row_start[b] + pos;
  }
  const bf16* w = p.word + static_cast<size_t>(tok) * H;
  const bf16* q = p.pos + static_cast<size_t>(pos) * H;
  const bf16* t = p.type + static_cast<size_t>(seg) * H;
  float x[V][8];
#pragma unroll
  for (int v = 0; v < V; ++v) {
    const int col = (v * 32 + lane) * 8;
    float a[8], c[8], d[8];
    unpack8(__ldg(reinterpret_cast<const uint4*>(w + col)), a);
    unpack8(__ldg(reinterpret_cast<const uint4*>(q + col)), c);
    unpack8(__ldg(reinterpret_cast<const uint4*>(t + col)), d);
#pragma unroll
    for (int i = 0; i < 8; ++i) x[v][i] = a[i] + c[i] + d[i];
  }
  float* out32 = p.out32 != nullptr ? p.out32 + static_cast<size_t>(out_row) * H : nullptr;
  normalise_store<V>(x, p.gamma, p.beta, p.out + static_cast<size_t>(out_row) * H, out32, lane, p.eps);
}

// Pooler + head, two launches.
//   pooler_kernel: one CTA = (32 pooled features, task, chunk of kSeqPerCta sequences).  The
//     position-0 rows of the chunk are staged in shared memory as fp32; each warp produces 4 features
//     for all sequences of the chunk at once (every pooler-matrix row is read once per CTA, 16-byte
//     loads), applies tanh and writes fp32 pooled vectors to the scratch buffer [task][B][H].
//   head_kernel: one CTA = (task, chunk); the C_t x chunk logits are warp-level dot products.
constexpr int kSeqPerCta = 8;
constexpr int kHeadThreads = 256;
constexpr int kPoolFeaturesPerCta = 32;

__global__ void __launch_bounds__(kHeadThreads) pooler_kernel(const HeadParams p) {
  extern __shared__ float cls[];  // [kSeqPerCta][H]
  const int H = p.hidden;
  const HeadTask tk = p.task[blockIdx.y];
  const int b0 = blockIdx.z * kSeqPerCta;
  const int nb = min(kSeqPerCta, p.batch - b0);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  grid_dependency_wait();
  grid_launch_dependents();

  for (int idx = threadIdx.x; idx < kSeqPerCta * (H / 8); idx += kHeadThreads) {
    const int s = idx / (H / 8), c = idx - s * (H / 8);
    float f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (s < nb) {
      const size_t row = tk.compact ? static_cast<size_t>(b0 + s)
                         : p.row_start != nullptr ? static_cast<size_t>(p.row_start[b0 + s])
                                                  : static_cast<size_t>(b0 + s) * p.seq;
      unpack8(*reinterpret_cast<const uint4*>(tk.hidden + row * H + c * 8), f);
    }
    *reinterpret_cast<float4*>(cls + s * H + c * 8) = make_float4(f[0], f[1], f[2], f[3]);
    *reinterpret_cast<float4*>(cls + s * H + c * 8 + 4) = make_float4(f[4], f[5], f[6], f[7]);
  }
  __syncthreads();

  const int vecs = H / 256;  // 16-byte vectors per lane per row
  float* pooled = p.pooled + static_cast<size_t>(blockIdx.y) * p.batch * H;
  constexpr int kPerWarp = kPoolFeaturesPerCta / (kHeadThreads / 32);
  const int j0 = blockIdx.x * kPoolFeaturesPerCta + warp * kPerWarp;
  float acc[kPerWarp][kSeqPerCta];
#pragma unroll
  for (int i = 0; i < kPerWarp; ++i)
#pragma unroll
    for (int s = 0; s < kSeqPerCta; ++s) acc[i][s] = 0.f;
  for (int v = 0; v < vecs; ++v) {
    const int col = (v * 32 + lane) * 8;
    // this lane's 8 columns of every staged row, read once for all of the warp's features
    float c[kSeqPerCta][8];
#pragma unroll
    for (int s = 0; s < kSeqPerCta; ++s) {
      const float4 c0 = *reinterpret_cast<const float4*>(cls + s * H + col);
      const float4 c1 = *reinterpret_cast<const float4*>(cls + s * H + col + 4);
      c[s][0] = c0.x; c[s][1] = c0.y; c[s][2] = c0.z; c[s][3] = c0.w;
      c[s][4] = c1.x; c[s][5] = c1.y; c[s][6] = c1.z; c[s][7] = c1.w;
    }
#pragma unroll
    for (int i = 0; i < kPerWarp; ++i) {
      float w[8];
      unpack8(__ldg(reinterpret_cast<const uint4*>(tk.pool_w + static_cast<size_t>(j0 + i) * H + col)), w);
#pragma unroll
      for (int s = 0; s < kSeqPerCta; ++s)
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[i][s] = fmaf(w[k], c[s][k], acc[i][s]);
    }
  }
#pragma unroll
  for (int i = 0; i < kPerWarp; ++i) {
    const float bias = __bfloat162float(tk.pool_b[j0 + i]);
#pragma unroll
    for (int s = 0; s < kSeqPerCta; ++s) {
      const float t = warp_sum(acc[i][s]);
      if (lane == 0 && s < nb) pooled[static_cast<size_t>(b0 + s) * H + j0 + i] = tanhf(t + bias);
    }
  }
}

__global__ void __launch_bounds__(kHeadThreads) head_kernel(const HeadParams p) {
  const int H = p.hidden;
  const HeadTask tk = p.task[blockIdx.y];
  const int b0 = blockIdx.x * kSeqPerCta;
  const int nb = min(kSeqPerCta, p.batch - b0);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float* pooled = p.pooled + static_cast<size_t>(blockIdx.y) * p.batch * H;
  grid_dependency_wait();
  grid_launch_dependents();
  for (int o = warp; o < tk.num_classes * nb; o += kHeadThreads / 32) {
    const int c = o / nb, s = o - c * nb;
    // eight consecutive columns per lane and step (H is a multiple of 256): every load of the dot
    // product is independent of the others, so they are all in flight together
    const bf16* wrow = tk.cls_w + static_cast<size_t>(c) * H;
    const float* prow = pooled + static_cast<size_t>(b0 + s) * H;
    float acc = 0.f;
    for (int k = lane * 8; k < H; k += 256) {
      float w[8];
      unpack8(__ldg(reinterpret_cast<const uint4*>(wrow + k)), w);
      const float4 p0 = *reinterpret_cast<const float4*>(prow + k);
      const float4 p1 = *reinterpret_cast<const float4*>(prow + k + 4);
      acc = fmaf(w[0], p0.x, acc); acc = fmaf(w[1], p0.y, acc); acc = fmaf(w[2], p0.z, acc); acc = fmaf(w[3], p0.w, acc);
      acc = fmaf(w[4], p1.x, acc); acc = fmaf(w[5], p1.y, acc); acc = fmaf(w[6], p1.z, acc); acc = fmaf(w[7], p1.w, acc);
    }
    acc = warp_sum(acc);
    if (lane == 0)
      p.logits[static_cast<size_t>(b0 + s) * p.logits_stride + tk.col0 + c] = acc + __bfloat162float(tk.cls_b[c]);
  }
}

// Row-wise E4M3 quantisation (QuantParams): one warp per row; the row is read twice (bf16 from L2), first for
// its largest magnitude, then to scale and convert.  Every decision is taken in fp32 with IEEE operations
// that no compiler option can change: scale = amax * (1/448), y = x / scale, code = cvt.rn.satfinite.e4m3.
__device__ __forceinline__ uint32_t cvt_e4m3x2(float hi, float lo) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
__global__ void __launch_bounds__(kRowThreads) quantize_rows_kernel(const QuantParams p) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = blockIdx.y;
  int rows = p.rows;
  if (p.rows_valid != nullptr) rows = min(rows, *p.rows_valid);   // (readable before the wait, as in layernorm_kernel)
  grid_dependency_wait();
  grid_launch_dependents();
  const int row = blockIdx.x * (kRowThreads / 32) + warp;
  if (row >= rows) return;
  const bf16* x = p.x[g] + static_cast<size_t>(row) * p.cols;
  float amax = 0.f;
  for (int c = lane * 8; c < p.cols; c += 256) {
    float f[8];
    unpack8(__ldg(reinterpret_cast<const uint4*>(x + c)), f);
#pragma unroll
    for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(f[i]));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  const float scale = amax == 0.f ? 1.0f : __fmul_rn(amax, 1.0f / 448.0f);
  if (lane == 0) p.scale[g][row] = scale;
  uint8_t* q = p.q[g] + static_cast<size_t>(row) * p.cols;
  for (int c = lane * 8; c < p.cols; c += 256) {
    float f[8];
    unpack8(__ldg(reinterpret_cast<const uint4*>(x + c)), f);
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] = __fdiv_rn(f[i], scale);
    uint2 out;
    out.x = cvt_e4m3x2(f[1], f[0]) | (cvt_e4m3x2(f[3], f[2]) << 16);
    out.y = cvt_e4m3x2(f[5], f[4]) | (cvt_e4m3x2(f[7], f[6]) << 16);
    *reinterpret_cast<uint2*>(q + c) = out;
  }
}

// One warp: inclusive scan of the clamped lengths in chunks of 32.
__global__ void row_starts_kernel(const int32_t* lengths, int32_t batch, int32_t seq, int32_t packed,
                                  int32_t* row_start, int32_t* rows_valid) {
  const int lane = threadIdx.x;
  grid_dependency_wait();
  grid_launch_dependents();
  int carry = 0;
  for (int base = 0; base < batch; base += 32) {
    const int b = base + lane;
    int n = 0;
    if (b < batch) {
      n = seq;
      if (packed) {
        n = lengths[b];
        n = n < 1 ? 1 : (n > seq ? seq : n);
      }
    }
    int incl = n;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += up;
    }
    if (b < batch) row_start[b] = carry + incl - n;
    carry += __shfl_sync(0xffffffffu, incl, 31);
  }
  if (lane == 0) {
    row_start[batch] = carry;
    *rows_valid = carry;
  }
}

// One warp per padded row.
__global__ void __launch_bounds__(kRowThreads) unpack_rows_kernel(const bf16* packed, const int32_t* lengths,
                                                                   const int32_t* row_start, bf16* padded, int32_t batch,
                                                                   int32_t seq, int32_t hidden, int32_t compact) {
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (kRowThreads / 32) + (threadIdx.x >> 5);
  if (row >= batch * seq) return;
  const int b = row / seq, pos = row - b * seq;
  int len = lengths[b];
  len = len < 1 ? 1 : (len > seq ? seq : len);
  const size_t src_row = compact ? static_cast<size_t>(b) : static_cast<size_t>(row_start[b] + pos);
  const bool present = compact ? pos == 0 : pos < len;
  const uint4* src = reinterpret_cast<const uint4*>(packed + src_row * hidden);
  uint4* dst = reinterpret_cast<uint4*>(padded + static_cast<size_t>(row) * hidden);
  for (int c = lane; c < hidden / 8; c += 32) dst[c] = present ? src[c] : make_uint4(0, 0, 0, 0);
}

}  // namespace

cudaError_t launch_quantize_rows(const QuantParams& p, cudaStream_t stream) {
  if (p.n_groups < 1 || p.n_groups > kMaxGroups || p.rows < 1 || p.cols < 256 || p.cols % 256 != 0) return cudaErrorInvalidValue;
  const int rows_per_cta = kRowThreads / 32;
  dim3 grid((p.rows + rows_per_cta - 1) / rows_per_cta, p.n_groups);
  return launch_kernel(quantize_rows_kernel, grid, dim3(kRowThreads), 0, stream, p);
}

cudaError_t launch_row_starts(const int32_t* lengths, int32_t batch, int32_t seq, int32_t packed, int32_t* row_start,
                              int32_t* rows_valid, cudaStream_t stream) {
  if (batch < 1 || seq < 1) return cudaErrorInvalidValue;
  row_starts_kernel<<<1, 32, 0, stream>>>(lengths, batch, seq, packed, row_start, rows_valid);
  return cudaGetLastError();
}

cudaError_t launch_unpack_rows(const bf16* packed, const int32_t* lengths, const int32_t* row_start, bf16* padded,
                               int32_t batch, int32_t seq, int32_t hidden, int32_t compact, cudaStream_t stream) {
  const int rows = batch * seq;
  if (rows < 1 || hidden % 8 != 0) return cudaErrorInvalidValue;
  unpack_rows_kernel<<<(rows + kRowThreads / 32 - 1) / (kRowThreads / 32), kRowThreads, 0, stream>>>(
      packed, lengths, row_start, padded, batch, seq, hidden, compact);
  return cudaGetLastError();
}

// Token-level heads: one warp per (task, sequence, position); the token's state is read once (16-byte
// loads, held in registers as fp32) and dotted with every class row of the head matrix, which stays in
// L1/L2; fp32 throughout.  HBM-bound on the states: 2 H bytes per token and task.
template <int V>
__global__ void __launch_bounds__(kRowThreads) token_head_kernel(const TokenHeadParams p) {
  constexpr int H = V * 256;
  const int lane = threadIdx.x & 31;
  const int pos = blockIdx.x * (kRowThreads / 32) + (threadIdx.x >> 5);
  const int b = blockIdx.y, t = blockIdx.z;
  grid_dependency_wait();
  grid_launch_dependents();
  int len = p.lengths[b];
  len = len < 1 ? 1 : (len > p.seq ? p.seq : len);
  if (pos >= len) return;
  const size_t row = p.row_start != nullptr ? static_cast<size_t>(p.row_start[b]) + pos : static_cast<size_t>(b) * p.seq + pos;
  const bf16* h = p.hidden_state[t] + row * H;
  float x[V][8];
#pragma unroll
  for (int v = 0; v < V; ++v) unpack8(*reinterpret_cast<const uint4*>(h + (v * 32 + lane) * 8), x[v]);
  float* out = p.logits + (static_cast<size_t>(b) * p.seq + pos) * p.logits_stride + p.col0[t];
  for (int c = 0; c < p.num_classes[t]; ++c) {
    const bf16* wrow = p.cls_w[t] + static_cast<size_t>(c) * H;
    float acc = 0.f;
#pragma unroll
    for (int v = 0; v < V; ++v) {
      float w[8];
      unpack8(__ldg(reinterpret_cast<const uint4*>(wrow + (v * 32 + lane) * 8)), w);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc = fmaf(x[v][i], w[i], acc);
    }
    acc = warp_sum(acc);
    if (lane == 0) out[c] = acc + __bfloat162float(p.cls_b[t][c]);
  }
}

cudaError_t launch_token_heads(const TokenHeadParams& p, cudaStream_t stream) {
  if (p.n_tasks < 1 || p.n_tasks > kMaxGroups || p.batch < 1 || p.seq < 1 || p.logits == nullptr || p.lengths == nullptr)
    return cudaErrorInvalidValue;
  dim3 grid((p.seq + kRowThreads / 32 - 1) / (kRowThreads / 32), p.batch, p.n_tasks);
  if (p.hidden == 768) return launch_kernel(token_head_kernel<3>, grid, dim3(kRowThreads), 0, stream, p);
  if (p.hidden == 1024) return launch_kernel(token_head_kernel<4>, grid, dim3(kRowThreads), 0, stream, p);
  return cudaErrorInvalidValue;
}

cudaError_t launch_layernorm(const LayerNormParams& p, cudaStream_t stream) {
  if (p.n_groups < 1 || p.n_groups > kMaxGroups || p.rows < 1 || p.n_parts < 0 || p.n_parts > kMaxParts) return cudaErrorInvalidValue;
  dim3 grid((p.rows + kRowThreads / 32 - 1) / (kRowThreads / 32), p.n_groups);
  if (p.n_parts > 0) {
    if (p.hidden == 768) return launch_kernel(layernorm_kernel<3, true>, grid, dim3(kRowThreads), 0, stream, p);
    if (p.hidden == 1024) return launch_kernel(layernorm_kernel<4, true>, grid, dim3(kRowThreads), 0, stream, p);
    return cudaErrorInvalidValue;
  }
  if (p.hidden == 768) return launch_kernel(layernorm_kernel<3, false>, grid, dim3(kRowThreads), 0, stream, p);
  if (p.hidden == 1024) return launch_kernel(layernorm_kernel<4, false>, grid, dim3(kRowThreads), 0, stream, p);
  return cudaErrorInvalidValue;
}

cudaError_t launch_embed(const EmbedParams& p, cudaStream_t stream) {
  const int rows = p.batch * p.seq;
  if (rows < 1) return cudaErrorInvalidValue;
  dim3 grid((rows + kRowThreads / 32 - 1) / (kRowThreads / 32));
  if (p.hidden == 768) return launch_kernel(embed_kernel<3>, grid, dim3(kRowThreads), 0, stream, p);
  if (p.hidden == 1024) return launch_kernel(embed_kernel<4>, grid, dim3(kRowThreads), 0, stream, p);
  return cudaErrorInvalidValue;
}

cudaError_t launch_pooler_head(const HeadParams& p, cudaStream_t stream) {
  if (p.n_tasks < 1 || p.n_tasks > kMaxGroups || p.batch < 1 || p.hidden % 256 != 0 || p.hidden > 1024 ||
      p.pooled == nullptr)
    return cudaErrorInvalidValue;
  const size_t smem = static_cast<size_t>(kSeqPerCta) * p.hidden * sizeof(float);  // <= 32 KB
  const int chunks = (p.batch + kSeqPerCta - 1) / kSeqPerCta;
  cudaError_t err = launch_kernel(pooler_kernel, dim3(p.hidden / kPoolFeaturesPerCta, p.n_tasks, chunks),
                                  dim3(kHeadThreads), smem, stream, p);
  if (err != cudaSuccess) return err;
  return launch_kernel(head_kernel, dim3(chunks, p.n_tasks), dim3(kHeadThreads), 0, stream, p);
}

cudaError_t launch_head(const HeadParams& p, cudaStream_t stream) {
  if (p.n_tasks < 1 || p.n_tasks > kMaxGroups || p.batch < 1 || p.hidden % 256 != 0 || p.hidden > 1024 ||
      p.pooled == nullptr)
    return cudaErrorInvalidValue;
  const int chunks = (p.batch + kSeqPerCta - 1) / kSeqPerCta;
  return launch_kernel(head_kernel, dim3(chunks, p.n_tasks), dim3(kHeadThreads), 0, stream, p);
}

}  // namespace mt
