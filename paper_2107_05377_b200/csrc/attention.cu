// Fused masked self-attention of the encoder layer:
//   ctx[i, head] = softmax_j( q_i . k_j / sqrt(64),  j < length ) . V        per (sequence, head)
// from the packed projection qkv[B*S, 3H] = [Q | K | V].  Keys at positions >= length get weight
// exactly 0 (their K/V rows are never read: zero-filled in shared memory), query rows >= length
// are written as 0, so padded rows stay finite and deterministic whatever they contained.
//
// One CTA = 64 query rows of one (group, sequence, head); 4 warps x 16 rows, four CTAs per SM.  Keys
// are visited in tiles of 64 (double buffered: tile t+1 is fetched while tile t is used, and V of a
// tile may still be in flight while its scores are computed) with an online softmax (running row maximum and sum in fp32, reduced across the four
// lanes that share a row with warp shuffles).  Q, K, V tiles are staged in shared memory with
// 16-byte cp.async copies into an XOR-swizzled layout and fed to the tensor cores through ldmatrix
// (mma.sync m16n8k16, bf16 inputs, fp32 accumulate); the probabilities are rounded to bf16 for the
// second product.  Several layers of one wave are the groups of a single launch.

#include "mt_kernels.h"

namespace mt {
namespace {

constexpr int kAttnThreads = 128;
constexpr int kTileQ = 64;
constexpr int kTileK = 64;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
// 16-byte async copy; copies nothing and zero-fills when !valid.
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, bool valid) {
  const int bytes = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_pending() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// A tile is 64 rows x 64 bf16 (128 bytes = eight 16-byte chunks per row); chunk c of row r lives at
// chunk position c ^ (r & 7), which makes both the row-wise cp.async writes and the 8-row ldmatrix
// reads free of bank conflicts.
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  return static_cast<uint32_t>(row * 128 + ((chunk ^ (row & 7)) << 4));
}

// Loads rows [row0, row0+64) x 64 columns starting at `col0` of a [*, ld] bf16 matrix; rows >= limit zero.
__device__ __forceinline__ void load_tile(uint32_t smem_tile, const bf16* base, int ld, int row0, int limit, int tid) {
#pragma unroll
  for (int i = 0; i < (kTileK * 8) / kAttnThreads; ++i) {
    const int idx = tid + i * kAttnThreads;
    const int r = idx >> 3;
    const int c = idx & 7;
    const bool valid = (row0 + r) < limit;
    const bf16* src = base + static_cast<size_t>(valid ? row0 + r : 0) * ld + c * 8;
    cp_async_16(smem_tile + tile_off(r, c), src, valid);
  }
}

__global__ void __launch_bounds__(kAttnThreads, 4) attention_kernel(const __grid_constant__ AttnParams p) {
  // Q tile, then two buffers of (K tile, V tile): the keys of tile t+1 are fetched while tile t is used
  __shared__ __align__(128) uint8_t smem[(kTileQ + 4 * kTileK) * 128];
  const uint32_t sQ = smem_u32(smem);
  const uint32_t sKV = sQ + kTileQ * 128;
  constexpr uint32_t kBufBytes = 2 * kTileK * 128;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  const int q0 = blockIdx.x * kTileQ;
  const int head = blockIdx.y;
  const int g = blockIdx.z / p.batch;
  const int b = blockIdx.z - g * p.batch;
  const int H = p.heads * kHeadDim;
  const int ld = 3 * H;

  grid_dependency_wait();
  grid_launch_dependents();
  int len = p.lengths[b];
  len = len < 1 ? 1 : (len > p.seq ? p.seq : len);

  const size_t row0 = p.row_start != nullptr ? static_cast<size_t>(p.row_start[b]) : static_cast<size_t>(b) * p.seq;
  const bf16* qkv = p.qkv[g] + row0 * ld + head * kHeadDim;
  bf16* ctx = p.ctx[g] + row0 * H + head * kHeadDim;
  // rows this tile may write: up to the sequence's length when packed (the next sequence follows
  // immediately), up to the padded length otherwise
  const int rows_here = min(kTileQ, (p.packed ? len : p.seq) - q0);

  if (q0 >= len) {
    if (p.packed) return;
    // the whole query tile is padding: write zeros
    for (int idx = tid; idx < rows_here * 8; idx += kAttnThreads) {
      const int r = idx >> 3, c = idx & 7;
      *reinterpret_cast<uint4*>(ctx + static_cast<size_t>(q0 + r) * H + c * 8) = make_uint4(0, 0, 0, 0);
    }
    return;
  }

  // copy groups, in order: {Q, K0}, {V0}, then {K(t+1)}, {V(t+1)} issued while tile t is being used
  load_tile(sQ, qkv, ld, q0, len, tid);
  load_tile(sKV, qkv + H, ld, 0, len, tid);
  cp_async_commit();
  load_tile(sKV + kTileK * 128, qkv + 2 * H, ld, 0, len, tid);
  cp_async_commit();

  float o[8][4];
#pragma unroll
  for (int n = 0; n < 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY};
  float l_run[2] = {0.f, 0.f};
  uint32_t qf[4][4];
  // scores are scaled by 1/sqrt(64) and moved to base 2 for exp2f
  const float scale_log2 = 0.125f * 1.4426950408889634f;

  const int n_key_tiles = (len + kTileK - 1) / kTileK;
  for (int kt = 0; kt < n_key_tiles; ++kt) {
    const int k0 = kt * kTileK;
    const uint32_t sK = sKV + (kt & 1) * kBufBytes;
    const uint32_t sV = sK + kTileK * 128;
    // K of this tile (and Q) have landed once at most one newer group (this tile's V) is pending;
    // the barrier also means every warp is done with the previous tile, whose buffer is refilled next
    cp_async_wait_pending<1>();
    __syncthreads();
    if (kt + 1 < n_key_tiles) {
      const uint32_t nK = sKV + ((kt + 1) & 1) * kBufBytes;
      load_tile(nK, qkv + H, ld, k0 + kTileK, len, tid);
      cp_async_commit();
      load_tile(nK + kTileK * 128, qkv + 2 * H, ld, k0 + kTileK, len, tid);
      cp_async_commit();
    } else {
      cp_async_commit();  // empty groups keep the pending-group arithmetic uniform
      cp_async_commit();
    }

    if (kt == 0) {
      // Q fragments: 16 rows of this warp x 64 dims = four k-steps of 16
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        const int r = warp * 16 + (lane & 15);
        const int c = ks * 2 + (lane >> 4);
        ldmatrix_x4(sQ + tile_off(r, c), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
      }
    }

    // Work is skipped at the granularity of the tensor-core fragments: a warp whose 16 query rows are
    // all padding computes nothing, n-tiles (8 keys) and k-steps (16 keys) beyond the length are
    // not multiplied.  All conditions are warp-uniform.
    const bool warp_has_rows = q0 + warp * 16 < len;
    const int keys_here = min(kTileK, len - k0);
    const int n_used = warp_has_rows ? (keys_here + 7) >> 3 : 0;
    const int ks_used = warp_has_rows ? (keys_here + 15) >> 4 : 0;

    // S = Q K^T : 16 x 64 per warp = eight n-tiles of 8 keys
    float s[8][4];
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
      if (n >= n_used) continue;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        // four 8x8 blocks of K rows (keys n*8..n*8+7), dims half*32 + {0,8,16,24}
        uint32_t k0r, k1r, k2r, k3r;
        const int r = n * 8 + (lane & 7);
        const int c = half * 4 + (lane >> 3);
        ldmatrix_x4(sK + tile_off(r, c), k0r, k1r, k2r, k3r);
        mma_bf16_16816(s[n], qf[half * 2], k0r, k1r);
        mma_bf16_16816(s[n], qf[half * 2 + 1], k2r, k3r);
      }
    }

    // mask keys >= len, online softmax.  Thread holds rows (lane/4) and (lane/4 + 8);
    // columns n*8 + 2*(lane%4) + {0,1}.
    float m_new[2] = {m_run[0], m_run[1]};
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      const int key = k0 + n * 8 + 2 * (lane & 3);
      if (key >= len) { s[n][0] = -INFINITY; s[n][2] = -INFINITY; }
      if (key + 1 >= len) { s[n][1] = -INFINITY; s[n][3] = -INFINITY; }
      m_new[0] = fmaxf(m_new[0], fmaxf(s[n][0], s[n][1]));
      m_new[1] = fmaxf(m_new[1], fmaxf(s[n][2], s[n][3]));
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      m_new[r] = fmaxf(m_new[r], __shfl_xor_sync(0xffffffffu, m_new[r], 1));
      m_new[r] = fmaxf(m_new[r], __shfl_xor_sync(0xffffffffu, m_new[r], 2));
    }
    // key 0 of the first tile is always valid (len >= 1), so m_new is finite from the first tile on
    float corr[2], sum[2] = {0.f, 0.f};
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      corr[r] = exp2f((m_run[r] - m_new[r]) * scale_log2);
      m_run[r] = m_new[r];
    }
    uint32_t pf[4][4];  // probabilities as A fragments: four k-steps of 16 keys
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      const float p0 = exp2f((s[n][0] - m_new[0]) * scale_log2);
      const float p1 = exp2f((s[n][1] - m_new[0]) * scale_log2);
      const float p2 = exp2f((s[n][2] - m_new[1]) * scale_log2);
      const float p3 = exp2f((s[n][3] - m_new[1]) * scale_log2);
      sum[0] += p0 + p1;
      sum[1] += p2 + p3;
      pf[n >> 1][(n & 1) * 2 + 0] = pack_bf16(p0, p1);
      pf[n >> 1][(n & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) l_run[r] = l_run[r] * corr[r] + sum[r];
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      o[n][0] *= corr[0]; o[n][1] *= corr[0];
      o[n][2] *= corr[1]; o[n][3] *= corr[1];
    }

    // V of this tile has landed once only the two groups of the next tile are pending
    cp_async_wait_pending<2>();
    __syncthreads();
    // O += P V : k = keys (four steps of 16), n = 64 dims (eight n-tiles)
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      if (ks >= ks_used) continue;
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        // V rows ks*16 .. +15, dims np*16 .. +15, transposed on load
        uint32_t v0, v1, v2, v3;
        const int r = ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int c = np * 2 + (lane >> 4);
        ldmatrix_x4_trans(sV + tile_off(r, c), v0, v1, v2, v3);
        mma_bf16_16816(o[np * 2], pf[ks], v0, v1);
        mma_bf16_16816(o[np * 2 + 1], pf[ks], v2, v3);
      }
    }
  }

  // row sums across the four lanes of a row, normalise, stage in this warp's rows of the Q tile
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }
  const float inv0 = 1.f / l_run[0];
  const float inv1 = 1.f / l_run[1];
  cp_async_wait_pending<0>();  // only empty groups can be left
  __syncwarp();
  uint8_t* sQg = smem;
#pragma unroll
  for (int n = 0; n < 8; ++n) {
    const int r0 = warp * 16 + (lane >> 2);
    const int byte_in_chunk = (lane & 3) * 4;
    *reinterpret_cast<uint32_t*>(sQg + tile_off(r0, n) + byte_in_chunk) = pack_bf16(o[n][0] * inv0, o[n][1] * inv0);
    *reinterpret_cast<uint32_t*>(sQg + tile_off(r0 + 8, n) + byte_in_chunk) = pack_bf16(o[n][2] * inv1, o[n][3] * inv1);
  }
  __syncwarp();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int idx = lane + i * 32;   // 16 rows x 8 chunks
    const int r = warp * 16 + (idx >> 3);
    const int c = idx & 7;
    if (r < rows_here) {
      uint4 val = *reinterpret_cast<const uint4*>(sQg + tile_off(r, c));
      if (q0 + r >= len) val = make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4*>(ctx + static_cast<size_t>(q0 + r) * H + c * 8) = val;
    }
  }
}

// First-token attention: one warp = one (sequence, head).  Lanes split the keys, for the scores
// (each lane a whole 128-byte K row per key) and for the weighted sum of V rows alike (each lane the
// whole V rows of its keys, then a butterfly sum over the lanes).  fp32 throughout; only the output
// is rounded to bf16.
constexpr int kClsWarps = 4;
constexpr int kClsMaxKeysPerLane = 16;  // sequences of up to 512 keys

__global__ void __launch_bounds__(kClsWarps * 32) cls_attention_kernel(const ClsAttnParams p) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int head = blockIdx.x * kClsWarps + warp;
  const int b = blockIdx.y, g = blockIdx.z;
  const int H = p.heads * kHeadDim, ld = 3 * H;
  grid_dependency_wait();
  grid_launch_dependents();
  int len = p.lengths[b];
  len = len < 1 ? 1 : (len > p.seq ? p.seq : len);
  const size_t row0 = p.row_start != nullptr ? static_cast<size_t>(p.row_start[b]) : static_cast<size_t>(b) * p.seq;

  // the block's share of the residual row: kClsWarps heads x 64 columns
  {
    const int col = blockIdx.x * kClsWarps * kHeadDim + threadIdx.x * 2;
    if (col < H) {
      const float2 r = *reinterpret_cast<const float2*>(p.in32[g] + row0 * H + col);
      *reinterpret_cast<float2*>(p.res[g] + static_cast<size_t>(b) * H + col) = r;
    }
  }
  if (head >= p.heads) return;

  const bf16* base = p.qkv[g] + row0 * ld + head * kHeadDim;
  float q[kHeadDim];
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const uint4 u = __ldg(reinterpret_cast<const uint4*>(base) + c);
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      q[c * 8 + 2 * i] = __uint_as_float(w[i] << 16);
      q[c * 8 + 2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  float sc[kClsMaxKeysPerLane];
  float mx = -INFINITY;
#pragma unroll
  for (int i = 0; i < kClsMaxKeysPerLane; ++i) {
    const int j = i * 32 + lane;
    sc[i] = -INFINITY;
    if (j < len) {
      const uint4* krow = reinterpret_cast<const uint4*>(base + static_cast<size_t>(j) * ld + H);
      float acc = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint4 u = krow[c];
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          acc = fmaf(q[c * 8 + 2 * t], __uint_as_float(w[t] << 16), acc);
          acc = fmaf(q[c * 8 + 2 * t + 1], __uint_as_float(w[t] & 0xFFFF0000u), acc);
        }
      }
      sc[i] = acc;
      mx = fmaxf(mx, acc);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  const float scale_log2 = 0.125f * 1.4426950408889634f;
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < kClsMaxKeysPerLane; ++i) {
    sc[i] = exp2f((sc[i] - mx) * scale_log2);   // 0 for keys beyond the length
    sum += sc[i];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);

  // P . V with the keys spread over the lanes exactly as for the scores: every lane accumulates
  // its own keys' rows of V (all of its loads are independent, so they are in flight together), then
  // the 32 partial rows of 64 columns are summed by a butterfly that halves the columns a lane keeps
  // at every step; lane l ends with columns 2l and 2l + 1.  The order of the additions is fixed.
  float o[kHeadDim];
#pragma unroll
  for (int c = 0; c < kHeadDim; ++c) o[c] = 0.f;
#pragma unroll
  for (int i = 0; i < kClsMaxKeysPerLane; ++i) {
    const int j = i * 32 + lane;
    if (j < len) {
      const uint4* vrow = reinterpret_cast<const uint4*>(base + static_cast<size_t>(j) * ld + 2 * H);
      const float pj = sc[i];
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint4 u = vrow[c];
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          o[c * 8 + 2 * t] = fmaf(pj, __uint_as_float(w[t] << 16), o[c * 8 + 2 * t]);
          o[c * 8 + 2 * t + 1] = fmaf(pj, __uint_as_float(w[t] & 0xFFFF0000u), o[c * 8 + 2 * t + 1]);
        }
      }
    }
  }
#pragma unroll
  for (int width = 32; width >= 2; width >>= 1) {   // columns kept after this step
    const bool upper = (lane & (width >> 1)) != 0;  // lane bit 4, 3, .. 0 for width 32, 16, .. 2
#pragma unroll
    for (int c = 0; c < width; ++c) {
      const float send = upper ? o[c] : o[c + width];
      const float keep = upper ? o[c + width] : o[c];
      o[c] = keep + __shfl_xor_sync(0xffffffffu, send, width >> 1);
    }
  }
  const float o0 = o[0], o1 = o[1];
  const float inv = 1.f / sum;
  *reinterpret_cast<uint32_t*>(p.ctx[g] + static_cast<size_t>(b) * H + head * kHeadDim + 2 * lane) =
      pack_bf16(o0 * inv, o1 * inv);
}

// The same for sequences of at most 128 tokens: one CTA of four warps = one (sequence, head), one key
// per lane.  A lane's K row and V row (128 bytes each) are requested together, before anything is
// computed, so the whole kernel is two trips to memory deep: (length, first row) and then (q, K, V).
// Maximum, sum and the 64 output columns are combined across the four warps through shared memory
// in warp order, so the result does not depend on timing.
constexpr int kClsShortMaxSeq = 128;

__global__ void __launch_bounds__(128) cls_attention_short_kernel(const ClsAttnParams p) {
  __shared__ float s_max[4], s_sum[4];
  __shared__ float s_out[4][kHeadDim];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int head = blockIdx.x, b = blockIdx.y, g = blockIdx.z;
  const int H = p.heads * kHeadDim, ld = 3 * H;
  grid_dependency_wait();
  grid_launch_dependents();
  int len = p.lengths[b];
  len = len < 1 ? 1 : (len > p.seq ? p.seq : len);
  const size_t row0 = p.row_start != nullptr ? static_cast<size_t>(p.row_start[b]) : static_cast<size_t>(b) * p.seq;
  const bf16* base = p.qkv[g] + row0 * ld + head * kHeadDim;
  const int j = warp * 32 + lane;   // this lane's key
  const bool valid = j < len;

  uint4 qv[8], kv[8], vv[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) qv[c] = __ldg(reinterpret_cast<const uint4*>(base) + c);
  if (valid) {
    const uint4* krow = reinterpret_cast<const uint4*>(base + static_cast<size_t>(j) * ld + H);
    const uint4* vrow = reinterpret_cast<const uint4*>(base + static_cast<size_t>(j) * ld + 2 * H);
#pragma unroll
    for (int c = 0; c < 8; ++c) kv[c] = krow[c];
#pragma unroll
    for (int c = 0; c < 8; ++c) vv[c] = vrow[c];
  }
  // this head's 64 columns of the first token's fp32 residual
  if (threadIdx.x < kHeadDim / 4) {
    const int col = head * kHeadDim + threadIdx.x * 4;
    *reinterpret_cast<float4*>(p.res[g] + static_cast<size_t>(b) * H + col) =
        *reinterpret_cast<const float4*>(p.in32[g] + row0 * H + col);
  }

  float score = -INFINITY;
  if (valid) {
    float acc = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const uint32_t qw[4] = {qv[c].x, qv[c].y, qv[c].z, qv[c].w};
      const uint32_t kw[4] = {kv[c].x, kv[c].y, kv[c].z, kv[c].w};
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        acc = fmaf(__uint_as_float(qw[t] << 16), __uint_as_float(kw[t] << 16), acc);
        acc = fmaf(__uint_as_float(qw[t] & 0xFFFF0000u), __uint_as_float(kw[t] & 0xFFFF0000u), acc);
      }
    }
    score = acc;
  }
  float mx = score;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) s_max[warp] = mx;
  __syncthreads();
  mx = fmaxf(fmaxf(s_max[0], s_max[1]), fmaxf(s_max[2], s_max[3]));   // key 0 is always valid: finite
  const float scale_log2 = 0.125f * 1.4426950408889634f;
  const float pj = valid ? exp2f((score - mx) * scale_log2) : 0.f;
  float sum = pj;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0) s_sum[warp] = sum;

  float o[kHeadDim];
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const uint32_t w[4] = {vv[c].x, vv[c].y, vv[c].z, vv[c].w};
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      o[c * 8 + 2 * t] = valid ? pj * __uint_as_float(w[t] << 16) : 0.f;
      o[c * 8 + 2 * t + 1] = valid ? pj * __uint_as_float(w[t] & 0xFFFF0000u) : 0.f;
    }
  }
#pragma unroll
  for (int width = 32; width >= 2; width >>= 1) {   // columns kept after this step; lane l ends with 2l, 2l + 1
    const bool upper = (lane & (width >> 1)) != 0;
#pragma unroll
    for (int c = 0; c < width; ++c) {
      const float send = upper ? o[c] : o[c + width];
      const float keep = upper ? o[c + width] : o[c];
      o[c] = keep + __shfl_xor_sync(0xffffffffu, send, width >> 1);
    }
  }
  s_out[warp][2 * lane] = o[0];
  s_out[warp][2 * lane + 1] = o[1];
  __syncthreads();
  if (warp == 0) {
    const float total = ((s_sum[0] + s_sum[1]) + s_sum[2]) + s_sum[3];
    const float inv = 1.f / total;
    const float o0 = ((s_out[0][2 * lane] + s_out[1][2 * lane]) + s_out[2][2 * lane]) + s_out[3][2 * lane];
    const float o1 = ((s_out[0][2 * lane + 1] + s_out[1][2 * lane + 1]) + s_out[2][2 * lane + 1]) + s_out[3][2 * lane + 1];
    *reinterpret_cast<uint32_t*>(p.ctx[g] + static_cast<size_t>(b) * H + head * kHeadDim + 2 * lane) =
        pack_bf16(o0 * inv, o1 * inv);
  }
}

}  // namespace

cudaError_t launch_cls_attention(const ClsAttnParams& p, cudaStream_t stream) {
  if (p.n_groups < 1 || p.n_groups > kMaxGroups || p.batch < 1 || p.seq < 1 || p.seq > 32 * kClsMaxKeysPerLane)
    return cudaErrorInvalidValue;
  if (p.seq <= kClsShortMaxSeq)
    return launch_kernel(cls_attention_short_kernel, dim3(p.heads, p.batch, p.n_groups), dim3(128), 0, stream, p);
  dim3 grid((p.heads + kClsWarps - 1) / kClsWarps, p.batch, p.n_groups);
  return launch_kernel(cls_attention_kernel, grid, dim3(kClsWarps * 32), 0, stream, p);
}

cudaError_t launch_attention(const AttnParams& p, cudaStream_t stream) {
  if (p.n_groups < 1 || p.n_groups > kMaxGroups || p.batch < 1 || p.seq < 1) return cudaErrorInvalidValue;
  if (p.tensor_memory) return launch_attention_tc(p, stream);
  dim3 grid((p.seq + kTileQ - 1) / kTileQ, p.heads, p.batch * p.n_groups);
  return launch_kernel(attention_kernel, grid, dim3(kAttnThreads), 0, stream, p);
}

}  // namespace mt
