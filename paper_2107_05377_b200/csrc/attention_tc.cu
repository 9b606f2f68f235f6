// Masked self-attention of the encoder layer on the tcgen05 tensor cores, for sequences of at most
// 128 tokens (the length the throughput configurations use):
//   ctx[i, head] = softmax_j( q_i . k_j / sqrt(64),  j < length ) . V        per (sequence, head)
// from the packed projection qkv[rows, 3H] = [Q | K | V].
//
// One CTA of 128 threads = one (layer of the wave, sequence, head); thread t owns query row t, which
// is lane t of tensor memory.  Steps:
//   1. an elected lane fetches the 128 x 64 Q, K and V tiles with three TMA loads (128-byte swizzle; rows
//      past the end of the buffer arrive as zeros, rows past the sequence's length are another
//      sequence's finite data or stale memory and are masked: V rows >= length are overwritten with
//      zeros in shared memory, score columns >= length never enter the softmax)
//   2. S = Q . K^T: four tcgen05.mma 128 x N x 16 (N = 64 when length <= 64, else 128) into tensor
//      memory columns [0, N), issued by the lane that saw the copies land while the others clear V
//   3. every thread reads its row of S twice with tcgen05.ld (maximum; then exponentials and their
//      fp32 sum), rounds the probabilities to bf16 and stores them K-major, 128-byte swizzled, over
//      the Q and K tiles, which are no longer needed
//   4. O = P . V: V is the MN-major B operand (its rows are keys = the K dimension), accumulated over
//      the S columns already consumed
//   5. O / sum, rounded to bf16, goes through shared memory and leaves as full 128-byte row segments.
// 50 KB of shared memory and 128 columns of tensor memory per CTA: four CTAs per SM.
//
// Both waits are bounded; a wait that runs out raises the timeout flag of the status word, the
// copies still in flight are given the same limit to land, tensor memory is freed and the CTA returns.

#include "tc_ptx.cuh"

namespace mt {
namespace {

constexpr int kTcThreads = 128;
constexpr int kTcRows = 128;  // queries and keys of one tile (one tcgen05 accumulator = 128 TMEM lanes)
constexpr int kTcTileBytes = kTcRows * 128;  // 128 rows of 64 bf16
constexpr uint32_t kTcTmemCols = 128;
constexpr int kTcSmemBytes = 3 * kTcTileBytes + 64 + 1024;  // Q, K, V + bookkeeping + alignment slack

// B operand in MN-major form (bit 16): the shared-memory rows of the tile run along K.
__host__ __device__ constexpr uint32_t umma_idesc_bf16_b_mn(int m, int n) { return umma_idesc_bf16(m, n) | (1u << 16); }

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(kTcThreads, 4) attention_tc_kernel(const __grid_constant__ AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sQ = smem_u32(smem);
  const uint32_t sK = sQ + kTcTileBytes;
  const uint32_t sV = sK + kTcTileBytes;
  uint8_t* book = smem + 3 * kTcTileBytes;
  const uint32_t bar_load = smem_u32(book);
  const uint32_t bar_mma = bar_load + 8;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(book + 16);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(book + 20);

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int head = blockIdx.x;
  const int b = blockIdx.y;
  const int g = blockIdx.z;
  const int H = p.heads * kHeadDim;
  // warp 1 is converged here: one of its lanes issues the copies and the MMAs (warp 0 allocates tensor memory)
  const bool leader = warp == 1 && elect_one();

  if (tid == 0) {
    mbar_init(bar_load, 1);
    mbar_init(bar_mma, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_shared();
    prefetch_tensormap(&p.tmap_qkv[g]);
    prefetch_tensormap(&p.tmap_qkv64[g]);
  }
  if (warp == 0) tmem_alloc(smem_u32(tmem_slot), kTcTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // The lengths are an input of the forward and the row starts were written by its first kernel: when this
  // kernel starts, every kernel but its immediate predecessor (the Q/K/V projection) has completed, so both
  // may be read before the dependency wait, off the critical path.
  int len = p.lengths[b];
  len = len < 1 ? 1 : (len > p.seq ? p.seq : len);   // as every kernel of the path: a bad length is clamped (and flagged by the embedding)
  const int row0 = p.row_start != nullptr ? p.row_start[b] : b * p.seq;

  grid_dependency_wait();
  grid_launch_dependents();
  const int rows_out = p.packed ? len : p.seq;   // the padded layout also gets its rows >= length, as zeros
  bf16* ctx = p.ctx[g];

  bool ok = true;
  bool loads_in_flight = false;
  {
    if (leader) {
      // a sequence of at most 64 tokens needs only the first 64 rows of each tile (the rest of the tiles
      // keeps whatever shared memory held: query rows and keys >= length never reach a result, and the V
      // rows >= length are overwritten with zeros below)
      const CUtensorMap* map = len <= 64 ? &p.tmap_qkv64[g] : &p.tmap_qkv[g];
      mbar_expect_tx(bar_load, len <= 64 ? 3 * kTcTileBytes / 2 : 3 * kTcTileBytes);
      tma_load_2d(sQ, map, head * kHeadDim, row0, bar_load);
      tma_load_2d(sK, map, H + head * kHeadDim, row0, bar_load);
      tma_load_2d(sV, map, 2 * H + head * kHeadDim, row0, bar_load);
    }
    const bool landed = mbar_wait(bar_load, 0, abort_flag);
    if (leader && landed) {
      // S = Q K^T at once: the thread that saw the barrier complete sees the tiles (no MMA is issued if
      // the copies never landed)
      tc_fence_after();
      const int key_tiles = len > 64 ? 2 : 1;   // 64 keys each
      const uint64_t dq = smem_desc_sw128(sQ);
      const uint64_t dk = smem_desc_sw128(sK);
      const uint32_t idesc = umma_idesc_bf16(kTcRows, 64 * key_tiles);
#pragma unroll
      for (int k = 0; k < kHeadDim / 16; ++k) umma_bf16(tmem_base, dq + 2 * k, dk + 2 * k, idesc, k > 0 ? 1u : 0u);
      umma_commit(bar_mma);
    }
    // meanwhile: keys >= length take no part (their probabilities are exactly 0), and 0 * V must stay finite;
    // the proxy fence after the probabilities are written covers these stores too
    if (landed && tid >= len) {
#pragma unroll
      for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4*>(smem + 2 * kTcTileBytes + tid * 128 + c * 16) = make_uint4(0, 0, 0, 0);
    }
    ok = __syncthreads_and(landed) != 0;
    loads_in_flight = !ok;
  }
  if (ok) ok = __syncthreads_and(mbar_wait(bar_mma, 0, abort_flag)) != 0;

  if (ok) {
    tc_fence_after();
    const int key_tiles = len > 64 ? 2 : 1;
    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
    const bool row_valid = tid < len;
    float row_max = -INFINITY;
    for (int c = 0; c < 2 * key_tiles; ++c) {
      uint32_t v[32];
      tmem_ld_32x32(t_row + c * 32, v);
      tmem_ld_wait();
      if (!row_valid) continue;
      if ((c + 1) * 32 <= len) {   // all 32 keys of the chunk are valid: no per-key test
#pragma unroll
        for (int j = 0; j < 32; ++j) row_max = fmaxf(row_max, __uint_as_float(v[j]));
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (c * 32 + j < len) row_max = fmaxf(row_max, __uint_as_float(v[j]));
      }
    }
    // exp((s - max) / 8) = 2^((s - max) * log2(e) / 8); the exponent is <= 0, so ex2.approx is in range
    const float k2 = 0.125f * 1.4426950408889634f;
    const float shift = row_max * k2;
    float row_sum = 0.0f;
    for (int c = 0; c < 2 * key_tiles; ++c) {
      uint32_t v[32];
      tmem_ld_32x32(t_row + c * 32, v);
      tmem_ld_wait();
      uint8_t* p_tile = smem + (c >> 1) * kTcTileBytes;   // probabilities replace the Q tile, then the K tile
      const bool chunk_full = (c + 1) * 32 <= len;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t w[4] = {0u, 0u, 0u, 0u};
        if (row_valid) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int key = c * 32 + q * 8 + 2 * j;
            float e0 = ex2_approx(fmaf(__uint_as_float(v[q * 8 + 2 * j]), k2, -shift));
            float e1 = ex2_approx(fmaf(__uint_as_float(v[q * 8 + 2 * j + 1]), k2, -shift));
            if (!chunk_full) {
              e0 = key < len ? e0 : 0.0f;
              e1 = key + 1 < len ? e1 : 0.0f;
            }
            row_sum += e0 + e1;
            w[j] = pack_bf16(e0, e1);
          }
        }
        *reinterpret_cast<uint4*>(p_tile + staging_off(tid, (c & 1) * 4 + q)) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
    const float inv_sum = row_valid ? 1.0f / row_sum : 0.0f;
    fence_async_shared();
    tc_fence_before();
    __syncthreads();

    if (leader) {
      tc_fence_after();
      const uint32_t idesc = umma_idesc_bf16_b_mn(kTcRows, kHeadDim);
      for (int t = 0; t < key_tiles; ++t) {
        const uint64_t dp = smem_desc_sw128(sQ + t * kTcTileBytes);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          // sixteen keys = sixteen 128-byte rows of the V tile: two groups of eight rows, 1024 bytes apart
          const uint64_t dv = smem_desc_sw128(sV + (t * 64 + k * 16) * 128);
          umma_bf16(tmem_base, dp + 2 * k, dv, idesc, (t | k) != 0 ? 1u : 0u);
        }
      }
      umma_commit(bar_mma);
    }
    ok = __syncthreads_and(mbar_wait(bar_mma, 1, abort_flag)) != 0;

    if (ok) {
      tc_fence_after();
      // O / sum -> bf16 -> the V tile's place (both products have completed), then out row by row
      uint8_t* o_tile = smem + 2 * kTcTileBytes;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t v[32];
        tmem_ld_32x32(t_row + half * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t w[4];
#pragma unroll
          for (int j = 0; j < 4; ++j)
            w[j] = pack_bf16(__uint_as_float(v[q * 8 + 2 * j]) * inv_sum, __uint_as_float(v[q * 8 + 2 * j + 1]) * inv_sum);
          *reinterpret_cast<uint4*>(o_tile + staging_off(tid, half * 4 + q)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      __syncthreads();
      const int chunk = tid & 7;
      for (int r = tid >> 3; r < rows_out; r += kTcThreads / 8) {
        const uint4 val = *reinterpret_cast<const uint4*>(o_tile + staging_off(r, chunk));
        *reinterpret_cast<uint4*>(ctx + static_cast<size_t>(row0 + r) * H + head * kHeadDim + chunk * 8) = val;
      }
    }
  }

  if (!ok && tid == 0) {
    if (loads_in_flight) {
      // shared memory must not be handed to another CTA while copies may still land in it
      const unsigned long long t0 = global_timer_ns();
      while (!mbar_try_wait(bar_load, 0)) {
        if (global_timer_ns() - t0 > kWaitLimitNs) break;
      }
    }
    if (p.status != nullptr) atomicOr(p.status, kFlagWaitTimeout);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, kTcTmemCols);
}


// ---- sequences of more than 128 tokens -----------------------------------------------------------
// One CTA of 128 threads = one (layer of the wave, sequence, head, tile of 128 queries).  The keys are walked
// in tiles of 128 with the running-maximum form of the softmax:
//   per key tile j:  S = Q . K_j^T (tcgen05.mma into tensor memory columns [0, 128));
//                    m' = max(m, rowmax S);  alpha = exp((m - m') / 8);  P = exp((S - m') / 8) (bf16, shared memory);
//                    l = l alpha + rowsum P;  T = P . V_j (tensor memory columns [128, 192));  O = O alpha + T
// with O (64 fp32 per query row) in registers; at the end O / l.  K_j and V_j are double buffered: the tiles of
// step j + 2 are requested as soon as the products of step j have completed.  The first 64 keys of P replace
// K_j (dead once S is complete), the other 64 have a tile of their own.  S of step j + 1 is issued right behind
// P . V of step j, so it runs while the threads fold T into O.
// Keys at positions >= length are excluded exactly as in the one-tile kernel (probability 0, V rows zeroed).
constexpr int kTlSmemBytes = 6 * kTcTileBytes + 64 + 1024;   // Q, K x 2, V x 2, upper half of P
constexpr uint32_t kTlTmemCols = 256;

__global__ void __launch_bounds__(kTcThreads, 2) attention_tc_tiled_kernel(const __grid_constant__ AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sQ = smem_u32(smem);
  const uint32_t sK = sQ + kTcTileBytes;            // two buffers; keys 0..63 of P replace the K tile of the step
  const uint32_t sV = sK + 2 * kTcTileBytes;        // two buffers
  const uint32_t sP1 = sV + 2 * kTcTileBytes;       // keys 64..127 of P; at the end the output tile
  uint8_t* k_ptr = smem + kTcTileBytes;
  uint8_t* v_ptr = smem + 3 * kTcTileBytes;
  uint8_t* p1_ptr = smem + 5 * kTcTileBytes;
  uint8_t* book = smem + 6 * kTcTileBytes;
  const uint32_t bar_q = smem_u32(book);
  const uint32_t bar_kv = bar_q + 8;                // two barriers
  const uint32_t bar_s = bar_kv + 16;               // S of a step is complete
  const uint32_t bar_pv = bar_s + 8;                // P . V of a step is complete
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(book + 40);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(book + 44);

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int head = blockIdx.x;
  const int q_tiles = (p.seq + kTcRows - 1) / kTcRows;
  const int b = blockIdx.y / q_tiles;
  const int q0 = (blockIdx.y - b * q_tiles) * kTcRows;   // first query of this CTA within the sequence
  const int g = blockIdx.z;
  const int H = p.heads * kHeadDim;

  // inputs of the forward and the output of its first kernel: readable before the dependency wait (see above)
  int len = p.lengths[b];
  len = len < 1 ? 1 : (len > p.seq ? p.seq : len);
  const int row0 = p.row_start != nullptr ? p.row_start[b] : b * p.seq;
  bf16* ctx = p.ctx[g];
  const int rows_in_seq = min(kTcRows, p.seq - q0);           // rows of this tile that exist in the padded layout
  const int rows_out = p.packed ? min(kTcRows, len - q0) : rows_in_seq;
  if (q0 >= len) {
    // a tile of padded query positions only: nothing in the packed layout, zeros in the padded one
    grid_dependency_wait();
    grid_launch_dependents();
    const int chunk = tid & 7;
    for (int r = tid >> 3; r < rows_out; r += kTcThreads / 8)
      *reinterpret_cast<uint4*>(ctx + static_cast<size_t>(row0 + q0 + r) * H + head * kHeadDim + chunk * 8) = make_uint4(0, 0, 0, 0);
    return;
  }

  if (tid == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_kv, 1);
    mbar_init(bar_kv + 8, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_pv, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_shared();
    prefetch_tensormap(&p.tmap_qkv[g]);
  }
  if (warp == 0) tmem_alloc(smem_u32(tmem_slot), kTlTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  grid_dependency_wait();
  grid_launch_dependents();

  const int n_kt = (len + kTcRows - 1) / kTcRows;   // key tiles
  const int rows_q = min(kTcRows, len - q0);         // valid query rows of this tile
  const CUtensorMap* map = &p.tmap_qkv[g];
  int kv_issued = 0;                                 // (thread 0) key tiles requested so far
  auto request_kv = [&](int j) {
    const int buf = j & 1;
    mbar_expect_tx(bar_kv + 8 * buf, 2 * kTcTileBytes);
    tma_load_2d(sK + buf * kTcTileBytes, map, H + head * kHeadDim, row0 + j * kTcRows, bar_kv + 8 * buf);
    tma_load_2d(sV + buf * kTcTileBytes, map, 2 * H + head * kHeadDim, row0 + j * kTcRows, bar_kv + 8 * buf);
  };
  // S = Q . K_j^T into tensor memory columns [0, 128) (thread 0; K_j has landed)
  auto issue_s = [&](int j) {
    tc_fence_after();
    const uint64_t dq = smem_desc_sw128(sQ);
    const uint64_t dk = smem_desc_sw128(sK + (j & 1) * kTcTileBytes);
    constexpr uint32_t idesc = umma_idesc_bf16(kTcRows, kTcRows);
#pragma unroll
    for (int k = 0; k < kHeadDim / 16; ++k) umma_bf16(tmem_base, dq + 2 * k, dk + 2 * k, idesc, k > 0 ? 1u : 0u);
    umma_commit(bar_s);
  };
  if (tid == 0) {
    mbar_expect_tx(bar_q, kTcTileBytes);
    tma_load_2d(sQ, map, head * kHeadDim, row0 + q0, bar_q);
    request_kv(0);
    if (n_kt > 1) request_kv(1);
    kv_issued = n_kt > 1 ? 2 : 1;
  }

  const uint32_t t_row = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
  const bool row_valid = tid < rows_q;
  const float k2 = 0.125f * 1.4426950408889634f;     // exp(x / 8) = 2^(x k2)
  float m_run = -INFINITY, l_run = 0.0f;
  float o[kHeadDim];
#pragma unroll
  for (int i = 0; i < kHeadDim; ++i) o[i] = 0.0f;
  bool ok = __syncthreads_and(mbar_wait(bar_q, 0, abort_flag)) != 0;
  if (ok) ok = __syncthreads_and(mbar_wait(bar_kv, 0, abort_flag)) != 0;
  if (ok && tid == 0) issue_s(0);

  for (int j = 0; j < n_kt && ok; ++j) {
    const int buf = j & 1;
    const int keys = min(kTcRows, len - j * kTcRows);   // valid keys of this tile
    // (K_j and V_j have landed: waited for by every thread before S of this step was issued)
    // keys >= length take no part: their probabilities are exactly 0, and 0 * V must stay finite
    if (tid >= keys) {
#pragma unroll
      for (int c = 0; c < 8; ++c)
        *reinterpret_cast<uint4*>(v_ptr + buf * kTcTileBytes + tid * 128 + c * 16) = make_uint4(0, 0, 0, 0);
    }
    ok = __syncthreads_and(mbar_wait(bar_s, static_cast<uint32_t>(j & 1), abort_flag)) != 0;
    if (!ok) break;
    tc_fence_after();

    // running maximum over this tile's valid keys
    float m_new = m_run;
    for (int c = 0; c < 4; ++c) {
      uint32_t v[32];
      tmem_ld_32x32(t_row + c * 32, v);
      tmem_ld_wait();
      if (!row_valid || c * 32 >= keys) continue;
      if ((c + 1) * 32 <= keys) {
#pragma unroll
        for (int i = 0; i < 32; ++i) m_new = fmaxf(m_new, __uint_as_float(v[i]));
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (c * 32 + i < keys) m_new = fmaxf(m_new, __uint_as_float(v[i]));
      }
    }
    // (a valid row has at least one valid key in every tile walked, so m_new is finite for it)
    const float alpha = row_valid ? ex2_approx((m_run - m_new) * k2) : 0.0f;   // 0 on the first tile (m_run = -inf)
    const float shift = m_new * k2;
    float tile_sum = 0.0f;
    for (int c = 0; c < 4; ++c) {
      uint32_t v[32];
      tmem_ld_32x32(t_row + c * 32, v);
      tmem_ld_wait();
      uint8_t* p_tile = c < 2 ? k_ptr + buf * kTcTileBytes : p1_ptr;   // S is complete: K_j is no longer needed
      const bool chunk_full = (c + 1) * 32 <= keys;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t w[4] = {0u, 0u, 0u, 0u};
        if (row_valid && c * 32 < keys) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int key = c * 32 + q * 8 + 2 * i;
            float e0 = ex2_approx(fmaf(__uint_as_float(v[q * 8 + 2 * i]), k2, -shift));
            float e1 = ex2_approx(fmaf(__uint_as_float(v[q * 8 + 2 * i + 1]), k2, -shift));
            if (!chunk_full) {
              e0 = key < keys ? e0 : 0.0f;
              e1 = key + 1 < keys ? e1 : 0.0f;
            }
            tile_sum += e0 + e1;
            w[i] = pack_bf16(e0, e1);
          }
        }
        *reinterpret_cast<uint4*>(p_tile + staging_off(tid, (c & 1) * 4 + q)) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
    l_run = fmaf(l_run, alpha, tile_sum);
    m_run = m_new;
    fence_async_shared();
    tc_fence_before();
    __syncthreads();

    if (tid == 0) {
      tc_fence_after();
      constexpr uint32_t idesc = umma_idesc_bf16_b_mn(kTcRows, kHeadDim);
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        const uint64_t dp = smem_desc_sw128(t == 0 ? sK + buf * kTcTileBytes : sP1);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          // sixteen keys = sixteen 128-byte rows of the V tile
          const uint64_t dv = smem_desc_sw128(sV + buf * kTcTileBytes + (t * 64 + k * 16) * 128);
          umma_bf16(tmem_base + kTcRows, dp + 2 * k, dv, idesc, (t | k) != 0 ? 1u : 0u);
        }
      }
      umma_commit(bar_pv);
      // S of the next step right behind it (every thread has read S of this step), once its K tile has landed
      if (j + 1 < n_kt && mbar_wait(bar_kv + 8 * (buf ^ 1), static_cast<uint32_t>(((j + 1) >> 1) & 1), abort_flag))
        issue_s(j + 1);
    }
    ok = __syncthreads_and(mbar_wait(bar_pv, static_cast<uint32_t>(j & 1), abort_flag)) != 0;
    if (!ok) break;
    tc_fence_after();
    // P . V of this step has completed (and S before it): its buffers may take the tiles of step j + 2
    if (tid == 0 && j + 2 < n_kt) {
      request_kv(j + 2);
      kv_issued = j + 3;
    }
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      uint32_t v[32];
      tmem_ld_32x32(t_row + kTcRows + half * 32, v);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 32; ++i) o[half * 32 + i] = fmaf(o[half * 32 + i], alpha, __uint_as_float(v[i]));
    }
    tc_fence_before();
    // V of the next step is written to (rows >= length) at the top of the loop: it must have landed for everyone
    if (j + 1 < n_kt)
      ok = __syncthreads_and(mbar_wait(bar_kv + 8 * (buf ^ 1), static_cast<uint32_t>(((j + 1) >> 1) & 1), abort_flag)) != 0;
  }

  if (ok) {
    // O / l -> bf16 -> the tile of P's upper half (all products have completed), then out row by row as full
    // 128-byte segments
    const float inv = row_valid ? 1.0f / l_run : 0.0f;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) w[i] = pack_bf16(o[q * 8 + 2 * i] * inv, o[q * 8 + 2 * i + 1] * inv);
      *reinterpret_cast<uint4*>(p1_ptr + staging_off(tid, q)) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    __syncthreads();
    const int chunk = tid & 7;
    for (int r = tid >> 3; r < rows_out; r += kTcThreads / 8) {
      const uint4 val = *reinterpret_cast<const uint4*>(p1_ptr + staging_off(r, chunk));
      *reinterpret_cast<uint4*>(ctx + static_cast<size_t>(row0 + q0 + r) * H + head * kHeadDim + chunk * 8) = val;
    }
  }

  if (!ok && tid == 0) {
    // shared memory must not be handed to another CTA while copies may still land in it: every tile that was
    // requested gets the usual limit to arrive
    const unsigned long long t0 = global_timer_ns();
    while (!mbar_try_wait(bar_q, 0)) {
      if (global_timer_ns() - t0 > kWaitLimitNs) break;
    }
    for (int j = max(0, kv_issued - 2); j < kv_issued; ++j) {
      while (!mbar_try_wait(bar_kv + 8 * (j & 1), static_cast<uint32_t>((j >> 1) & 1))) {
        if (global_timer_ns() - t0 > 2 * kWaitLimitNs) break;
      }
    }
    if (p.status != nullptr) atomicOr(p.status, kFlagWaitTimeout);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, kTlTmemCols);
}

}  // namespace

cudaError_t launch_attention_tc(const AttnParams& p, cudaStream_t stream) {
  if (p.n_groups < 1 || p.n_groups > kMaxGroups || p.batch < 1 || p.seq < 1 || p.seq > kAttnTensorMemoryMaxSeq)
    return cudaErrorInvalidValue;
  static PerDeviceOnce once;
  cudaError_t e = per_device_once(once, [&](int) {
    cudaError_t r = cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemBytes);
    if (r != cudaSuccess) return r;
    return cudaFuncSetAttribute(attention_tc_tiled_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTlSmemBytes);
  });
  if (e != cudaSuccess) return e;
  if (p.seq <= kTcRows) {
    dim3 grid(p.heads, p.batch, p.n_groups);
    return launch_kernel(attention_tc_kernel, grid, dim3(kTcThreads), kTcSmemBytes, stream, p);
  }
  const int q_tiles = (p.seq + kTcRows - 1) / kTcRows;
  dim3 grid(p.heads, p.batch * q_tiles, p.n_groups);
  return launch_kernel(attention_tc_tiled_kernel, grid, dim3(kTcThreads), kTlSmemBytes, stream, p);
}

}  // namespace mt
