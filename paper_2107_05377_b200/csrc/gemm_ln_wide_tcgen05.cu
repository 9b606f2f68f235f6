// Residual GEMM fused with the LayerNorm that follows it, on 256-column accumulator tiles:
//
//   Y_g = LN( X_g[M,K] . W_g[N,K]^T + bias_g + residual_g ) * gamma_g + beta_g        N = hidden
//
// A tcgen05.mma over 128 rows occupies the same issue slot whether it is 128 or 256 columns wide, so launches
// with many row blocks (several layers of a wave) want 128 x 256 tiles; the cluster that holds the columns of
// one block of 128 rows then has N / 256 CTAs (3 for N = 768, 4 for 1024).  gemm_ln_tcgen05 (128-column tiles,
// clusters of N / 128) has twice the CTAs per row block and is the better choice when a launch has few row
// blocks.  Both sum over K in one sequence and define the row statistics over the same 64-column segments with
// the same additions in the same order, so they - and the separate GEMM and LayerNorm launches - give identical
// bits, and the choice between them may depend on the size of a launch.
//
// Epilogue (eight warps; a thread owns one row and 128 of its CTA's 256 columns, as two segments of 64):
//   pass 1, per segment: accumulator (tcgen05.ld) + bias + fp32 residual -> x; mean and centred sum of squares
//           of the 64 values.  The residual of the first segment is read into registers while the MMAs run, that
//           of the second arrives by TMA in the warp's staging buffers.  x of the first segment is written back
//           over the accumulator (tcgen05.st), x of the second stays in registers;
//   the two (mean, M2) pairs go into slots of EVERY CTA of the cluster (st.async, counted on the receiver's
//           mbarrier: no fence, no arrival); after the wait the 2 N / 128 pairs of the row are merged in column order;
//   pass 2: the second segment is normalised from registers, the first is read back from tensor memory (which
//           frees the accumulator) and normalised; results leave, bf16 and fp32, through the staging buffers
//           and TMA stores.
// The statistics slots are single buffered: a warp writes the next tile's only after every warp of the cluster
// has reported (second mbarrier, off the critical path) that it has read this tile's.
// Main loop as in gemm_bf16_tcgen05 (TMA producer warp, one MMA thread, accumulator double buffered in tensor
// memory, so the epilogue of a tile overlaps the main loop of the next).  Every wait is bounded.

#include "cluster_ptx.cuh"
#include "rowwise.cuh"

namespace mt {
namespace {

constexpr int kLwEpilogueWarps = 8;
constexpr int kLwThreads = 32 * (2 + kLwEpilogueWarps);
constexpr int kLwTileN = 256;
constexpr int kLwStages = 3;
constexpr int kLwMaxCluster = 4;
constexpr int kLwABytes = kGemmBlockM * kGemmBlockK * 2;    // 16 KB
constexpr int kLwBBytes = kLwTileN * kGemmBlockK * 2;       // 32 KB
constexpr int kLwStagingBytes = 4096;                       // 32 rows x 128 bytes
constexpr int kLwStatsBytes = kLwMaxCluster * 4 * kGemmBlockM * 8;   // [rank][segment of 64][row] float2
constexpr uint32_t kLwTmemCols = 512;                       // two 128 x 256 fp32 accumulators
constexpr int kLwSmemBytes = kLwStages * (kLwABytes + kLwBBytes) + kLwEpilogueWarps * 2 * kLwStagingBytes +
                             kLwStatsBytes + 512 + 1024;
static_assert(kLwSmemBytes <= 227 * 1024, "shared memory of one CTA");

__global__ void __launch_bounds__(kLwThreads, 1) gemm_ln_wide_tcgen05(const __grid_constant__ GemmLnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sA = smem_u32(smem);
  const uint32_t sB = sA + kLwStages * kLwABytes;
  const uint32_t sStage = sB + kLwStages * kLwBBytes;
  uint8_t* stage_ptr = smem + kLwStages * (kLwABytes + kLwBBytes);
  uint8_t* stats_ptr = stage_ptr + kLwEpilogueWarps * 2 * kLwStagingBytes;
  const uint32_t sStats = smem_u32(stats_ptr);
  uint8_t* book = stats_ptr + kLwStatsBytes;
  const uint32_t bar_full = smem_u32(book);                   // kLwStages x 8 bytes
  const uint32_t bar_empty = bar_full + 8 * kLwStages;
  const uint32_t bar_acc_full = bar_empty + 8 * kLwStages;    // 2 x 8 bytes
  const uint32_t bar_acc_empty = bar_acc_full + 16;
  const uint32_t bar_res = bar_acc_empty + 16;                // kLwEpilogueWarps x 8 bytes: the warp's residual box pair
  const uint32_t bar_stats = bar_res + 8 * kLwEpilogueWarps;  // all statistics of the tile are here
  const uint32_t bar_sfree = bar_stats + 8;                   // every warp of the cluster has read them
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(book + 8 * (2 * kLwStages + 4 + kLwEpilogueWarps + 2));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int rank = static_cast<int>(cluster_cta_rank());      // column block (of 256) of this CTA
  const int cluster_size = p.N / kLwTileN;
  const int cluster = static_cast<int>(cluster_id_x());
  const int n_clusters = static_cast<int>(cluster_count_x());
  const int k_blocks = p.K / kGemmBlockK;
  const int n0 = rank * kLwTileN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kLwStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_acc_full + 8 * a, 1);
      mbar_init(bar_acc_empty + 8 * a, kLwEpilogueWarps);
    }
    for (int i = 0; i < kLwEpilogueWarps; ++i) mbar_init(bar_res + 8 * i, 1);
    mbar_init(bar_stats, 1);   // armed per tile by one thread with the bytes of all statistics
    mbar_init(bar_sfree, static_cast<uint32_t>(cluster_size * kLwEpilogueWarps));
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kLwTmemCols);
  tc_fence_before();
  __syncwarp();
  cluster_sync_all();   // the peers' barriers exist before anything can signal them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // rows in use: all M, or fewer when the token layout is packed (a device-side count written by the forward's
  // first kernel).  When this kernel starts, every kernel of the stream but its immediate predecessor has
  // completed (each waits for its own predecessor before it lets its dependents start), and the immediate
  // predecessor is never the one that writes the count: it is read before the dependency wait, off the
  // critical path.
  int m_rows = p.M;
  if (p.m_valid != nullptr) m_rows = min(m_rows, *p.m_valid);

  grid_dependency_wait();
  grid_launch_dependents();
  const int total_tiles = ((m_rows + kGemmBlockM - 1) / kGemmBlockM) * p.n_groups;   // (row block, group) pairs

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    // the warp stays converged (all lanes wait on the barriers); the elected lane issues the copies
    const bool leader = elect_one();
    {
      int stage = 0;
      uint32_t phase = 0;
      long long issued = 0;
      bool ok = true;
      for (int tile = cluster; tile < total_tiles && ok; tile += n_clusters) {
        const int m0 = (tile / p.n_groups) * kGemmBlockM;
        const int g = tile % p.n_groups;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
          if (leader) {
            mbar_expect_tx(bar_full + 8 * stage, kLwABytes + kLwBBytes);
            tma_load_2d(sA + stage * kLwABytes, &p.tmap_x[g], kb * kGemmBlockK, m0, bar_full + 8 * stage);
            tma_load_2d(sB + stage * kLwBBytes, &p.tmap_w256[g], kb * kGemmBlockK, n0, bar_full + 8 * stage);
          }
          ++issued;
          if (++stage == kLwStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok && leader) {
        // aborting: give the copies still in flight the same limit to land before the CTA retires
        int s = stage;
        uint32_t ph = phase;
        const int pending = issued < kLwStages ? static_cast<int>(issued) : kLwStages;
        for (int i = 0; i < pending; ++i) {
          if (s == 0) { s = kLwStages; ph ^= 1u; }
          --s;
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(bar_full + 8 * s, ph)) {
            if (global_timer_ns() - t0 > kWaitLimitNs) break;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------
    // (the same: a converged warp, the elected lane issues the MMAs and the commits)
    const bool leader = elect_one();
    {
      constexpr uint32_t idesc = umma_idesc_bf16(kGemmBlockM, kLwTileN);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = cluster; tile < total_tiles && ok; tile += n_clusters) {
        if (!mbar_wait(bar_acc_empty + 8 * acc, acc_phase ^ 1u, abort_flag)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kLwTileN);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          if (leader) {
            const uint64_t da = smem_desc_sw128(sA + stage * kLwABytes);
            const uint64_t db = smem_desc_sw128(sB + stage * kLwBBytes);
#pragma unroll
            for (int k = 0; k < kGemmBlockK / 16; ++k)
              umma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
            umma_commit(bar_empty + 8 * stage);
          }
          if (++stage == kLwStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (leader) umma_commit(bar_acc_full + 8 * acc);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------ epilogue ----------------------------------
    const int e = warp - 2;
    const int quarter = warp & 3;     // TMEM lanes this warp may read: rows quarter * 32 .. + 31 of the tile
    const int half = e >> 2;          // which 128 of the CTA's 256 columns
    const int row_in_tile = quarter * 32 + lane;
    const uint32_t my_stage = sStage + static_cast<uint32_t>(e * 2 * kLwStagingBytes);
    uint8_t* my_stage_ptr = stage_ptr + e * 2 * kLwStagingBytes;
    const uint32_t my_res_bar = bar_res + 8 * e;
    const float inv_n = 1.0f / static_cast<float>(p.N);
    int acc = 0;
    uint32_t acc_phase = 0, res_phase = 0, s_phase = 0;

    // x = residual + (accumulator + bias) for 8 columns: the order of the plain residual epilogue
    auto combine8 = [](float* x, const float4& r0, const float4& r1, const uint4& b) {
      const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
      x[0] = r0.x + (x[0] + bf16_lo(bw[0]));
      x[1] = r0.y + (x[1] + bf16_hi(bw[0]));
      x[2] = r0.z + (x[2] + bf16_lo(bw[1]));
      x[3] = r0.w + (x[3] + bf16_hi(bw[1]));
      x[4] = r1.x + (x[4] + bf16_lo(bw[2]));
      x[5] = r1.y + (x[5] + bf16_hi(bw[2]));
      x[6] = r1.z + (x[6] + bf16_lo(bw[3]));
      x[7] = r1.w + (x[7] + bf16_hi(bw[3]));
    };
    // mean and centred sum of squares of a segment of 64 values, with the additions of the row-wise LayerNorm
    // kernel (eight sums of 8 in order, then a balanced tree)
    auto segment_stats = [](const float* v, float* mean_out, float* m2_out) {
      float sub[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) sub[j] = sum8_in_order(*reinterpret_cast<const float(*)[8]>(v + 8 * j));
      const float mean_l = (((sub[0] + sub[1]) + (sub[2] + sub[3])) + ((sub[4] + sub[5]) + (sub[6] + sub[7]))) * (1.0f / 64.0f);
#pragma unroll
      for (int j = 0; j < 8; ++j) sub[j] = sumsq8_in_order(*reinterpret_cast<const float(*)[8]>(v + 8 * j), mean_l);
      *mean_out = mean_l;
      *m2_out = ((sub[0] + sub[1]) + (sub[2] + sub[3])) + ((sub[4] + sub[5]) + (sub[6] + sub[7]));
    };

    for (int tile = cluster; tile < total_tiles; tile += n_clusters) {
      const int m0 = (tile / p.n_groups) * kGemmBlockM;
      const int g = tile % p.n_groups;
      const int row0 = m0 + quarter * 32;
      const int col0 = n0 + half * 128;       // first of this thread's 128 columns
      const bool rows_in_range = row0 < m_rows;
      if (lane == 0) {
        tma_store_wait_read<0>();   // the previous tile's stores have read the staging buffers
        // the residual of the SECOND segment (32 rows x 64 columns) by TMA into the two staging buffers
        mbar_expect_tx(my_res_bar, 2 * kLwStagingBytes);
        tma_load_2d(my_stage, &p.tmap_res[g], col0 + 64, row0, my_res_bar);
        tma_load_2d(my_stage + kLwStagingBytes, &p.tmap_res[g], col0 + 96, row0, my_res_bar);
        // this tile's statistics: (one thread of the CTA) the bytes of all segments of the 128 rows
        if (e == 0) mbar_expect_tx(bar_stats, static_cast<uint32_t>(cluster_size * 4 * kGemmBlockM * 8));
      }
      // the residual of the FIRST segment into registers, while the MMAs run (rows past the buffer read as zero)
      float v[64];
      {
        const int row = row0 + lane;
        if (row < p.M) {
          const float4* src = reinterpret_cast<const float4*>(p.residual[g] + static_cast<size_t>(row) * p.N + col0);
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const float4 t = __ldg(src + c);
            v[4 * c] = t.x; v[4 * c + 1] = t.y; v[4 * c + 2] = t.z; v[4 * c + 3] = t.w;
          }
        } else {
#pragma unroll
          for (int c = 0; c < 64; ++c) v[c] = 0.f;
        }
      }
      if (lane < 6) {   // bias, gamma and beta of this thread's columns (two 128-byte lines each) into L1
        const bf16* line = (lane < 2 ? p.bias[g] : (lane < 4 ? p.gamma[g] : p.beta[g])) + col0 + (lane & 1) * 64;
        asm volatile("prefetch.global.L1 [%0];" ::"l"(line));
      }
      if (!__all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8 * acc, acc_phase, abort_flag))) break;
      tc_fence_after();
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                             static_cast<uint32_t>(acc * kLwTileN + half * 128);
      float mean_s[2], m2_s[2];
      // ---- pass 1, first segment: x = residual (registers) + (accumulator + bias), written back over the accumulator
      {
        const bf16* bias = p.bias[g] + col0;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          uint32_t r[32];
          tmem_ld_32x32(t_row + hh * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint4 b = __ldg(reinterpret_cast<const uint4*>(bias + hh * 32) + q);
            float* x = v + hh * 32 + q * 8;
            const float4 r0 = make_float4(x[0], x[1], x[2], x[3]);
            const float4 r1 = make_float4(x[4], x[5], x[6], x[7]);
#pragma unroll
            for (int i = 0; i < 8; ++i) x[i] = __uint_as_float(r[q * 8 + i]);
            combine8(x, r0, r1, b);
#pragma unroll
            for (int i = 0; i < 8; ++i) r[q * 8 + i] = __float_as_uint(x[i]);
          }
          tmem_st_32x32(t_row + hh * 32, r);
        }
        segment_stats(v, &mean_s[0], &m2_s[0]);
        tmem_st_wait();
      }
      // ---- pass 1, second segment: residual from the staging buffers; x stays in registers
      if (!__all_sync(0xffffffffu, mbar_wait(my_res_bar, res_phase, abort_flag))) break;
      res_phase ^= 1u;
      {
        const bf16* bias = p.bias[g] + col0 + 64;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          uint32_t r[32];
          tmem_ld_32x32(t_row + 64 + hh * 32, r);
          tmem_ld_wait();
          const uint8_t* sbuf = my_stage_ptr + hh * kLwStagingBytes;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint4 b = __ldg(reinterpret_cast<const uint4*>(bias + hh * 32) + q);
            const float4 r0 = *reinterpret_cast<const float4*>(sbuf + staging_off(lane, 2 * q));
            const float4 r1 = *reinterpret_cast<const float4*>(sbuf + staging_off(lane, 2 * q + 1));
            float* x = v + hh * 32 + q * 8;
#pragma unroll
            for (int i = 0; i < 8; ++i) x[i] = __uint_as_float(r[q * 8 + i]);
            combine8(x, r0, r1, b);
          }
        }
        segment_stats(v, &mean_s[1], &m2_s[1]);
      }
      __syncwarp();   // every lane has read the residual: the staging buffers now serve the stores
      // every warp of the cluster has read the previous tile's statistics
      if (!__all_sync(0xffffffffu, mbar_wait_cluster(bar_sfree, s_phase ^ 1u, abort_flag))) break;
      // into slots [rank][segment][row] of every CTA of the cluster, counted on that CTA's barrier
#pragma unroll
      for (int sgm = 0; sgm < 2; ++sgm) {
        const uint32_t slot = sStats + static_cast<uint32_t>(((rank * 4 + half * 2 + sgm) * kGemmBlockM + row_in_tile) * 8);
        for (int peer = 0; peer < cluster_size; ++peer)
          st_async_f2(map_to_cta(slot, static_cast<uint32_t>(peer)), mean_s[sgm], m2_s[sgm],
                      map_to_cta(bar_stats, static_cast<uint32_t>(peer)));
      }
      if (!__all_sync(0xffffffffu, mbar_wait_cluster(bar_stats, s_phase, abort_flag))) break;
      s_phase ^= 1u;
      // merge the 4 * cluster_size segment statistics of this row, in column order
      float mean, rstd;
      {
        const uint8_t* base = stats_ptr + row_in_tile * 8;
        if (cluster_size == 3) {
          float sm[12], sq[12];
#pragma unroll
          for (int i = 0; i < 12; ++i) {
            const float2 part = *reinterpret_cast<const float2*>(base + i * kGemmBlockM * 8);
            sm[i] = part.x; sq[i] = part.y;
          }
          merge_segments<12>(sm, sq, inv_n, p.eps, &mean, &rstd);
        } else {
          float sm[16], sq[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float2 part = *reinterpret_cast<const float2*>(base + i * kGemmBlockM * 8);
            sm[i] = part.x; sq[i] = part.y;
          }
          merge_segments<16>(sm, sq, inv_n, p.eps, &mean, &rstd);
        }
      }

      // ---- pass 2: normalise and store, the second segment (in registers) first, then the first (read back)
      uint8_t* buf0 = my_stage_ptr;
      uint8_t* buf1 = my_stage_ptr + kLwStagingBytes;
#pragma unroll 1
      for (int sgm = 1; sgm >= 0; --sgm) {
        const int colS = col0 + sgm * 64;
        if (sgm == 0) {
          // x of the first segment back from tensor memory; after this the MMA thread may reuse the accumulator
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            uint32_t r[32];
            tmem_ld_32x32(t_row + hh * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) v[hh * 32 + i] = __uint_as_float(r[i]);
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(bar_acc_empty + 8 * acc);
            tma_store_wait_read<0>();   // the second segment's stores have read the staging buffers
          }
          __syncwarp();
        }
        const bf16* gamma = p.gamma[g] + colS;
        const bf16* beta = p.beta[g] + colS;
        // bf16 copy of all 64 columns -> buffer 0, fp32 of the first 32 -> buffer 1, stores; then fp32 of the
        // other 32 -> buffer 0 once the bf16 store has read it
#pragma unroll
        for (int c = 0; c < 8; ++c) {   // 8 columns at a time
          const uint4 gq = __ldg(reinterpret_cast<const uint4*>(gamma) + c);
          const uint4 bq = __ldg(reinterpret_cast<const uint4*>(beta) + c);
          const uint32_t gw[4] = {gq.x, gq.y, gq.z, gq.w};
          const uint32_t bw[4] = {bq.x, bq.y, bq.z, bq.w};
          float* x = v + c * 8;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            x[2 * j] = fmaf(__fmul_rn(x[2 * j] - mean, rstd), bf16_lo(gw[j]), bf16_lo(bw[j]));
            x[2 * j + 1] = fmaf(__fmul_rn(x[2 * j + 1] - mean, rstd), bf16_hi(gw[j]), bf16_hi(bw[j]));
          }
          *reinterpret_cast<uint4*>(buf0 + staging_off(lane, c)) =
              make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]), pack_bf16(x[6], x[7]));
          if (c < 4) {
            *reinterpret_cast<float4*>(buf1 + staging_off(lane, 2 * c)) = make_float4(x[0], x[1], x[2], x[3]);
            *reinterpret_cast<float4*>(buf1 + staging_off(lane, 2 * c + 1)) = make_float4(x[4], x[5], x[6], x[7]);
          }
        }
        fence_async_shared();
        __syncwarp();
        if (lane == 0) {
          if (rows_in_range) {
            tma_store_2d(&p.tmap_y[g], my_stage, colS, row0);
            tma_store_2d(&p.tmap_y32[g], my_stage + kLwStagingBytes, colS, row0);
          }
          tma_store_commit();
          tma_store_wait_read<0>();
        }
        __syncwarp();
#pragma unroll
        for (int c = 4; c < 8; ++c) {
          const float* x = v + c * 8;
          *reinterpret_cast<float4*>(buf0 + staging_off(lane, 2 * (c - 4))) = make_float4(x[0], x[1], x[2], x[3]);
          *reinterpret_cast<float4*>(buf0 + staging_off(lane, 2 * (c - 4) + 1)) = make_float4(x[4], x[5], x[6], x[7]);
        }
        fence_async_shared();
        __syncwarp();
        if (lane == 0) {
          if (rows_in_range) tma_store_2d(&p.tmap_y32[g], my_stage, colS + 32, row0);
          tma_store_commit();
        }
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      if (lane == 0) {
        // (off the critical path) the statistics slots may be overwritten once every warp of the cluster has said
        // that it has read them: one release fence, then an arrival on every CTA's barrier
        fence_acq_rel_cluster();
        for (int peer = 0; peer < cluster_size; ++peer)
          mbar_arrive_cluster_relaxed(map_to_cta(bar_sfree, static_cast<uint32_t>(peer)));
      }
    }
    if (lane == 0) tma_store_wait_read<0>();   // shared memory must outlive the stores that still read it
    __syncwarp();
  }

  // ------------------------------ teardown ------------------------------------
  // No CTA may retire while a peer can still write its statistics slots or signal its barriers: every
  // thread of every CTA of the cluster gets here (all waits above are bounded).
  tc_fence_before();
  __syncwarp();
  cluster_sync_all();
  if (threadIdx.x == 0 && *abort_flag && p.status != nullptr) atomicOr(p.status, kFlagWaitTimeout);
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, kLwTmemCols);
  }
}

}  // namespace

bool gemm_ln_wide_supported(int N) { return N == 768 || N == 1024; }

cudaError_t launch_gemm_ln_wide(const GemmLnParams& p, cudaStream_t stream) {
  if (p.n_groups < 1 || p.n_groups > kMaxGroups || !gemm_ln_wide_supported(p.N) || p.K % kGemmBlockK != 0 ||
      p.K < kGemmBlockK || p.M < 1)
    return cudaErrorInvalidValue;
  const int cluster_size = p.N / kLwTileN;
  // per device: shared-memory opt-in and, per cluster size, the number of clusters that fit the GPU at once
  static PerDeviceOnce once;
  static int max_clusters[kMaxDevices][2] = {};
  int dev = 0;
  cudaError_t err = per_device_once(once, [&](int d) {
    cudaError_t r = cudaFuncSetAttribute(gemm_ln_wide_tcgen05, cudaFuncAttributeMaxDynamicSharedMemorySize, kLwSmemBytes);
    if (r != cudaSuccess) return r;
    for (int which = 0; which < 2; ++which) {
      const int cs = which == 0 ? 3 : 4;
      cudaLaunchConfig_t q = {};
      q.gridDim = dim3(cs * 64);
      q.blockDim = dim3(kLwThreads);
      q.dynamicSmemBytes = kLwSmemBytes;
      cudaLaunchAttribute a[1];
      a[0].id = cudaLaunchAttributeClusterDimension;
      a[0].val.clusterDim.x = cs;
      a[0].val.clusterDim.y = 1;
      a[0].val.clusterDim.z = 1;
      q.attrs = a;
      q.numAttrs = 1;
      int n = 0;
      r = cudaOccupancyMaxActiveClusters(&n, gemm_ln_wide_tcgen05, &q);
      if (r != cudaSuccess) return r;
      max_clusters[d][which] = n;
    }
    return cudaSuccess;
  }, &dev);
  if (err != cudaSuccess) return err;
  const int fit = max_clusters[dev][cluster_size == 4 ? 1 : 0];
  if (fit < 1) return cudaErrorLaunchOutOfResources;
  const int tiles = ((p.M + kGemmBlockM - 1) / kGemmBlockM) * p.n_groups;
  const int clusters = tiles < fit ? tiles : fit;
  return launch_kernel(gemm_ln_wide_tcgen05, dim3(clusters * cluster_size), dim3(kLwThreads), kLwSmemBytes, stream, p,
                       static_cast<unsigned>(cluster_size));
}

}  // namespace mt
