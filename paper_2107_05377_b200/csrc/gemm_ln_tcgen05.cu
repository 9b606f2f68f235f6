// Residual GEMM fused with the LayerNorm that follows it (the attention-output projection with the first
// LayerNorm of the layer, the FFN-down projection with the second):
//
//   Y_g = LN( X_g[M,K] . W_g[N,K]^T + bias_g + residual_g ) * gamma_g + beta_g        N = hidden
//
// LayerNorm needs whole rows, a CTA holds 128 of the N columns (one tcgen05 accumulator, 128 x 128,
// double buffered in tensor memory).  So the N / 128 CTAs that hold the column blocks of the same 128
// rows are launched as one thread-block cluster (6 CTAs for N = 768, 8 for 1024) and exchange per-row
// partial statistics through distributed shared memory:
//   * every epilogue thread owns one row and 64 of its CTA's columns; it adds bias and the fp32 residual
//     (fetched by TMA while the MMAs run) to the accumulator, keeps the 64 sums in registers, and
//     computes their mean and centred sum of squares;
//   * it stores that pair into a slot of EVERY CTA of the cluster (st.shared::cluster), and each warp
//     then arrives (release, cluster scope) on every CTA's "statistics full" mbarrier;
//   * after the wait, the 2 N / 128 pairs of a row are merged in column order (equal counts:
//     mean = average of the means, M2 = sum of M2_i + 64 (mean_i - mean)^2), the thread normalises
//     its 64 values and the results leave, bf16 and fp32, through swizzled staging and TMA stores.
// The row-wise LayerNorm kernel defines its statistics over the same 64-column segments with the same
// additions in the same order, so this launch and the separate GEMM and LayerNorm launches give
// identical bits, and the choice between them may depend on the size of a launch.
// The pre-normalisation sum never goes to global memory and no LayerNorm launch follows.  The statistics
// are double buffered by tile parity: a CTA can be at most one tile ahead of a peer, because its next
// "statistics full" needs that peer's arrival.
//
// The main loop is that of gemm_bf16_tcgen05: warp 0 streams 128 x 64 X tiles and 128 x 64 W tiles by
// TMA into a ring of stages, one thread of warp 1 issues tcgen05.mma 128 x 128 x 16, eight epilogue
// warps.  A cluster walks over the (row block, group) pairs; clusters do not wait for one another.
// Every wait is bounded (mbarrier waits by %globaltimer): when one runs out the CTA raises its abort
// flag and the status word, all roles leave their loops, the peers' waits run out in turn, and every
// CTA reaches the closing cluster barrier, after which tensor memory is freed.

#include "cluster_ptx.cuh"
#include "rowwise.cuh"

namespace mt {
namespace {

constexpr int kLnEpilogueWarps = 8;
constexpr int kLnThreads = 32 * (2 + kLnEpilogueWarps);
constexpr int kLnBlockN = 128;
constexpr int kLnStages = 4;
constexpr int kLnMaxCluster = 8;
constexpr int kLnABytes = kGemmBlockM * kGemmBlockK * 2;   // 16 KB
constexpr int kLnBBytes = kLnBlockN * kGemmBlockK * 2;     // 16 KB
constexpr int kLnStagingBytes = 4096;                      // 32 rows x 128 bytes
constexpr int kLnStatsBytes = 2 * kLnMaxCluster * 2 * kGemmBlockM * 8;   // [parity][rank][half][row] float2
constexpr uint32_t kLnTmemCols = 256;
constexpr int kLnSmemBytes = kLnStages * (kLnABytes + kLnBBytes) + kLnEpilogueWarps * 2 * kLnStagingBytes +
                             kLnStatsBytes + 512 + 1024;

__global__ void __launch_bounds__(kLnThreads, 1) gemm_ln_tcgen05(const __grid_constant__ GemmLnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sA = smem_u32(smem);
  const uint32_t sB = sA + kLnStages * kLnABytes;
  const uint32_t sStage = sB + kLnStages * kLnBBytes;
  uint8_t* stage_ptr = smem + kLnStages * (kLnABytes + kLnBBytes);
  uint8_t* stats_ptr = stage_ptr + kLnEpilogueWarps * 2 * kLnStagingBytes;
  const uint32_t sStats = smem_u32(stats_ptr);
  uint8_t* book = stats_ptr + kLnStatsBytes;
  const uint32_t bar_full = smem_u32(book);                   // kLnStages x 8 bytes
  const uint32_t bar_empty = bar_full + 8 * kLnStages;
  const uint32_t bar_acc_full = bar_empty + 8 * kLnStages;    // 2 x 8 bytes
  const uint32_t bar_acc_empty = bar_acc_full + 16;
  const uint32_t bar_res = bar_acc_empty + 16;                // kLnEpilogueWarps x 2 x 8 bytes
  const uint32_t bar_stats = bar_res + 16 * kLnEpilogueWarps; // 2 x 8 bytes: statistics of a tile parity are all there
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(book + 8 * (2 * kLnStages + 4 + 2 * kLnEpilogueWarps + 2));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int rank = static_cast<int>(cluster_cta_rank());      // column block of this CTA
  const int cluster_size = p.N / kLnBlockN;
  const int cluster = static_cast<int>(cluster_id_x());
  const int n_clusters = static_cast<int>(cluster_count_x());
  const int k_blocks = p.K / kGemmBlockK;
  const int n0 = rank * kLnBlockN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kLnStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_acc_full + 8 * a, 1);
      mbar_init(bar_acc_empty + 8 * a, kLnEpilogueWarps);
      mbar_init(bar_stats + 8 * a, 1);   // armed per tile by one thread with the bytes of all statistics
    }
    for (int i = 0; i < 2 * kLnEpilogueWarps; ++i) mbar_init(bar_res + 8 * i, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kLnTmemCols);
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
            mbar_expect_tx(bar_full + 8 * stage, kLnABytes + kLnBBytes);
            tma_load_2d(sA + stage * kLnABytes, &p.tmap_x[g], kb * kGemmBlockK, m0, bar_full + 8 * stage);
            tma_load_2d(sB + stage * kLnBBytes, &p.tmap_w[g], kb * kGemmBlockK, n0, bar_full + 8 * stage);
          }
          ++issued;
          if (++stage == kLnStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok && leader) {
        // aborting: give the copies still in flight the same limit to land before the CTA retires
        int s = stage;
        uint32_t ph = phase;
        const int pending = issued < kLnStages ? static_cast<int>(issued) : kLnStages;
        for (int i = 0; i < pending; ++i) {
          if (s == 0) { s = kLnStages; ph ^= 1u; }
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
      constexpr uint32_t idesc = umma_idesc_bf16(kGemmBlockM, kLnBlockN);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = cluster; tile < total_tiles && ok; tile += n_clusters) {
        if (!mbar_wait(bar_acc_empty + 8 * acc, acc_phase ^ 1u, abort_flag)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kLnBlockN);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          if (leader) {
            const uint64_t da = smem_desc_sw128(sA + stage * kLnABytes);
            const uint64_t db = smem_desc_sw128(sB + stage * kLnBBytes);
#pragma unroll
            for (int k = 0; k < kGemmBlockK / 16; ++k)
              umma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
            umma_commit(bar_empty + 8 * stage);
          }
          if (++stage == kLnStages) { stage = 0; phase ^= 1u; }
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
    const int half = e >> 2;          // which 64 of the CTA's 128 columns
    const int row_in_tile = quarter * 32 + lane;
    const uint32_t my_stage = sStage + static_cast<uint32_t>(e * 2 * kLnStagingBytes);
    uint8_t* my_stage_ptr = stage_ptr + e * 2 * kLnStagingBytes;
    const uint32_t my_res_bar = bar_res + 16 * e;
    const float inv_n = 1.0f / static_cast<float>(p.N);
    int acc = 0;
    uint32_t acc_phase = 0;
    uint32_t res_phase = 0;           // both residual barriers complete once per tile
    uint32_t stats_phase[2] = {0, 0};
    int parity = 0;                   // statistics buffer of this tile

    for (int tile = cluster; tile < total_tiles; tile += n_clusters) {
      const int m0 = (tile / p.n_groups) * kGemmBlockM;
      const int g = tile % p.n_groups;
      const int row0 = m0 + quarter * 32;
      const int col0 = n0 + half * 64;
      // the residual of this warp's 32 x 64 block, while the MMAs run
      if (lane == 0) {
        // (one thread of the CTA) this tile's statistics: 8 bytes from every epilogue thread of the cluster
        if (e == 0) mbar_expect_tx(bar_stats + 8 * parity, static_cast<uint32_t>(cluster_size * kLnEpilogueWarps * 32 * 8));
        tma_store_wait_read<0>();   // the previous tile's stores have read the staging buffers
        mbar_expect_tx(my_res_bar, kLnStagingBytes);
        tma_load_2d(my_stage, &p.tmap_res[g], col0, row0, my_res_bar);
        mbar_expect_tx(my_res_bar + 8, kLnStagingBytes);
        tma_load_2d(my_stage + kLnStagingBytes, &p.tmap_res[g], col0 + 32, row0, my_res_bar + 8);
      }
      // this warp's 64 columns of bias, gamma and beta (128 bytes each) into L1 ahead of their use
      if (lane < 3) {
        const bf16* line = (lane == 0 ? p.bias[g] : (lane == 1 ? p.gamma[g] : p.beta[g])) + col0;
        asm volatile("prefetch.global.L1 [%0];" ::"l"(line));
      }
      if (!__all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8 * acc, acc_phase, abort_flag))) break;
      tc_fence_after();
      float v[64];
      {
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                               static_cast<uint32_t>(acc * kLnBlockN + half * 64);
        uint32_t r[32];
        tmem_ld_32x32(taddr, r);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
        tmem_ld_32x32(taddr + 32, r);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) v[32 + i] = __uint_as_float(r[i]);
      }
      // the accumulator is in registers: the MMA thread may reuse it
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_acc_empty + 8 * acc);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }

      bool res_ok = mbar_wait(my_res_bar, res_phase, abort_flag);
      res_ok = mbar_wait(my_res_bar + 8, res_phase, abort_flag) && res_ok;
      if (!__all_sync(0xffffffffu, res_ok)) break;
      res_phase ^= 1u;
      const bf16* bias = p.bias[g] + col0;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint8_t* sbuf = my_stage_ptr + h * kLnStagingBytes;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint4 b = __ldg(reinterpret_cast<const uint4*>(bias + h * 32) + q);
          const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
          const float4 r0 = *reinterpret_cast<const float4*>(sbuf + staging_off(lane, 2 * q));
          const float4 r1 = *reinterpret_cast<const float4*>(sbuf + staging_off(lane, 2 * q + 1));
          float* x = v + h * 32 + q * 8;
          // residual + (accumulator + bias): the order of the plain residual epilogue
          x[0] = r0.x + (x[0] + bf16_lo(bw[0]));
          x[1] = r0.y + (x[1] + bf16_hi(bw[0]));
          x[2] = r0.z + (x[2] + bf16_lo(bw[1]));
          x[3] = r0.w + (x[3] + bf16_hi(bw[1]));
          x[4] = r1.x + (x[4] + bf16_lo(bw[2]));
          x[5] = r1.y + (x[5] + bf16_hi(bw[2]));
          x[6] = r1.z + (x[6] + bf16_lo(bw[3]));
          x[7] = r1.w + (x[7] + bf16_hi(bw[3]));
        }
      }
      // this thread's segment of 64 values: mean and centred sum of squares, with the additions of the
      // row-wise LayerNorm kernel (eight sums of 8 in order, then a balanced tree)
      float mean_l, m2_l;
      {
        float sub[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) sub[j] = sum8_in_order(*reinterpret_cast<const float(*)[8]>(v + 8 * j));
        mean_l = (((sub[0] + sub[1]) + (sub[2] + sub[3])) + ((sub[4] + sub[5]) + (sub[6] + sub[7]))) * (1.0f / 64.0f);
#pragma unroll
        for (int j = 0; j < 8; ++j) sub[j] = sumsq8_in_order(*reinterpret_cast<const float(*)[8]>(v + 8 * j), mean_l);
        m2_l = ((sub[0] + sub[1]) + (sub[2] + sub[3])) + ((sub[4] + sub[5]) + (sub[6] + sub[7]));
      }
      // into slot [parity][rank][half][row] of every CTA of the cluster
      const uint32_t slot = sStats + static_cast<uint32_t>((((parity * kLnMaxCluster + rank) * 2 + half) * kGemmBlockM + row_in_tile) * 8);
      // (asynchronous stores that count their bytes on the receiver's barrier: its wait is all the synchronisation)
      for (int peer = 0; peer < cluster_size; ++peer)
        st_async_f2(map_to_cta(slot, static_cast<uint32_t>(peer)), mean_l, m2_l,
                    map_to_cta(bar_stats + 8 * parity, static_cast<uint32_t>(peer)));
      if (!__all_sync(0xffffffffu, mbar_wait_cluster(bar_stats + 8 * parity, stats_phase[parity], abort_flag))) break;
      stats_phase[parity] ^= 1u;
      // merge the 2 * cluster_size segment statistics of this row, in column order
      float mean, rstd;
      {
        const uint8_t* base = stats_ptr + static_cast<size_t>(parity) * kLnMaxCluster * 2 * kGemmBlockM * 8 + row_in_tile * 8;
        if (cluster_size == 6) {
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
      parity ^= 1;

      // normalise; bf16 copy of all 64 columns -> buffer 0, fp32 of the first 32 -> buffer 1, stores;
      // then fp32 of the other 32 -> buffer 0 once the bf16 store has read it
      const bf16* gamma = p.gamma[g] + col0;
      const bf16* beta = p.beta[g] + col0;
      const bool rows_in_range = row0 < m_rows;
      uint8_t* buf0 = my_stage_ptr;
      uint8_t* buf1 = my_stage_ptr + kLnStagingBytes;
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
          tma_store_2d(&p.tmap_y[g], my_stage, col0, row0);
          tma_store_2d(&p.tmap_y32[g], my_stage + kLnStagingBytes, col0, row0);
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
        if (rows_in_range) tma_store_2d(&p.tmap_y32[g], my_stage, col0 + 32, row0);
        tma_store_commit();
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
    tmem_dealloc(tmem_base, kLnTmemCols);
  }
}

}  // namespace

bool gemm_ln_supported(int N) { return N == 768 || N == 1024; }

cudaError_t launch_gemm_ln(const GemmLnParams& p, cudaStream_t stream) {
  if (p.n_groups < 1 || p.n_groups > kMaxGroups || !gemm_ln_supported(p.N) || p.K % kGemmBlockK != 0 || p.K < kGemmBlockK ||
      p.M < 1)
    return cudaErrorInvalidValue;
  const int cluster_size = p.N / kLnBlockN;
  // per device: shared-memory opt-in and, per cluster size, the number of clusters that fit the GPU at once
  static PerDeviceOnce once;
  static int max_clusters[kMaxDevices][2] = {};
  int dev = 0;
  cudaError_t err = per_device_once(once, [&](int d) {
    cudaError_t r = cudaFuncSetAttribute(gemm_ln_tcgen05, cudaFuncAttributeMaxDynamicSharedMemorySize, kLnSmemBytes);
    if (r != cudaSuccess) return r;
    for (int which = 0; which < 2; ++which) {
      const int cs = which == 0 ? 6 : 8;
      cudaLaunchConfig_t q = {};
      q.gridDim = dim3(cs * 64);
      q.blockDim = dim3(kLnThreads);
      q.dynamicSmemBytes = kLnSmemBytes;
      cudaLaunchAttribute a[1];
      a[0].id = cudaLaunchAttributeClusterDimension;
      a[0].val.clusterDim.x = cs;
      a[0].val.clusterDim.y = 1;
      a[0].val.clusterDim.z = 1;
      q.attrs = a;
      q.numAttrs = 1;
      int n = 0;
      r = cudaOccupancyMaxActiveClusters(&n, gemm_ln_tcgen05, &q);
      if (r != cudaSuccess) return r;
      max_clusters[d][which] = n;
    }
    return cudaSuccess;
  }, &dev);
  if (err != cudaSuccess) return err;
  const int fit = max_clusters[dev][cluster_size == 8 ? 1 : 0];
  if (fit < 1) return cudaErrorLaunchOutOfResources;
  const int tiles = ((p.M + kGemmBlockM - 1) / kGemmBlockM) * p.n_groups;
  const int clusters = tiles < fit ? tiles : fit;
  return launch_kernel(gemm_ln_tcgen05, dim3(clusters * cluster_size), dim3(kLnThreads), kLnSmemBytes, stream, p,
                       static_cast<unsigned>(cluster_size));
}

}  // namespace mt
