// Grouped bf16 GEMM on the 5th-generation tensor cores (tcgen05) of sm_100a.
//
//   Y_g[M,N] = epilogue( X_g[M,K] . W_g[N,K]^T + bias_g )        g = 0 .. n_groups-1
//
// These are the linear maps of the encoder layer (QKV, attention output, FFN up, FFN down).
// The layers that are ready in the same wave of the task tree (the trunk layer and the branch
// layers of several tasks) are the groups of ONE launch, so their tiles fill the machine together.
//
// One persistent CTA per SM walks over the tiles (128 x BN) of all groups.  Warp roles:
//   warp 0      : TMA producer - streams 128x64 X tiles and BNx64 W tiles (128-byte swizzle) into
//                 a ring of shared-memory stages, signalling "full" mbarriers by transaction count
//   warp 1      : allocates tensor memory; one thread issues tcgen05.mma (128 x BN x 16 per
//                 instruction) with the accumulator in TMEM, and tcgen05.commit to release stages
//   warps 2..   : epilogue - tcgen05.ld the fp32 accumulator (each warp its own 32-lane quarter),
//                 add bias (+GELU) and round once to bf16, or add bias + fp32 residual and keep
//                 fp32.  Each warp owns small 128-byte-swizzled staging buffers in shared memory:
//                 results leave through TMA stores (and the fp32 residual arrives through TMA
//                 loads, prefetched one chunk ahead), so every global access is a full 128-byte
//                 row segment and no epilogue thread ever waits on a global load
// The accumulator is double buffered in TMEM (2 x BN columns) so the epilogue of tile i overlaps
// the MMAs of tile i+1.  Every output element is the sum over K in a fixed order inside a single
// tile, so a result never depends on which other groups share the launch.
//
// Every mbarrier wait is bounded: after kWaitLimitNs the waiting thread raises the CTA's abort
// flag, the status word gets kFlagWaitTimeout, all roles leave their loops, the producer drains
// the copies it still has in flight, TMEM is freed and the CTA returns.

#include "tc_ptx.cuh"

namespace mt {
namespace {

constexpr int kNumEpilogueWarps = 8;
constexpr int kGemmThreads = 32 * (2 + kNumEpilogueWarps);

constexpr int kStagingBytes = 4096;  // 32 rows x 128 bytes, one epilogue chunk of one warp
// Shared memory of a CTA: the ring of operand stages, the epilogue warps' staging buffers, bookkeeping.
// The ring is what bounds a CTA's throughput (bytes in flight over the load latency), so it gets all the
// room the staging leaves.  The residual epilogue prefetches its fp32 residual chunk while it works on
// the previous one and needs two staging buffers per warp; the other epilogues take one or two
// (MT_GEMM_NBUF) - with one, a warp waits for its last store to have read the buffer before refilling it.
#ifndef MT_GEMM_NBUF
#define MT_GEMM_NBUF 2
#endif
constexpr int kSmemLimit = 227 * 1024;
constexpr int kBookBytes = 512 + 1024;   // barriers/bookkeeping + slack for manual 1024-byte alignment
__host__ __device__ constexpr int gemm_a_bytes() { return kGemmBlockM * kGemmBlockK * 2; }
// A CTA of a pair stages only its half of the W tile.
__host__ __device__ constexpr int gemm_b_bytes(int bn, bool pair) { return (pair ? bn / 2 : bn) * kGemmBlockK * 2; }
__host__ __device__ constexpr int gemm_staging_bufs(int bn, bool pair, int epi) {
  return epi == kEpiBiasResidual ? 2 : ((bn == 256 && !pair) ? 1 : MT_GEMM_NBUF);
}
__host__ __device__ constexpr int gemm_stages(int bn, bool pair, int epi) {
  const int room = kSmemLimit - kBookBytes - kNumEpilogueWarps * gemm_staging_bufs(bn, pair, epi) * kStagingBytes;
  const int s = room / (gemm_a_bytes() + gemm_b_bytes(bn, pair));
  return s > 8 ? 8 : s;
}
__host__ __device__ constexpr int gemm_smem_bytes(int bn, bool pair, int epi) {
  return gemm_stages(bn, pair, epi) * (gemm_a_bytes() + gemm_b_bytes(bn, pair)) +
         kNumEpilogueWarps * gemm_staging_bufs(bn, pair, epi) * kStagingBytes + kBookBytes;
}

// ---- the kernel -------------------------------------------------------------------------------

// PAIR: the kernel runs as clusters of two CTAs that share 256 x BN tiles (tcgen05 cta_group::2).
// CTA `rank` of a pair owns rows rank*128.. of the tile (its A rows, its accumulator, its epilogue)
// and stages half of the W tile; the MMA, issued by rank 0, reads both halves.  Per 128 x BN x 64
// of tensor work a CTA then pulls 16 KB + BN/2 x 128 B from L2 instead of 16 KB + BN x 128 B, which
// is what bounds the single-CTA kernel (an SM takes in roughly 64 bytes per clock).
// FP8: the operands are E4M3 bytes with one fp32 scale per row of X and per row of W (GemmParams::scale_x,
// scale_w); a shared-memory row of 128 bytes then holds 128 elements of K, an instruction covers 32 of them,
// and the epilogue multiplies the accumulator by scale_x[row] * scale_w[column] before the bias.
template <int BN, int EPI, bool PAIR, bool FP8 = false>
__global__ void __launch_bounds__(kGemmThreads, 1) gemm_bf16_tcgen05(const __grid_constant__ GemmParams p) {
  static_assert(!FP8 || !PAIR, "the 8-bit operands run as single CTAs");
  constexpr int KB_ELEMS = FP8 ? 2 * kGemmBlockK : kGemmBlockK;   // elements of K in a 128-byte row
  constexpr int STAGES = gemm_stages(BN, PAIR, EPI);
  constexpr int A_BYTES = gemm_a_bytes();
  constexpr int B_BYTES = gemm_b_bytes(BN, PAIR);   // this CTA's part of the W tile
  constexpr int NBUF = gemm_staging_bufs(BN, PAIR, EPI);
  constexpr int TILE_M = PAIR ? 2 * kGemmBlockM : kGemmBlockM;
  constexpr int ACC_ARRIVALS = PAIR ? 2 * kNumEpilogueWarps : kNumEpilogueWarps;
  constexpr uint32_t TMEM_COLS = BN == 64 ? 128 : (BN == 128 ? 256 : 512);  // two accumulators; a power of two >= 32
  static_assert(BN == 64 || BN == 128 || BN == 192 || BN == 256, "tile widths implemented: 64, 128, 192, 256");
  static_assert(BN != 64 || !PAIR, "64-wide tiles (launches of a few rows) run as single CTAs");
  static_assert(EPI != kEpiBiasResidual || NBUF == 2, "the residual epilogue prefetches: two staging buffers");

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sA = smem_u32(smem);
  const uint32_t sB = sA + STAGES * A_BYTES;
  const uint32_t sStage = sB + STAGES * B_BYTES;          // kNumEpilogueWarps x NBUF x 4 KB
  uint8_t* book = smem + STAGES * (A_BYTES + B_BYTES) + kNumEpilogueWarps * NBUF * kStagingBytes;
  const uint32_t bar_full = smem_u32(book);               // STAGES x 8 bytes
  const uint32_t bar_empty = bar_full + 8 * STAGES;       // STAGES x 8 bytes
  const uint32_t bar_acc_full = bar_empty + 8 * STAGES;   // 2 x 8 bytes
  const uint32_t bar_acc_empty = bar_acc_full + 16;       // 2 x 8 bytes
  const uint32_t bar_res = bar_acc_empty + 16;            // kNumEpilogueWarps x 2 x 8 bytes
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(book + 8 * (2 * STAGES + 4 + 2 * kNumEpilogueWarps));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = PAIR ? cluster_cta_rank() : 0u;           // 0 = the CTA that issues the MMAs
  const int worker = PAIR ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
  const int n_workers = PAIR ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);

  const int n_tiles_n = p.N / BN;
  const int k_splits = p.k_splits > 1 ? p.k_splits : 1;   // ranges of K (> 1 only with the partial-sum epilogue)
  const int k_blocks = p.K / KB_ELEMS / k_splits;         // k-blocks of one tile

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_acc_full + 8 * a, 1);
      mbar_init(bar_acc_empty + 8 * a, ACC_ARRIVALS);
    }
    for (int i = 0; i < 2 * kNumEpilogueWarps; ++i) mbar_init(bar_res + 8 * i, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    if (PAIR) tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS); else tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
  }
  tc_fence_before();
  // the partner's barriers must exist before anything of this CTA can signal them
  __syncwarp();
  if (PAIR) cluster_sync_all(); else __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // where the "stage full" barriers are counted: in rank 0 of a pair
  const uint32_t bar_full_count = PAIR ? map_to_cta(bar_full, 0) : bar_full;
  // Tiles are numbered m-tile outermost: tile = ((m_tile * n_groups + g) * n_tiles_n + n_tile) * k_splits + range,
  // so the group, the column block and the K range of a tile do not depend on the (device-side) number of rows.
  const int tiles_per_m = p.n_groups * n_tiles_n * k_splits;
  // Everything above touched no global data.  The weights do not depend on the previous kernel
  // either: the producer thread starts the W tiles of this CTA's first tile before it waits for
  // that kernel, so their trip from HBM overlaps its tail.  From the wait on, the previous kernel
  // has completed and its writes are visible.
  int prefetched = 0;   // stages whose W tile is already on its way (producer warp only)
  bool producer_leader = false;
  if (warp == 0) {
    producer_leader = elect_one();   // the warp stays converged; this lane issues the copies
    const int rem_s = worker % tiles_per_m;
    const int kb0 = (rem_s % k_splits) * k_blocks;   // first k-block of the tile's range of K
    const int rem = rem_s / k_splits;
    const int g = rem / n_tiles_n;
    const int n0 = (rem - g * n_tiles_n) * BN + static_cast<int>(rank) * (PAIR ? BN / 2 : 0);
    prefetched = k_blocks < STAGES ? k_blocks : STAGES;
    if (producer_leader) {
      prefetch_tensormap(&p.tmap_x[g]);
      prefetch_tensormap(&p.tmap_w[g]);
      for (int s = 0; s < prefetched; ++s) {
        if (PAIR) {
          // rank 0 announces the bytes of both CTAs' W parts on its barrier; either CTA's copy may land first
          if (rank == 0) mbar_add_tx(bar_full + 8 * s, 2 * B_BYTES);
          tma_load_2d_pair(sB + s * B_BYTES, &p.tmap_w[g], (kb0 + s) * KB_ELEMS, n0, bar_full_count + 8 * s);
        } else {
          mbar_add_tx(bar_full + 8 * s, B_BYTES);
          tma_load_2d(sB + s * B_BYTES, &p.tmap_w[g], (kb0 + s) * KB_ELEMS, n0, bar_full + 8 * s);
        }
      }
    }
  }
  // rows in use: all M, or fewer when the token layout is packed (a device-side count written by the forward's
  // first kernel).  When this kernel starts, every kernel of the stream but its immediate predecessor has
  // completed (each waits for its own predecessor before it lets its dependents start), and the immediate
  // predecessor is never the one that writes the count: it is read before the dependency wait, off the
  // critical path.
  int m_rows = p.M;
  if (p.m_valid != nullptr) m_rows = min(m_rows, *p.m_valid);
  grid_dependency_wait();
  grid_launch_dependents();
  const int n_tiles_m = (m_rows + TILE_M - 1) / TILE_M;
  const int total_tiles = n_tiles_m * tiles_per_m;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    {
      int stage = 0;
      uint32_t phase = 0;
      long long issued = 0;
      bool ok = true;
      if (worker >= total_tiles && rank == 0 && producer_leader) {
        // no tile for this CTA (pair) after all (fewer rows in use than the grid was sized for): let
        // the early W tiles land before the CTA retires (in a pair, rank 1 is held by the exit barrier)
        for (int s = 0; s < prefetched; ++s) {
          mbar_arrive(bar_full + 8 * s);
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(bar_full + 8 * s, 0)) {
            if (global_timer_ns() - t0 > kWaitLimitNs) break;
          }
        }
      }
      for (int tile = worker; tile < total_tiles && ok; tile += n_workers) {
        const int m0 = (tile / tiles_per_m) * TILE_M + static_cast<int>(rank) * kGemmBlockM;
        const int rem_s = tile % tiles_per_m;
        const int kb0 = (rem_s % k_splits) * k_blocks;
        const int rem = rem_s / k_splits;
        const int g = rem / n_tiles_n;
        const int n0 = (rem - g * n_tiles_n) * BN + static_cast<int>(rank) * (PAIR ? BN / 2 : 0);
        for (int kb = 0; kb < k_blocks; ++kb) {
          // this CTA's stage is free once the MMAs that read it (in both CTAs of a pair) are done
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
          const bool w_on_its_way = prefetched > 0;
          if (w_on_its_way) --prefetched;
          if (!producer_leader) {
            // the other lanes only keep the warp together
          } else if (PAIR) {
            if (rank == 0)
              mbar_expect_tx(bar_full + 8 * stage, 2 * A_BYTES + (w_on_its_way ? 0 : 2 * B_BYTES));
            tma_load_2d_pair(sA + stage * A_BYTES, &p.tmap_x[g], (kb0 + kb) * KB_ELEMS, m0, bar_full_count + 8 * stage);
            if (!w_on_its_way)
              tma_load_2d_pair(sB + stage * B_BYTES, &p.tmap_w[g], (kb0 + kb) * KB_ELEMS, n0, bar_full_count + 8 * stage);
          } else {
            mbar_expect_tx(bar_full + 8 * stage, A_BYTES + (w_on_its_way ? 0 : B_BYTES));
            tma_load_2d(sA + stage * A_BYTES, &p.tmap_x[g], (kb0 + kb) * KB_ELEMS, m0, bar_full + 8 * stage);
            if (!w_on_its_way)
              tma_load_2d(sB + stage * B_BYTES, &p.tmap_w[g], (kb0 + kb) * KB_ELEMS, n0, bar_full + 8 * stage);
          }
          ++issued;
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok && rank == 0 && producer_leader) {
        // Aborting: wait (bounded) until the copies still in flight have landed, so that the
        // CTA does not retire underneath them.  The last min(issued, STAGES) fills are the ones
        // that may be pending; walk back over them.
        int s = stage;
        uint32_t ph = phase;
        const int pending = issued < STAGES ? static_cast<int>(issued) : STAGES;
        for (int i = 0; i < pending; ++i) {
          if (s == 0) { s = STAGES; ph ^= 1u; }
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
    // The whole warp walks the loop and waits on the barriers (it stays converged); the elected lane issues.
    const bool leader = elect_one();
    if (rank == 0) {
      constexpr uint32_t idesc = FP8 ? umma_idesc_e4m3(TILE_M, BN) : umma_idesc_bf16(TILE_M, BN);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = worker; tile < total_tiles && ok; tile += n_workers) {
        // the epilogue warps (of both CTAs of a pair) have drained this accumulator
        if (!mbar_wait(bar_acc_empty + 8 * acc, acc_phase ^ 1u, abort_flag)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          if (leader) {
            const uint64_t da = smem_desc_sw128(sA + stage * A_BYTES);
            const uint64_t db = smem_desc_sw128(sB + stage * B_BYTES);
#pragma unroll
            for (int k = 0; k < kGemmBlockK / 16; ++k) {
              // advancing one instruction along K (16 bf16 or 32 E4M3 = 32 bytes) inside the swizzled row: +2 in the address field
              if (FP8) umma_e4m3(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
              else if (PAIR) umma_bf16_pair(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
              else umma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
            }
            if (PAIR) umma_commit_pair(bar_empty + 8 * stage); else umma_commit(bar_empty + 8 * stage);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (leader) {
          if (PAIR) umma_commit_pair(bar_acc_full + 8 * acc); else umma_commit(bar_acc_full + 8 * acc);
        }
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------ epilogue ----------------------------------
    // A chunk is 32 rows (this warp's TMEM lanes) x 128 bytes of output: 32 fp32 columns for the
    // residual epilogue, 64 bf16 columns otherwise.  Thread t owns row t of the chunk.
    const int e = warp - 2;
    const int quarter = warp & 3;                       // TMEM lanes this warp may read
    const int col_group = e >> 2;                       // which share of the column chunks
    constexpr int COL_GROUPS = kNumEpilogueWarps / 4;
    constexpr int CHUNK_COLS = (EPI == kEpiBiasResidual || EPI == kEpiBiasTanhF32 || EPI == kEpiPartialF32) ? 32 : 64;
    constexpr int CHUNKS = BN / CHUNK_COLS;
    const uint32_t my_stage = sStage + static_cast<uint32_t>(e * NBUF * kStagingBytes);
    const uint32_t my_res_bar = bar_res + 16 * e;       // two barriers, one per staging buffer
    uint8_t* my_stage_ptr = smem + STAGES * (A_BYTES + B_BYTES) + e * NBUF * kStagingBytes;
    int acc = 0;
    uint32_t acc_phase = 0;
    int buf = 0;                  // staging buffer of the next chunk
    uint32_t res_phase[2] = {0, 0};
    bool ok = true;

    // (residual epilogue) asks for the residual chunk `chunk` of tile `tile` into staging buffer b
    auto prefetch_residual = [&](int tile, int chunk, int b) {
      const int rem = (tile % tiles_per_m) / k_splits;
      const int g = rem / n_tiles_n;
      const int row0 = (tile / tiles_per_m) * TILE_M + static_cast<int>(rank) * kGemmBlockM + quarter * 32;
      const int col0 = (rem - g * n_tiles_n) * BN + chunk * CHUNK_COLS;
      // the store issued last read this very buffer: it must be done with it before TMA refills it
      tma_store_wait_read<0>();
      mbar_expect_tx(my_res_bar + 8 * b, kStagingBytes);
      tma_load_2d(my_stage + b * kStagingBytes, &p.tmap_res[g], col0, row0, my_res_bar + 8 * b);
    };

    // (residual epilogue, lane 0) This warp's chunks, in the order it works through them, use the two staging
    // buffers alternately.  A buffer can take the residual of the chunk two places on as soon as the store of
    // its present chunk has read it, so up to two requests are kept in flight: both chunks of a 128-wide tile
    // are asked for before the tile's main loop ends (at the kernel's start for a CTA's first tile) instead of
    // the second one only when the first is being worked on.
    int req_tile = worker, req_chunk = col_group;   // the next chunk to ask for
    int n_req = 0, n_done = 0;                      // chunks asked for / chunks whose store has been issued
    auto refill = [&]() {
      while (n_req < n_done + 2 && req_tile < total_tiles) {
        prefetch_residual(req_tile, req_chunk, n_req & 1);
        ++n_req;
        req_chunk += COL_GROUPS;
        if (req_chunk >= CHUNKS) { req_chunk = col_group; req_tile += n_workers; }
      }
    };
    if (EPI == kEpiBiasResidual && lane == 0) refill();
    // a pair's accumulator is free again when the epilogue warps of both CTAs are done with it
    const uint32_t bar_acc_empty_count = (PAIR && rank != 0) ? map_to_cta(bar_acc_empty, 0) : bar_acc_empty;

    for (int tile = worker; tile < total_tiles && ok; tile += n_workers) {
      const int m0 = (tile / tiles_per_m) * TILE_M + static_cast<int>(rank) * kGemmBlockM;
      const int rem_s = tile % tiles_per_m;
      const int rem = rem_s / k_splits;
      const int g = rem / n_tiles_n;
      const int n0 = (rem - g * n_tiles_n) * BN;
      // (partial sums) the tile's range of K writes its own rows of the output
      const int out_row0 = m0 + quarter * 32 + (EPI == kEpiPartialF32 ? (rem_s % k_splits) * p.split_pitch : 0);
      // warp-uniform decisions: the TMEM loads below are warp-collective
      if (!__all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8 * acc, acc_phase, abort_flag))) break;
      tc_fence_after();
      const bf16* bias = p.group[g].bias;
      const bool rows_in_range = m0 + quarter * 32 < m_rows;
      float row_scale = 1.0f;          // (8-bit operands) scale of this thread's row of X
      const float* col_scale = nullptr;
      if (FP8) {
        const int row = m0 + quarter * 32 + lane;
        row_scale = row < p.M ? __ldg(p.group[g].scale_x + row) : 0.0f;
        col_scale = p.group[g].scale_w;
      }
#pragma unroll 1
      for (int chunk = col_group; chunk < CHUNKS; chunk += COL_GROUPS) {
        const int col = n0 + chunk * CHUNK_COLS;
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                               static_cast<uint32_t>(acc * BN + chunk * CHUNK_COLS);
        uint8_t* sbuf = my_stage_ptr + buf * kStagingBytes;
        if (EPI == kEpiBiasResidual) {
          uint32_t v[32];
          tmem_ld_32x32(taddr, v);
          // the other buffer is free once the store before this chunk has read it
          if (lane == 0) refill();
          __syncwarp();
          tmem_ld_wait();
          if (!__all_sync(0xffffffffu, mbar_wait(my_res_bar + 8 * buf, res_phase[buf], abort_flag))) {
            ok = false;
            break;
          }
          res_phase[buf] ^= 1u;
          if (FP8) {
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const float4 sc = __ldg(reinterpret_cast<const float4*>(col_scale + col) + q);
              v[q * 4 + 0] = __float_as_uint(__uint_as_float(v[q * 4 + 0]) * (row_scale * sc.x));
              v[q * 4 + 1] = __float_as_uint(__uint_as_float(v[q * 4 + 1]) * (row_scale * sc.y));
              v[q * 4 + 2] = __float_as_uint(__uint_as_float(v[q * 4 + 2]) * (row_scale * sc.z));
              v[q * 4 + 3] = __float_as_uint(__uint_as_float(v[q * 4 + 3]) * (row_scale * sc.w));
            }
          }
          const uint4* bias4 = reinterpret_cast<const uint4*>(bias + col);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint4 b = __ldg(bias4 + q);
            const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
            float4* s0 = reinterpret_cast<float4*>(sbuf + staging_off(lane, 2 * q));
            float4* s1 = reinterpret_cast<float4*>(sbuf + staging_off(lane, 2 * q + 1));
            float4 r0 = *s0, r1 = *s1;
            r0.x += __uint_as_float(v[q * 8 + 0]) + bf16_lo(bw[0]);
            r0.y += __uint_as_float(v[q * 8 + 1]) + bf16_hi(bw[0]);
            r0.z += __uint_as_float(v[q * 8 + 2]) + bf16_lo(bw[1]);
            r0.w += __uint_as_float(v[q * 8 + 3]) + bf16_hi(bw[1]);
            r1.x += __uint_as_float(v[q * 8 + 4]) + bf16_lo(bw[2]);
            r1.y += __uint_as_float(v[q * 8 + 5]) + bf16_hi(bw[2]);
            r1.z += __uint_as_float(v[q * 8 + 6]) + bf16_lo(bw[3]);
            r1.w += __uint_as_float(v[q * 8 + 7]) + bf16_hi(bw[3]);
            *s0 = r0;
            *s1 = r1;
          }
        } else if (EPI == kEpiPartialF32) {
          // the store that last read this staging buffer must be done with it
          if (lane == 0) {
            if (NBUF == 2) tma_store_wait_read<1>(); else tma_store_wait_read<0>();
          }
          __syncwarp();
          uint32_t v[32];
          tmem_ld_32x32(taddr, v);
          tmem_ld_wait();
#pragma unroll
          for (int q = 0; q < 8; ++q)
            *reinterpret_cast<uint4*>(sbuf + staging_off(lane, q)) = make_uint4(v[q * 4 + 0], v[q * 4 + 1], v[q * 4 + 2], v[q * 4 + 3]);
        } else if (EPI == kEpiBiasTanhF32) {
          // the store that last read this staging buffer must be done with it
          if (lane == 0) {
            if (NBUF == 2) tma_store_wait_read<1>(); else tma_store_wait_read<0>();
          }
          __syncwarp();
          uint32_t v[32];
          tmem_ld_32x32(taddr, v);
          tmem_ld_wait();
          const uint4* bias4 = reinterpret_cast<const uint4*>(bias + col);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint4 b = __ldg(bias4 + q);
            const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
            float4 r0, r1;
            r0.x = tanhf(__uint_as_float(v[q * 8 + 0]) + bf16_lo(bw[0]));
            r0.y = tanhf(__uint_as_float(v[q * 8 + 1]) + bf16_hi(bw[0]));
            r0.z = tanhf(__uint_as_float(v[q * 8 + 2]) + bf16_lo(bw[1]));
            r0.w = tanhf(__uint_as_float(v[q * 8 + 3]) + bf16_hi(bw[1]));
            r1.x = tanhf(__uint_as_float(v[q * 8 + 4]) + bf16_lo(bw[2]));
            r1.y = tanhf(__uint_as_float(v[q * 8 + 5]) + bf16_hi(bw[2]));
            r1.z = tanhf(__uint_as_float(v[q * 8 + 6]) + bf16_lo(bw[3]));
            r1.w = tanhf(__uint_as_float(v[q * 8 + 7]) + bf16_hi(bw[3]));
            *reinterpret_cast<float4*>(sbuf + staging_off(lane, 2 * q)) = r0;
            *reinterpret_cast<float4*>(sbuf + staging_off(lane, 2 * q + 1)) = r1;
          }
        } else {
          // the store that last read this staging buffer must be done with it
          if (lane == 0) {
            if (NBUF == 2) tma_store_wait_read<1>(); else tma_store_wait_read<0>();
          }
          __syncwarp();
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t v[32];
            tmem_ld_32x32(taddr + half * 32, v);
            tmem_ld_wait();
            if (FP8) {
#pragma unroll
              for (int q = 0; q < 8; ++q) {
                const float4 sc = __ldg(reinterpret_cast<const float4*>(col_scale + col + half * 32) + q);
                v[q * 4 + 0] = __float_as_uint(__uint_as_float(v[q * 4 + 0]) * (row_scale * sc.x));
                v[q * 4 + 1] = __float_as_uint(__uint_as_float(v[q * 4 + 1]) * (row_scale * sc.y));
                v[q * 4 + 2] = __float_as_uint(__uint_as_float(v[q * 4 + 2]) * (row_scale * sc.z));
                v[q * 4 + 3] = __float_as_uint(__uint_as_float(v[q * 4 + 3]) * (row_scale * sc.w));
              }
            }
            const uint4* bias4 = reinterpret_cast<const uint4*>(bias + col + half * 32);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint4 b = __ldg(bias4 + q);
              const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
              uint32_t ow[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                float x0 = __uint_as_float(v[q * 8 + 2 * j]) + bf16_lo(bw[j]);
                float x1 = __uint_as_float(v[q * 8 + 2 * j + 1]) + bf16_hi(bw[j]);
                if (EPI == kEpiBiasGelu) {
                  x0 = gelu_fitted(x0);
                  x1 = gelu_fitted(x1);
                }
                ow[j] = pack_bf16(x0, x1);
              }
              *reinterpret_cast<uint4*>(sbuf + staging_off(lane, half * 4 + q)) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
            }
          }
        }
        fence_async_shared();
        __syncwarp();
        if (lane == 0 && rows_in_range) {
          tma_store_2d(&p.tmap_out[g], my_stage + buf * kStagingBytes, col, out_row0);
          tma_store_commit();
        }
        ++n_done;
        if (NBUF == 2) buf ^= 1;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR && rank != 0) mbar_arrive_cluster(bar_acc_empty_count + 8 * acc);
        else mbar_arrive(bar_acc_empty + 8 * acc);
        // the tile's last store frees its buffer for the next tile's residual while that tile's main loop runs
        if (EPI == kEpiBiasResidual) refill();
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    // shared memory must outlive the stores that still read it, and (when the CTA is giving up) the residual
    // copies that were asked for and never used: those get the same limit to land
    if (lane == 0) {
      tma_store_wait_read<0>();
      for (int i = n_done; i < n_req; ++i) {
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(my_res_bar + 8 * (i & 1), res_phase[i & 1])) {
          if (global_timer_ns() - t0 > kWaitLimitNs) break;
        }
      }
    }
    __syncwarp();
  }

  // ------------------------------ teardown ------------------------------------
  tc_fence_before();
  // In a pair neither CTA may retire (or free tensor memory) while the other can still signal its
  // barriers or while MMAs that read its shared memory may be in flight: every thread of both CTAs
  // gets here (all waits above are bounded), so this barrier completes.
  __syncwarp();
  if (PAIR) cluster_sync_all(); else __syncthreads();
  if (threadIdx.x == 0 && *abort_flag && p.status != nullptr) atomicOr(p.status, kFlagWaitTimeout);
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    if (PAIR) tmem_dealloc_pair(tmem_base, TMEM_COLS); else tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

template <int BN, int EPI, bool PAIR, bool FP8 = false>
cudaError_t launch_one(const GemmParams& p, int sm_count, cudaStream_t stream) {
  auto kernel = gemm_bf16_tcgen05<BN, EPI, PAIR, FP8>;
  static PerDeviceOnce once;   // per instantiation
  cudaError_t err = per_device_once(once, [&](int) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, gemm_smem_bytes(BN, PAIR, EPI));
  });
  if (err != cudaSuccess) return err;
  constexpr int tile_m = PAIR ? 2 * kGemmBlockM : kGemmBlockM;
  const int tiles = ((p.M + tile_m - 1) / tile_m) * (p.N / BN) * p.n_groups * (p.k_splits > 1 ? p.k_splits : 1);
  const int workers_max = PAIR ? sm_count / 2 : sm_count;
  const int workers = tiles < workers_max ? tiles : workers_max;
  if (workers <= 0) return cudaSuccess;
  return launch_kernel(kernel, dim3(PAIR ? 2 * workers : workers), dim3(kGemmThreads), gemm_smem_bytes(BN, PAIR, EPI), stream,
                       p, PAIR ? 2u : 1u);
}

template <int BN, bool PAIR>
cudaError_t launch_bn(const GemmParams& p, int epilogue, int sm_count, cudaStream_t stream) {
  switch (epilogue) {
    case kEpiBias: return launch_one<BN, kEpiBias, PAIR>(p, sm_count, stream);
    case kEpiBiasGelu: return launch_one<BN, kEpiBiasGelu, PAIR>(p, sm_count, stream);
    case kEpiBiasResidual:
      if constexpr (BN != 256 || PAIR) return launch_one<BN, kEpiBiasResidual, PAIR>(p, sm_count, stream);
      return cudaErrorInvalidValue;  // single CTAs: 256-wide stages and two fp32 staging buffers do not fit
    case kEpiBiasTanhF32:   // the pooler: a few rows, single CTAs on 128-wide tiles only
      if constexpr (BN == 128 && !PAIR) return launch_one<BN, kEpiBiasTanhF32, PAIR>(p, sm_count, stream);
      return cudaErrorInvalidValue;
    case kEpiPartialF32:    // partial sums of a split K: launches of few rows, single CTAs on 64- or 128-wide tiles
      if constexpr ((BN == 128 || BN == 64) && !PAIR) return launch_one<BN, kEpiPartialF32, PAIR>(p, sm_count, stream);
      return cudaErrorInvalidValue;
    default: return cudaErrorInvalidValue;
  }
}

template <bool PAIR>
cudaError_t launch_any(const GemmParams& p, int epilogue, int sm_count, cudaStream_t stream) {
  switch (p.block_n) {
    case 256: return launch_bn<256, PAIR>(p, epilogue, sm_count, stream);
    case 192: return launch_bn<192, PAIR>(p, epilogue, sm_count, stream);
    case 128: return launch_bn<128, PAIR>(p, epilogue, sm_count, stream);
    case 64:
      if constexpr (!PAIR) return launch_bn<64, PAIR>(p, epilogue, sm_count, stream);
      return cudaErrorInvalidValue;
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

int gemm_block_n(int N, int epilogue, int64_t rows, int groups, bool pair, int sm_count) {
  if (epilogue == kEpiBiasTanhF32) return 128;
  if (epilogue == kEpiPartialF32) {
    // (`groups` counts the ranges of K too) 64-wide tiles while they all run at once, else 128-wide (measured at
    // N = 768, K = 3072 in four ranges: 128 rows 5.4 against 6.0 us, 512 rows 8.8 against 6.7 us)
    const int64_t tiles64 = ((rows + kGemmBlockM - 1) / kGemmBlockM) * (N / 64) * groups;
    return (N % 128 != 0 || tiles64 <= sm_count) ? 64 : 128;
  }
  // (64: only ever the cheapest where a launch has so few rows that even 128-wide tiles leave most SMs
  // without work - the first-token tails - and each CTA would stream a long K by itself)
  const int candidates[4] = {256, 192, 128, 64};
  const int64_t tile_m = pair ? 2 * kGemmBlockM : kGemmBlockM;
  const int64_t workers = pair ? (sm_count / 2 > 0 ? sm_count / 2 : 1) : (sm_count > 0 ? sm_count : 1);
  const int64_t m_tiles = (rows + tile_m - 1) / tile_m;
  int best = 128;
  int64_t best_cost = -1;
  for (int bn : candidates) {
    if (N % bn != 0) continue;
    if (bn == 256 && epilogue == kEpiBiasResidual && !pair) continue;   // not instantiated: two fp32 staging buffers do not fit
    if (bn == 64 && pair) continue;
    const int64_t tiles = m_tiles * (N / bn) * groups;
    const int64_t rounds = (tiles + workers - 1) / workers;
    // per 64 of K a CTA stages 128 rows of X and bn (a pair's CTA: bn / 2) rows of W, and its tensor
    // core needs about bn of the same units
    const int64_t staged = 128 + (pair ? bn / 2 : bn);
    const int64_t cost = rounds * (staged > bn ? staged : bn);
    if (best_cost < 0 || cost < best_cost) {   // candidates run from wide to narrow: ties keep the wider tile
      best_cost = cost;
      best = bn;
    }
  }
  return best;
}
int gemm_out_box_cols(int epilogue) {
  return (epilogue == kEpiBiasResidual || epilogue == kEpiBiasTanhF32 || epilogue == kEpiPartialF32) ? 32 : 64;
}

cudaError_t launch_gemm(const GemmParams& p, int epilogue, int sm_count, cudaStream_t stream) {
  if (p.n_groups < 1 || p.n_groups > kMaxGroups || p.K % kGemmBlockK != 0 || p.block_n < 1 || p.N % p.block_n != 0 ||
      p.M < 1)
    return cudaErrorInvalidValue;
  // a split K only with the partial-sum epilogue (single CTAs, bf16): equal ranges of whole k-blocks, and the
  // ranges' outputs a whole number of row blocks apart so that no store box reaches into the next range's rows
  if (p.k_splits > 1 &&
      (epilogue != kEpiPartialF32 || p.fp8 || p.pair || (p.K / kGemmBlockK) % p.k_splits != 0 ||
       p.split_pitch < p.M || p.split_pitch % kGemmBlockM != 0))
    return cudaErrorInvalidValue;
  if (p.fp8) {
    if (p.pair || p.K % (2 * kGemmBlockK) != 0) return cudaErrorInvalidValue;
    if (epilogue == kEpiBias && p.block_n == 256) return launch_one<256, kEpiBias, false, true>(p, sm_count, stream);
    if (epilogue == kEpiBiasGelu && p.block_n == 256) return launch_one<256, kEpiBiasGelu, false, true>(p, sm_count, stream);
    if (epilogue == kEpiBiasResidual && p.block_n == 128) return launch_one<128, kEpiBiasResidual, false, true>(p, sm_count, stream);
    return cudaErrorInvalidValue;
  }
  return p.pair ? launch_any<true>(p, epilogue, sm_count, stream) : launch_any<false>(p, epilogue, sm_count, stream);
}

}  // namespace mt
