// The encoder layer after attention, as ONE persistent launch per wave of the task tree:
//
//   phase 0  u  = ctx . Wo^T + bo + x      fp32        -> h1  = LN(u)  (bf16 + fp32)
//   phase 1  f  = GELU(h1 . W1^T + b1)     bf16
//   phase 2  u  = f . W2^T + b2 + h1       fp32        -> out = LN(u)  (bf16 + fp32)
//
// for all layers (groups) of the wave.  At the sizes of one serving batch each of the three GEMMs has
// about as many tiles as the GPU has SMs, so as separate launches every one of them pays its own
// pipeline ramp, a last round that fills part of the machine, and a drain, and LayerNorm pays two more
// launches.  Here the tiles of the three GEMMs form one ordered list (phase-major, then row block,
// group, column block) dealt out round-robin to one persistent CTA per SM, and dependencies are
// tracked per block of 128 rows in global memory:
//   * every epilogue warp of a tile arrives on its row block's counter once the stores it issued for the
//     tile have completed (the arrival is deferred until the warp has stored the first chunk of its next
//     tile, so that the round trip of the last store is hidden, unless it would idle anyway),
//   * six more warps per CTA only normalise rows: their work items are pairs of rows of a (phase, row
//     block, group), dealt round-robin over all such warps of the grid; an item waits until all tiles of
//     its row block have arrived, and in phase 0 adds itself to "h1 ready",
//   * a phase-1 tile waits until "h1 ready" of its row block is complete,
//   * a phase-2 tile waits until all phase-1 tiles of its row block have arrived.
// A tile only ever waits for tiles (and LayerNorm items) that precede it in the list, every CTA takes
// its tiles in list order and all CTAs are resident (grid <= number of SMs, one CTA per SM), so the earliest unfinished
// tile can always proceed: the waits cannot deadlock.  They are bounded all the same: after
// kDepWaitLimitNs a waiting thread raises the CTA's abort flag, the status word gets
// kFlagWaitTimeout, every role leaves its loop, copies in flight are drained, TMEM is freed.
//
// The tile machinery is that of gemm_bf16_tcgen05 (TMA producer warp, one MMA-issuing thread with the
// accumulator double buffered in tensor memory, eight epilogue warps that stage 128-byte rows for TMA
// stores), with the tile width a run-time property of the phase, and every output element is the
// same fixed-order sum over K: results are bit-identical to the separate launches.
//
// Memory ordering between CTAs.  Producers write u and f with TMA stores (async proxy) and h1 / out
// with ordinary stores; consumers read h1 and f with TMA loads and u with ordinary loads.  A writer
// waits for the completion of its bulk stores (cp.async.bulk.wait_group), fences, and only then
// arrives on the counter with a release at GPU scope; a reader acquires the counter at GPU scope and
// issues fence.proxy.async before its TMA loads; ordinary loads of produced data bypass L1 (ld.cg),
// because the same addresses are read again in a later phase of the same launch.

#include "rowwise.cuh"
#include "tc_ptx.cuh"

namespace mt {
namespace {

constexpr int kChainEpilogueWarps = 8;
constexpr int kChainLnWarps = 6;          // warps that only normalise rows
constexpr int kChainLnRows = 2;           // rows of one LayerNorm work item (both in flight in one warp)
constexpr int kChainLnSlices = kGemmBlockM / kChainLnRows;   // work items per block of 128 rows
constexpr int kChainFirstEpilogueWarp = 2 + kChainLnWarps;
constexpr int kChainThreads = 32 * (2 + kChainLnWarps + kChainEpilogueWarps);
// (an epilogue warp w reads the TMEM lanes of quarter w % 4: any four consecutive warps cover all quarters)
constexpr int kChainStages = 4;
constexpr int kChainStagingBytes = 4096;                                  // 32 rows x 128 bytes
constexpr int kChainABytes = kGemmBlockM * kGemmBlockK * 2;               // 16 KB
constexpr int kChainBBytesMax = kChainMaxBlockN * kGemmBlockK * 2;        // 24 KB
constexpr int kChainAccStride = 256;                                      // TMEM columns between the two accumulators
constexpr uint32_t kChainTmemCols = 512;
constexpr int kChainSmemBytes = kChainStages * (kChainABytes + kChainBBytesMax) +
                                kChainEpilogueWarps * 2 * kChainStagingBytes + 512 + 1024;
constexpr unsigned long long kDepWaitLimitNs = 2000000000ull;             // 2 s

// words of the sync array per (group, row block)
enum { kSyncArrive0 = 0, kSyncH1Ready = 1, kSyncArrive1 = 2, kSyncArrive2 = 3 };

__device__ __forceinline__ uint32_t ld_acquire_gpu(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t atom_add_acq_rel_gpu(uint32_t* p, uint32_t v) {
  uint32_t old;
  asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}
// Orders this thread's earlier (acquired) view of global memory before its later TMA operations, and its
// earlier ordinary writes before later async-proxy accesses.
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
// All of this thread's bulk stores have completed (their writes are performed), not just read their source.
__device__ __forceinline__ void tma_store_wait_complete() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// ... all but the N most recently committed groups of them.
template <int N>
__device__ __forceinline__ void tma_store_wait_complete_but() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }
// Bounded wait until *word >= target.  False once the CTA is aborting.
__device__ __forceinline__ bool dep_wait(const uint32_t* word, uint32_t target, volatile int* abort_flag) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (ld_acquire_gpu(word) >= target) return true;
    __nanosleep(40);
    if ((it & 0x3Fu) == 0x3Fu) {
      if (*abort_flag) return false;
      const unsigned long long now = global_timer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > kDepWaitLimitNs) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

// Optional timeline of one launch (compiled in with -DMT_CHAIN_TRACE, for tuning only): per CTA and per
// tile of that CTA, %globaltimer at the points of interest.
#ifdef MT_CHAIN_TRACE
constexpr int kTraceSlots = 16;    // tiles per CTA recorded
constexpr int kTracePoints = 12;
__device__ unsigned long long g_chain_trace[160 * kTraceSlots * kTracePoints];
__device__ int g_chain_trace_on;
#define CHAIN_TRACE(slot, point)                                                                   \
  do {                                                                                             \
    if (g_chain_trace_on && (slot) < kTraceSlots && blockIdx.x < 160)                              \
      g_chain_trace[(blockIdx.x * kTraceSlots + (slot)) * kTracePoints + (point)] = global_timer_ns(); \
  } while (0)
#else
#define CHAIN_TRACE(slot, point) do { } while (0)
#endif

// A tile of the list.
struct Item {
  int phase, g, m0, n0, row_block;
};

struct PhaseShape {
  int bn, n_tiles_n, k_blocks, tiles_per_m, first;   // first = index of the phase's first tile in the list
};

// One row of the pre-normalisation sum into registers; L1 is bypassed because the same addresses hold
// another phase's sum later in the same launch.
template <int V>
__device__ __forceinline__ void load_row(const float* xin, int lane, float (&x)[V][8]) {
#pragma unroll
  for (int v = 0; v < V; ++v) {
    const float4 a = __ldcg(reinterpret_cast<const float4*>(xin + (v * 32 + lane) * 8));
    const float4 b = __ldcg(reinterpret_cast<const float4*>(xin + (v * 32 + lane) * 8 + 4));
    x[v][0] = a.x; x[v][1] = a.y; x[v][2] = a.z; x[v][3] = a.w;
    x[v][4] = b.x; x[v][5] = b.y; x[v][6] = b.z; x[v][7] = b.w;
  }
}
// LayerNorm of rows [row0, row_end), at most kChainLnRows = 2 of them, by one warp; both rows are loaded
// before either is reduced, so their trips to L2 overlap.
template <int V>
__device__ __forceinline__ void layernorm_rows(const LayerNormParams& ln, int g, int row0, int row_end, int lane) {
  constexpr int H = V * 256;
  if (row0 >= row_end) return;
  const float* xbase = ln.x[g];
  bf16* ybase = ln.y[g];
  float* y32base = ln.y32[g];
  const int row_b = row0 + 1;
  const bool two = row_b < row_end;
  float xa[V][8], xb[V][8];
  load_row<V>(xbase + static_cast<size_t>(row0) * H, lane, xa);
  if (two) load_row<V>(xbase + static_cast<size_t>(row_b) * H, lane, xb);
  normalise_store<V>(xa, ln.gamma[g], ln.beta[g], ybase + static_cast<size_t>(row0) * H,
                     y32base != nullptr ? y32base + static_cast<size_t>(row0) * H : nullptr, lane, ln.eps);
  if (two)
    normalise_store<V>(xb, ln.gamma[g], ln.beta[g], ybase + static_cast<size_t>(row_b) * H,
                       y32base != nullptr ? y32base + static_cast<size_t>(row_b) * H : nullptr, lane, ln.eps);
}

__global__ void __launch_bounds__(kChainThreads, 1) layer_chain_tcgen05(const __grid_constant__ ChainParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sA = smem_u32(smem);
  const uint32_t sB = sA + kChainStages * kChainABytes;
  const uint32_t sStage = sB + kChainStages * kChainBBytesMax;
  uint8_t* stage_ptr = smem + kChainStages * (kChainABytes + kChainBBytesMax);
  uint8_t* book = stage_ptr + kChainEpilogueWarps * 2 * kChainStagingBytes;
  const uint32_t bar_full = smem_u32(book);                       // kChainStages x 8 bytes
  const uint32_t bar_empty = bar_full + 8 * kChainStages;
  const uint32_t bar_acc_full = bar_empty + 8 * kChainStages;     // 2 x 8 bytes
  const uint32_t bar_acc_empty = bar_acc_full + 16;
  const uint32_t bar_res = bar_acc_empty + 16;                    // kChainEpilogueWarps x 2 x 8 bytes
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(book + 8 * (2 * kChainStages + 4 + 2 * kChainEpilogueWarps));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int worker = static_cast<int>(blockIdx.x);
  const int n_workers = static_cast<int>(gridDim.x);
  const int n_groups = p.gemm[0].n_groups;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kChainStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_acc_full + 8 * a, 1);
      mbar_init(bar_acc_empty + 8 * a, kChainEpilogueWarps);
    }
    for (int i = 0; i < 2 * kChainEpilogueWarps; ++i) mbar_init(bar_res + 8 * i, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kChainTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // Nothing above touched global memory; from here on the previous kernel has completed.
  grid_dependency_wait();
  grid_launch_dependents();

  int m_rows = p.gemm[0].M;
  if (p.gemm[0].m_valid != nullptr) m_rows = min(m_rows, *p.gemm[0].m_valid);
  const int n_tiles_m = (m_rows + kGemmBlockM - 1) / kGemmBlockM;
  PhaseShape shape[3];
  int total_items = 0;
#pragma unroll
  for (int ph = 0; ph < 3; ++ph) {
    shape[ph].bn = p.gemm[ph].block_n;
    shape[ph].n_tiles_n = p.gemm[ph].N / shape[ph].bn;
    shape[ph].k_blocks = p.gemm[ph].K / kGemmBlockK;
    shape[ph].tiles_per_m = n_groups * shape[ph].n_tiles_n;
    shape[ph].first = total_items;
    total_items += n_tiles_m * shape[ph].tiles_per_m;
  }
  auto decode = [&](int item) {
    Item it;
    it.phase = item >= shape[2].first ? 2 : (item >= shape[1].first ? 1 : 0);
    const PhaseShape& s = shape[it.phase];
    const int t = item - s.first;
    it.row_block = t / s.tiles_per_m;
    const int rem = t - it.row_block * s.tiles_per_m;
    it.g = rem / s.n_tiles_n;
    it.m0 = it.row_block * kGemmBlockM;
    it.n0 = (rem - it.g * s.n_tiles_n) * s.bn;
    return it;
  };
  auto sync_word = [&](int g, int row_block, int which) {
    return p.sync + (static_cast<size_t>(g) * p.sync_blocks + row_block) * 4 + which;
  };
  // what a tile's operands wait for: the word and the value it must reach (null = nothing produced in this launch)
  auto dependency = [&](const Item& it, uint32_t* target) -> const uint32_t* {
    if (it.phase == 1) { *target = static_cast<uint32_t>(kChainLnSlices); return sync_word(it.g, it.row_block, kSyncH1Ready); }
    if (it.phase == 2) {
      *target = static_cast<uint32_t>(shape[1].n_tiles_n * kChainEpilogueWarps);
      return sync_word(it.g, it.row_block, kSyncArrive1);
    }
    return nullptr;
  };

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      long long issued = 0;
      bool ok = true;
      for (int item = worker; item < total_items && ok; item += n_workers) {
        const Item it = decode(item);
        const PhaseShape& s = shape[it.phase];
        const GemmParams& gp = p.gemm[it.phase];
        uint32_t target = 0;
        const uint32_t* dep = dependency(it, &target);
        CHAIN_TRACE((item - worker) / n_workers, 0);
        if (dep != nullptr) {
          if (!dep_wait(dep, target, abort_flag)) { ok = false; break; }
          fence_proxy_async_all();
        }
        CHAIN_TRACE((item - worker) / n_workers, 1);
        const uint32_t b_bytes = static_cast<uint32_t>(s.bn) * kGemmBlockK * 2;
        for (int kb = 0; kb < s.k_blocks; ++kb) {
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
          mbar_expect_tx(bar_full + 8 * stage, kChainABytes + b_bytes);
          tma_load_2d(sA + stage * kChainABytes, &gp.tmap_x[it.g], kb * kGemmBlockK, it.m0, bar_full + 8 * stage);
          tma_load_2d(sB + stage * kChainBBytesMax, &gp.tmap_w[it.g], kb * kGemmBlockK, it.n0, bar_full + 8 * stage);
          ++issued;
          if (++stage == kChainStages) { stage = 0; phase ^= 1u; }
        }
        CHAIN_TRACE((item - worker) / n_workers, 2);
      }
      if (!ok) {
        // aborting: give the copies still in flight the same limit to land before the CTA retires
        int s = stage;
        uint32_t ph = phase;
        const int pending = issued < kChainStages ? static_cast<int>(issued) : kChainStages;
        for (int i = 0; i < pending; ++i) {
          if (s == 0) { s = kChainStages; ph ^= 1u; }
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
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int item = worker; item < total_items && ok; item += n_workers) {
        const Item it = decode(item);
        const PhaseShape& s = shape[it.phase];
        const uint32_t idesc = umma_idesc_bf16(kGemmBlockM, s.bn);
        if (!mbar_wait(bar_acc_empty + 8 * acc, acc_phase ^ 1u, abort_flag)) break;
        tc_fence_after();
        CHAIN_TRACE((item - worker) / n_workers, 3);
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kChainAccStride);
        for (int kb = 0; kb < s.k_blocks; ++kb) {
          if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = smem_desc_sw128(sA + stage * kChainABytes);
          const uint64_t db = smem_desc_sw128(sB + stage * kChainBBytesMax);
#pragma unroll
          for (int k = 0; k < kGemmBlockK / 16; ++k)
            umma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit(bar_empty + 8 * stage);
          if (++stage == kChainStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        CHAIN_TRACE((item - worker) / n_workers, 4);
        umma_commit(bar_acc_full + 8 * acc);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else if (warp < kChainFirstEpilogueWarp) {
    // ------------------------------ LayerNorm warps ---------------------------
    // Work items: kChainLnRows rows of one (phase, row block, group), phase 0 before phase 2, dealt
    // round-robin over all LayerNorm warps of the grid.  An item waits until every epilogue warp of every
    // tile of its row block has arrived (u complete), normalises its rows and, in phase 0, adds itself
    // to "h1 ready".  Items without valid rows still count, so the target is the same for every block.
    const int ln_warp = worker * kChainLnWarps + (warp - 2);
    const int n_ln_warps = n_workers * kChainLnWarps;
    const int items_per_block = n_groups * kChainLnSlices;
    const int items_per_phase = n_tiles_m * items_per_block;
    for (int j = ln_warp; j < 2 * items_per_phase; j += n_ln_warps) {
      const int ph = j >= items_per_phase ? 2 : 0;
      const int t = ph == 0 ? j : j - items_per_phase;
      const int row_block = t / items_per_block;
      const int rem = t - row_block * items_per_block;
      const int g = rem / kChainLnSlices;
      const int row0 = row_block * kGemmBlockM + (rem - g * kChainLnSlices) * kChainLnRows;
      const LayerNormParams& ln = p.ln[ph == 0 ? 0 : 1];
      {
        // while the tiles are still on their way: bring this layer's gamma and beta into L1
        const int line = lane * 64;   // 128-byte lines of bf16
        if (line < ln.hidden) {
          asm volatile("prefetch.global.L1 [%0];" ::"l"(ln.gamma[g] + line));
          asm volatile("prefetch.global.L1 [%0];" ::"l"(ln.beta[g] + line));
        }
      }
      int all_here = 1;
      if (lane == 0)
        all_here = dep_wait(sync_word(g, row_block, ph == 0 ? kSyncArrive0 : kSyncArrive2),
                            static_cast<uint32_t>(shape[ph].n_tiles_n * kChainEpilogueWarps), abort_flag) ? 1 : 0;
      if (__shfl_sync(0xffffffffu, all_here, 0) == 0) break;
      const int row_end = min(row0 + kChainLnRows, m_rows);
      if (ln.hidden == 768) layernorm_rows<3>(ln, g, row0, row_end, lane);
      else layernorm_rows<4>(ln, g, row0, row_end, lane);
      if (ph == 0) {
        __syncwarp();
        if (lane == 0) {
          __threadfence();
          fence_proxy_async_all();
          atom_add_acq_rel_gpu(sync_word(g, row_block, kSyncH1Ready), 1u);
        }
      }
    }
  } else {
    // ------------------------------ epilogue ----------------------------------
    const int e = warp - kChainFirstEpilogueWarp;
    const int quarter = warp & 3;       // TMEM lanes this warp may read
    const int col_group = e >> 2;       // which share of the column chunks
    constexpr int COL_GROUPS = kChainEpilogueWarps / 4;
    const uint32_t my_stage = sStage + static_cast<uint32_t>(e * 2 * kChainStagingBytes);
    uint8_t* my_stage_ptr = stage_ptr + e * 2 * kChainStagingBytes;
    const uint32_t my_res_bar = bar_res + 16 * e;
    int acc = 0;
    uint32_t acc_phase = 0;
    int buf = 0;
    uint32_t res_phase[2] = {0, 0};
    bool ok = true;
    // A tile's arrival is published by each epilogue warp on its own, once the stores it issued for
    // the tile have completed.  Waiting for that right away would stall the warp for the round trip of
    // its last store, so the arrival is deferred until the first chunk of the warp's next tile has been
    // stored (by then the wait is over) - unless that tile's accumulator is not there yet, in which case
    // the warp would idle anyway, and it must not hold the arrival back: the tile it waits for may
    // itself depend on it.
    uint32_t* pending_arrival = nullptr;
    auto publish = [&](uint32_t* word) {
      fence_proxy_async_all();
      __threadfence();
      atom_add_acq_rel_gpu(word, 1u);
    };

    for (int item = worker; item < total_items && ok; item += n_workers) {
      const Item it = decode(item);
      const PhaseShape& s = shape[it.phase];
      const GemmParams& gp = p.gemm[it.phase];
      const bool residual = it.phase != 1;
      const int chunk_cols = residual ? 32 : 64;
      const int chunks = s.bn / chunk_cols;
      const int row0 = it.m0 + quarter * 32;

      auto prefetch_residual = [&](int chunk, int b) {
        tma_store_wait_read<0>();   // the store issued last read this very buffer
        mbar_expect_tx(my_res_bar + 8 * b, kChainStagingBytes);
        tma_load_2d(my_stage + b * kChainStagingBytes, &gp.tmap_res[it.g], it.n0 + chunk * 32, row0, my_res_bar + 8 * b);
      };
      if (pending_arrival != nullptr) {   // lane 0 only
        if (!mbar_try_wait(bar_acc_full + 8 * acc, acc_phase)) {
          tma_store_wait_complete();
          publish(pending_arrival);
          pending_arrival = nullptr;
        }
      }
      // The residual of the first chunk is requested before the accumulator is awaited when it is
      // known to be there: always in phase 0 (the layer input), in phase 2 (h1) if the row block's
      // counter already says so; otherwise right after the accumulator (whose operands waited for it).
      bool first_requested = false;
      if (e == 0 && lane == 0) CHAIN_TRACE((item - worker) / n_workers, 5);
      if (residual && lane == 0) {
        uint32_t target = 0;
        const uint32_t* dep = dependency(it, &target);
        if (dep == nullptr || ld_acquire_gpu(dep) >= target) {
          fence_proxy_async_all();
          prefetch_residual(col_group, buf);
          first_requested = true;
        }
      }
      if (!__all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8 * acc, acc_phase, abort_flag))) break;
      tc_fence_after();
      if (e == 0 && lane == 0) CHAIN_TRACE((item - worker) / n_workers, 6);
      if (residual && lane == 0 && !first_requested) {
        fence_proxy_async_all();
        prefetch_residual(col_group, buf);
      }
      const bf16* bias = gp.group[it.g].bias;
      const bool rows_in_range = row0 < m_rows;
#pragma unroll 1
      for (int chunk = col_group; chunk < chunks; chunk += COL_GROUPS) {
        const int col = it.n0 + chunk * chunk_cols;
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                               static_cast<uint32_t>(acc * kChainAccStride + chunk * chunk_cols);
        uint8_t* sbuf = my_stage_ptr + buf * kChainStagingBytes;
        if (residual) {
          if (lane == 0 && chunk + COL_GROUPS < chunks) prefetch_residual(chunk + COL_GROUPS, buf ^ 1);
          __syncwarp();
          uint32_t v[32];
          tmem_ld_32x32(taddr, v);
          tmem_ld_wait();
          if (!__all_sync(0xffffffffu, mbar_wait(my_res_bar + 8 * buf, res_phase[buf], abort_flag))) {
            ok = false;
            break;
          }
          res_phase[buf] ^= 1u;
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
        } else {
          if (lane == 0) tma_store_wait_read<1>();   // the store that last read this staging buffer
          __syncwarp();
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t v[32];
            tmem_ld_32x32(taddr + half * 32, v);
            tmem_ld_wait();
            const uint4* bias4 = reinterpret_cast<const uint4*>(bias + col + half * 32);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint4 b = __ldg(bias4 + q);
              const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
              uint32_t ow[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float x0 = gelu_erf(__uint_as_float(v[q * 8 + 2 * j]) + bf16_lo(bw[j]));
                const float x1 = gelu_erf(__uint_as_float(v[q * 8 + 2 * j + 1]) + bf16_hi(bw[j]));
                ow[j] = pack_bf16(x0, x1);
              }
              *reinterpret_cast<uint4*>(sbuf + staging_off(lane, half * 4 + q)) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
            }
          }
        }
        fence_async_shared();
        __syncwarp();
        if (lane == 0) {
          // (a warp whose rows all lie beyond the rows in use stores nothing but still arrives)
          if (rows_in_range) tma_store_2d(&gp.tmap_out[it.g], my_stage + buf * kChainStagingBytes, col, row0);
          tma_store_commit();
          if (pending_arrival != nullptr) {
            // the previous tile's stores precede the group just committed
            tma_store_wait_complete_but<1>();
            publish(pending_arrival);
            pending_arrival = nullptr;
          }
        }
        buf ^= 1;
      }
      if (!ok) break;
      // the accumulator is drained: the MMA thread may reuse it
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_acc_empty + 8 * acc);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      if (e == 0 && lane == 0) CHAIN_TRACE((item - worker) / n_workers, 7);
      if (lane == 0)
        pending_arrival = sync_word(it.g, it.row_block,
                                    it.phase == 0 ? kSyncArrive0 : (it.phase == 1 ? kSyncArrive1 : kSyncArrive2));
    }
    if (lane == 0) {
      tma_store_wait_complete();   // also: shared memory must outlive the stores that still read it
      if (pending_arrival != nullptr && !*abort_flag) publish(pending_arrival);
    }
    __syncwarp();
  }

  // ------------------------------ teardown ------------------------------------
  tc_fence_before();
  __syncwarp();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag && p.gemm[0].status != nullptr) atomicOr(p.gemm[0].status, kFlagWaitTimeout);
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, kChainTmemCols);
  }
}

}  // namespace

#ifdef MT_CHAIN_TRACE
}  // namespace mt
// Tuning aid: switch the timeline on or off for the launches that follow / copy it out (host buffer of
// 160 * 16 * 12 uint64).
extern "C" int mt_debug_chain_trace_enable(int on) {
  return cudaMemcpyToSymbol(mt::g_chain_trace_on, &on, sizeof(int)) == cudaSuccess ? 0 : 1;
}
extern "C" int mt_debug_chain_trace_read(unsigned long long* host) {
  return cudaMemcpyFromSymbol(host, mt::g_chain_trace, sizeof(mt::g_chain_trace)) == cudaSuccess ? 0 : 1;
}
namespace mt {
#endif

size_t chain_sync_bytes(int groups, int64_t rows) {
  const int64_t blocks = (rows + kGemmBlockM - 1) / kGemmBlockM;
  return static_cast<size_t>(groups) * static_cast<size_t>(blocks) * 4 * sizeof(uint32_t);
}

bool chain_supported(int hidden, int ffn) {
  return (hidden == 768 || hidden == 1024) && hidden % 128 == 0 && ffn % 128 == 0;
}

int chain_block_n(int phase, int N, int64_t rows, int groups, int sm_count) {
  // 192-wide tiles stage fewer bytes per FLOP; 128-wide ones cut the list finer, which matters for the
  // last phase (nothing follows it that could fill the machine while its last tiles finish) and
  // whenever a phase has fewer tiles than there are SMs.
  if (N % 192 != 0) return 128;
  if (phase == 1) return 192;
  const int64_t m_tiles = (rows + kGemmBlockM - 1) / kGemmBlockM;
  const int64_t tiles_192 = m_tiles * (N / 192) * groups;
  return tiles_192 >= 3 * static_cast<int64_t>(sm_count > 0 ? sm_count : 1) ? 192 : 128;
}

cudaError_t launch_chain(const ChainParams& p, int sm_count, cudaStream_t stream) {
  const int groups = p.gemm[0].n_groups;
  if (groups < 1 || groups > kMaxGroups || p.sync == nullptr) return cudaErrorInvalidValue;
  int64_t items = 0;
  for (int ph = 0; ph < 3; ++ph) {
    const GemmParams& g = p.gemm[ph];
    if (g.n_groups != groups || g.M != p.gemm[0].M || g.m_valid != p.gemm[0].m_valid || g.pair != 0 || g.M < 1 ||
        g.K % kGemmBlockK != 0 || (g.block_n != 128 && g.block_n != 192) || g.N % g.block_n != 0)
      return cudaErrorInvalidValue;
    items += static_cast<int64_t>((g.M + kGemmBlockM - 1) / kGemmBlockM) * (g.N / g.block_n) * groups;
  }
  if (p.sync_blocks < (p.gemm[0].M + kGemmBlockM - 1) / kGemmBlockM) return cudaErrorInvalidValue;
  if ((p.ln[0].hidden != 768 && p.ln[0].hidden != 1024) || p.ln[1].hidden != p.ln[0].hidden ||
      p.gemm[0].N != p.ln[0].hidden || p.gemm[2].N != p.ln[0].hidden)
    return cudaErrorInvalidValue;
  static bool configured = false;
  static int configured_device = -1;
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (!configured || configured_device != dev) {
    err = cudaFuncSetAttribute(layer_chain_tcgen05, cudaFuncAttributeMaxDynamicSharedMemorySize, kChainSmemBytes);
    if (err != cudaSuccess) return err;
    configured = true;
    configured_device = dev;
  }
  // one CTA per SM and never more CTAs than SMs: every CTA of the grid is resident, which the
  // dependency waits rely on
  const int workers = static_cast<int>(items < sm_count ? items : sm_count);
  if (workers <= 0) return cudaSuccess;
  return launch_kernel(layer_chain_tcgen05, dim3(workers), dim3(kChainThreads), kChainSmemBytes, stream, p);
}

}  // namespace mt
