// Internal interface between the host-side scheduler and the sm_100a kernels.
// Every launcher enqueues on the given stream and returns the cudaError_t of the launch.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

namespace mt {

typedef __nv_bfloat16 bf16;

constexpr int kMaxGroups = 8;      // layers fused into one grouped launch
constexpr int kHeadDim = 64;       // the only head width implemented
constexpr int kGemmBlockM = 128;   // rows of one GEMM tile (one tcgen05 accumulator = 128 TMEM lanes)
constexpr int kGemmBlockK = 64;    // bf16 elements per 128-byte swizzled shared-memory row

constexpr uint32_t kFlagBadToken = 0x1u;
constexpr uint32_t kFlagBadSegment = 0x2u;
constexpr uint32_t kFlagBadLength = 0x4u;
constexpr uint32_t kFlagWaitTimeout = 0x8u;

// Programmatic dependent launch.  Every kernel of the path is launched with the "programmatic stream
// serialization" attribute and begins with grid_dependency_wait(): it may be scheduled, and run the
// part of its prologue that touches no global data, while the previous kernel in the stream is still
// draining, and only proceeds once that kernel has completed and its writes are visible.  Because
// every kernel waits (before its first global read or write), completion is transitive along the
// stream, exactly as with ordinary stream order.  g_use_pdl = false falls back to plain launches.
extern bool g_use_pdl;
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Per-function launch set-up (the opt-in to large dynamic shared memory, occupancy queries) is per device: this runs
// `setup(dev)` once per device and call site, under a lock, so that launches from several host threads or on
// several devices of one process never race on it.
constexpr int kMaxDevices = 64;
struct PerDeviceOnce {
  std::mutex mu;
  bool done[kMaxDevices] = {};
};
template <typename F>
cudaError_t per_device_once(PerDeviceOnce& state, F&& setup, int* device_out = nullptr) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (device_out != nullptr) *device_out = dev;
  std::lock_guard<std::mutex> lock(state.mu);
  if (!state.done[dev]) {
    e = setup(dev);
    if (e != cudaSuccess) return e;
    state.done[dev] = true;
  }
  return cudaSuccess;
}

// cluster_x > 1 launches the grid as thread-block clusters of that many CTAs along x.
template <typename Param>
cudaError_t launch_kernel(void (*kernel)(Param), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                          const Param& param, unsigned cluster_x = 1) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  if (g_use_pdl) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster_x;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, param);
}
#endif

enum GemmEpilogue { kEpiBias = 0, kEpiBiasGelu = 1, kEpiBiasResidual = 2, kEpiBiasTanhF32 = 3, kEpiPartialF32 = 4 };

// One problem of a grouped GEMM: Y_g[M,N] = epi(X_g[M,K] . W_g[N,K]^T + bias_g (+ residual_g)).
// All groups of a launch share M, N, K and the epilogue.  kEpiBias and kEpiBiasGelu write bf16;
// kEpiBiasResidual adds an fp32 residual and writes fp32 (the pre-LayerNorm sum is never rounded);
// kEpiBiasTanhF32 writes tanh(.) in fp32 (the pooler; single CTAs on 128-wide tiles only).
// kEpiPartialF32 writes the bare fp32 accumulator (no bias): the launch may then split K into k_splits equal
// ranges, one tile per (row block, group, column block, range); range s of group g writes rows
// [s * split_pitch, s * split_pitch + M) of that group's output, and whoever reads the partial sums adds them
// in the order s = 0, 1, ... (the LayerNorm kernel does, with the bias and the residual).  For launches of so
// few rows that most SMs would have no tile while each tile walks a long K by itself (64- and 128-wide
// tiles, single CTAs, bf16 operands only).
// The output and the residual are reached through the tensor maps of GemmParams.
struct GemmGroup {
  const bf16* bias;
  const float* scale_x;  // (8-bit operands) one scale per row of X, [M]
  const float* scale_w;  // (8-bit operands) one scale per row of W, [N]
};

struct alignas(64) GemmParams {
  CUtensorMap tmap_x[kMaxGroups];    // X_g: dims {K, M}, box {64, 128}, 128-byte swizzle
  CUtensorMap tmap_w[kMaxGroups];    // W_g: dims {K, N}, box {64, block_n}, 128-byte swizzle
  CUtensorMap tmap_out[kMaxGroups];  // Y_g: dims {N, M}, box {64 bf16 | 32 fp32, 32}, 128-byte swizzle
  CUtensorMap tmap_res[kMaxGroups];  // residual_g (fp32): dims {N, M}, box {32, 32}; kEpiBiasResidual only
  GemmGroup group[kMaxGroups];
  int32_t n_groups;
  int32_t M, N, K;
  const int32_t* m_valid;  // device scalar: rows actually in use (<= M); null = all M rows
  int32_t pair;            // 1: run as pairs of CTAs on 256-row tiles (the W maps then fetch half a tile's rows)
  int32_t block_n;         // tile width along N: 128, 192 or 256 (gemm_block_n); N % block_n == 0
  int32_t k_splits;        // ranges K is split into (kEpiPartialF32 only; otherwise 1): (K / 64) % k_splits == 0
  int32_t split_pitch;     // rows between the outputs of consecutive ranges (a multiple of 128, >= M)
  int32_t fp8;             // 1: X and W are E4M3 bytes (maps of uint8, boxes of 128 bytes of K) with row scales;
                           // single CTAs, block_n 256 (128 for the residual epilogue), K % 128 == 0
  uint32_t* status;        // sticky device status word (may be null)
};

// Tile width along N for a launch of `groups` problems with about `rows` rows in use each, from a cost
// model of the kernel: the tiles are dealt out in rounds over the SMs (or SM pairs), and a round costs
// about (128 + width) per 64 of K because a CTA is bound by the bytes it stages.  Fewer, wider tiles
// re-read X less; narrower ones waste less of the last round.  Every output element is accumulated
// over K in the same order whatever the width, so the choice never changes a result.
int gemm_block_n(int N, int epilogue, int64_t rows, int groups, bool pair, int sm_count);
// Width in elements of the 128-byte output box (64 bf16 or 32 fp32 columns; 32 rows).
int gemm_out_box_cols(int epilogue);
cudaError_t launch_gemm(const GemmParams& p, int epilogue, int sm_count, cudaStream_t stream);

// Token layout.  The rows of sequence b start at row_start[b] (device array of batch + 1 ints written
// by launch_row_starts: b * seq for the padded layout, the running sum of the lengths for the packed
// layout, in which only valid tokens exist).  A null row_start means the padded layout.
struct alignas(64) AttnParams {
  CUtensorMap tmap_qkv[kMaxGroups];  // qkv_g: dims {3H, rows}, box {64, 128}, 128-byte swizzle (tensor-memory kernel only)
  CUtensorMap tmap_qkv64[kMaxGroups];  // the same with a box of 64 rows: sequences of at most 64 tokens fetch half
  const bf16* qkv[kMaxGroups];  // [rows, 3*H] = [Q | K | V]
  bf16* ctx[kMaxGroups];        // [rows, H]
  const int32_t* lengths;       // [B]
  const int32_t* row_start;     // [B + 1] or null
  int32_t packed;               // 1: no padded rows exist, nothing is written beyond a sequence's length
  int32_t n_groups, batch, seq, heads;
  int32_t tensor_memory;        // 1: the tcgen05 kernel (seq <= 128, tmap_qkv filled); 0: the mma.sync kernel
  uint32_t* status;             // sticky device status word (may be null)
};
// Longest sequence the tensor-memory attention kernels handle (up to 128 tokens: one CTA holds all keys of a
// sequence; longer: tiles of 128 queries walk the keys in tiles of 128).
constexpr int kAttnTensorMemoryMaxSeq = 512;
constexpr int kAttnTileRows = 128;   // rows of the Q/K/V boxes of the tensor maps
cudaError_t launch_attention(const AttnParams& p, cudaStream_t stream);
cudaError_t launch_attention_tc(const AttnParams& p, cudaStream_t stream);

// Attention of the first token of every sequence only (the last layer of a task branch: its head
// reads nothing but that row).  Writes the context compactly, ctx[b, :], and gathers the fp32
// residual of that row from the layer input, res[b, :] = in32[row_start[b], :].
struct ClsAttnParams {
  const bf16* qkv[kMaxGroups];   // [rows, 3*H]
  const float* in32[kMaxGroups]; // [rows, H] fp32 layer input
  bf16* ctx[kMaxGroups];         // [B, H]
  float* res[kMaxGroups];        // [B, H]
  const int32_t* lengths;
  const int32_t* row_start;      // [B + 1] or null (padded layout)
  int32_t n_groups, batch, seq, heads;
};
cudaError_t launch_cls_attention(const ClsAttnParams& p, cudaStream_t stream);

// y = LN(x): x fp32; y is written as bf16 (the next GEMM's operand) and, if y32 is not null, also
// as fp32 (the residual of the next sub-layer, so the residual stream is never rounded to bf16).
// y = LayerNorm(x) row by row.  With n_parts > 0 the row is first put together from the partial sums of a GEMM
// whose K was split (kEpiPartialF32): x = residual + ((part_0 + part_1 + ... in this order) + bias), the
// arithmetic of the residual epilogue with the sum over K taken range by range; `x` is then not read.
struct LayerNormParams {
  const float* x[kMaxGroups];
  const float* part[kMaxGroups];      // [n_parts][part_pitch rows][hidden] fp32
  const float* residual[kMaxGroups];  // [rows][hidden] fp32
  const bf16* bias[kMaxGroups];       // [hidden]
  int32_t n_parts, part_pitch;
  const bf16* gamma[kMaxGroups];
  const bf16* beta[kMaxGroups];
  bf16* y[kMaxGroups];
  float* y32[kMaxGroups];
  int32_t n_groups, rows, hidden;
  const int32_t* rows_valid;  // device scalar: rows actually in use (<= rows); null = all
  float eps;
};
cudaError_t launch_layernorm(const LayerNormParams& p, cudaStream_t stream);

// Residual GEMM with the LayerNorm that follows it, in one launch:
//   Y_g = LN( X_g[M,K] . W_g[N,K]^T + bias_g + residual_g ) * gamma_g + beta_g      N = hidden
// written twice, bf16 (the next GEMM's operand) and fp32 (the next residual).  The N / 128 CTAs that hold
// the column blocks of one block of 128 rows form a thread-block cluster and exchange per-row partial
// statistics through distributed shared memory, so the pre-normalisation sum never goes to global memory.
struct alignas(64) GemmLnParams {
  CUtensorMap tmap_x[kMaxGroups];     // X_g: dims {K, M}, box {64, 128}
  CUtensorMap tmap_w[kMaxGroups];     // W_g: dims {K, N}, box {64, 128}
  CUtensorMap tmap_w256[kMaxGroups];  // W_g with a box of 256 rows (the kernel on 256-column tiles)
  CUtensorMap tmap_res[kMaxGroups];   // residual_g fp32: dims {N, M}, box {32, 32}
  CUtensorMap tmap_y[kMaxGroups];     // Y_g bf16: dims {N, M}, box {64, 32}
  CUtensorMap tmap_y32[kMaxGroups];   // Y_g fp32: dims {N, M}, box {32, 32}
  const float* residual[kMaxGroups];  // the same residual by pointer (fp32 [M, N]; the kernel on 256-column tiles)
  const bf16* bias[kMaxGroups];
  const bf16* gamma[kMaxGroups];
  const bf16* beta[kMaxGroups];
  int32_t n_groups;
  int32_t M, N, K;
  const int32_t* m_valid;  // device scalar: rows actually in use (<= M); null = all M rows
  float eps;
  uint32_t* status;        // sticky device status word (may be null)
};
// N must be 768 or 1024 (clusters of 6 or 8 CTAs), K a multiple of 64.
bool gemm_ln_supported(int N);
cudaError_t launch_gemm_ln(const GemmLnParams& p, cudaStream_t stream);
// The same on 128 x 256 accumulator tiles, clusters of N / 256 CTAs (tmap_w256 and residual filled): identical bits,
// half the CTAs per row block and full-rate tcgen05.mma - for launches with many row blocks.
bool gemm_ln_wide_supported(int N);
cudaError_t launch_gemm_ln_wide(const GemmLnParams& p, cudaStream_t stream);

struct EmbedParams {
  const int32_t* token_ids;
  const int32_t* segment_ids;
  const int32_t* lengths;
  const bf16 *word, *pos, *type, *gamma, *beta;
  bf16* out;
  float* out32;  // may be null
  const int32_t* row_start;  // [B + 1] or null (padded layout)
  int32_t packed;            // 1: positions >= length are skipped
  int32_t batch, seq, hidden, vocab, type_vocab;
  float eps;
  uint32_t* status;
};
cudaError_t launch_embed(const EmbedParams& p, cudaStream_t stream);

struct HeadTask {
  const bf16* hidden;  // final state of the task, [rows, H]; the first row of every sequence is pooled
  const bf16 *pool_w, *pool_b, *cls_w, *cls_b;
  int32_t num_classes, col0;
  int32_t compact;  // 1: `hidden` is [B, H], one row per sequence (last branch layer computed for that row only)
};
struct HeadParams {
  HeadTask task[kMaxGroups];
  float* logits;
  float* pooled;  // scratch, fp32 [n_tasks][batch][hidden]: tanh pooler outputs between the two launches
  const int32_t* row_start;  // [B + 1] or null (padded layout: sequence b starts at row b * seq)
  int32_t n_tasks, batch, seq, hidden, logits_stride;
};

// Token-level heads: logits[(b * seq + pos) * logits_stride + col0_t + c] = cls_w_t[c, :] . h_t[row(b, pos), :] + cls_b_t[c]
// for every valid position of every sequence; positions >= length are not written.
struct TokenHeadParams {
  const bf16* hidden_state[kMaxGroups];  // final state of the task, [rows, H]
  const bf16* cls_w[kMaxGroups];
  const bf16* cls_b[kMaxGroups];
  int32_t num_classes[kMaxGroups], col0[kMaxGroups];
  float* logits;             // fp32 [batch, seq, logits_stride]
  const int32_t* lengths;
  const int32_t* row_start;  // [B + 1] or null (padded layout)
  int32_t n_tasks, batch, seq, hidden, logits_stride;
};
cudaError_t launch_token_heads(const TokenHeadParams& p, cudaStream_t stream);

// Row-wise quantisation to E4M3 for the 8-bit GEMMs: scale[r] = max|x[r, :]| * (1 / 448) (1 for a row of zeros),
// q[r, c] = the E4M3 value nearest to x[r, c] / scale[r] (ties to even, saturating), all in fp32.
struct QuantParams {
  const bf16* x[kMaxGroups];   // [rows, cols]
  uint8_t* q[kMaxGroups];      // [rows, cols]
  float* scale[kMaxGroups];    // [rows]
  int32_t n_groups, rows, cols;   // cols a multiple of 256
  const int32_t* rows_valid;   // device scalar: rows actually in use (<= rows); null = all
};
cudaError_t launch_quantize_rows(const QuantParams& p, cudaStream_t stream);

// The kernels' bounded mbarrier wait run on a barrier that nothing completes (arrive == 0) or that is complete
// (arrive != 0), with a limit of the caller's choosing: waited_ns[2] and ok_out[2] (device) receive, per warp, how
// long the wait took and whether it succeeded; status gets kFlagWaitTimeout when a wait ran out (wait_probe.cu).
cudaError_t launch_wait_probe(unsigned long long limit_ns, int arrive, uint32_t* status, unsigned long long* waited_ns,
                              int* ok_out, cudaStream_t stream);

// row_start[b] for b = 0..batch and *rows_valid = row_start[batch]: b * seq (padded) or the running sum
// of the lengths clamped to [1, seq] (packed).
cudaError_t launch_row_starts(const int32_t* lengths, int32_t batch, int32_t seq, int32_t packed, int32_t* row_start,
                              int32_t* rows_valid, cudaStream_t stream);
// padded[b*seq + pos] = packed[row_start[b] + pos] for pos < length, 0 elsewhere (bf16 rows of `hidden`).
// With compact != 0 the source is [B, H] (first tokens only) and only position 0 of a sequence is filled.
cudaError_t launch_unpack_rows(const bf16* packed, const int32_t* lengths, const int32_t* row_start, bf16* padded,
                               int32_t batch, int32_t seq, int32_t hidden, int32_t compact, cudaStream_t stream);
// Two launches: pooler (tanh features into `pooled`), then head (logits).
cudaError_t launch_pooler_head(const HeadParams& p, cudaStream_t stream);
// The head alone, for a caller that has filled `pooled` itself (the pooler as a grouped GEMM).
cudaError_t launch_head(const HeadParams& p, cudaStream_t stream);

}  // namespace mt
