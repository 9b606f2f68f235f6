// C-ABI boundary, weight arena and tree scheduler of the merged multi-task forward pass.
//
// Model merging (paper Section 3.3) = one weight arena holding the shared trunk once and every
// task's own layers, plus a static schedule over the resulting tree: wave w runs trunk layer w
// together with every branch layer whose input is ready (branch layer j of a task that forks at
// depth d runs in wave d + j), all as groups of the same kernel launches.  The trunk state at a
// fork depth stays resident until the wave after it has consumed it (two ping-pong trunk buffers
// are enough because every reader of depth d runs in wave d + 1); tasks masked off by task_mask
// contribute no branch, no head, and do not extend the trunk depth.

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <tuple>
#include <vector>

#include "../../include/mt_bert.h"
#include "mt_kernels.h"

using namespace mt;

namespace mt {
bool g_use_pdl = true;
}
static int g_force_block_n = 0;   // tile width forced on mt_kernel_linear (tuning aid), 0 = chosen by gemm_block_n

namespace {

constexpr uint32_t kBlobMagic = 0x4D544257u;
constexpr uint32_t kBlobVersion = 1u;
constexpr size_t kAlign = 256;
constexpr size_t kHeaderBytes = 256;
// rows between the partial sums of consecutive ranges of K: whole 128-row blocks
constexpr size_t split_pitch(size_t rows) { return (rows + 127) / 128 * 128; }
// The FFN-down projection of a launch of few rows is split into this many ranges of K (option "ffn_down_split").
constexpr int32_t kDownSplits = 4;
// "Few rows": at most this many per layer (batch 4 x 128 tokens; the first-token tails of batches up to 512).
constexpr int32_t kSplitRowsMax = 512;

inline size_t pad256(size_t n) { return (n + kAlign - 1) / kAlign * kAlign; }

// Offsets (bytes from the start of the arena = start of the blob payload) of one layer's tensors.
struct LayerOffsets {
  size_t wq, wk, wv, bq, bk, bv, wo, bo, ln1_g, ln1_b, w1, b1, w2, b2, ln2_g, ln2_b;
  // 8-bit copies (option "fp8_gemm"), behind the payload of the blob: E4M3 bytes and one fp32 scale per output row
  size_t q_qkv, s_qkv, q_w1, s_w1, q_w2, s_w2;
};

struct TaskEntry {
  mt_task_config cfg;
  std::vector<LayerOffsets> layers;
  size_t pool_w, pool_b, cls_w, cls_b;
  size_t section_begin, section_bytes;
  int32_t col0;
  bool loaded;
};

struct BlobHeader {
  uint32_t magic, version, kind;
  int32_t hidden, heads, ffn, trunk_layers, vocab, max_position, type_vocab;
  int32_t n_tasks, task_index, fork_depth, branch_layers, num_classes, reserved;
  uint64_t payload_bytes;
};

// ---- logical schedule (no device pointers) -----------------------------------------------------

struct OpDesc {
  int32_t task;   // -1 = trunk
  int32_t layer;  // trunk: depth produced (1..D); branch: 1..k_t
};
struct Schedule {
  int32_t trunk_depth = 0;
  int32_t n_layers = 0;
  std::vector<std::vector<OpDesc>> waves;       // waves[w-1] = layers of wave w
  std::vector<std::vector<int32_t>> heads;      // heads[w] = tasks whose head runs after wave w (0 = after embedding)
};

// ---- bound plan (device pointers, tensor maps) --------------------------------------------------

// Everything of a layer after the QKV projection, for a set of layers that share the row count.
struct LayerTail {
  GemmParams attn_out, ffn_up, ffn_down;
  LayerNormParams ln1, ln2;
  int32_t count = 0;
  // each residual GEMM together with the LayerNorm after it, as one cluster launch (option "fused_ln")
  bool ln_fused = false;
  bool ln_wide = false;      // ... on 128 x 256 accumulator tiles (clusters of N / 256): launches with many row blocks
  bool down_fused = false;   // the FFN-down projection too (not with 8-bit operands: that GEMM is the plain kernel)
  // launches of few rows: the FFN-down projection as partial sums over `down_splits` ranges of K, put together
  // (ranges in order, bias, residual) by the LayerNorm kernel after it
  int32_t down_splits = 1;
  GemmLnParams attn_out_ln, ffn_down_ln;
  // 8-bit operands: the inputs of the FFN-up and FFN-down projections are quantised row by row first
  bool fp8 = false;
  QuantParams q_h1, q_f;
};
struct DumpCopy {
  const bf16* src;
  int32_t slot;
  bool compact;  // [B, H]: first tokens only
};
// One chunk of a wave: the QKV projection of all its layers in one launch, then the rest of the
// layer for the layers computed on every token (`full`).  The last layers of task branches are
// needed for the first token of every sequence only: in their wave they get the QKV projection (keys
// and values of all tokens) and the first-token attention (`attn_cls`, `n_cls` groups); the rest of
// those layers, a few rows each, is run for all tasks together after the last wave (a `cls tail` step).
struct Chunk {
  QuantParams q_in;   // 8-bit operands: the layers' inputs, quantised row by row before the Q/K/V projection
  GemmParams qkv;
  AttnParams attn;
  ClsAttnParams attn_cls;
  LayerTail full;
  int32_t n_cls = 0;
  std::vector<DumpCopy> dumps;
};
struct PlanStep {
  int kind;  // 0 = chunk, 1 = heads, 2 = cls tail, 3 = token-level heads
  TokenHeadParams token_heads;
  Chunk chunk;
  HeadParams heads;
  bool pool_gemm = false;           // heads step: the pooler runs as a grouped GEMM (`pool`), then the head kernel
  GemmParams pool;
  std::vector<int32_t> head_tasks;  // tasks of a heads step, in group order
  LayerTail tail;
  std::vector<DumpCopy> dumps;
};
struct Plan {
  std::vector<PlanStep> steps;
  int32_t launches = 0;
  uint64_t last_use = 0;  // stamp of the last forward that ran this plan (least recently used goes first)
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

std::mutex g_driver_mutex;
EncodeTiledFn g_encode = nullptr;

cudaError_t get_encoder(EncodeTiledFn* out) {
  std::lock_guard<std::mutex> lock(g_driver_mutex);
  if (g_encode == nullptr) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t err = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (err != cudaSuccess) return err;
    if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return cudaErrorNotSupported;
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  *out = g_encode;
  return cudaSuccess;
}

// Tensor map of a row-major matrix [rows, cols] (bf16, or fp32 when `fp32`) accessed in boxes of
// box_rows x box_cols whose rows are 128 bytes, with the 128-byte swizzle; out-of-range parts of a
// box read as zero and are skipped on stores.
cudaError_t make_tmap(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int box_rows, int box_cols,
                      bool fp32) {
  EncodeTiledFn enc = nullptr;
  cudaError_t err = get_encoder(&enc);
  if (err != cudaSuccess) return err;
  const size_t elem_bytes = fp32 ? sizeof(float) : sizeof(bf16);
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * elem_bytes};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t elem[2] = {1, 1};
  CUresult r = enc(map, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                   const_cast<void*>(base), dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// Tensor map of a row-major matrix [rows, cols] of bytes (E4M3 operands) accessed in boxes of box_rows x 128.
cudaError_t make_tmap_u8(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int box_rows) {
  EncodeTiledFn enc = nullptr;
  cudaError_t err = get_encoder(&enc);
  if (err != cudaSuccess) return err;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols)};
  const cuuint32_t box[2] = {128u, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t elem[2] = {1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, elem,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// Fills group i of a grouped GEMM Y = epi(X[M,K] . W[N,K]^T + bias (+ residual)): operand maps, the
// output map (bf16, or fp32 for the residual epilogue) and the fp32 residual map.
cudaError_t set_gemm_group(GemmParams* g, int i, int epilogue, const void* x, const void* w, const bf16* bias,
                           const float* residual, void* y) {
  const int M = g->M, N = g->N, K = g->K;
  const bool res = epilogue == kEpiBiasResidual;
  const bool f32_out = res || epilogue == kEpiBiasTanhF32 || epilogue == kEpiPartialF32;
  cudaError_t e;
  if (g->fp8 != 0) {
    if ((e = make_tmap_u8(&g->tmap_x[i], x, M, K, kGemmBlockM)) != cudaSuccess) return e;
    if ((e = make_tmap_u8(&g->tmap_w[i], w, N, K, g->block_n)) != cudaSuccess) return e;
  } else {
    if ((e = make_tmap(&g->tmap_x[i], x, M, K, kGemmBlockM, kGemmBlockK, false)) != cudaSuccess) return e;
    if ((e = make_tmap(&g->tmap_w[i], w, N, K, g->block_n / (g->pair != 0 ? 2 : 1), kGemmBlockK, false)) != cudaSuccess) return e;
  }
  if ((e = make_tmap(&g->tmap_out[i], y, M, N, 32, gemm_out_box_cols(epilogue), f32_out)) != cudaSuccess) return e;
  if (res && (e = make_tmap(&g->tmap_res[i], residual, M, N, 32, 32, true)) != cudaSuccess) return e;
  g->group[i].bias = bias;
  return cudaSuccess;
}

}  // namespace

struct mt_model {
  mt_trunk_config trunk;
  std::vector<TaskEntry> tasks;
  int32_t max_batch, max_seq, c_total, ct_total;  // columns of the sequence-level / of the token-level tasks

  // arena
  size_t emb_word, emb_pos, emb_type, emb_ln_g, emb_ln_b;
  std::vector<LayerOffsets> trunk_layers;
  size_t payload_bytes;   // the blob's payload = the bf16 part of the arena
  size_t weights_bytes;   // payload + (option "fp8_gemm") the 8-bit copies
  bool trunk_loaded;

  // options
  int32_t max_groups;
  bool debug_capture;
  bool pack_tokens;  // packed token layout: only valid tokens are stored and computed
  bool cls_only;     // the last layer of a task branch is evaluated for the first token of a sequence only
  int64_t expected_tokens;  // caller's estimate of the valid tokens per batch (0 = every row); tunes tile shapes only
  bool attention_tc;  // attention on tcgen05 with tensor-memory accumulators when seq <= 128 (else mma.sync)
  int32_t gemm_pair;  // GEMMs as pairs of CTAs on 256-row tiles (cta_group::2): 0 never, 1 always, 2 by launch size
  bool early_heads;  // every task's head (and first-token tail) runs right after the wave that finishes its branch
  int32_t fused_ln;  // each residual GEMM and the LayerNorm after it as one cluster launch: 0 never, 1 always on
                     // 128-column tiles, 3 always on 256-column tiles, 2 by the launch (fused_ln_kind)
  int32_t fused_ln_max_groups;
  int32_t ffn_down_split;   // 0: never; 1: launches of few rows split the K of the FFN-down projection (default)
  int32_t fused_ln_max_rows;
  // The first-token attention of the branches that end in a wave depends on the wave's QKV projection only
  // and feeds nothing before the first-token tails, so it runs on a stream of the library's own beside the
  // wave's other kernels (fork after the projection, join before the next step); option "overlap_cls".
  bool overlap_cls;
  cudaStream_t side_stream;
  cudaEvent_t ev_fork, ev_join;
  bool fp8;          // Q/K/V, FFN-up and FFN-down projections on E4M3 operands (set before mt_bind_memory)
  bool pool_gemm;    // the pooler of tasks with a compact final state runs as a grouped GEMM on the tensor cores

  // device memory (caller-owned)
  uint8_t* d_weights;
  uint8_t* d_workspace;
  size_t ws_bytes_bound;
  int sm_count;    // SMs the persistent GEMM grids are sized for: all of the device's, or option "sm_limit"
  int sm_device, sm_limit;

  // workspace layout (byte offsets)
  size_t ws_status, ws_rows_valid, ws_row_start, ws_tok, ws_seg, ws_len, ws_logits, ws_pooled, ws_partial, ws_trunk[2], ws_task0,
      ws_slot0, ws_cls0, ws_dump0;
  size_t slot_q_off, cls_q_off;   // 8-bit scratch inside a slot / inside a task's first-token scratch
  size_t cls_bytes, cls_h_bytes, cls_h32_bytes;  // per-task first-token scratch and its [B,H] bf16 / fp32 pieces
  size_t act_bytes;    // max_batch*max_seq*hidden bf16
  size_t act32_bytes;  // the same tensor in fp32
  size_t state_bytes;  // one hidden state = its bf16 copy (GEMM operand) followed by its fp32 copy (residual)
  size_t slot_bytes;
  int32_t n_slots, n_dump;
  size_t ws_total;

  std::map<std::tuple<uint64_t, int32_t, int32_t>, Plan> plans;  // at most plan_cache entries
  int32_t plan_cache;
  uint64_t use_clock;
  int32_t last_batch, last_seq;
  const int32_t* last_lengths;  // device lengths of the last forward (for mt_debug_copy_hidden)

  // optional per-launch timing (option "profile"): event pairs recorded around every launch
  bool profile;
  std::vector<cudaEvent_t> events;                 // pool, two per recorded launch
  std::vector<int32_t> event_class;                // class of the i-th recorded launch
  size_t events_used;
  std::string last_error;
};

namespace {

int fail(const mt_model* m, int code, const std::string& msg) {
  if (m != nullptr) const_cast<mt_model*>(m)->last_error = msg;
  return code;
}
int fail_cuda(const mt_model* m, cudaError_t e, const char* what) {
  return fail(m, MT_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

size_t place_layer(const mt_trunk_config& c, size_t off, LayerOffsets* lo) {
  const size_t H = c.hidden, F = c.ffn, e = sizeof(bf16);
  auto take = [&](size_t elems) { size_t at = off; off += pad256(elems * e); return at; };
  lo->wq = take(H * H); lo->wk = take(H * H); lo->wv = take(H * H);
  lo->bq = take(H); lo->bk = take(H); lo->bv = take(H);
  lo->wo = take(H * H); lo->bo = take(H);
  lo->ln1_g = take(H); lo->ln1_b = take(H);
  lo->w1 = take(F * H); lo->b1 = take(F);
  lo->w2 = take(H * F); lo->b2 = take(H);
  lo->ln2_g = take(H); lo->ln2_b = take(H);
  return off;
}

// The 8-bit copies live behind the blob's payload, so the bf16 part of the arena stays a verbatim copy of it.
void layout_fp8_weights(mt_model* m) {
  size_t off = m->payload_bytes;
  if (m->fp8) {
    const size_t H = m->trunk.hidden, F = m->trunk.ffn;
    auto take = [&](size_t bytes) { size_t at = off; off += pad256(bytes); return at; };
    auto place = [&](LayerOffsets* lo) {
      lo->q_qkv = take(3 * H * H); lo->s_qkv = take(3 * H * 4);
      lo->q_w1 = take(F * H); lo->s_w1 = take(F * 4);
      lo->q_w2 = take(H * F); lo->s_w2 = take(H * 4);
    };
    for (LayerOffsets& lo : m->trunk_layers) place(&lo);
    for (TaskEntry& t : m->tasks)
      for (LayerOffsets& lo : t.layers) place(&lo);
  }
  m->weights_bytes = off;
}

// Quantises the Q/K/V, FFN-up and FFN-down matrices of `layers` (already in the arena as bf16) into their 8-bit
// copies: one scale per output channel = per row of W[N, K].  Grouped launches of up to kMaxGroups layers.
cudaError_t quantize_layer_weights(const mt_model* m, const std::vector<const LayerOffsets*>& layers, cudaStream_t stream) {
  const int32_t H = m->trunk.hidden, F = m->trunk.ffn;
  for (size_t first = 0; first < layers.size(); first += kMaxGroups) {
    const size_t count = std::min<size_t>(kMaxGroups, layers.size() - first);
    for (int which = 0; which < 3; ++which) {
      QuantParams q;
      memset(&q, 0, sizeof(q));
      q.n_groups = static_cast<int32_t>(count);
      q.rows = which == 0 ? 3 * H : (which == 1 ? F : H);
      q.cols = which == 2 ? F : H;
      for (size_t i = 0; i < count; ++i) {
        const LayerOffsets* lo = layers[first + i];
        const size_t src = which == 0 ? lo->wq : (which == 1 ? lo->w1 : lo->w2);
        const size_t dst = which == 0 ? lo->q_qkv : (which == 1 ? lo->q_w1 : lo->q_w2);
        const size_t sc = which == 0 ? lo->s_qkv : (which == 1 ? lo->s_w1 : lo->s_w2);
        q.x[i] = reinterpret_cast<const bf16*>(m->d_weights + src);
        q.q[i] = m->d_weights + dst;
        q.scale[i] = reinterpret_cast<float*>(m->d_weights + sc);
      }
      cudaError_t e = launch_quantize_rows(q, stream);
      if (e != cudaSuccess) return e;
    }
  }
  return cudaSuccess;
}

void layout_workspace(mt_model* m) {
  const size_t M = static_cast<size_t>(m->max_batch) * m->max_seq;
  const size_t H = m->trunk.hidden, F = m->trunk.ffn;
  m->act_bytes = pad256(M * H * sizeof(bf16));
  m->act32_bytes = pad256(M * H * sizeof(float));
  m->state_bytes = m->act_bytes + m->act32_bytes;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t at = off; off += pad256(bytes); return at; };
  m->ws_status = take(256);
  m->ws_rows_valid = take(256);
  m->ws_row_start = take((static_cast<size_t>(m->max_batch) + 1) * 4);
  m->ws_tok = take(M * 4);
  m->ws_seg = take(M * 4);
  m->ws_len = take(static_cast<size_t>(m->max_batch) * 4);
  m->ws_logits = take(static_cast<size_t>(m->max_batch) * m->c_total * 4);
  // tanh pooler outputs of the tasks of one head launch: fp32 [kMaxGroups][max_batch][H]
  m->ws_pooled = take(static_cast<size_t>(kMaxGroups) * m->max_batch * H * sizeof(float));
  // partial sums of the FFN-down projection in launches of few rows: fp32 [group][range of K][row pitch][H]
  m->ws_partial = take(static_cast<size_t>(kMaxGroups) * kDownSplits * split_pitch(std::min<size_t>(M, kSplitRowsMax)) * H * sizeof(float));
  m->ws_trunk[0] = take(m->state_bytes);
  m->ws_trunk[1] = take(m->state_bytes);
  m->ws_task0 = off;
  off += m->state_bytes * m->tasks.size();
  m->n_slots = std::min<int32_t>(m->max_groups, static_cast<int32_t>(m->tasks.size()) + 1);
  // slot = qkv [M,3H] bf16 + ctx [M,H] bf16 + u [M,H] fp32 + h1 [M,H] bf16 and fp32 + f [M,F] bf16
  m->slot_bytes = pad256(M * 3 * H * 2) + m->act_bytes + m->act32_bytes + m->state_bytes + pad256(M * F * 2);
  m->slot_q_off = m->slot_bytes;
  // 8-bit operands: E4M3 copies of the layer input and of h1 ([M,H]) and of f ([M,F]), each with a scale per row
  if (m->fp8) m->slot_bytes += 2 * pad256(M * H) + pad256(M * F) + 3 * pad256(M * 4);
  m->ws_slot0 = off;
  off += m->slot_bytes * m->n_slots;
  // per task, for its last branch layer on first tokens: ctx bf16, residual fp32, u fp32, h1 bf16 + fp32 (all
  // [B,H]) and f bf16 [B,F]
  m->cls_h_bytes = pad256(static_cast<size_t>(m->max_batch) * H * 2);
  m->cls_h32_bytes = pad256(static_cast<size_t>(m->max_batch) * H * 4);
  m->cls_bytes = 2 * m->cls_h_bytes + 3 * m->cls_h32_bytes + pad256(static_cast<size_t>(m->max_batch) * F * 2);
  m->cls_q_off = m->cls_bytes;
  if (m->fp8) {
    const size_t B = static_cast<size_t>(m->max_batch);
    m->cls_bytes += pad256(B * H) + pad256(B * F) + 2 * pad256(B * 4);
  }
  m->ws_cls0 = off;
  off += m->cls_bytes * m->tasks.size();
  m->n_dump = 0;
  m->ws_dump0 = off;
  if (m->debug_capture) {
    m->n_dump = m->trunk.trunk_layers + 1;
    for (const TaskEntry& t : m->tasks) m->n_dump += t.cfg.branch_layers;
    off += m->act_bytes * m->n_dump;
  }
  m->ws_total = off;
}

int32_t dump_slot(const mt_model* m, int32_t task, int32_t layer) {
  if (task < 0) return layer;  // 0..trunk_layers
  int32_t idx = m->trunk.trunk_layers + 1;
  for (int32_t t = 0; t < task; ++t) idx += m->tasks[t].cfg.branch_layers;
  return idx + layer - 1;
}

bool build_schedule(const mt_model* m, uint64_t mask, Schedule* s) {
  const int32_t T = static_cast<int32_t>(m->tasks.size());
  if (T < 64) mask &= (uint64_t(1) << T) - 1;
  if (mask == 0) return false;
  int32_t depth = 0, last_wave = 0, layers = 0;
  for (int32_t t = 0; t < T; ++t) {
    if (!((mask >> t) & 1)) continue;
    const mt_task_config& c = m->tasks[t].cfg;
    depth = std::max(depth, c.fork_depth);
    last_wave = std::max(last_wave, c.fork_depth + c.branch_layers);
    layers += c.branch_layers;
  }
  s->trunk_depth = depth;
  s->n_layers = depth + layers;
  s->waves.assign(last_wave, {});
  s->heads.assign(last_wave + 1, {});
  for (int32_t w = 1; w <= last_wave; ++w) {
    if (w <= depth) s->waves[w - 1].push_back({-1, w});
    for (int32_t t = 0; t < T; ++t) {
      if (!((mask >> t) & 1)) continue;
      const mt_task_config& c = m->tasks[t].cfg;
      const int32_t j = w - c.fork_depth;
      if (j >= 1 && j <= c.branch_layers) s->waves[w - 1].push_back({t, j});
    }
  }
  // Heads: a task without branch layers pools the trunk state, which lives in a ping-pong buffer, so
  // its head runs right after the wave that produced that state; every other task keeps its final
  // state in its own buffer and, for throughput, all of those heads share one launch after the last
  // wave.  With option early_heads every head runs right after the wave that finishes its task, so
  // that shallow tasks deliver before the deep ones are done (the latency limitation of Section 5.2).
  for (int32_t t = 0; t < T; ++t) {
    if (!((mask >> t) & 1)) continue;
    const mt_task_config& c = m->tasks[t].cfg;
    // (a token-level head reads every row of the final state and has no tail to share: it runs at once too)
    const bool now = c.branch_layers == 0 || m->early_heads || c.head_kind == MT_HEAD_TOKEN;
    s->heads[now ? c.fork_depth + c.branch_layers : last_wave].push_back(t);
  }
  return true;
}

bf16* ws_ptr(const mt_model* m, size_t off) { return reinterpret_cast<bf16*>(m->d_workspace + off); }
const bf16* w_ptr(const mt_model* m, size_t off) { return reinterpret_cast<const bf16*>(m->d_weights + off); }

// Where the state of a stream lives: trunk depth d in ping-pong buffer d & 1, a task in its own buffer.
bf16* trunk_buf(const mt_model* m, int32_t depth) { return ws_ptr(m, m->ws_trunk[depth & 1]); }
bf16* task_buf(const mt_model* m, int32_t task) { return ws_ptr(m, m->ws_task0 + m->state_bytes * task); }
// fp32 copy of a state: stored right after its bf16 copy
float* f32_of(const mt_model* m, bf16* state) {
  return reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(state) + m->act_bytes);
}

// 8-bit scratch of a slot (rows = max_batch * max_seq; xq/sx: the layer input) or of a task's first-token
// scratch (rows = max_batch; no xq).
struct QuantScratch {
  uint8_t* xq; float* sx;
  uint8_t* h1q; float* sh1;
  uint8_t* fq; float* sf;
};
QuantScratch slot_quant(const mt_model* m, uint8_t* slot) {
  const size_t M = static_cast<size_t>(m->max_batch) * m->max_seq, H = m->trunk.hidden, F = m->trunk.ffn;
  uint8_t* p = slot + m->slot_q_off;
  QuantScratch q;
  q.xq = p; p += pad256(M * H);
  q.sx = reinterpret_cast<float*>(p); p += pad256(M * 4);
  q.h1q = p; p += pad256(M * H);
  q.sh1 = reinterpret_cast<float*>(p); p += pad256(M * 4);
  q.fq = p; p += pad256(M * F);
  q.sf = reinterpret_cast<float*>(p);
  return q;
}
QuantScratch cls_quant(const mt_model* m, uint8_t* cs) {
  const size_t B = static_cast<size_t>(m->max_batch), H = m->trunk.hidden, F = m->trunk.ffn;
  uint8_t* p = cs + m->cls_q_off;
  QuantScratch q;
  q.xq = nullptr; q.sx = nullptr;
  q.h1q = p; p += pad256(B * H);
  q.sh1 = reinterpret_cast<float*>(p); p += pad256(B * 4);
  q.fq = p; p += pad256(B * F);
  q.sf = reinterpret_cast<float*>(p);
  return q;
}

// True when the final state of a task is [B, H], one row per sequence.
bool is_token_task(const mt_model* m, int32_t task) { return m->tasks[task].cfg.head_kind == MT_HEAD_TOKEN; }
bool is_compact_task(const mt_model* m, int32_t task) {
  return m->cls_only && m->tasks[task].cfg.branch_layers > 0 && !is_token_task(m, task);
}
// True for the last layer of a task branch when only the first token's state is needed downstream.
bool is_cls_op(const mt_model* m, const OpDesc& op) {
  return m->cls_only && op.task >= 0 && op.layer == m->tasks[op.task].cfg.branch_layers && !is_token_task(m, op.task);
}

// Whether a grouped GEMM launch of `groups` problems of `rows` (padded) rows runs as CTA pairs.  Pairs
// stage half as many weight bytes per CTA but tile rows by 256: measured faster from about three
// layers' worth of the 32 x 128 batch per launch, slower below.  The result is the same bits either way.
int32_t use_pair(const mt_model* m, int64_t rows, int64_t groups) {
  if (m->gemm_pair != 2) return m->gemm_pair;
  return rows * groups >= 12288 ? 1 : 0;
}
// Tile width of a grouped GEMM launch (see gemm_block_n).  `rows` are the rows the launch is sized for;
// with the packed token layout only the valid tokens are in use, and the caller's estimate of their
// number (option "expected_tokens"), when given, replaces it.
void choose_block_n(const mt_model* m, GemmParams* g, int epilogue, bool all_rows_valid, int32_t groups) {
  int64_t rows = g->M;
  if (!all_rows_valid && m->pack_tokens && m->expected_tokens > 0 && m->expected_tokens < rows) rows = m->expected_tokens;
  g->block_n = gemm_block_n(g->N, epilogue, rows, groups < 1 ? 1 : groups, g->pair != 0, m->sm_count);
}

// Whether the residual GEMMs of `groups` layers carry their LayerNorm (see GemmLnParams): 0 no, 1 on 128-column
// tiles (clusters of N / 128 CTAs), 2 on 256-column tiles (clusters of N / 256).  All three ways give the same bits,
// so the default chooses by the launch.  The fused epilogue is a chain of latencies (statistics through the
// cluster, staged stores) run by eight warps per CTA; it only beats the separate LayerNorm launch, which hides the
// same latencies behind full occupancy, while the whole launch is a single round of tiles.  Measured on the
// 32 x 128 batch (about 2409 valid rows per layer): one layer per launch - narrow tiles, 12.5 + 23.4 us against
// 8.8 + 6 + 20.1 + 6 us; two layers - wide tiles, 18.2 + 32.8 us against 18.9 + 40.1 us for the narrow ones; three
// layers - separate launches, 15 + 8 + 40 + 8 us against 25 + 60 us (narrow) or 31 + 62 us (wide).
// The first-token tails (a few rows per layer) keep the separate launches unless fused_ln_max_rows says otherwise.
int fused_ln_kind(const mt_model* m, int32_t groups, int64_t rows) {
  if (groups < 1 || !gemm_ln_supported(m->trunk.hidden) || m->fused_ln == 0) return 0;
  if (m->fused_ln == 1) return 1;
  if (m->fused_ln == 3) return 2;
  if (rows <= m->fused_ln_max_rows) return 1;
  if (rows <= m->max_batch || groups > m->fused_ln_max_groups) return 0;   // a first-token tail, or many layers
  // few rows in all (small batches): the row-wise LayerNorm is a 3 us launch and the plain GEMM has the shorter
  // epilogue (measured at 128 and 512 rows: 6.9 + 2.7 against 10.8 us, 17.1 + 2.7 against 21.3 us)
  int64_t in_use = rows;
  if (m->pack_tokens && m->expected_tokens > 0 && m->expected_tokens < in_use) in_use = m->expected_tokens;
  if (in_use * groups <= 1024) return 0;
  return groups == 1 ? 1 : 2;
}
bool use_fused_ln(const mt_model* m, int32_t groups, int64_t rows) { return fused_ln_kind(m, groups, rows) != 0; }
// Ranges the K of the FFN-down projection is split into.  A launch of few rows has few tiles, and each walks
// K = F by itself (48 k-blocks one after the other for BERT-base) while most SMs have none: four ranges, each a
// tile of its own, shorten that chain fourfold, and the LayerNorm kernel that follows adds the four partial
// sums in a fixed order.  The sum over K is then taken range by range, so the bits differ from the unsplit
// projection; the choice depends only on the rows of one layer (batch x seq, or the batch for a first-token
// tail) and on options, which are the same for a merged model and for its tasks run alone, never on how many
// layers share the launch or on which tasks are asked for.
// (Nor on option "fused_ln", whose settings all give the same bits: where the projection is split it keeps its
// LayerNorm as a launch of its own, and only the attention-output projection is fused when that option says so.)
int32_t down_split_count(const mt_model* m, int64_t rows) {
  if (m->ffn_down_split == 0 || m->fp8 || rows > kSplitRowsMax) return 1;
  return (m->trunk.ffn / kGemmBlockK) % kDownSplits == 0 ? kDownSplits : 1;
}
// Launches of steps 3-7 for `groups` layers.
int32_t tail_launches(const mt_model* m, int32_t groups, int64_t rows) {
  const bool fused = use_fused_ln(m, groups, rows);
  // 8-bit operands: two quantisations, and the FFN-down projection keeps its LayerNorm as a launch of its own;
  // so does a projection whose K is split
  return (fused ? 3 : 5) + (m->fp8 ? 2 + (fused ? 1 : 0) : 0) + (fused && down_split_count(m, rows) > 1 ? 1 : 0);
}

void init_tail(const mt_model* m, LayerTail* t, int32_t rows, bool all_rows_valid, int32_t groups) {
  const int32_t H = m->trunk.hidden, F = m->trunk.ffn;
  const int32_t* rows_valid =
      all_rows_valid ? nullptr : reinterpret_cast<const int32_t*>(m->d_workspace + m->ws_rows_valid);
  auto init_gemm = [&](GemmParams* g, int32_t N, int32_t K, int epilogue) {
    memset(g, 0, sizeof(*g));
    g->M = rows; g->N = N; g->K = K;
    g->pair = use_pair(m, rows, groups);
    choose_block_n(m, g, epilogue, all_rows_valid, groups);
    g->m_valid = rows_valid;
    g->status = reinterpret_cast<uint32_t*>(m->d_workspace + m->ws_status);
  };
  init_gemm(&t->attn_out, H, H, kEpiBiasResidual);
  init_gemm(&t->ffn_up, F, H, kEpiBiasGelu);
  t->down_splits = down_split_count(m, rows);
  if (t->down_splits > 1) {
    init_gemm(&t->ffn_down, H, F, kEpiPartialF32);
    t->ffn_down.k_splits = t->down_splits;
    t->ffn_down.split_pitch = static_cast<int32_t>(split_pitch(rows));
    t->ffn_down.block_n = gemm_block_n(H, kEpiPartialF32, rows, groups * t->down_splits, false, m->sm_count);
    t->ffn_down.pair = 0;
  } else {
    init_gemm(&t->ffn_down, H, F, kEpiBiasResidual);
  }
  t->fp8 = m->fp8;
  if (m->fp8) {
    // E4M3 operands: single CTAs, 256-wide tiles (128 with the residual epilogue)
    t->ffn_up.fp8 = t->ffn_down.fp8 = 1;
    t->ffn_up.pair = t->ffn_down.pair = 0;
    t->ffn_up.block_n = 256;
    t->ffn_down.block_n = 128;
    memset(&t->q_h1, 0, sizeof(t->q_h1));
    memset(&t->q_f, 0, sizeof(t->q_f));
    t->q_h1.rows = t->q_f.rows = rows;
    t->q_h1.cols = H;
    t->q_f.cols = F;
    t->q_h1.rows_valid = t->q_f.rows_valid = rows_valid;
  }
  memset(&t->ln1, 0, sizeof(t->ln1));
  memset(&t->ln2, 0, sizeof(t->ln2));
  t->ln1.rows_valid = t->ln2.rows_valid = rows_valid;
  t->ln1.rows = t->ln2.rows = rows;
  t->ln1.hidden = t->ln2.hidden = H;
  t->ln1.eps = t->ln2.eps = m->trunk.ln_eps;
  t->count = 0;
  t->ln_fused = use_fused_ln(m, groups, rows);
  t->ln_wide = fused_ln_kind(m, groups, rows) == 2;
  t->down_fused = t->ln_fused && !m->fp8 && t->down_splits == 1;
  if (t->ln_fused) {
    auto init_ln = [&](GemmLnParams* g, int32_t K) {
      memset(g, 0, sizeof(*g));
      g->M = rows; g->N = H; g->K = K;
      g->m_valid = rows_valid;
      g->eps = m->trunk.ln_eps;
      g->status = reinterpret_cast<uint32_t*>(m->d_workspace + m->ws_status);
    };
    init_ln(&t->attn_out_ln, H);
    init_ln(&t->ffn_down_ln, F);
  }
}

// Steps 3-7 of a layer for one group of a tail: u = ctx Wo^T + bo + residual; h1 = LN(u);
// f = GELU(h1 W1^T + b1); u = f W2^T + b2 + h1; out = LN(u).
cudaError_t add_to_tail(const mt_model* m, LayerTail* t, const LayerOffsets* lo, const bf16* ctx, const float* residual,
                        float* u, bf16* h1, float* h1_32, bf16* f, bf16* out, float* out32, const QuantScratch* qs) {
  const int i = t->count;
  cudaError_t e;
  if ((e = set_gemm_group(&t->attn_out, i, kEpiBiasResidual, ctx, w_ptr(m, lo->wo), w_ptr(m, lo->bo), residual, u)) !=
      cudaSuccess)
    return e;
  t->ln1.x[i] = u; t->ln1.gamma[i] = w_ptr(m, lo->ln1_g); t->ln1.beta[i] = w_ptr(m, lo->ln1_b);
  t->ln1.y[i] = h1; t->ln1.y32[i] = h1_32;
  if (t->fp8) {
    // h1 and f are quantised row by row into the scratch; the projections read those and the 8-bit weights
    t->q_h1.x[i] = h1; t->q_h1.q[i] = qs->h1q; t->q_h1.scale[i] = qs->sh1;
    t->q_f.x[i] = f; t->q_f.q[i] = qs->fq; t->q_f.scale[i] = qs->sf;
    t->q_h1.n_groups = t->q_f.n_groups = i + 1;
    if ((e = set_gemm_group(&t->ffn_up, i, kEpiBiasGelu, qs->h1q, m->d_weights + lo->q_w1, w_ptr(m, lo->b1), nullptr, f)) !=
        cudaSuccess)
      return e;
    t->ffn_up.group[i].scale_x = qs->sh1;
    t->ffn_up.group[i].scale_w = reinterpret_cast<const float*>(m->d_weights + lo->s_w1);
    if ((e = set_gemm_group(&t->ffn_down, i, kEpiBiasResidual, qs->fq, m->d_weights + lo->q_w2, w_ptr(m, lo->b2), h1_32,
                            u)) != cudaSuccess)
      return e;
    t->ffn_down.group[i].scale_x = qs->sf;
    t->ffn_down.group[i].scale_w = reinterpret_cast<const float*>(m->d_weights + lo->s_w2);
  } else {
    if ((e = set_gemm_group(&t->ffn_up, i, kEpiBiasGelu, h1, w_ptr(m, lo->w1), w_ptr(m, lo->b1), nullptr, f)) !=
        cudaSuccess)
      return e;
    if (t->down_splits > 1) {
      // partial sums: range s of this group writes rows [s * pitch, s * pitch + rows) of the group's piece of the
      // partial-sum scratch; the LayerNorm kernel adds the ranges, the bias and the residual
      const size_t pitch = static_cast<size_t>(t->ffn_down.split_pitch);
      float* part = reinterpret_cast<float*>(m->d_workspace + m->ws_partial) +
                    static_cast<size_t>(i) * t->down_splits * pitch * m->trunk.hidden;
      if ((e = set_gemm_group(&t->ffn_down, i, kEpiPartialF32, f, w_ptr(m, lo->w2), nullptr, nullptr, part)) != cudaSuccess)
        return e;
      if ((e = make_tmap(&t->ffn_down.tmap_out[i], part, static_cast<int>(t->down_splits * pitch), t->ffn_down.N, 32, 32,
                         true)) != cudaSuccess)
        return e;
      t->ln2.part[i] = part; t->ln2.residual[i] = h1_32; t->ln2.bias[i] = w_ptr(m, lo->b2);
      t->ln2.n_parts = t->down_splits; t->ln2.part_pitch = static_cast<int32_t>(pitch);
    } else if ((e = set_gemm_group(&t->ffn_down, i, kEpiBiasResidual, f, w_ptr(m, lo->w2), w_ptr(m, lo->b2), h1_32, u)) !=
               cudaSuccess) {
      return e;
    }
  }
  t->ln2.x[i] = u; t->ln2.gamma[i] = w_ptr(m, lo->ln2_g); t->ln2.beta[i] = w_ptr(m, lo->ln2_b);
  t->ln2.y[i] = out; t->ln2.y32[i] = out32;
  t->count = i + 1;
  t->attn_out.n_groups = t->ffn_up.n_groups = t->ffn_down.n_groups = t->ln1.n_groups = t->ln2.n_groups = t->count;
  if (t->ln_fused) {
    auto set_ln = [&](GemmLnParams* g, const void* x, size_t w, size_t b, size_t gamma, size_t beta, const float* res,
                      bf16* y, float* y32) -> cudaError_t {
      cudaError_t err;
      if ((err = make_tmap(&g->tmap_x[i], x, g->M, g->K, kGemmBlockM, kGemmBlockK, false)) != cudaSuccess) return err;
      if ((err = make_tmap(&g->tmap_w[i], w_ptr(m, w), g->N, g->K, 128, kGemmBlockK, false)) != cudaSuccess) return err;
      if ((err = make_tmap(&g->tmap_w256[i], w_ptr(m, w), g->N, g->K, 256, kGemmBlockK, false)) != cudaSuccess) return err;
      g->residual[i] = res;
      if ((err = make_tmap(&g->tmap_res[i], res, g->M, g->N, 32, 32, true)) != cudaSuccess) return err;
      if ((err = make_tmap(&g->tmap_y[i], y, g->M, g->N, 32, 64, false)) != cudaSuccess) return err;
      if ((err = make_tmap(&g->tmap_y32[i], y32, g->M, g->N, 32, 32, true)) != cudaSuccess) return err;
      g->bias[i] = w_ptr(m, b); g->gamma[i] = w_ptr(m, gamma); g->beta[i] = w_ptr(m, beta);
      g->n_groups = i + 1;
      return cudaSuccess;
    };
    // (a state is its bf16 copy followed by room for its fp32 copy: the fp32 result always has a home)
    float* out32_home = out32 != nullptr ? out32 : f32_of(m, out);
    if ((e = set_ln(&t->attn_out_ln, ctx, lo->wo, lo->bo, lo->ln1_g, lo->ln1_b, residual, h1, h1_32)) != cudaSuccess) return e;
    if (t->down_fused &&
        (e = set_ln(&t->ffn_down_ln, f, lo->w2, lo->b2, lo->ln2_g, lo->ln2_b, h1_32, out, out32_home)) != cudaSuccess)
      return e;
  }
  return cudaSuccess;
}

cudaError_t build_chunk(const mt_model* m, const std::vector<OpDesc>& ops, size_t first, size_t count, int32_t batch,
                        int32_t seq, Chunk* ck) {
  const int32_t M = batch * seq, H = m->trunk.hidden;
  const size_t act = m->act_bytes;
  const size_t qkv_bytes = pad256(static_cast<size_t>(m->max_batch) * m->max_seq * 3 * H * 2);
  const int32_t* row_start = reinterpret_cast<const int32_t*>(m->d_workspace + m->ws_row_start);
  memset(&ck->qkv, 0, sizeof(ck->qkv));
  ck->qkv.n_groups = static_cast<int32_t>(count);
  ck->qkv.M = M; ck->qkv.N = 3 * H; ck->qkv.K = H;
  ck->qkv.pair = use_pair(m, M, static_cast<int64_t>(count));
  choose_block_n(m, &ck->qkv, kEpiBias, false, static_cast<int32_t>(count));
  memset(&ck->q_in, 0, sizeof(ck->q_in));
  if (m->fp8) {
    ck->qkv.fp8 = 1;
    ck->qkv.pair = 0;
    ck->qkv.block_n = 256;
    ck->q_in.n_groups = static_cast<int32_t>(count);
    ck->q_in.rows = M;
    ck->q_in.cols = H;
    ck->q_in.rows_valid = reinterpret_cast<const int32_t*>(m->d_workspace + m->ws_rows_valid);
  }
  ck->qkv.m_valid = reinterpret_cast<const int32_t*>(m->d_workspace + m->ws_rows_valid);
  ck->qkv.status = reinterpret_cast<uint32_t*>(m->d_workspace + m->ws_status);
  int32_t n_full = 0;
  for (size_t i = 0; i < count; ++i) n_full += is_cls_op(m, ops[first + i]) ? 0 : 1;
  init_tail(m, &ck->full, M, false, n_full);
  ck->n_cls = 0;
  memset(&ck->attn, 0, sizeof(ck->attn));
  memset(&ck->attn_cls, 0, sizeof(ck->attn_cls));
  ck->attn.batch = ck->attn_cls.batch = batch;
  ck->attn.seq = ck->attn_cls.seq = seq;
  ck->attn.heads = ck->attn_cls.heads = m->trunk.heads;
  ck->attn.row_start = ck->attn_cls.row_start = row_start;  // lengths are patched per call
  ck->attn.packed = m->pack_tokens ? 1 : 0;
  ck->attn.tensor_memory = (m->attention_tc && seq <= kAttnTensorMemoryMaxSeq) ? 1 : 0;
  ck->attn.status = ck->qkv.status;

  for (size_t i = 0; i < count; ++i) {
    const OpDesc& op = ops[first + i];
    const LayerOffsets* lo;
    bf16 *in, *out;
    if (op.task < 0) {
      lo = &m->trunk_layers[op.layer - 1];
      in = trunk_buf(m, op.layer - 1);
      out = trunk_buf(m, op.layer);
    } else {
      const TaskEntry& te = m->tasks[op.task];
      lo = &te.layers[op.layer - 1];
      in = op.layer == 1 ? trunk_buf(m, te.cfg.fork_depth) : task_buf(m, op.task);
      out = task_buf(m, op.task);
    }
    uint8_t* slot = m->d_workspace + m->ws_slot0 + m->slot_bytes * i;
    bf16* qkv = reinterpret_cast<bf16*>(slot);
    bf16* ctx = reinterpret_cast<bf16*>(slot + qkv_bytes);
    float* u = reinterpret_cast<float*>(slot + qkv_bytes + act);
    bf16* h1 = reinterpret_cast<bf16*>(slot + qkv_bytes + act + m->act32_bytes);
    bf16* f = reinterpret_cast<bf16*>(slot + qkv_bytes + act + m->act32_bytes + m->state_bytes);

    cudaError_t e;
    // 1. qkv = in . [Wq;Wk;Wv]^T + [bq;bk;bv] on every token (the three matrices and biases are
    //    contiguous in the arena); keys and values are needed for all tokens even in a `cls` layer
    const QuantScratch qs = m->fp8 ? slot_quant(m, slot) : QuantScratch{};
    if (m->fp8) {
      ck->q_in.x[i] = in; ck->q_in.q[i] = qs.xq; ck->q_in.scale[i] = qs.sx;
      if ((e = set_gemm_group(&ck->qkv, static_cast<int>(i), kEpiBias, qs.xq, m->d_weights + lo->q_qkv, w_ptr(m, lo->bq),
                              nullptr, qkv)) != cudaSuccess)
        return e;
      ck->qkv.group[i].scale_x = qs.sx;
      ck->qkv.group[i].scale_w = reinterpret_cast<const float*>(m->d_weights + lo->s_qkv);
    } else if ((e = set_gemm_group(&ck->qkv, static_cast<int>(i), kEpiBias, in, w_ptr(m, lo->wq), w_ptr(m, lo->bq), nullptr,
                                   qkv)) != cudaSuccess) {
      return e;
    }
    const bool cls = is_cls_op(m, op);
    if (!cls) {
      // 2. ctx = attention(qkv) for every token; 3-7 on every token
      const int a = ck->full.count;
      ck->attn.qkv[a] = qkv;
      ck->attn.ctx[a] = ctx;
      ck->attn.n_groups = a + 1;
      if (ck->attn.tensor_memory &&
          ((e = make_tmap(&ck->attn.tmap_qkv[a], qkv, M, 3 * H, kAttnTileRows, kHeadDim, false)) != cudaSuccess ||
           (e = make_tmap(&ck->attn.tmap_qkv64[a], qkv, M, 3 * H, kAttnTileRows / 2, kHeadDim, false)) != cudaSuccess))
        return e;
      if ((e = add_to_tail(m, &ck->full, lo, ctx, f32_of(m, in), u, h1, f32_of(m, h1), f, out, f32_of(m, out), &qs)) !=
          cudaSuccess)
        return e;
      if (m->debug_capture) ck->dumps.push_back({out, dump_slot(m, op.task, op.layer), false});
    } else {
      // 2'. first-token attention into the task's compact [B, H] scratch, which also gathers the first
      //     tokens' fp32 residual; steps 3-7 of these layers follow after the last wave
      const int a = ck->n_cls;
      uint8_t* cs = m->d_workspace + m->ws_cls0 + m->cls_bytes * op.task;
      ck->attn_cls.qkv[a] = qkv;
      ck->attn_cls.in32[a] = f32_of(m, in);
      ck->attn_cls.ctx[a] = reinterpret_cast<bf16*>(cs);
      ck->attn_cls.res[a] = reinterpret_cast<float*>(cs + m->cls_h_bytes);
      ck->attn_cls.n_groups = ck->n_cls = a + 1;
    }
  }
  return cudaSuccess;
}

// Steps 3-7 of the last branch layers of `tasks` on their first tokens ([B, H] rows), one group per task.
cudaError_t build_cls_tail(const mt_model* m, const std::vector<int32_t>& tasks, size_t first, size_t count,
                           int32_t batch, PlanStep* st) {
  init_tail(m, &st->tail, batch, true, static_cast<int32_t>(count));
  for (size_t i = 0; i < count; ++i) {
    const int32_t t = tasks[first + i];
    const TaskEntry& te = m->tasks[t];
    const LayerOffsets* lo = &te.layers[te.cfg.branch_layers - 1];
    uint8_t* cs = m->d_workspace + m->ws_cls0 + m->cls_bytes * t;
    bf16* ctx = reinterpret_cast<bf16*>(cs);
    float* res = reinterpret_cast<float*>(cs + m->cls_h_bytes);
    float* u = reinterpret_cast<float*>(cs + m->cls_h_bytes + m->cls_h32_bytes);
    bf16* h1 = reinterpret_cast<bf16*>(cs + m->cls_h_bytes + 2 * m->cls_h32_bytes);
    float* h1_32 = reinterpret_cast<float*>(cs + 2 * m->cls_h_bytes + 2 * m->cls_h32_bytes);
    bf16* f = reinterpret_cast<bf16*>(cs + 2 * m->cls_h_bytes + 3 * m->cls_h32_bytes);
    bf16* out = task_buf(m, t);  // the task's state becomes [B, H]
    const QuantScratch qs = m->fp8 ? cls_quant(m, cs) : QuantScratch{};
    cudaError_t e = add_to_tail(m, &st->tail, lo, ctx, res, u, h1, h1_32, f, out, nullptr, &qs);
    if (e != cudaSuccess) return e;
    if (m->debug_capture) st->dumps.push_back({out, dump_slot(m, t, te.cfg.branch_layers), true});
  }
  return cudaSuccess;
}

int32_t chunk_launches(const mt_model* m, const std::vector<OpDesc>& ops, size_t first, size_t count, int64_t rows) {
  size_t n_cls = 0;
  for (size_t i = 0; i < count; ++i) n_cls += is_cls_op(m, ops[first + i]) ? 1 : 0;
  return 1 + (m->fp8 ? 1 : 0) + (n_cls < count ? 1 + tail_launches(m, static_cast<int32_t>(count - n_cls), rows) : 0) +
         (n_cls > 0 ? 1 : 0);
}
// Active tasks whose last branch layer is finished on first tokens right after wave w (1-based):
// those whose last layer is in wave w with option early_heads, otherwise all of them after the last wave.
std::vector<int32_t> cls_tasks_after_wave(const mt_model* m, const Schedule& s, size_t w) {
  std::vector<int32_t> out;
  for (size_t v = 1; v <= s.waves.size(); ++v) {
    if (m->early_heads ? v != w : w != s.waves.size()) continue;
    for (const OpDesc& op : s.waves[v - 1])
      if (is_cls_op(m, op)) out.push_back(op.task);
  }
  std::sort(out.begin(), out.end());
  return out;
}

cudaError_t build_plan(const mt_model* m, const Schedule& s, int32_t batch, int32_t seq, Plan* plan) {
  plan->steps.clear();
  plan->launches = 2;  // row starts, embedding
  // Pooler + head of a set of tasks.  Tasks whose final state is compact ([B, H], one row per sequence:
  // the last branch layer was evaluated on first tokens only) get their pooler as one grouped GEMM on
  // the tensor cores, Y_t = tanh(X_t . Wp_t^T + bp_t) in fp32, followed by the head kernel; the others
  // pool rows gathered by row_start with the two row-wise kernels.  The split is per task, so a task's
  // logits never depend on which other tasks are active.
  cudaError_t heads_error = cudaSuccess;
  auto add_heads_of = [&](const std::vector<int32_t>& tasks, bool compact) {
    for (size_t first = 0; first < tasks.size(); first += kMaxGroups) {
      const size_t count = std::min<size_t>(kMaxGroups, tasks.size() - first);
      PlanStep st;
      st.kind = 1;
      memset(&st.heads, 0, sizeof(st.heads));
      st.heads.n_tasks = static_cast<int32_t>(count);
      st.heads.batch = batch; st.heads.seq = seq; st.heads.hidden = m->trunk.hidden;
      st.heads.logits_stride = m->c_total;
      st.heads.pooled = reinterpret_cast<float*>(m->d_workspace + m->ws_pooled);
      st.heads.row_start = reinterpret_cast<const int32_t*>(m->d_workspace + m->ws_row_start);
      st.pool_gemm = compact && m->pool_gemm;
      if (st.pool_gemm) {
        memset(&st.pool, 0, sizeof(st.pool));
        st.pool.n_groups = static_cast<int32_t>(count);
        st.pool.M = batch; st.pool.N = m->trunk.hidden; st.pool.K = m->trunk.hidden;
        st.pool.pair = 0;
        st.pool.block_n = gemm_block_n(st.pool.N, kEpiBiasTanhF32, batch, static_cast<int>(count), false, m->sm_count);
        st.pool.m_valid = nullptr;
        st.pool.status = reinterpret_cast<uint32_t*>(m->d_workspace + m->ws_status);
      }
      for (size_t i = 0; i < count; ++i) {
        const int32_t t = tasks[first + i];
        const TaskEntry& te = m->tasks[t];
        HeadTask& ht = st.heads.task[i];
        ht.hidden = te.cfg.branch_layers == 0 ? trunk_buf(m, te.cfg.fork_depth) : task_buf(m, t);
        ht.pool_w = w_ptr(m, te.pool_w); ht.pool_b = w_ptr(m, te.pool_b);
        ht.cls_w = w_ptr(m, te.cls_w); ht.cls_b = w_ptr(m, te.cls_b);
        ht.num_classes = te.cfg.num_classes; ht.col0 = te.col0;
        ht.compact = compact ? 1 : 0;
        st.head_tasks.push_back(t);
        if (st.pool_gemm) {
          cudaError_t e = set_gemm_group(&st.pool, static_cast<int>(i), kEpiBiasTanhF32, ht.hidden, ht.pool_w, ht.pool_b,
                                         nullptr, st.heads.pooled + i * static_cast<size_t>(batch) * m->trunk.hidden);
          if (e != cudaSuccess) heads_error = e;
        }
      }
      plan->steps.push_back(std::move(st));
      plan->launches += 2;
    }
  };
  // Token-level tasks: one linear map on every valid token of the final state, written by position.
  auto add_token_heads = [&](const std::vector<int32_t>& tasks) {
    for (size_t first = 0; first < tasks.size(); first += kMaxGroups) {
      const size_t count = std::min<size_t>(kMaxGroups, tasks.size() - first);
      PlanStep st;
      st.kind = 3;
      memset(&st.heads, 0, sizeof(st.heads));
      memset(&st.token_heads, 0, sizeof(st.token_heads));
      TokenHeadParams& th = st.token_heads;
      th.n_tasks = static_cast<int32_t>(count);
      th.batch = batch; th.seq = seq; th.hidden = m->trunk.hidden;
      th.logits_stride = m->ct_total;
      th.row_start = reinterpret_cast<const int32_t*>(m->d_workspace + m->ws_row_start);
      for (size_t i = 0; i < count; ++i) {
        const int32_t t = tasks[first + i];
        const TaskEntry& te = m->tasks[t];
        th.hidden_state[i] = te.cfg.branch_layers == 0 ? trunk_buf(m, te.cfg.fork_depth) : task_buf(m, t);
        th.cls_w[i] = w_ptr(m, te.cls_w); th.cls_b[i] = w_ptr(m, te.cls_b);
        th.num_classes[i] = te.cfg.num_classes; th.col0[i] = te.col0;
        st.head_tasks.push_back(t);
      }
      plan->steps.push_back(std::move(st));
      plan->launches += 1;
    }
  };
  auto add_heads = [&](const std::vector<int32_t>& tasks) {
    std::vector<int32_t> compact, gathered, token;
    for (int32_t t : tasks) (is_token_task(m, t) ? token : (is_compact_task(m, t) ? compact : gathered)).push_back(t);
    add_token_heads(token);
    add_heads_of(gathered, false);
    add_heads_of(compact, true);
  };
  add_heads(s.heads[0]);
  for (size_t w = 1; w <= s.waves.size(); ++w) {
    const std::vector<OpDesc>& ops = s.waves[w - 1];
    for (size_t first = 0; first < ops.size(); first += m->n_slots) {
      const size_t count = std::min<size_t>(m->n_slots, ops.size() - first);
      PlanStep st;
      st.kind = 0;
      cudaError_t e = build_chunk(m, ops, first, count, batch, seq, &st.chunk);
      if (e != cudaSuccess) return e;
      plan->steps.push_back(std::move(st));
      plan->launches += chunk_launches(m, ops, first, count, static_cast<int64_t>(batch) * seq);
    }
    {
      // first-token tails: of the tasks finishing in this wave (early_heads), or of all tasks after the last wave
      const std::vector<int32_t> tasks = cls_tasks_after_wave(m, s, w);
      for (size_t first = 0; first < tasks.size(); first += kMaxGroups) {
        PlanStep st;
        st.kind = 2;
        cudaError_t e = build_cls_tail(m, tasks, first, std::min<size_t>(kMaxGroups, tasks.size() - first), batch, &st);
        if (e != cudaSuccess) return e;
        plan->launches += tail_launches(m, st.tail.count, batch);
        plan->steps.push_back(std::move(st));
      }
    }
    add_heads(s.heads[w]);
  }
  return heads_error;
}

cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

}  // namespace

// =================================================================================================
// C ABI
// =================================================================================================

extern "C" {

int mt_create(const mt_trunk_config* trunk, const mt_task_config* tasks, int32_t n_tasks, int32_t max_batch,
              int32_t max_seq, mt_model** out) {
  if (out == nullptr) return MT_ERR_INVALID_ARG;
  *out = nullptr;
  if (trunk == nullptr || tasks == nullptr || n_tasks < 1 || n_tasks > 64 || max_batch < 1 || max_seq < 1)
    return MT_ERR_INVALID_ARG;
  if (trunk->hidden != trunk->heads * kHeadDim || (trunk->hidden != 768 && trunk->hidden != 1024) ||
      trunk->ffn % 256 != 0 || trunk->ffn < 256 || trunk->activation != 0 || max_seq > 512)
    return MT_ERR_UNSUPPORTED;
  if (trunk->vocab_size < 1 || trunk->type_vocab < 1 || trunk->trunk_layers < 0 || max_seq > trunk->max_position ||
      !(trunk->ln_eps >= 0.f))
    return MT_ERR_INVALID_ARG;
  if (static_cast<int64_t>(max_batch) * max_seq > (int64_t(1) << 24)) return MT_ERR_SHAPE;
  for (int32_t t = 0; t < n_tasks; ++t) {
    if (tasks[t].fork_depth < 0 || tasks[t].fork_depth > trunk->trunk_layers || tasks[t].branch_layers < 0 ||
        tasks[t].num_classes < 1 || (tasks[t].head_kind != MT_HEAD_SEQUENCE && tasks[t].head_kind != MT_HEAD_TOKEN))
      return MT_ERR_INVALID_ARG;
  }
  mt_model* m = new mt_model();
  m->trunk = *trunk;
  m->max_batch = max_batch;
  m->max_seq = max_seq;
  m->max_groups = kMaxGroups;
  m->plan_cache = 32;
  m->use_clock = 0;
  m->debug_capture = false;
  m->pack_tokens = true;
  m->cls_only = true;
  m->early_heads = false;
  m->gemm_pair = 2;
  m->attention_tc = true;
  m->expected_tokens = 0;
  m->pool_gemm = true;
  m->overlap_cls = true;
  m->side_stream = nullptr;
  m->ev_fork = m->ev_join = nullptr;
  m->fused_ln = 2;
  m->fused_ln_max_groups = 2;
  m->ffn_down_split = 1;
  m->fused_ln_max_rows = 0;
  m->last_lengths = nullptr;
  m->d_weights = m->d_workspace = nullptr;
  m->ws_bytes_bound = 0;
  m->sm_count = 0;
  m->sm_device = 0;
  m->sm_limit = 0;
  m->trunk_loaded = false;
  m->last_batch = m->last_seq = 0;
  m->profile = false;
  m->events_used = 0;

  const size_t H = trunk->hidden, e = sizeof(bf16);
  size_t off = 0;
  auto take = [&](size_t elems) { size_t at = off; off += pad256(elems * e); return at; };
  m->emb_word = take(static_cast<size_t>(trunk->vocab_size) * H);
  m->emb_pos = take(static_cast<size_t>(trunk->max_position) * H);
  m->emb_type = take(static_cast<size_t>(trunk->type_vocab) * H);
  m->emb_ln_g = take(H);
  m->emb_ln_b = take(H);
  m->trunk_layers.resize(trunk->trunk_layers);
  for (int32_t l = 0; l < trunk->trunk_layers; ++l) off = place_layer(*trunk, off, &m->trunk_layers[l]);
  int32_t col = 0, col_tok = 0;
  m->tasks.resize(n_tasks);
  for (int32_t t = 0; t < n_tasks; ++t) {
    TaskEntry& te = m->tasks[t];
    te.cfg = tasks[t];
    te.section_begin = off;
    te.layers.resize(tasks[t].branch_layers);
    for (int32_t j = 0; j < tasks[t].branch_layers; ++j) off = place_layer(*trunk, off, &te.layers[j]);
    te.pool_w = take(H * H);
    te.pool_b = take(H);
    te.cls_w = take(static_cast<size_t>(tasks[t].num_classes) * H);
    te.cls_b = take(tasks[t].num_classes);
    te.section_bytes = off - te.section_begin;
    // sequence-level and token-level tasks have output arrays, and column counts, of their own
    if (tasks[t].head_kind == MT_HEAD_TOKEN) {
      te.col0 = col_tok;
      col_tok += tasks[t].num_classes;
    } else {
      te.col0 = col;
      col += tasks[t].num_classes;
    }
    te.loaded = false;
  }
  m->payload_bytes = off;
  m->fp8 = false;
  layout_fp8_weights(m);
  m->c_total = col;
  m->ct_total = col_tok;
  layout_workspace(m);
  *out = m;
  return MT_OK;
}

void mt_destroy(mt_model* m) {
  if (m == nullptr) return;
  for (cudaEvent_t ev : m->events) cudaEventDestroy(ev);
  if (m->ev_fork != nullptr) cudaEventDestroy(m->ev_fork);
  if (m->ev_join != nullptr) cudaEventDestroy(m->ev_join);
  if (m->side_stream != nullptr) cudaStreamDestroy(m->side_stream);
  delete m;
}

size_t mt_weights_bytes(const mt_model* m) { return m ? m->weights_bytes : 0; }
size_t mt_workspace_bytes(const mt_model* m) { return m ? m->ws_total : 0; }
size_t mt_blob_bytes(const mt_model* m) { return m ? m->payload_bytes + kHeaderBytes : 0; }
size_t mt_task_blob_bytes(const mt_model* m, int32_t task) {
  if (m == nullptr || task < 0 || task >= static_cast<int32_t>(m->tasks.size())) return 0;
  return m->tasks[task].section_bytes + kHeaderBytes;
}

const char* mt_last_error_string(const mt_model* m) { return m ? m->last_error.c_str() : "null model"; }

int mt_set_option(mt_model* m, const char* key, int64_t value) {
  if (m == nullptr || key == nullptr) return MT_ERR_INVALID_ARG;
  if (strcmp(key, "gemm_pair") == 0) {
    if (value < 0 || value > 2) return fail(m, MT_ERR_INVALID_ARG, "gemm_pair must be 0, 1 or 2");
    m->gemm_pair = static_cast<int32_t>(value);
    m->plans.clear();
    return MT_OK;
  }
  if (strcmp(key, "expected_tokens") == 0) {
    if (value < 0) return fail(m, MT_ERR_INVALID_ARG, "expected_tokens must be >= 0");
    if (value != m->expected_tokens) m->plans.clear();
    m->expected_tokens = value;
    return MT_OK;
  }
  if (strcmp(key, "fused_ln") == 0) {
    if (value < 0 || value > 3) return fail(m, MT_ERR_INVALID_ARG, "fused_ln must be 0, 1, 2 or 3");
    m->fused_ln = static_cast<int32_t>(value);
    m->plans.clear();
    return MT_OK;
  }
  if (strcmp(key, "sm_limit") == 0) {
    if (value < 0) return fail(m, MT_ERR_INVALID_ARG, "sm_limit must be >= 0");
    m->sm_limit = static_cast<int>(value);
    if (m->sm_device > 0) m->sm_count = (m->sm_limit > 0 && m->sm_limit < m->sm_device) ? m->sm_limit : m->sm_device;
    m->plans.clear();
    return MT_OK;
  }
  if (strcmp(key, "fused_ln_max_rows") == 0) {
    if (value < 0) return fail(m, MT_ERR_INVALID_ARG, "fused_ln_max_rows must be >= 0");
    m->fused_ln_max_rows = static_cast<int32_t>(value);
    m->plans.clear();
    return MT_OK;
  }
  if (strcmp(key, "ffn_down_split") == 0) {
    if (value != 0 && value != 1) return fail(m, MT_ERR_INVALID_ARG, "ffn_down_split must be 0 or 1");
    m->ffn_down_split = static_cast<int32_t>(value);
    m->plans.clear();
    return MT_OK;
  }
  if (strcmp(key, "fused_ln_max_groups") == 0) {
    if (value < 1) return fail(m, MT_ERR_INVALID_ARG, "fused_ln_max_groups must be >= 1");
    m->fused_ln_max_groups = static_cast<int32_t>(value);
    m->plans.clear();
    return MT_OK;
  }
  if (strcmp(key, "plan_cache") == 0) {
    if (value < 1) return fail(m, MT_ERR_INVALID_ARG, "plan_cache must be >= 1");
    m->plan_cache = static_cast<int32_t>(value > 4096 ? 4096 : value);
    m->plans.clear();
    return MT_OK;
  }
  if (strcmp(key, "overlap_cls") == 0) {
    m->overlap_cls = value != 0;
    return MT_OK;
  }
  if (strcmp(key, "pool_gemm") == 0) {
    m->pool_gemm = value != 0;
    m->plans.clear();
    return MT_OK;
  }
  if (strcmp(key, "attention_tc") == 0) {
    m->attention_tc = value != 0;
    m->plans.clear();
    return MT_OK;
  }
  if (strcmp(key, "pdl") == 0) {  // process-wide: programmatic dependent launch on or off
    g_use_pdl = value != 0;
    return MT_OK;
  }
  if (strcmp(key, "early_heads") == 0) {
    m->early_heads = value != 0;
    m->plans.clear();
    return MT_OK;
  }
  if (strcmp(key, "cls_only_last_layer") == 0) {
    m->cls_only = value != 0;
    m->plans.clear();
    return MT_OK;
  }
  if (strcmp(key, "pack_tokens") == 0) {
    m->pack_tokens = value != 0;
    m->plans.clear();
    return MT_OK;
  }
  if (strcmp(key, "profile") == 0) {
    m->profile = value != 0;
    m->events_used = 0;
    m->event_class.clear();
    return MT_OK;
  }
  if (m->d_workspace != nullptr) return fail(m, MT_ERR_INVALID_ARG, "options must be set before mt_bind_memory");
  if (strcmp(key, "max_groups") == 0) {
    if (value < 1 || value > kMaxGroups) return fail(m, MT_ERR_INVALID_ARG, "max_groups must be in 1..8");
    m->max_groups = static_cast<int32_t>(value);
  } else if (strcmp(key, "debug_capture") == 0) {
    m->debug_capture = value != 0;
  } else if (strcmp(key, "fp8_gemm") == 0) {
    m->fp8 = value != 0;
    layout_fp8_weights(m);
  } else {
    return fail(m, MT_ERR_INVALID_ARG, std::string("unknown option ") + key);
  }
  layout_workspace(m);
  m->plans.clear();
  return MT_OK;
}

int mt_bind_memory(mt_model* m, void* d_weights, size_t weights_bytes, void* d_workspace, size_t workspace_bytes) {
  if (m == nullptr) return MT_ERR_INVALID_ARG;
  if (d_weights == nullptr || d_workspace == nullptr) return fail(m, MT_ERR_INVALID_ARG, "null arena");
  if ((reinterpret_cast<uintptr_t>(d_weights) | reinterpret_cast<uintptr_t>(d_workspace)) & (kAlign - 1))
    return fail(m, MT_ERR_INVALID_ARG, "arenas must be 256-byte aligned");
  if (weights_bytes < m->weights_bytes || workspace_bytes < m->ws_total)
    return fail(m, MT_ERR_INVALID_ARG, "arena smaller than mt_weights_bytes / mt_workspace_bytes");
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return fail_cuda(m, e, "querying the device");
  int major = 0;
  e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (e != cudaSuccess) return fail_cuda(m, e, "querying the device");
  if (major != 10) return fail(m, MT_ERR_UNSUPPORTED, "the kernels are built for sm_100a only");
  m->sm_device = sms;
  m->sm_count = (m->sm_limit > 0 && m->sm_limit < sms) ? m->sm_limit : sms;
  m->d_weights = static_cast<uint8_t*>(d_weights);
  m->d_workspace = static_cast<uint8_t*>(d_workspace);
  m->ws_bytes_bound = workspace_bytes;
  m->plans.clear();
  m->trunk_loaded = false;
  for (TaskEntry& t : m->tasks) t.loaded = false;
  e = cudaMemset(m->d_workspace + m->ws_status, 0, 256);
  if (e != cudaSuccess) return fail_cuda(m, e, "clearing the status word");
  // the stream beside the caller's (option "overlap_cls") and its fork/join events: created here, once, so
  // that a forward never creates anything
  if (m->side_stream == nullptr) {
    if ((e = cudaStreamCreateWithFlags(&m->side_stream, cudaStreamNonBlocking)) != cudaSuccess ||
        (e = cudaEventCreateWithFlags(&m->ev_fork, cudaEventDisableTiming)) != cudaSuccess ||
        (e = cudaEventCreateWithFlags(&m->ev_join, cudaEventDisableTiming)) != cudaSuccess)
      return fail_cuda(m, e, "creating the side stream");
  }
  return MT_OK;
}

static int check_header(const mt_model* m, const void* blob, size_t bytes, uint32_t kind, int32_t task, size_t payload) {
  if (blob == nullptr) return fail(m, MT_ERR_INVALID_ARG, "null blob");
  if (bytes < kHeaderBytes) return fail(m, MT_ERR_BLOB_MISMATCH, "blob shorter than its header");
  BlobHeader h;
  memcpy(&h, blob, sizeof(h));
  const mt_trunk_config& c = m->trunk;
  if (h.magic != kBlobMagic || h.version != kBlobVersion) return fail(m, MT_ERR_BLOB_MISMATCH, "bad magic or version");
  if (h.kind != kind) return fail(m, MT_ERR_BLOB_MISMATCH, "blob kind (full model / single task) mismatch");
  if (h.hidden != c.hidden || h.heads != c.heads || h.ffn != c.ffn || h.trunk_layers != c.trunk_layers ||
      h.vocab != c.vocab_size || h.max_position != c.max_position || h.type_vocab != c.type_vocab ||
      h.n_tasks != static_cast<int32_t>(m->tasks.size()))
    return fail(m, MT_ERR_BLOB_MISMATCH, "blob was written for another configuration");
  if (kind == 1) {
    const mt_task_config& tc = m->tasks[task].cfg;
    if (h.task_index != task || h.fork_depth != tc.fork_depth || h.branch_layers != tc.branch_layers ||
        h.num_classes != tc.num_classes)
      return fail(m, MT_ERR_BLOB_MISMATCH, "task blob does not match this task's configuration");
  }
  if (h.payload_bytes != payload || bytes != payload + kHeaderBytes)
    return fail(m, MT_ERR_BLOB_MISMATCH, "blob size disagrees with the configuration");
  return MT_OK;
}

int mt_load_weights(mt_model* m, const void* host_blob, size_t bytes, void* stream) {
  if (m == nullptr) return MT_ERR_INVALID_ARG;
  if (m->d_weights == nullptr) return fail(m, MT_ERR_NOT_BOUND, "mt_bind_memory has not been called");
  int rc = check_header(m, host_blob, bytes, 0, -1, m->payload_bytes);
  if (rc != MT_OK) return rc;
  cudaError_t e = cudaMemcpyAsync(m->d_weights, static_cast<const uint8_t*>(host_blob) + kHeaderBytes, m->payload_bytes,
                                  cudaMemcpyHostToDevice, as_stream(stream));
  if (e != cudaSuccess) return fail_cuda(m, e, "copying weights");
  if (m->fp8) {
    std::vector<const LayerOffsets*> layers;
    for (const LayerOffsets& lo : m->trunk_layers) layers.push_back(&lo);
    for (const TaskEntry& t : m->tasks)
      for (const LayerOffsets& lo : t.layers) layers.push_back(&lo);
    if ((e = quantize_layer_weights(m, layers, as_stream(stream))) != cudaSuccess) return fail_cuda(m, e, "quantising weights");
  }
  m->trunk_loaded = true;
  for (TaskEntry& t : m->tasks) t.loaded = true;
  return MT_OK;
}

int mt_adopt_weights(mt_model* m, const mt_model* src) {
  if (m == nullptr || src == nullptr) return MT_ERR_INVALID_ARG;
  if (m->d_weights == nullptr || src->d_weights == nullptr) return fail(m, MT_ERR_NOT_BOUND, "both models must be bound");
  if (m->d_weights != src->d_weights) return fail(m, MT_ERR_INVALID_ARG, "the two models are bound to different weight arenas");
  bool same = m->weights_bytes == src->weights_bytes && m->fp8 == src->fp8 && m->tasks.size() == src->tasks.size() &&
              memcmp(&m->trunk, &src->trunk, sizeof(m->trunk)) == 0;
  for (size_t t = 0; same && t < m->tasks.size(); ++t)
    same = memcmp(&m->tasks[t].cfg, &src->tasks[t].cfg, sizeof(mt_task_config)) == 0;
  if (!same) return fail(m, MT_ERR_BLOB_MISMATCH, "the two models were created from different configurations");
  m->trunk_loaded = src->trunk_loaded;
  for (size_t t = 0; t < m->tasks.size(); ++t) m->tasks[t].loaded = src->tasks[t].loaded;
  return MT_OK;
}

int mt_load_task_weights(mt_model* m, int32_t task, const void* host_blob, size_t bytes, void* stream) {
  if (m == nullptr) return MT_ERR_INVALID_ARG;
  if (task < 0 || task >= static_cast<int32_t>(m->tasks.size())) return fail(m, MT_ERR_INVALID_ARG, "task out of range");
  if (m->d_weights == nullptr) return fail(m, MT_ERR_NOT_BOUND, "mt_bind_memory has not been called");
  TaskEntry& te = m->tasks[task];
  int rc = check_header(m, host_blob, bytes, 1, task, te.section_bytes);
  if (rc != MT_OK) return rc;
  cudaError_t e = cudaMemcpyAsync(m->d_weights + te.section_begin, static_cast<const uint8_t*>(host_blob) + kHeaderBytes,
                                  te.section_bytes, cudaMemcpyHostToDevice, as_stream(stream));
  if (e != cudaSuccess) return fail_cuda(m, e, "copying task weights");
  if (m->fp8) {
    std::vector<const LayerOffsets*> layers;
    for (const LayerOffsets& lo : te.layers) layers.push_back(&lo);
    if ((e = quantize_layer_weights(m, layers, as_stream(stream))) != cudaSuccess) return fail_cuda(m, e, "quantising task weights");
  }
  te.loaded = true;
  return MT_OK;
}

int mt_plan_summary(const mt_model* m, uint64_t task_mask, int32_t* n_layers, int32_t* n_waves, int32_t* trunk_depth,
                    int32_t* groups_per_wave) {
  if (m == nullptr) return MT_ERR_INVALID_ARG;
  Schedule s;
  if (!build_schedule(m, task_mask, &s)) return fail(m, MT_ERR_INVALID_ARG, "task_mask selects no task");
  if (n_layers) *n_layers = s.n_layers;
  if (n_waves) *n_waves = static_cast<int32_t>(s.waves.size());
  if (trunk_depth) *trunk_depth = s.trunk_depth;
  if (groups_per_wave)
    for (size_t w = 0; w < s.waves.size(); ++w) groups_per_wave[w] = static_cast<int32_t>(s.waves[w].size());
  return MT_OK;
}

int mt_plan_cache_size(const mt_model* m) { return m == nullptr ? MT_ERR_INVALID_ARG : static_cast<int>(m->plans.size()); }

int mt_plan_launches(const mt_model* m, uint64_t task_mask, int32_t* n_launches) {
  if (m == nullptr || n_launches == nullptr) return MT_ERR_INVALID_ARG;
  Schedule s;
  if (!build_schedule(m, task_mask, &s)) return fail(m, MT_ERR_INVALID_ARG, "task_mask selects no task");
  int32_t n = 2;  // row starts, embedding
  for (size_t w = 0; w <= s.waves.size(); ++w) {
    if (w >= 1) {
      const std::vector<OpDesc>& ops = s.waves[w - 1];
      for (size_t first = 0; first < ops.size(); first += m->n_slots)
        n += chunk_launches(m, ops, first, std::min<size_t>(m->n_slots, ops.size() - first),
                            static_cast<int64_t>(m->max_batch) * m->max_seq);
      const size_t n_cls_tasks = cls_tasks_after_wave(m, s, w).size();
      for (size_t first = 0; first < n_cls_tasks; first += kMaxGroups)
        n += tail_launches(m, static_cast<int32_t>(std::min<size_t>(kMaxGroups, n_cls_tasks - first)), m->max_batch);
    }
    size_t n_compact = 0, n_token = 0;
    for (int32_t t : s.heads[w]) {
      n_compact += is_compact_task(m, t) ? 1 : 0;
      n_token += is_token_task(m, t) ? 1 : 0;
    }
    n += static_cast<int32_t>((n_token + kMaxGroups - 1) / kMaxGroups);
    n += 2 * static_cast<int32_t>((n_compact + kMaxGroups - 1) / kMaxGroups +
                                  (s.heads[w].size() - n_compact - n_token + kMaxGroups - 1) / kMaxGroups);
  }
  *n_launches = n;
  return MT_OK;
}

int mt_forward(mt_model* m, const int32_t* d_token_ids, const int32_t* d_segment_ids, const int32_t* d_lengths,
               uint64_t task_mask, int32_t batch, int32_t seq, float* d_logits, void* stream_) {
  return mt_forward_events(m, d_token_ids, d_segment_ids, d_lengths, task_mask, batch, seq, d_logits, nullptr, stream_);
}

int mt_forward_events(mt_model* m, const int32_t* d_token_ids, const int32_t* d_segment_ids, const int32_t* d_lengths,
                      uint64_t task_mask, int32_t batch, int32_t seq, float* d_logits, void* const* task_events,
                      void* stream_) {
  return mt_forward_tokens(m, d_token_ids, d_segment_ids, d_lengths, task_mask, batch, seq, d_logits, nullptr, task_events,
                           stream_);
}

int mt_forward_tokens(mt_model* m, const int32_t* d_token_ids, const int32_t* d_segment_ids, const int32_t* d_lengths,
                      uint64_t task_mask, int32_t batch, int32_t seq, float* d_logits, float* d_token_logits,
                      void* const* task_events, void* stream_) {
  if (m == nullptr) return MT_ERR_INVALID_ARG;
  if (d_token_ids == nullptr || d_segment_ids == nullptr || d_lengths == nullptr)
    return fail(m, MT_ERR_INVALID_ARG, "null input pointer");
  for (size_t t = 0; t < m->tasks.size(); ++t) {
    if (!((task_mask >> t) & 1)) continue;
    const bool token = m->tasks[t].cfg.head_kind == MT_HEAD_TOKEN;
    if (token && d_token_logits == nullptr)
      return fail(m, MT_ERR_INVALID_ARG, "a token-level task is active: its logits need d_token_logits (mt_forward_tokens)");
    if (!token && d_logits == nullptr) return fail(m, MT_ERR_INVALID_ARG, "null output pointer");
  }
  if (batch < 1 || seq < 1) return fail(m, MT_ERR_INVALID_ARG, "batch and seq must be positive");
  if (batch > m->max_batch || seq > m->max_seq) return fail(m, MT_ERR_SHAPE, "batch/seq beyond the limits of mt_create");
  if (m->d_workspace == nullptr) return fail(m, MT_ERR_NOT_BOUND, "mt_bind_memory has not been called");
  const int32_t T = static_cast<int32_t>(m->tasks.size());
  if (T < 64) task_mask &= (uint64_t(1) << T) - 1;
  if (task_mask == 0) return fail(m, MT_ERR_INVALID_ARG, "task_mask selects no task");
  if (!m->trunk_loaded) return fail(m, MT_ERR_NOT_LOADED, "mt_load_weights has not been called");
  for (int32_t t = 0; t < T; ++t)
    if (((task_mask >> t) & 1) && !m->tasks[t].loaded) return fail(m, MT_ERR_NOT_LOADED, "an active task has no weights");
  cudaStream_t stream = as_stream(stream_);

  const auto key = std::make_tuple(task_mask, batch, seq);
  auto it = m->plans.find(key);
  if (it == m->plans.end()) {
    Schedule s;
    build_schedule(m, task_mask, &s);
    Plan plan;
    cudaError_t e = build_plan(m, s, batch, seq, &plan);
    if (e != cudaSuccess) return fail_cuda(m, e, "building the launch plan");
    // a plan holds hundreds of tensor maps: keep the most recently used ones only
    while (static_cast<int32_t>(m->plans.size()) >= m->plan_cache) {
      auto oldest = m->plans.begin();
      for (auto p = m->plans.begin(); p != m->plans.end(); ++p)
        if (p->second.last_use < oldest->second.last_use) oldest = p;
      m->plans.erase(oldest);
    }
    it = m->plans.emplace(key, std::move(plan)).first;
  }
  Plan& plan = it->second;
  plan.last_use = ++m->use_clock;
  uint32_t* status = reinterpret_cast<uint32_t*>(m->d_workspace + m->ws_status);
  const size_t act_used = static_cast<size_t>(batch) * seq * m->trunk.hidden * sizeof(bf16);
  cudaError_t e;
#define MT_LAUNCH(call, what)                          \
  do {                                                 \
    e = (call);                                        \
    if (e != cudaSuccess) return fail_cuda(m, e, what); \
  } while (0)
  // With option "profile" every kernel launch sits between two events of a pool that grows on the host.
#define MT_TIMED(cls, call, what)                                                            \
  do {                                                                                       \
    if (m->profile) {                                                                        \
      while (m->events.size() < m->events_used + 2) {                                        \
        cudaEvent_t ev;                                                                      \
        MT_LAUNCH(cudaEventCreate(&ev), "creating a timing event");                          \
        m->events.push_back(ev);                                                             \
      }                                                                                      \
      MT_LAUNCH(cudaEventRecord(m->events[m->events_used], stream), "recording an event");   \
    }                                                                                        \
    MT_LAUNCH(call, what);                                                                   \
    if (m->profile) {                                                                        \
      MT_LAUNCH(cudaEventRecord(m->events[m->events_used + 1], stream), "recording an event"); \
      m->events_used += 2;                                                                   \
      m->event_class.push_back(cls);                                                         \
    }                                                                                        \
  } while (0)

  // Steps 3-7 of the layers of a wave: three launches (each residual GEMM carries its LayerNorm) or five.
#define MT_TAIL(tail)                                                                                                  \
  do {                                                                                                                 \
    LayerTail* t_ = (tail);                                                                                            \
    if (t_->ln_fused) {                                                                                                \
      MT_TIMED(MT_CLASS_ATTN_OUT, t_->ln_wide ? launch_gemm_ln_wide(t_->attn_out_ln, stream)                          \
                                              : launch_gemm_ln(t_->attn_out_ln, stream),                              \
               "attention output GEMM + LayerNorm");                                                                   \
    } else {                                                                                                           \
      MT_TIMED(MT_CLASS_ATTN_OUT, launch_gemm(t_->attn_out, kEpiBiasResidual, m->sm_count, stream), "attention output GEMM"); \
      MT_TIMED(MT_CLASS_LN1, launch_layernorm(t_->ln1, stream), "LayerNorm 1");                                        \
    }                                                                                                                  \
    if (t_->fp8) MT_TIMED(MT_CLASS_QUANT, launch_quantize_rows(t_->q_h1, stream), "quantising the FFN input");         \
    MT_TIMED(MT_CLASS_FFN_UP, launch_gemm(t_->ffn_up, kEpiBiasGelu, m->sm_count, stream), "FFN up GEMM");              \
    if (t_->fp8) MT_TIMED(MT_CLASS_QUANT, launch_quantize_rows(t_->q_f, stream), "quantising the FFN intermediate");   \
    if (t_->down_fused) {                                                                                              \
      MT_TIMED(MT_CLASS_FFN_DOWN, t_->ln_wide ? launch_gemm_ln_wide(t_->ffn_down_ln, stream)                          \
                                              : launch_gemm_ln(t_->ffn_down_ln, stream),                              \
               "FFN down GEMM + LayerNorm");                                                                           \
    } else {                                                                                                           \
      MT_TIMED(MT_CLASS_FFN_DOWN, launch_gemm(t_->ffn_down, t_->down_splits > 1 ? kEpiPartialF32 : kEpiBiasResidual,   \
                                              m->sm_count, stream), "FFN down GEMM");                                  \
      MT_TIMED(MT_CLASS_LN2, launch_layernorm(t_->ln2, stream), "LayerNorm 2");                                        \
    }                                                                                                                  \
  } while (0)

  int32_t* row_start = reinterpret_cast<int32_t*>(m->d_workspace + m->ws_row_start);
  MT_LAUNCH(launch_row_starts(d_lengths, batch, seq, m->pack_tokens ? 1 : 0, row_start,
                              reinterpret_cast<int32_t*>(m->d_workspace + m->ws_rows_valid), stream),
            "row-start kernel");
  EmbedParams ep;
  ep.row_start = row_start;
  ep.packed = m->pack_tokens ? 1 : 0;
  ep.token_ids = d_token_ids; ep.segment_ids = d_segment_ids; ep.lengths = d_lengths;
  ep.word = w_ptr(m, m->emb_word); ep.pos = w_ptr(m, m->emb_pos); ep.type = w_ptr(m, m->emb_type);
  ep.gamma = w_ptr(m, m->emb_ln_g); ep.beta = w_ptr(m, m->emb_ln_b);
  ep.out = trunk_buf(m, 0);
  ep.out32 = f32_of(m, ep.out);
  ep.batch = batch; ep.seq = seq; ep.hidden = m->trunk.hidden; ep.vocab = m->trunk.vocab_size;
  ep.type_vocab = m->trunk.type_vocab; ep.eps = m->trunk.ln_eps; ep.status = status;
  MT_TIMED(MT_CLASS_EMBED, launch_embed(ep, stream), "embedding kernel");
  if (m->debug_capture)
    MT_LAUNCH(cudaMemcpyAsync(m->d_workspace + m->ws_dump0, ep.out, act_used, cudaMemcpyDeviceToDevice, stream),
              "debug capture");

  bool side_pending = false;   // work on the side stream that the caller's stream has not waited for yet
  for (PlanStep& st : plan.steps) {
    if (side_pending) {
      MT_LAUNCH(cudaStreamWaitEvent(stream, m->ev_join, 0), "joining the side stream");
      side_pending = false;
    }
    if (st.kind == 0) {
      Chunk& ck = st.chunk;
      ck.attn.lengths = d_lengths;
      ck.attn_cls.lengths = d_lengths;
      if (m->fp8) MT_TIMED(MT_CLASS_QUANT, launch_quantize_rows(ck.q_in, stream), "quantising the layer inputs");
      MT_TIMED(MT_CLASS_QKV, launch_gemm(ck.qkv, kEpiBias, m->sm_count, stream), "QKV GEMM");
      const bool beside = m->overlap_cls && m->side_stream != nullptr && !m->profile && ck.n_cls > 0 && ck.full.count > 0;
      if (beside) {
        MT_LAUNCH(cudaEventRecord(m->ev_fork, stream), "forking the side stream");
        MT_LAUNCH(cudaStreamWaitEvent(m->side_stream, m->ev_fork, 0), "forking the side stream");
        MT_LAUNCH(launch_cls_attention(ck.attn_cls, m->side_stream), "first-token attention kernel");
        MT_LAUNCH(cudaEventRecord(m->ev_join, m->side_stream), "joining the side stream");
        side_pending = true;
      }
      if (ck.full.count > 0) MT_TIMED(MT_CLASS_ATTENTION, launch_attention(ck.attn, stream), "attention kernel");
      if (ck.n_cls > 0 && !beside)
        MT_TIMED(MT_CLASS_ATTENTION, launch_cls_attention(ck.attn_cls, stream), "first-token attention kernel");
      if (ck.full.count > 0) MT_TAIL(&ck.full);
      for (const DumpCopy& d : ck.dumps)
        MT_LAUNCH(cudaMemcpyAsync(m->d_workspace + m->ws_dump0 + m->act_bytes * d.slot, d.src,
                                  d.compact ? static_cast<size_t>(batch) * m->trunk.hidden * sizeof(bf16) : act_used,
                                  cudaMemcpyDeviceToDevice, stream),
                  "debug capture");
    } else if (st.kind == 2) {
      MT_TAIL(&st.tail);
      for (const DumpCopy& d : st.dumps)
        MT_LAUNCH(cudaMemcpyAsync(m->d_workspace + m->ws_dump0 + m->act_bytes * d.slot, d.src,
                                  static_cast<size_t>(batch) * m->trunk.hidden * sizeof(bf16), cudaMemcpyDeviceToDevice,
                                  stream),
                  "debug capture");
    } else {
      if (st.kind == 3) {
        st.token_heads.logits = d_token_logits;
        st.token_heads.lengths = d_lengths;
        MT_TIMED(MT_CLASS_HEAD, launch_token_heads(st.token_heads, stream), "token-level head kernel");
      } else if (st.pool_gemm) {
        st.heads.logits = d_logits;
        MT_TIMED(MT_CLASS_HEAD, launch_gemm(st.pool, kEpiBiasTanhF32, m->sm_count, stream), "pooler GEMM");
        MT_TIMED(MT_CLASS_HEAD, launch_head(st.heads, stream), "head kernel");
      } else {
        st.heads.logits = d_logits;
        MT_TIMED(MT_CLASS_HEAD, launch_pooler_head(st.heads, stream), "pooler/head kernel");
      }
      if (task_events != nullptr)
        for (int32_t t : st.head_tasks)
          if (task_events[t] != nullptr)
            MT_LAUNCH(cudaEventRecord(reinterpret_cast<cudaEvent_t>(task_events[t]), stream), "recording a task event");
    }
  }
  if (side_pending) MT_LAUNCH(cudaStreamWaitEvent(stream, m->ev_join, 0), "joining the side stream");
#undef MT_TAIL
#undef MT_TIMED
#undef MT_LAUNCH
  m->last_batch = batch;
  m->last_seq = seq;
  m->last_lengths = d_lengths;
  return MT_OK;
}

int mt_forward_host(mt_model* m, const int32_t* h_token_ids, const int32_t* h_segment_ids, const int32_t* h_lengths,
                    uint64_t task_mask, int32_t batch, int32_t seq, float* h_logits, void* stream_) {
  int rc = mt_forward_host_async(m, h_token_ids, h_segment_ids, h_lengths, task_mask, batch, seq, h_logits, stream_);
  if (rc != MT_OK) return rc;
  cudaError_t e = cudaStreamSynchronize(as_stream(stream_));
  return e == cudaSuccess ? MT_OK : fail_cuda(m, e, "waiting for the logits");
}

int mt_forward_host_async(mt_model* m, const int32_t* h_token_ids, const int32_t* h_segment_ids, const int32_t* h_lengths,
                          uint64_t task_mask, int32_t batch, int32_t seq, float* h_logits, void* stream_) {
  if (m == nullptr) return MT_ERR_INVALID_ARG;
  if (h_token_ids == nullptr || h_segment_ids == nullptr || h_lengths == nullptr || h_logits == nullptr)
    return fail(m, MT_ERR_INVALID_ARG, "null input or output pointer");
  if (batch < 1 || seq < 1) return fail(m, MT_ERR_INVALID_ARG, "batch and seq must be positive");
  if (batch > m->max_batch || seq > m->max_seq) return fail(m, MT_ERR_SHAPE, "batch/seq beyond the limits of mt_create");
  if (m->d_workspace == nullptr) return fail(m, MT_ERR_NOT_BOUND, "mt_bind_memory has not been called");
  cudaStream_t stream = as_stream(stream_);
  int32_t* d_tok = reinterpret_cast<int32_t*>(m->d_workspace + m->ws_tok);
  int32_t* d_seg = reinterpret_cast<int32_t*>(m->d_workspace + m->ws_seg);
  int32_t* d_len = reinterpret_cast<int32_t*>(m->d_workspace + m->ws_len);
  float* d_logits = reinterpret_cast<float*>(m->d_workspace + m->ws_logits);
  const size_t n = static_cast<size_t>(batch) * seq * 4;
  const size_t out_bytes = static_cast<size_t>(batch) * m->c_total * 4;
  cudaError_t e;
  if ((e = cudaMemcpyAsync(d_tok, h_token_ids, n, cudaMemcpyHostToDevice, stream)) != cudaSuccess ||
      (e = cudaMemcpyAsync(d_seg, h_segment_ids, n, cudaMemcpyHostToDevice, stream)) != cudaSuccess ||
      (e = cudaMemcpyAsync(d_len, h_lengths, static_cast<size_t>(batch) * 4, cudaMemcpyHostToDevice, stream)) != cudaSuccess ||
      (e = cudaMemsetAsync(d_logits, 0, out_bytes, stream)) != cudaSuccess)
    return fail_cuda(m, e, "copying inputs to the device");
  int rc = mt_forward(m, d_tok, d_seg, d_len, task_mask, batch, seq, d_logits, stream_);
  if (rc != MT_OK) return rc;
  if ((e = cudaMemcpyAsync(h_logits, d_logits, out_bytes, cudaMemcpyDeviceToHost, stream)) != cudaSuccess)
    return fail_cuda(m, e, "copying logits to the host");
  return MT_OK;
}

int mt_poll_status(mt_model* m, void* stream_, uint32_t* flags) {
  if (m == nullptr) return MT_ERR_INVALID_ARG;
  if (m->d_workspace == nullptr) return fail(m, MT_ERR_NOT_BOUND, "mt_bind_memory has not been called");
  cudaStream_t stream = as_stream(stream_);
  uint32_t word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, m->d_workspace + m->ws_status, 4, cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(m->d_workspace + m->ws_status, 0, 4, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return fail_cuda(m, e, "reading the status word");
  if (flags) *flags = word;
  if (word != 0) {
    char buf[64];
    snprintf(buf, sizeof(buf), "device status word 0x%x", word);
    return fail(m, MT_ERR_DEVICE_FLAG, buf);
  }
  return MT_OK;
}

int mt_profile_read(mt_model* m, double* ms_by_class, int64_t* launches_by_class) {
  if (m == nullptr || ms_by_class == nullptr || launches_by_class == nullptr) return MT_ERR_INVALID_ARG;
  for (int c = 0; c < MT_NUM_CLASSES; ++c) { ms_by_class[c] = 0.0; launches_by_class[c] = 0; }
  for (size_t i = 0; i < m->event_class.size(); ++i) {
    cudaError_t e = cudaEventSynchronize(m->events[2 * i + 1]);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, m->events[2 * i], m->events[2 * i + 1]);
    if (e != cudaSuccess) return fail_cuda(m, e, "reading a timing event");
    ms_by_class[m->event_class[i]] += ms;
    launches_by_class[m->event_class[i]] += 1;
  }
  m->events_used = 0;
  m->event_class.clear();
  return MT_OK;
}

int mt_debug_copy_hidden(mt_model* m, int32_t task, int32_t layer, void* d_out, void* stream_) {
  if (m == nullptr || d_out == nullptr) return MT_ERR_INVALID_ARG;
  if (!m->debug_capture) return fail(m, MT_ERR_INVALID_ARG, "option debug_capture is off");
  if (m->d_workspace == nullptr || m->last_batch == 0) return fail(m, MT_ERR_NOT_BOUND, "no forward has run");
  const int32_t T = static_cast<int32_t>(m->tasks.size());
  if (task < -1 || task >= T) return fail(m, MT_ERR_INVALID_ARG, "task out of range");
  if (task < 0 ? (layer < 0 || layer > m->trunk.trunk_layers) : (layer < 1 || layer > m->tasks[task].cfg.branch_layers))
    return fail(m, MT_ERR_INVALID_ARG, "layer out of range");
  // the captured state is in the layout of the forward (packed or padded): hand it back padded
  cudaError_t e = launch_unpack_rows(
      reinterpret_cast<const bf16*>(m->d_workspace + m->ws_dump0 + m->act_bytes * dump_slot(m, task, layer)),
      m->last_lengths, reinterpret_cast<const int32_t*>(m->d_workspace + m->ws_row_start),
      static_cast<bf16*>(d_out), m->last_batch, m->last_seq, m->trunk.hidden,
      (task >= 0 && is_compact_task(m, task) && layer == m->tasks[task].cfg.branch_layers) ? 1 : 0, as_stream(stream_));
  if (e != cudaSuccess) return fail_cuda(m, e, "copying a captured hidden state");
  return MT_OK;
}

// ---- single steps ------------------------------------------------------------------------------

void mt_kernel_linear_force_block_n(int32_t block_n) { g_force_block_n = block_n; }

int mt_kernel_linear(const void* d_x, const void* d_w, const void* d_bias, const void* d_residual, void* d_y, int32_t M,
                     int32_t N, int32_t K, int32_t epilogue, int32_t cta_pair, uint32_t* d_status, void* stream) {
  if (d_x == nullptr || d_w == nullptr || d_bias == nullptr || d_y == nullptr || M < 1 || N < 128 || N % 128 != 0 ||
      K < 64 || K % 64 != 0 || epilogue < 0 || epilogue > 2 || (epilogue == 2 && d_residual == nullptr))
    return MT_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return MT_ERR_CUDA;
  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.n_groups = 1; p.M = M; p.N = N; p.K = K; p.status = d_status;
  p.pair = cta_pair != 0 ? 1 : 0;
  p.block_n = gemm_block_n(N, epilogue, M, 1, p.pair != 0, sms);
  if (g_force_block_n > 0 && N % g_force_block_n == 0) p.block_n = g_force_block_n;
  if (set_gemm_group(&p, 0, epilogue, d_x, d_w, static_cast<const bf16*>(d_bias), static_cast<const float*>(d_residual),
                     d_y) != cudaSuccess)
    return MT_ERR_CUDA;
  return launch_gemm(p, epilogue, sms, as_stream(stream)) == cudaSuccess ? MT_OK : MT_ERR_CUDA;
}

int mt_kernel_linear_partial(const void* d_x, const void* d_w, void* d_part, int32_t M, int32_t N, int32_t K,
                             int32_t k_splits, int32_t split_pitch, uint32_t* d_status, void* stream) {
  if (d_x == nullptr || d_w == nullptr || d_part == nullptr || M < 1 || N < 128 || N % 128 != 0 || K < 64 ||
      K % 64 != 0 || k_splits < 1 || (K / 64) % k_splits != 0 || split_pitch < M || split_pitch % 128 != 0)
    return MT_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return MT_ERR_CUDA;
  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.n_groups = 1; p.M = M; p.N = N; p.K = K; p.status = d_status;
  p.k_splits = k_splits; p.split_pitch = split_pitch;
  p.block_n = gemm_block_n(N, kEpiPartialF32, M, k_splits, false, sms);
  if (g_force_block_n == 64 || g_force_block_n == 128) p.block_n = g_force_block_n;
  if (set_gemm_group(&p, 0, kEpiPartialF32, d_x, d_w, nullptr, nullptr, d_part) != cudaSuccess) return MT_ERR_CUDA;
  if (make_tmap(&p.tmap_out[0], d_part, static_cast<int64_t>(k_splits) * split_pitch, N, 32, 32, true) != cudaSuccess)
    return MT_ERR_CUDA;
  return launch_gemm(p, kEpiPartialF32, sms, as_stream(stream)) == cudaSuccess ? MT_OK : MT_ERR_CUDA;
}

int mt_kernel_quantize_rows(const void* d_x, void* d_q, float* d_scale, int32_t rows, int32_t cols, void* stream) {
  if (d_x == nullptr || d_q == nullptr || d_scale == nullptr || rows < 1 || cols < 256 || cols % 256 != 0)
    return MT_ERR_INVALID_ARG;
  QuantParams p;
  memset(&p, 0, sizeof(p));
  p.x[0] = static_cast<const bf16*>(d_x); p.q[0] = static_cast<uint8_t*>(d_q); p.scale[0] = d_scale;
  p.n_groups = 1; p.rows = rows; p.cols = cols;
  return launch_quantize_rows(p, as_stream(stream)) == cudaSuccess ? MT_OK : MT_ERR_CUDA;
}

int mt_kernel_linear_fp8(const void* d_xq, const float* d_scale_x, const void* d_wq, const float* d_scale_w,
                         const void* d_bias, const void* d_residual, void* d_y, int32_t M, int32_t N, int32_t K,
                         int32_t epilogue, uint32_t* d_status, void* stream) {
  if (d_xq == nullptr || d_scale_x == nullptr || d_wq == nullptr || d_scale_w == nullptr || d_bias == nullptr ||
      d_y == nullptr || M < 1 || K < 128 || K % 128 != 0 || epilogue < 0 || epilogue > 2 ||
      (epilogue == 2 && d_residual == nullptr))
    return MT_ERR_INVALID_ARG;
  if (N < 128 || N % (epilogue == 2 ? 128 : 256) != 0) return MT_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return MT_ERR_CUDA;
  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.n_groups = 1; p.M = M; p.N = N; p.K = K; p.status = d_status;
  p.fp8 = 1;
  p.block_n = epilogue == 2 ? 128 : 256;
  if (set_gemm_group(&p, 0, epilogue, d_xq, d_wq, static_cast<const bf16*>(d_bias), static_cast<const float*>(d_residual),
                     d_y) != cudaSuccess)
    return MT_ERR_CUDA;
  p.group[0].scale_x = d_scale_x;
  p.group[0].scale_w = d_scale_w;
  return launch_gemm(p, epilogue, sms, as_stream(stream)) == cudaSuccess ? MT_OK : MT_ERR_CUDA;
}

int mt_kernel_linear_layernorm(const void* d_x, const void* d_w, const void* d_bias, const void* d_residual,
                               const void* d_gamma, const void* d_beta, void* d_y, void* d_y_f32, int32_t M, int32_t N,
                               int32_t K, float eps, uint32_t* d_status, void* stream) {
  return mt_kernel_linear_layernorm_tiles(d_x, d_w, d_bias, d_residual, d_gamma, d_beta, d_y, d_y_f32, M, N, K, eps, 128,
                                          d_status, stream);
}

int mt_kernel_linear_layernorm_tiles(const void* d_x, const void* d_w, const void* d_bias, const void* d_residual,
                                     const void* d_gamma, const void* d_beta, void* d_y, void* d_y_f32, int32_t M,
                                     int32_t N, int32_t K, float eps, int32_t tile_cols, uint32_t* d_status, void* stream) {
  if (tile_cols != 128 && tile_cols != 256) return MT_ERR_INVALID_ARG;
  if (d_x == nullptr || d_w == nullptr || d_bias == nullptr || d_residual == nullptr || d_gamma == nullptr ||
      d_beta == nullptr || d_y == nullptr || d_y_f32 == nullptr || M < 1 || !gemm_ln_supported(N) || K < 64 || K % 64 != 0 ||
      !(eps >= 0.f))
    return MT_ERR_INVALID_ARG;
  GemmLnParams p;
  memset(&p, 0, sizeof(p));
  p.n_groups = 1; p.M = M; p.N = N; p.K = K; p.eps = eps; p.status = d_status;
  if (make_tmap(&p.tmap_x[0], d_x, M, K, kGemmBlockM, kGemmBlockK, false) != cudaSuccess ||
      make_tmap(&p.tmap_w[0], d_w, N, K, 128, kGemmBlockK, false) != cudaSuccess ||
      make_tmap(&p.tmap_w256[0], d_w, N, K, 256, kGemmBlockK, false) != cudaSuccess ||
      make_tmap(&p.tmap_res[0], d_residual, M, N, 32, 32, true) != cudaSuccess ||
      make_tmap(&p.tmap_y[0], d_y, M, N, 32, 64, false) != cudaSuccess ||
      make_tmap(&p.tmap_y32[0], d_y_f32, M, N, 32, 32, true) != cudaSuccess)
    return MT_ERR_CUDA;
  p.bias[0] = static_cast<const bf16*>(d_bias);
  p.gamma[0] = static_cast<const bf16*>(d_gamma);
  p.beta[0] = static_cast<const bf16*>(d_beta);
  p.residual[0] = static_cast<const float*>(d_residual);
  const cudaError_t e = tile_cols == 256 ? launch_gemm_ln_wide(p, as_stream(stream)) : launch_gemm_ln(p, as_stream(stream));
  return e == cudaSuccess ? MT_OK : MT_ERR_CUDA;
}

int mt_kernel_attention(const void* d_qkv, const int32_t* d_lengths, void* d_ctx, int32_t batch, int32_t seq,
                        int32_t heads, int32_t tensor_memory, uint32_t* d_status, void* stream) {
  if (d_qkv == nullptr || d_lengths == nullptr || d_ctx == nullptr || batch < 1 || seq < 1 || heads < 1 ||
      (tensor_memory != 0 && seq > kAttnTensorMemoryMaxSeq))
    return MT_ERR_INVALID_ARG;
  AttnParams p;
  memset(&p, 0, sizeof(p));
  p.qkv[0] = static_cast<const bf16*>(d_qkv);
  p.ctx[0] = static_cast<bf16*>(d_ctx);
  p.lengths = d_lengths;
  p.n_groups = 1; p.batch = batch; p.seq = seq; p.heads = heads;
  p.status = d_status;
  if (tensor_memory != 0) {
    p.tensor_memory = 1;
    if (make_tmap(&p.tmap_qkv[0], d_qkv, static_cast<int64_t>(batch) * seq, 3 * static_cast<int64_t>(heads) * kHeadDim,
                  kAttnTileRows, kHeadDim, false) != cudaSuccess ||
        make_tmap(&p.tmap_qkv64[0], d_qkv, static_cast<int64_t>(batch) * seq, 3 * static_cast<int64_t>(heads) * kHeadDim,
                  kAttnTileRows / 2, kHeadDim, false) != cudaSuccess)
      return MT_ERR_CUDA;
  }
  return launch_attention(p, as_stream(stream)) == cudaSuccess ? MT_OK : MT_ERR_CUDA;
}

int mt_kernel_layernorm(const void* d_x, const void* d_gamma, const void* d_beta, void* d_y, void* d_y_f32,
                        int32_t rows, int32_t hidden, float eps, void* stream) {
  if (d_x == nullptr || d_gamma == nullptr || d_beta == nullptr || d_y == nullptr || rows < 1) return MT_ERR_INVALID_ARG;
  if (hidden != 768 && hidden != 1024) return MT_ERR_UNSUPPORTED;
  LayerNormParams p;
  memset(&p, 0, sizeof(p));
  p.x[0] = static_cast<const float*>(d_x); p.gamma[0] = static_cast<const bf16*>(d_gamma);
  p.beta[0] = static_cast<const bf16*>(d_beta); p.y[0] = static_cast<bf16*>(d_y);
  p.y32[0] = static_cast<float*>(d_y_f32);
  p.n_groups = 1; p.rows = rows; p.hidden = hidden; p.eps = eps;
  return launch_layernorm(p, as_stream(stream)) == cudaSuccess ? MT_OK : MT_ERR_CUDA;
}

int mt_kernel_layernorm_partial(const float* d_part, int32_t n_parts, int32_t part_pitch, const float* d_residual,
                                const void* d_bias, const void* d_gamma, const void* d_beta, void* d_y, void* d_y_f32,
                                int32_t rows, int32_t hidden, float eps, void* stream) {
  if (d_part == nullptr || d_residual == nullptr || d_bias == nullptr || d_gamma == nullptr || d_beta == nullptr ||
      d_y == nullptr || rows < 1 || n_parts < 1 || n_parts > 4 || part_pitch < rows)
    return MT_ERR_INVALID_ARG;
  if (hidden != 768 && hidden != 1024) return MT_ERR_UNSUPPORTED;
  LayerNormParams p;
  memset(&p, 0, sizeof(p));
  p.part[0] = d_part; p.residual[0] = d_residual; p.bias[0] = static_cast<const bf16*>(d_bias);
  p.n_parts = n_parts; p.part_pitch = part_pitch;
  p.gamma[0] = static_cast<const bf16*>(d_gamma); p.beta[0] = static_cast<const bf16*>(d_beta);
  p.y[0] = static_cast<bf16*>(d_y); p.y32[0] = static_cast<float*>(d_y_f32);
  p.n_groups = 1; p.rows = rows; p.hidden = hidden; p.eps = eps;
  return launch_layernorm(p, as_stream(stream)) == cudaSuccess ? MT_OK : MT_ERR_CUDA;
}

int mt_debug_wait_probe(uint64_t limit_ns, int32_t arrive, uint32_t* d_status, uint64_t* d_waited_ns, int32_t* d_ok,
                        void* stream) {
  // (at most a second: the second warp's own limit is 64 times the first's)
  if (limit_ns < 1000 || limit_ns > 15000000ull || d_waited_ns == nullptr || d_ok == nullptr) return MT_ERR_INVALID_ARG;
  return launch_wait_probe(limit_ns, arrive != 0 ? 1 : 0, d_status, reinterpret_cast<unsigned long long*>(d_waited_ns),
                           d_ok, as_stream(stream)) == cudaSuccess ? MT_OK : MT_ERR_CUDA;
}

int mt_kernel_embed(const int32_t* d_token_ids, const int32_t* d_segment_ids, const int32_t* d_lengths,
                    const void* d_word, const void* d_pos, const void* d_type, const void* d_gamma, const void* d_beta,
                    void* d_h0, void* d_h0_f32, int32_t batch, int32_t seq, int32_t hidden, int32_t vocab,
                    int32_t type_vocab, float eps, uint32_t* d_status, void* stream) {
  if (d_token_ids == nullptr || d_segment_ids == nullptr || d_lengths == nullptr || d_word == nullptr ||
      d_pos == nullptr || d_type == nullptr || d_gamma == nullptr || d_beta == nullptr || d_h0 == nullptr ||
      batch < 1 || seq < 1 || vocab < 1 || type_vocab < 1)
    return MT_ERR_INVALID_ARG;
  if (hidden != 768 && hidden != 1024) return MT_ERR_UNSUPPORTED;
  EmbedParams p;
  p.token_ids = d_token_ids; p.segment_ids = d_segment_ids; p.lengths = d_lengths;
  p.word = static_cast<const bf16*>(d_word); p.pos = static_cast<const bf16*>(d_pos);
  p.type = static_cast<const bf16*>(d_type); p.gamma = static_cast<const bf16*>(d_gamma);
  p.beta = static_cast<const bf16*>(d_beta); p.out = static_cast<bf16*>(d_h0);
  p.out32 = static_cast<float*>(d_h0_f32);
  p.batch = batch; p.seq = seq; p.hidden = hidden; p.vocab = vocab; p.type_vocab = type_vocab; p.eps = eps;
  p.status = d_status;
  p.row_start = nullptr;
  p.packed = 0;
  return launch_embed(p, as_stream(stream)) == cudaSuccess ? MT_OK : MT_ERR_CUDA;
}

int mt_kernel_pooler_head(const void* d_hidden, const void* d_pool_w, const void* d_pool_b, const void* d_cls_w,
                          const void* d_cls_b, float* d_pooled_scratch, float* d_logits, int32_t batch, int32_t seq,
                          int32_t hidden, int32_t num_classes, int32_t logits_stride, int32_t col0, void* stream) {
  if (d_pooled_scratch == nullptr) return MT_ERR_INVALID_ARG;
  if (d_hidden == nullptr || d_pool_w == nullptr || d_pool_b == nullptr || d_cls_w == nullptr || d_cls_b == nullptr ||
      d_logits == nullptr || batch < 1 || seq < 1 || num_classes < 1 || col0 < 0 || logits_stride < col0 + num_classes)
    return MT_ERR_INVALID_ARG;
  if (hidden != 768 && hidden != 1024) return MT_ERR_UNSUPPORTED;
  HeadParams p;
  memset(&p, 0, sizeof(p));
  p.task[0] = {static_cast<const bf16*>(d_hidden), static_cast<const bf16*>(d_pool_w),
               static_cast<const bf16*>(d_pool_b), static_cast<const bf16*>(d_cls_w),
               static_cast<const bf16*>(d_cls_b), num_classes, col0};
  p.logits = d_logits;
  p.pooled = d_pooled_scratch;
  p.n_tasks = 1; p.batch = batch; p.seq = seq; p.hidden = hidden; p.logits_stride = logits_stride;
  return launch_pooler_head(p, as_stream(stream)) == cudaSuccess ? MT_OK : MT_ERR_CUDA;
}

}  // extern "C"
