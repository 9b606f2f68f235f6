/*
 * mt_bert.h - C ABI of the merged multi-task BERT forward pass for NVIDIA B200 (sm_100a).
 *
 * The paper (Section 3.3, Fig. 1(c)) merges several single-task student models - each made of
 * x frozen bottom layers of one pre-trained BERT encoder plus y task-specific transformer layers,
 * Table 2's "(x, y)" - into ONE computation graph whose frozen layers are evaluated once per
 * request and shared by all tasks.  Every task reads the shared trunk after its own depth
 * (Section 5.1), runs its own layers, and a request yields the output of every task (Section 5.2).
 * This library is that serving-time graph: mt_create() builds the tree, mt_load_weights() loads
 * the checkpoints into it, mt_forward() evaluates it.
 *
 * Conventions
 *  - All device memory and all streams belong to the caller.  The library allocates only host
 *    metadata.  Pointers named d_* are DEVICE pointers, everything else is a HOST pointer.
 *  - cudaStream_t is passed as a plain `void*` (the value of the stream handle; NULL = default stream).
 *  - Weights and the operands of every matrix product are bf16; accumulation, LayerNorm statistics
 *    and the residual stream (every LayerNorm input and the residual it is added to) are fp32; logits
 *    are fp32.
 *  - Every entry point returns an mt_status (0 = OK, negative = error); nothing throws, aborts or
 *    traps.  mt_last_error_string() describes the most recent failure on that model.
 *  - Encoder layer (the published post-LayerNorm BERT layer the paper builds on, Section 3):
 *        u  = x + (softmax(QK^T/sqrt(64) over valid keys) V) Wo^T + bo ;  h1 = LN(u)
 *        h2 = LN(h1 + GELU_erf(h1 W1^T + b1) W2^T + b2)
 *    with Q,K,V = x W{q,k,v}^T + b, every W stored [out, in], LN with biased variance.
 *  - There is no CPU fallback: without a CUDA device every compute entry point fails with MT_ERR_CUDA.
 */
#ifndef MT_BERT_H_
#define MT_BERT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MT_OK = 0,
  MT_ERR_INVALID_ARG = -1,   /* null pointer, bad index, empty task mask ...              */
  MT_ERR_SHAPE = -2,         /* batch/seq beyond the limits given to mt_create             */
  MT_ERR_NOT_BOUND = -3,     /* mt_bind_memory has not been called                         */
  MT_ERR_NOT_LOADED = -4,    /* weights of the trunk or of an active task are not loaded   */
  MT_ERR_BLOB_MISMATCH = -5, /* weight blob header/size disagrees with the configuration   */
  MT_ERR_CUDA = -6,          /* a CUDA runtime/driver call failed                          */
  MT_ERR_UNSUPPORTED = -7,   /* configuration outside what the kernels implement           */
  MT_ERR_DEVICE_FLAG = -8    /* mt_poll_status: the device status word is non-zero         */
} mt_status;

/* Bits of the sticky device status word returned through mt_poll_status(). */
#define MT_FLAG_BAD_TOKEN    0x1u  /* a token id was outside [0, vocab): clamped              */
#define MT_FLAG_BAD_SEGMENT  0x2u  /* a segment id was outside [0, type_vocab): clamped       */
#define MT_FLAG_BAD_LENGTH   0x4u  /* a length was outside [1, seq]: clamped                  */
#define MT_FLAG_WAIT_TIMEOUT 0x8u  /* a pipeline wait inside a kernel gave up (results invalid) */

/* Encoder shared by trunk and branches: the paper uses 12-layer uncased BERT-base (Section 3). */
typedef struct {
  int32_t vocab_size;    /* 30522 */
  int32_t max_position;  /* 512: learned absolute positions */
  int32_t type_vocab;    /* 2 */
  int32_t hidden;        /* 768 or 1024; must be heads * 64 */
  int32_t heads;         /* 12 or 16 */
  int32_t ffn;           /* 3072 or 4096 */
  int32_t trunk_layers;  /* number of frozen layers loaded (12 for BERT-base) */
  float   ln_eps;        /* 1e-12 */
  int32_t activation;    /* 0 = GELU of the exact form x * Phi(x); nothing else is implemented.  The kernels evaluate
                            it through a fitted sigmoid argument, absolute error <= 2.6e-5 before bf16 rounding */
} mt_trunk_config;

/* One student model before merging, Table 2's (x, y): x = fork_depth frozen layers, y = branch_layers. */
typedef struct {
  int32_t fork_depth;     /* 0..trunk_layers; 0 forks off the embedding output */
  int32_t branch_layers;  /* >= 0; 0 pools the trunk state directly            */
  int32_t num_classes;    /* >= 1; 1 = regression head (raw output)            */
  int32_t head_kind;      /* MT_HEAD_SEQUENCE or MT_HEAD_TOKEN                 */
} mt_task_config;
/* Output layer of a task.  The paper's GLUE tasks are sequence-level: tanh pooler on the first token,
 * then a linear head.  Its production system (Appendix E) also serves token-level tasks and gives no
 * formula for them; the reading here is one linear map on every token's final state, no pooler (the
 * task's pooler tensors stay in the blob, unused). */
#define MT_HEAD_SEQUENCE 0
#define MT_HEAD_TOKEN    1

typedef struct mt_model mt_model;

/* ---- model merging (Section 3.3) ------------------------------------------------------------ */

/* Builds the merged tree for n_tasks (1..64) students over one trunk.  No GPU work.
 * max_batch*max_seq bounds every later mt_forward; max_seq <= max_position and <= 512.
 * *out receives a heap object owned by the caller until mt_destroy().
 * Errors: INVALID_ARG (nulls, depths out of range), UNSUPPORTED (hidden != heads*64, hidden/ffn not
 * multiples of 256, activation != 0). */
int mt_create(const mt_trunk_config* trunk, const mt_task_config* tasks, int32_t n_tasks,
              int32_t max_batch, int32_t max_seq, mt_model** out);
void mt_destroy(mt_model* m);

/* Sizes (bytes) of the two caller-provided device arenas.  The workspace size grows when the
 * debug capture is enabled (mt_set_option "debug_capture") - query it after setting that option. */
size_t mt_weights_bytes(const mt_model* m);
size_t mt_workspace_bytes(const mt_model* m);

/* Hands the library its two device arenas (both 256-byte aligned, at least the sizes above).
 * The caller keeps ownership and must keep them alive while the model is used. */
int mt_bind_memory(mt_model* m, void* d_weights, size_t weights_bytes, void* d_workspace, size_t workspace_bytes);

/* Size and layout of the host weight blob: a 256-byte header followed by bf16 tensors, each padded
 * to 256 bytes, in this order: word/position/type embedding tables, embedding LN gamma/beta; for
 * every trunk layer: wq wk wv bq bk bv wo bo ln1_g ln1_b w1 b1 w2 b2 ln2_g ln2_b; then for every task
 * its branch layers (same 16 tensors each), pool_w [H,H], pool_b, cls_w [C,H], cls_b.
 * Header (little endian): u32 magic 'MTBW'=0x4D544257, u32 version=1, u32 kind (0 full, 1 one task),
 * i32 hidden, heads, ffn, trunk_layers, vocab, max_position, type_vocab, n_tasks, task_index (-1 for
 * full), fork_depth, branch_layers, num_classes (of that task; 0 for full), i32 reserved = 0,
 * u64 payload_bytes (at byte 64). */
size_t mt_blob_bytes(const mt_model* m);
size_t mt_task_blob_bytes(const mt_model* m, int32_t task);

/* Model merging (Section 3.3): the students' checkpoints, packed into one blob, are loaded into the one
 * merged graph.
 * Validates the header against the configuration, then copies the payload to the weights arena
 * with cudaMemcpyAsync on `stream` (host_blob must stay valid until the stream reaches that point;
 * pinned memory makes the copy asynchronous).  Errors: NOT_BOUND, BLOB_MISMATCH, CUDA. */
int mt_load_weights(mt_model* m, const void* host_blob, size_t bytes, void* stream);

/* Per-task update (Sections 1 and 5.1: a task is modified without affecting the others):
 * replaces the branch layers, pooler and head of one task; nothing else in the arena is touched. */
int mt_load_task_weights(mt_model* m, int32_t task, const void* host_blob, size_t bytes, void* stream);

/* Several models over ONE weights arena: a server that keeps more than one batch in flight (one model and
 * one stream per batch in flight; the kernels of independent forwards fill one another's ramps and tails,
 * +11 % sequences/s with two at batch 32 x seq 128) needs a workspace per model but the weights only
 * once.  Create the second model from the same configuration, bind it with the FIRST model's d_weights
 * and a workspace of its own, then call this instead of mt_load_weights: it marks as loaded whatever
 * `src` has loaded.  Later mt_load_weights / mt_load_task_weights on either model write the shared
 * arena; repeat the call on the other one.  Errors: NOT_BOUND, INVALID_ARG (different arenas),
 * BLOB_MISMATCH (different configurations). */
int mt_adopt_weights(mt_model* m, const mt_model* src);

/* ---- the hot path ---------------------------------------------------------------------------- */

/* Merged multi-task forward of one padded batch.
 *   d_token_ids, d_segment_ids : int32 [batch, seq] row-major (device)
 *   d_lengths                  : int32 [batch], valid tokens per sequence, 1..seq (device)
 *   task_mask                  : bit t set = task t is evaluated; 0 is an error
 *   d_logits                   : fp32 [batch, C_total] row-major (device), task t in columns
 *                                [off_t, off_t + C_t), off_t = sum of C of the tasks before it;
 *                                columns of tasks not in the mask are left untouched
 * The shared trunk runs once, to the deepest fork among the active tasks only; each active task's
 * branch starts from the trunk state at its fork depth; keys at positions >= length are excluded
 * from every softmax; the pooler reads position 0.  Asynchronous: only enqueues kernels on `stream`,
 * never synchronises, never allocates device memory.  The first call for a given
 * (batch, seq, task_mask) builds and caches a launch plan on the host (host memory and tensor-map
 * encoding only; the model's own second stream and its two events exist since mt_bind_memory) - make one
 * warm-up call before capturing mt_forward into a CUDA graph.  Option "profile" creates CUDA events here.
 * One mt_model serves one caller at a time: the cached plans carry per-call pointers.
 * Errors: INVALID_ARG, SHAPE, NOT_BOUND, NOT_LOADED, CUDA. */
int mt_forward(mt_model* m, const int32_t* d_token_ids, const int32_t* d_segment_ids,
               const int32_t* d_lengths, uint64_t task_mask, int32_t batch, int32_t seq,
               float* d_logits, void* stream);

/* mt_forward that also tells the caller when each task is done.  task_events: NULL, or an array of
 * n_tasks entries, each NULL or a cudaEvent_t (passed as void*) owned by the caller; the event of
 * task t is recorded on `stream` right after the launch that writes that task's logits, so a second
 * stream (cudaStreamWaitEvent) or the host (cudaEventSynchronize) can pick up task t's columns of
 * d_logits before the other tasks have finished.  The paper notes that in the merged model no task's
 * output is available before all are computed (Section 5.2); with option "early_heads" = 1 every task's
 * head is scheduled right after the wave that completes its branch, so tasks that fork low and have
 * short branches finish first.  Without that option all heads of tasks with branch layers share one
 * launch at the end (higher throughput) and their events are recorded together. */
int mt_forward_events(mt_model* m, const int32_t* d_token_ids, const int32_t* d_segment_ids,
                      const int32_t* d_lengths, uint64_t task_mask, int32_t batch, int32_t seq,
                      float* d_logits, void* const* task_events, void* stream);

/* mt_forward_events for trees with token-level tasks (mt_task_config.head_kind = MT_HEAD_TOKEN).
 *   d_logits       : fp32 [batch, C_total], C_total counted over the sequence-level tasks only, task t in
 *                    columns [off_t, off_t + C_t) among them (may be NULL if none is active)
 *   d_token_logits : fp32 [batch, seq, Ct_total], Ct_total counted over the token-level tasks only;
 *                    element (b, pos, off_t + c) for pos < length(b); positions >= length and columns of
 *                    tasks not in the mask are left untouched (may be NULL if no token-level task is active)
 * A token-level task's last branch layer is evaluated on all tokens (nothing to skip), and its head
 * runs right after the wave that completes its branch.  mt_forward and mt_forward_events are this call
 * with d_token_logits = NULL: they fail with INVALID_ARG if the mask selects a token-level task. */
int mt_forward_tokens(mt_model* m, const int32_t* d_token_ids, const int32_t* d_segment_ids,
                      const int32_t* d_lengths, uint64_t task_mask, int32_t batch, int32_t seq,
                      float* d_logits, float* d_token_logits, void* const* task_events, void* stream);

/* Same computation from HOST buffers: copies the three inputs to the workspace, runs mt_forward,
 * copies the logits back to h_logits ([batch, C_total] fp32) and synchronises the stream.
 * Pinned host buffers make the copies asynchronous with respect to the host. */
int mt_forward_host(mt_model* m, const int32_t* h_token_ids, const int32_t* h_segment_ids,
                    const int32_t* h_lengths, uint64_t task_mask, int32_t batch, int32_t seq,
                    float* h_logits, void* stream);
/* The same without the final synchronisation: everything (three copies in, the forward, one copy out)
 * is only enqueued on `stream`; the host buffers must stay valid, and h_logits must not be read, until
 * the stream has reached that point.  With pinned buffers nothing here blocks the host, so the whole
 * call can also be captured into a CUDA graph and replayed. */
int mt_forward_host_async(mt_model* m, const int32_t* h_token_ids, const int32_t* h_segment_ids,
                          const int32_t* h_lengths, uint64_t task_mask, int32_t batch, int32_t seq,
                          float* h_logits, void* stream);

/* Synchronises `stream`, reads the sticky device status word into *flags (may be NULL) and clears
 * it.  Returns MT_ERR_DEVICE_FLAG if it was non-zero. */
int mt_poll_status(mt_model* m, void* stream, uint32_t* flags);

/* ---- scheduler introspection (host only, no GPU needed) --------------------------------------- */

/* The tree scheduler runs trunk layer w and every branch layer whose input is ready as one
 * "wave" of grouped launches.  These report the plan for a task mask: the number of transformer
 * layers executed (the paper's overhead measure, Section 4.1: shared depth + sum of task layers),
 * the number of waves, and per wave the number of layers grouped in it (groups_per_wave may be NULL;
 * otherwise room for trunk_layers + max branch_layers + 1 ints). */
int mt_plan_summary(const mt_model* m, uint64_t task_mask, int32_t* n_layers, int32_t* n_waves,
                    int32_t* trunk_depth, int32_t* groups_per_wave);
/* Kernel launches one mt_forward at batch = max_batch, seq = max_seq enqueues for this mask. */
int mt_plan_launches(const mt_model* m, uint64_t task_mask, int32_t* n_launches);

/* Launch plans currently cached (host side; no device access).  mt_forward keeps one plan per distinct
 * (task_mask, batch, seq), at most option "plan_cache" of them (default 32, >= 1, any time; setting it
 * clears the cache); beyond that the least recently used plan is dropped and rebuilt on its next use.
 * Serving many request shapes (Section 5.2: per-request task subsets) therefore costs bounded host memory.
 * Returns the count, or MT_ERR_INVALID_ARG for a null model. */
int mt_plan_cache_size(const mt_model* m);

/* Options.  key "max_groups" (1..8): upper bound on layers fused into one grouped launch;
 * key "debug_capture" (0/1): keep a copy of every layer output for mt_debug_copy_hidden (changes
 * mt_workspace_bytes); both must be set before mt_bind_memory.  key "profile" (0/1): see
 * mt_profile_read.  key "cls_only_last_layer" (0/1, default 1, any time): the last
 * layer of every task branch is evaluated for the first token of each sequence only (keys and values
 * still for all tokens) because the pooler reads nothing else; mt_debug_copy_hidden then returns that
 * layer's state at position 0 and zeros elsewhere.  key "early_heads" (0/1, default 0, any time): see mt_forward_events.
 * key "pack_tokens" (0/1, default 1, any time): store
 * and compute only the valid tokens of every sequence (rows of sequence b follow those of b-1) instead
 * of batch*seq padded rows; logits agree to rounding either way.  key "gemm_pair" (0 never, 1 always, 2 = by launch size, the default; any
 * time): run GEMM launches as pairs of CTAs on 256-row tiles (tcgen05 cta_group::2, each CTA stages half
 * of a weight tile) instead of single CTAs on 128-row tiles; faster on large launches (+11 % at 8192^3),
 * slower on small ones; the results are bit-identical.  key "attention_tc" (0/1, default 1, any time): attention
 * for seq <= 128 runs on tcgen05 with its accumulators in tensor memory (1) or on mma.sync (0, also
 * used for every longer seq).  key "expected_tokens" (>= 0, default 0 = every row, any time): the caller's
 * estimate of the valid tokens per batch; with the packed layout the GEMM tile widths are chosen for
 * that many rows instead of batch*seq; it never changes a result.
 * key "fp8_gemm" (0/1, default 0; before mt_bind_memory, it enlarges both arenas): reduced precision in the
 * sense of Appendix E.  The Q/K/V, FFN-up and FFN-down projections run on E4M3 operands (tcgen05 kind::f8f6f4,
 * fp32 accumulation) with one fp32 scale per operand row: weights are quantised once per output channel when
 * they are loaded (8-bit copies behind the bf16 payload in the weights arena), activations per token by a
 * row-wise kernel before each of those projections; see mt_kernel_quantize_rows.  Everything else (attention,
 * the attention-output projection, LayerNorm, the fp32 residual stream, pooler, heads) is unchanged.  Against
 * the unquantised fp64 definition the hidden states then agree to about 4e-2 relative L2 and the logits to
 * about 3e-2 (measured on the 8-task tree; the tests state the bounds); merged == stand-alone still holds bit
 * for bit.
 * key "sm_limit" (>= 0, default 0 = all; any time): size the persistent GEMM grids for at most this many SMs
 * (for callers that share the GPU between several streams and want to leave room; measured no gain).
 * key "fused_ln" (0 never; 1 always, on 128-column tiles; 3 always, on 256-column tiles; 2 = chosen per launch, the
 * default: launches of at most "fused_ln_max_groups" (default 2) layers on all tokens - one layer on 128-column
 * tiles, more on 256-column tiles - and launches of at most "fused_ln_max_rows" (default 0) rows per layer; any
 * time): the attention-output and FFN-down projections carry the LayerNorm that follows them: the CTAs holding the
 * column blocks of the same 128 rows form a thread-block cluster and exchange per-row statistics through
 * distributed shared memory, so the pre-normalisation sum never goes to global memory and no LayerNorm launch
 * follows.  All settings give the same bits (every LayerNorm of the library sums its row statistics over the same
 * 64-column segments in the same order, every projection sums over K in one sequence).  Measured: faster than the
 * separate launches while the launch is a single round of tiles (one or two layers of the 32 x 128 batch), slower
 * beyond, where the separate LayerNorm hides the same latencies behind full occupancy.
 * key "ffn_down_split" (0/1, default 1, any time): launches of at most 512 rows per layer (batch x seq up to
 * 4 x 128, and the first-token rows of the last branch layers for batches up to 512) run the FFN-down projection
 * as partial sums over four ranges of K - four times as many tiles, each a quarter as long - and the LayerNorm
 * kernel after it adds the ranges in order, then the bias and the residual.  Such a launch has so few tiles that
 * the chain of k-blocks one CTA walks is what it costs.  The sum over K is then taken range by range: results
 * differ in the last bits from the unsplit projection, within every tolerance of the tests; the choice depends on
 * the rows of one layer and on options only, never on the tasks asked for or on how many layers share a launch,
 * so a merged model and its tasks run alone still agree bit for bit.  Not with "fp8_gemm".
 * key "overlap_cls" (0/1, default 1, any time): where a wave holds layers on all tokens and last branch
 * layers, the first-token attention of the latter runs on a stream the library creates for itself (in
 * mt_bind_memory), forked from the caller's stream after the wave's Q/K/V projection and joined before the next
 * step, so that it overlaps the wave's other kernels; the caller sees ordinary single-stream semantics,
 * also under stream capture.  Same results.
 * key "pool_gemm" (0/1, default 1, any time): the pooler of tasks whose last branch layer was evaluated on
 * first tokens only runs as one grouped GEMM with a tanh epilogue on the tensor cores (1) or in the
 * row-wise pooler kernel (0, also used for every other task); logits agree to rounding.
 * key "pdl" (0/1, default 1, applies to the whole process): launch every kernel
 * with programmatic stream serialization, so that a kernel's set-up overlaps the previous kernel's
 * tail; results are identical either way. */
int mt_set_option(mt_model* m, const char* key, int64_t value);

/* Per-launch timing.  With option "profile" = 1 (may be toggled at any time) every kernel launch of
 * mt_forward is bracketed by two CUDA events on the caller's stream (events are created on the host
 * on first use).  mt_profile_read waits for the recorded events, adds the elapsed milliseconds and the
 * launch counts per kernel class since the last read into the two arrays (MT_NUM_CLASSES entries
 * each) and forgets them.  Classes follow the steps of the encoder layer. */
#define MT_CLASS_EMBED     0  /* embedding gather + LayerNorm                       */
#define MT_CLASS_QKV       1  /* GEMM: Q,K,V projections                            */
#define MT_CLASS_ATTENTION 2  /* masked softmax attention                           */
#define MT_CLASS_ATTN_OUT  3  /* GEMM: attention output projection + residual       */
#define MT_CLASS_LN1       4  /* LayerNorm after attention                          */
#define MT_CLASS_FFN_UP    5  /* GEMM: FFN up projection + GELU                     */
#define MT_CLASS_FFN_DOWN  6  /* GEMM: FFN down projection + residual               */
#define MT_CLASS_LN2       7  /* LayerNorm after the FFN                            */
#define MT_CLASS_HEAD      8  /* pooler + head                                      */
#define MT_CLASS_QUANT     9  /* row-wise E4M3 quantisation (option "fp8_gemm")        */
#define MT_NUM_CLASSES     10
int mt_profile_read(mt_model* m, double* ms_by_class, int64_t* launches_by_class);

/* Copies the hidden state [batch*seq, hidden] bf16 captured by the LAST mt_forward to d_out (padded
 * layout, rows at positions >= length are zero; the d_lengths of that forward must still be valid).
 * task = -1: trunk state after `layer` layers (0 = embedding output); task >= 0: state after branch
 * layer `layer` (1-based) of that task.  Requires option debug_capture = 1. */
int mt_debug_copy_hidden(mt_model* m, int32_t task, int32_t layer, void* d_out_bf16, void* stream);

const char* mt_last_error_string(const mt_model* m);

/* ---- the individual steps, callable on their own (used by the per-kernel parity tests) -------- */
/* All pointers are device pointers; d_status may be NULL or point to one uint32 status word.      */

/* Y[M,N] = epilogue(X[M,K] . W[N,K]^T + bias[N]) on tcgen05 tensor cores (X, W, bias bf16; fp32
 * accumulate).  epilogue 0: +bias, Y bf16; 1: +bias then GELU x * Phi(x) (fitted evaluation, absolute error <= 2.6e-5, then one rounding), Y bf16; 2: +bias +residual with
 * residual fp32 [M,N] and Y fp32 [M,N] (the LayerNorm input).  K % 64 == 0, N % 128 == 0, all
 * pointers 16-byte aligned.  cta_pair != 0 runs it as pairs of CTAs (see option "gemm_pair").  This is
 * one linear map of the layer above. */
int mt_kernel_linear(const void* d_x, const void* d_w, const void* d_bias, const void* d_residual,
                     void* d_y, int32_t M, int32_t N, int32_t K, int32_t epilogue, int32_t cta_pair,
                     uint32_t* d_status, void* stream);
/* Tuning aid for the kernel micro-benchmark: forces the tile width (64, 128, 192, 256; must divide N) of the
 * following mt_kernel_linear calls of this process; 0 returns to the automatic choice.  Never changes a
 * result: every output element is one fixed-order sum over K whatever the tile. */
void mt_kernel_linear_force_block_n(int32_t block_n);

/* Reduced precision (Appendix E: the production model ran at reduced precision; the paper gives no recipe, the
 * reading here is 8-bit E4M3 operands with one fp32 scale per operand row).  Row-wise quantisation of a bf16
 * matrix X[rows, cols] (cols % 256 == 0): d_scale[r] = max|X[r,:]| / 448 (1 for a row of zeros), d_q[r,c] = the
 * E4M3 value nearest to X[r,c] / d_scale[r] (ties to even, saturating at +-448), decided in fp32.  Used for
 * activations (a scale per token) and, once at load time, for weights [N, K] (a scale per output channel). */
int mt_kernel_quantize_rows(const void* d_x, void* d_q, float* d_scale, int32_t rows, int32_t cols, void* stream);
/* Y[M,N] = epilogue((Xq[M,K] . Wq[N,K]^T) * scale_x[row] * scale_w[column] + bias[N]) on tcgen05 (kind::f8f6f4,
 * fp32 accumulate): Xq, Wq E4M3 bytes as written by mt_kernel_quantize_rows, scales fp32, bias bf16.  Epilogues
 * as mt_kernel_linear (0: bf16; 1: GELU, bf16; 2: + fp32 residual, fp32).  K % 128 == 0; N % 256 == 0 (N % 128 == 0
 * for epilogue 2); pointers 16-byte aligned. */
int mt_kernel_linear_fp8(const void* d_xq, const float* d_scale_x, const void* d_wq, const float* d_scale_w,
                         const void* d_bias, const void* d_residual, void* d_y, int32_t M, int32_t N, int32_t K,
                         int32_t epilogue, uint32_t* d_status, void* stream);

/* What a kernel of the path does when one of its pipeline waits never ends.  Every mbarrier wait of the tensor-core
 * kernels is bounded: after its limit (4 s in the kernels) the waiting role raises its CTA's abort flag, the other
 * roles see the flag at their next look and leave too, and MT_FLAG_WAIT_TIMEOUT is set in the status word.  This
 * call runs that same wait in a two-warp kernel with a limit of the caller's choosing (1 us .. 15 ms): warp 0 waits
 * on a barrier with limit_ns, warp 1 on another with 64 * limit_ns.  arrive == 0: nothing ever completes the
 * barriers - warp 0's wait runs out, warp 1 leaves through the abort flag, d_status (device, may be NULL) gets
 * MT_FLAG_WAIT_TIMEOUT; arrive != 0: both barriers are complete, the waits succeed at once.  d_waited_ns[2] and
 * d_ok[2] (device) receive per warp the nanoseconds waited and 1 / 0 for success.  Nothing faults and the
 * context stays usable. */
int mt_debug_wait_probe(uint64_t limit_ns, int32_t arrive, uint32_t* d_status, uint64_t* d_waited_ns, int32_t* d_ok,
                        void* stream);

/* Partial sums of X[M,K] . W[N,K]^T with K split into k_splits equal ranges (a launch of few rows then has
 * k_splits times as many tiles, each walking a k_splits-th of K): range s writes its fp32 sum, without bias, to rows
 * [s * split_pitch, s * split_pitch + M) of d_part (fp32 [k_splits * split_pitch, N], device).  X, W bf16;
 * (K / 64) % k_splits == 0; split_pitch >= M and a multiple of 128; N % 128 == 0.  This is how the FFN-down
 * projection (Section 3: the second linear map of the feed-forward sub-layer) runs for launches of at most 512
 * rows per layer (option "ffn_down_split"); mt_kernel_layernorm_partial puts the row together. */
int mt_kernel_linear_partial(const void* d_x, const void* d_w, void* d_part, int32_t M, int32_t N, int32_t K,
                             int32_t k_splits, int32_t split_pitch, uint32_t* d_status, void* stream);

/* Y = LN(X[M,K] . W[N,K]^T + bias[N] + residual[M,N]) * gamma[N] + beta[N] in one launch: the residual
 * sub-layer followed by LayerNorm, as the encoder layer has it twice (after attention, after the FFN).
 * X, W, bias, gamma, beta bf16; residual fp32; Y is written twice, d_y bf16 [M,N] and d_y_f32 fp32 [M,N].
 * N = 768 or 1024 (the CTAs of a row block form a cluster of N / 128), K % 64 == 0, all pointers 16-byte
 * aligned.  The result has the bits of mt_kernel_linear(epilogue 2) followed by mt_kernel_layernorm.
 * d_status (device, may be NULL) receives MT_FLAG_WAIT_TIMEOUT. */
int mt_kernel_linear_layernorm(const void* d_x, const void* d_w, const void* d_bias, const void* d_residual,
                               const void* d_gamma, const void* d_beta, void* d_y, void* d_y_f32, int32_t M,
                               int32_t N, int32_t K, float eps, uint32_t* d_status, void* stream);
/* The same with the accumulator tile width chosen by the caller: 128 (clusters of N / 128 CTAs, as above) or 256
 * (clusters of N / 256 CTAs; tcgen05.mma at its full rate, for launches with many row blocks).  Identical bits. */
int mt_kernel_linear_layernorm_tiles(const void* d_x, const void* d_w, const void* d_bias, const void* d_residual,
                                     const void* d_gamma, const void* d_beta, void* d_y, void* d_y_f32, int32_t M,
                                     int32_t N, int32_t K, float eps, int32_t tile_cols, uint32_t* d_status, void* stream);

/* ctx[B*S, heads*64] = softmax(QK^T/8 masked to keys < length) V per (sequence, head), from the
 * packed projection qkv[B*S, 3*heads*64] = [Q | K | V].  Rows at positions >= length are written as 0.
 * tensor_memory != 0 (seq <= 128 only, else MT_ERR_INVALID_ARG) selects the tcgen05 kernel, whose
 * score and output accumulators live in tensor memory; 0 the mma.sync kernel, which takes any seq
 * (see option "attention_tc").  d_status (device, may be NULL) receives MT_FLAG_WAIT_TIMEOUT. */
int mt_kernel_attention(const void* d_qkv, const int32_t* d_lengths, void* d_ctx,
                        int32_t batch, int32_t seq, int32_t heads, int32_t tensor_memory,
                        uint32_t* d_status, void* stream);

/* y[rows, hidden] = LayerNorm(x) * gamma + beta (fp32 statistics, biased variance) for fp32 x;
 * written as bf16 to d_y and, when d_y_f32 is not NULL, as fp32 too.  hidden in {768, 1024}. */
int mt_kernel_layernorm(const void* d_x, const void* d_gamma, const void* d_beta, void* d_y, void* d_y_f32,
                        int32_t rows, int32_t hidden, float eps, void* stream);

/* The same LayerNorm on x = residual + ((part_0 + part_1 + ... + part_{n_parts-1}) + bias), the ranges added in
 * this order: the residual sub-layer after a projection whose K was split (mt_kernel_linear_partial).  d_part fp32
 * [n_parts * part_pitch, hidden] (range s at row s * part_pitch; n_parts <= 4), d_residual fp32 [rows, hidden], bias bf16. */
int mt_kernel_layernorm_partial(const float* d_part, int32_t n_parts, int32_t part_pitch, const float* d_residual,
                                const void* d_bias, const void* d_gamma, const void* d_beta, void* d_y, void* d_y_f32,
                                int32_t rows, int32_t hidden, float eps, void* stream);

/* h0[B*S, hidden] = LayerNorm(word[tok] + pos[position] + type[seg]), bf16 (and fp32 if d_h0_f32 != NULL). */
int mt_kernel_embed(const int32_t* d_token_ids, const int32_t* d_segment_ids, const int32_t* d_lengths,
                    const void* d_word, const void* d_pos, const void* d_type,
                    const void* d_gamma, const void* d_beta, void* d_h0, void* d_h0_f32,
                    int32_t batch, int32_t seq, int32_t hidden, int32_t vocab, int32_t type_vocab,
                    float eps, uint32_t* d_status, void* stream);

/* logits[b, col0 + c] = cls_w[c,:] . tanh(pool_w . h[b*seq, :] + pool_b) + cls_b[c], c < num_classes.
 * Two launches (pooler, head); d_pooled_scratch is caller-provided scratch of batch*hidden floats that
 * carries the tanh features between them (contents afterwards: those features). */
int mt_kernel_pooler_head(const void* d_hidden, const void* d_pool_w, const void* d_pool_b,
                          const void* d_cls_w, const void* d_cls_b, float* d_pooled_scratch, float* d_logits,
                          int32_t batch, int32_t seq, int32_t hidden, int32_t num_classes,
                          int32_t logits_stride, int32_t col0, void* stream);

/* The same pooler + head for callers that cannot allocate device memory (no counterpart in the
 * paper: it is a convenience of this library).  Meant for code that lives inside a process whose
 * device memory is owned by someone else - an inference server that handed all of it out at start-up,
 * a plug-in that only ever sees input and output pointers - or that must not call cudaMalloc because
 * it stalls the device.  The tanh pooler features, which mt_kernel_pooler_head passes through
 * d_pooled_scratch, go through an array built into the library instead: MT_STATIC_POOLER_MAX_FLOATS
 * floats (1 MiB) that every GPU loading the library keeps until the process ends.
 *  - batch * hidden must not exceed MT_STATIC_POOLER_MAX_FLOATS, else MT_ERR_SHAPE (nothing is launched).
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *    that device current); make that first call before starting any stream capture.
 *  - It calls no cudaMalloc/cudaFree and no allocating library routine.
 *  - All calls on a device share the one array, which keeps the previous call's features (the pooler
 *    launch overwrites every entry the head launch reads, so nothing needs clearing).  Two calls whose
 *    kernels can overlap on the GPU - different streams, no ordering between them - race on it:
 *    order them, or use mt_kernel_pooler_head with separate scratch buffers.
 * All other arguments, results and errors are those of mt_kernel_pooler_head. */
#define MT_STATIC_POOLER_MAX_FLOATS (256 * 1024)
int mt_kernel_pooler_head_static(const void* d_hidden, const void* d_pool_w, const void* d_pool_b,
                                 const void* d_cls_w, const void* d_cls_b, float* d_logits,
                                 int32_t batch, int32_t seq, int32_t hidden, int32_t num_classes,
                                 int32_t logits_stride, int32_t col0, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MT_BERT_H_ */
