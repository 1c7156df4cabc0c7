/*
 * dkv.h -- C ABI of the dKV-Cache denoising step for masked diffusion
 * language models on NVIDIA B200 (sm_100a).
 *
 * The library runs, for a bidirectional pre-norm decoder (RMSNorm, rotate-half
 * RoPE, SwiGLU, MHA or GQA, untied vocabulary head), ONE denoising step in
 * which only the ACTIVE rows are recomputed and every other row's key/value
 * states are served from a persistent per-layer cache ("dKV-Cache: The Cache
 * for Diffusion Language Models", Sec. 3.3 Eq. 4, Sec. 3.4, Algorithm 1), and
 * ends the step with confidence-based unmasking (Sec. 3.1).
 *
 * Conventions
 *  - Every function returns an int status: DKV_OK (0) or a negative DKV_E_*.
 *    Nothing throws, aborts or prints.
 *  - Unless a parameter is marked HOST, tensor pointers are DEVICE pointers
 *    owned by the caller (the caller allocates; the library never calls
 *    cudaMalloc).  The library owns only the small host-side handles.
 *  - `stream` is a cudaStream_t passed as void*.  Calls enqueue work on it and
 *    return without synchronising, except where stated.
 *  - Matrices are row-major.  Weight matrices are [out_features, in_features].
 *  - dtype DKV_F32: weights, activations and the cache are float; all kernels
 *    are plain FMA kernels (the check mode).  dtype DKV_BF16: weights are
 *    bfloat16, GEMMs run on tcgen05 tensor cores with fp32 accumulation in
 *    tensor memory, the residual stream and every norm / softmax statistic
 *    stay in fp32, and the GEMM row operands (normalised activations,
 *    attention output, SwiGLU product), the queries and the K/V cache are
 *    16-bit: act_dtype DKV_F16 (11-bit significand: the mode whose logits
 *    stay within 2e-2 sigma of an exact evaluation) or DKV_BF16 (fp32's
 *    exponent range, 8-bit significand).
 *  - Positions are 0-based; step numbers t are 1-based as in the paper.
 *  - A handle is used from one host thread at a time.  A handle argument that
 *    is not a live handle (never created, already destroyed, or a cache whose
 *    model was destroyed) yields DKV_E_STATE; nothing is read through it.
 *  - The kernels of this library size themselves to the whole GPU, and in some
 *    launches the thread blocks of one launch wait for each other (bounded
 *    waits).  Launches of the library on ONE device must therefore not overlap:
 *    drive a device from one stream at a time.
 *  - Device-side problems (a row bound that was exceeded, fewer candidates
 *    than k, a wait inside a kernel that ran out) set a sticky status word
 *    that dkv_status() reads; kernels never trap.
 */
#ifndef DKV_H_
#define DKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DKV_OK 0
#define DKV_E_INVALID_ARG (-1)
#define DKV_E_SHAPE (-2)
#define DKV_E_STATE (-3)
#define DKV_E_NOMEM (-4)
#define DKV_E_CUDA (-5)
#define DKV_E_UNSUPPORTED (-6)
#define DKV_E_DEVICE (-7) /* a kernel reported a problem through the status word */

#define DKV_F32 0
#define DKV_BF16 1
#define DKV_F16 2

/* Cache policies (Sec. 3.3 and 3.4). */
#define DKV_POLICY_NONE 0    /* no cache: every row recomputed every step          */
#define DKV_POLICY_DECODE 1  /* Eq. 4: active rows = masked set of the previous step */
#define DKV_POLICY_PREFILL 2 /* prompt K/V computed at step 1 and kept; every
                                generation row recomputed every step               */
#define DKV_POLICY_PD 3      /* prompt as PREFILL; decoded rows as DECODE, refresh
                                recomputes the generation rows only                */
#define DKV_POLICY_GREEDY 4  /* Sec. 3.4: active rows = D_t, D_{t-1} and a window    */

#define DKV_CENTER_PREV 0 /* window centred on D_{t-1} (the paper's better choice) */
#define DKV_CENTER_CUR 1  /* window centred on D_t                                 */

/* Remasking scores of Sec. 3.1: the largest softmax probability; the margin
 * between the two most probable values; minus the entropy (sum p log p). */
#define DKV_SCORE_MAXPROB 0
#define DKV_SCORE_MARGIN 1
#define DKV_SCORE_NEG_ENTROPY 2

#define DKV_REFRESH_ALL 0          /* next step recomputes every row               */
#define DKV_REFRESH_DECODED_ONLY 1 /* next step recomputes the generation rows     */

typedef struct dkv_model dkv_model;
typedef struct dkv_cache dkv_cache;

typedef struct dkv_model_desc {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab, mask_id;
  float rope_theta; /* RoPE base, e.g. 10000 */
  float rms_eps;    /* RMSNorm epsilon, e.g. 1e-5 */
  int32_t dtype;    /* weights: DKV_F32 or DKV_BF16 */
  int32_t act_dtype; /* activations and K/V cache: DKV_F32 with F32 weights; DKV_F16 or DKV_BF16 with BF16 weights */
} dkv_model_desc;

/* Weights of one layer (device pointers; matrices in the model dtype, norm
 * gains always float).  wqkv stacks the rows of W_q, W_k, W_v; wgu stacks the
 * rows of W_gate and W_up. */
typedef struct dkv_layer_weights {
  const void* wqkv;        /* [d_q + 2 d_kv, d_model] */
  const void* wo;          /* [d_model, d_q]          */
  const void* wgu;         /* [2 d_ffn, d_model]      */
  const void* wd;          /* [d_model, d_ffn]        */
  const float* attn_norm;  /* [d_model] */
  const float* ffn_norm;   /* [d_model] */
} dkv_layer_weights;

typedef struct dkv_weights {
  const void* embed;                /* [vocab, d_model] */
  const void* head;                 /* [vocab, d_model] */
  const float* final_norm;          /* [d_model] */
  const dkv_layer_weights* layers;  /* HOST array of n_layers entries */
} dkv_weights;

typedef struct dkv_policy {
  int32_t kind;             /* DKV_POLICY_* */
  int32_t refresh_interval; /* N >= 1: 0-based step s is a full step when s mod N == 0; 0 = never after step 1 */
  int32_t delay;            /* 1 = one-step delayed caching (Eq. 4); 0 = cache at the unmask step (Eq. 3) */
  int32_t window;           /* w of the Greedy local window [c - ceil(w/2), c + floor(w/2)] */
  int32_t window_center;    /* DKV_CENTER_* */
  int32_t max_head_rows;    /* most rows per sequence that need logits in one step; 0 = generation length */
  int32_t max_k;            /* most positions unmasked per sequence per step; 0 = 1 */
  int32_t shift;            /* 1: shifted outputs (models adapted from autoregressive ones, Appendix B,
                               "Un-Shift"): the logits of position j are read at row j-1, which is
                               computed in addition to the policy's rows; K/V are cached unshifted.
                               2: the same, and a row is served from the cache only when the policy
                               would cache both its own position and the one to its right, i.e. its
                               input is fixed and the token it predicts is decoded (Appendix B,
                               "Un&Right-Shift"). Needs cand_lo >= 1 */
  int32_t score;            /* DKV_SCORE_*: what `conf` holds and the top-k selection ranks */
  int32_t isolated_prefill; /* Prefill / PD only (Sec. 3.3, prefill tokens mostly attend to each other;
                               prefill / decode disaggregation): 1 = at step 1 the prompt rows are computed
                               in a pass of their own in which they attend to the prompt slots only; the
                               generation rows follow in the same step over all slots. 0 = step 1 is the
                               joint full step. DKV_E_UNSUPPORTED with the other policies */
} dkv_policy;

typedef struct dkv_stats {
  int64_t steps;            /* dkv_step calls since dkv_init_cache */
  int64_t refresh_steps;    /* of which full (or generation-only) recomputes */
  int64_t active_rows;      /* sum over steps of the number of active rows, all sequences (counted on the device) */
  int64_t total_rows;       /* steps * batch * seq_len */
  double cache_ratio;       /* 1 - active_rows / total_rows (the paper's cache-ratio metric, Sec. 4.1) */
  int64_t cache_bytes;      /* bytes of K/V slots */
  int64_t kernel_launches;  /* kernels launched by this handle */
} dkv_stats;

const char* dkv_strerror(int status);

/* The problem statement's model (Algorithm 1's transformer T).  Records the
 * descriptor and the weight pointers and, with bf16 weights, builds the TMA
 * descriptors of the weight matrices.  With act_dtype DKV_F16 the projection
 * and head matrices are first copied to fp16 into `arena` (caller-owned
 * device memory, 256-byte aligned, at least dkv_model_bytes(desc) bytes, kept
 * alive until dkv_model_destroy): tcgen05 MMAs need both operands in one
 * 16-bit format.  (The copies of the layers' matrices and of the head are laid out in blocks
 * of 128 rows x 64 columns, zero-padded; the size includes the padding.)  The copy is exact for |w| >= 2^-14 and within 2^-25
 * absolute below; afterwards only embed and the norm gains of the caller's
 * weights are still read.  In the other modes arena may be NULL and the
 * caller keeps all weights alive and unchanged until dkv_model_destroy.
 * Errors: INVALID_ARG (NULL), SHAPE (head_dim not in {64,128}; d_model,
 * d_ffn not multiples of 8), UNSUPPORTED (dtype), NOMEM (arena), CUDA. */
size_t dkv_model_bytes(const dkv_model_desc* desc);
int dkv_model_create(const dkv_model_desc* desc, const dkv_weights* weights, void* arena, size_t arena_bytes,
                     void* stream, dkv_model** out);
int dkv_model_destroy(dkv_model* model);

/* Bytes of device memory dkv_init_cache needs for `batch` sequences of
 * `seq_len` positions: the K/V slots [layer][batch][kv_head][pos][head_dim]
 * (the cached Key and Value of Algorithm 1's Require line), the index maps,
 * and the per-step workspace.  0 on invalid arguments. */
size_t dkv_cache_bytes(const dkv_model* model, int batch, int seq_len, const dkv_policy* policy);

/* Start a generation: all slots invalid, step counter 0, so the first
 * dkv_step is a full step (Sec. 3.3, refresh: "revert back to the normal
 * calculation").  `arena` is caller-owned device memory of at least
 * dkv_cache_bytes(), 256-byte aligned, kept alive until dkv_cache_destroy.
 * May be called again on a fresh handle with the same arena to restart.
 * Errors: INVALID_ARG, SHAPE (prompt_len > seq_len, batch < 1), NOMEM
 * (arena too small), CUDA. */
int dkv_init_cache(const dkv_model* model, int batch, int seq_len, int prompt_len, const dkv_policy* policy,
                   void* arena, size_t arena_bytes, void* stream, dkv_cache** out);
int dkv_cache_destroy(dkv_cache* cache);

/* One denoising step (Algorithm 1 with Eq. 4; Sec. 3.4 for GREEDY):
 *   1. active rows A_t from the policy, the previous step's mask, `masked`
 *      and the step number; ascending compaction;
 *   2. embedding gather, then per layer: RMSNorm, QKV projection, RoPE at the
 *      original positions, fresh K/V written into the rows' own cache slots,
 *      bidirectional attention of the active queries over all seq_len slots,
 *      output projection, SwiGLU FFN;
 *   3. for the head rows (masked positions inside [cand_lo, cand_hi); for
 *      GREEDY the positions `next_pos`): final norm, vocabulary head, and per
 *      row the most probable token (mask_id excluded, lowest id on ties) and
 *      its softmax probability, written at the ORIGINAL positions.
 * tokens  [batch, seq_len] int32  x_t; masked positions must hold mask_id (its
 *                                 embedding row is what the model reads there)
 * masked  [batch, seq_len] uint8  M_t, 1 = masked
 * next_pos[batch, k] int32        D_t, required for GREEDY, else NULL
 * rows_bound                      promise: no sequence has more than this many
 *                                 masked positions in `masked`; -1 = unknown
 *                                 (the library then sizes for seq_len)
 * conf    [batch, seq_len] float  out: the policy's score (default: max softmax
 *                                 probability), -inf where the position is
 *                                 not a head row
 * pred    [batch, seq_len] int32  out: argmax token, -1 where not a head row
 * logits_dbg [head rows, vocab] float, or NULL.  When given it receives the
 *                                 logits of the head rows in head-row order
 *                                 (sequence-major, ascending position), row
 *                                 stride = vocab; it must hold batch *
 *                                 max_head_rows rows
 * Updates the cache slots of A_t, the provenance stamps, the stored previous
 * mask and the step / refresh counters.  Errors: INVALID_ARG, STATE (not a
 * live handle), SHAPE (k > max_k, cand range outside the sequence; GREEDY: k
 * differs from the previous step's, whose D_{t-1} the window rule reads). */
int dkv_step(dkv_cache* cache, const int32_t* tokens, const uint8_t* masked, const int32_t* next_pos, int k,
             int cand_lo, int cand_hi, int rows_bound, float* conf, int32_t* pred, float* logits_dbg,
             void* stream);

/* Mark the cache stale (Sec. 3.3, cache refreshing): the next dkv_step
 * recomputes every row (DKV_REFRESH_ALL) or every generation row
 * (DKV_REFRESH_DECODED_ONLY) and the interval counter restarts there. */
int dkv_refresh(dkv_cache* cache, int scope);

/* Confidence-based unmasking (Sec. 3.1, "keeping the most confident ones"):
 * per sequence, the k positions with the largest conf among the masked
 * positions inside [cand_lo, cand_hi); ties go to the lower position; NaN
 * counts as -inf.  For each chosen position p (in order of decreasing conf):
 * tokens[p] = pred[p], masked[p] = 0, chosen_pos[b][j] = p.  If a sequence has
 * fewer than k candidates the missing entries are -1 and, when `status` is
 * not NULL, bit 1 of *status (device int32) is set.  All pointers device. */
int dkv_select_unmask(const float* conf, const int32_t* pred, int batch, int seq_len, int cand_lo, int cand_hi,
                      int k, int32_t* tokens, uint8_t* masked, int32_t* chosen_pos, int32_t* status,
                      void* stream);

/* The same step driven from HOST buffers (pinned or pageable): copies
 * tokens / masked (and next_pos) to the device, runs dkv_step and, unless
 * policy GREEDY supplies the positions, dkv_select_unmask, copies the updated
 * tokens, masked and chosen positions back, and synchronises the stream.
 * tokens_host / masked_host are updated in place; chosen_host [batch,k]. */
int dkv_step_host(dkv_cache* cache, int32_t* tokens_host, uint8_t* masked_host, const int32_t* next_pos_host,
                  int k, int cand_lo, int cand_hi, int rows_bound, int32_t* chosen_host, void* stream);

/* The sampling loop of Sec. 3.1 (predict every masked position, keep the most
 * confident, leave the rest masked) with the semi-autoregressive blocks of the
 * paper's generation settings (appendix table of L, T and block size), as a
 * whole generation on the device with no host synchronisation: T = gen_len/k
 * steps of dkv_step + dkv_select_unmask over `tokens` / `masked` (device,
 * updated in place), semi-autoregressive blocks of block_len positions
 * (block_len = 0: one block).  order_dev [T, batch, k] int32 is required for
 * GREEDY (the predefined decoding order), otherwise NULL.  chosen_dev
 * [T, batch, k] int32 (or NULL) receives every step's D_t.  n_steps <= T
 * limits the number of steps run (0 = all). */
int dkv_generate(dkv_cache* cache, int32_t* tokens, uint8_t* masked, const int32_t* order_dev, int k,
                 int block_len, int n_steps, int32_t* chosen_dev, void* stream);

/* Bookkeeping.  dkv_get_stats synchronises the stream of the last step. */
int dkv_get_stats(const dkv_cache* cache, dkv_stats* out);
/* Step number at which each slot was last written (0 = never): device
 * int32 [batch, seq_len].  Appendix A: the tokens that newly enter the cache at
 * step t are those decoded at step t-1, so under Eq. 4 a decoded position shows
 * its unmask step + 1 until the next refresh (with delay = 0, Eq. 3: its
 * unmask step); prompt positions under PREFILL / PD show 1. */
int dkv_get_provenance(const dkv_cache* cache, int32_t* written_step, void* stream);
/* The token-level index maps of the last step (Appendix A: the reordering is
 * done once per model evaluation on [B, L] indices and shared by all layers;
 * Algorithm 1's x' = x[M_{t-1}] and the scatter of the outputs back to their
 * original positions): act_idx [batch*seq_len] (flattened
 * b*seq_len+pos, ascending; entries past the count are undefined), row_off
 * [batch+1] and inv [batch, seq_len] (compact row of a position, -1 if
 * inactive).  Any pointer may be NULL. */
int dkv_get_index_maps(const dkv_cache* cache, int32_t* act_idx, int32_t* row_off, int32_t* inv, void* stream);
/* Synchronises the stream of the last call and returns DKV_OK, or
 * DKV_E_DEVICE if a kernel set the status word (the word is in *word). */
int dkv_status(dkv_cache* cache, int32_t* word);
/* Direct read access to a layer's slots (Algorithm 1's cached Key and Value
 * states, after RoPE): device pointers to K and V of layer `layer`, layout
 * [batch][kv_head][pos][head_dim] in the activation type. */
int dkv_cache_slots(const dkv_cache* cache, int layer, void** k_slots, void** v_slots);

/* Checkpoint / resume of a generation.  What Algorithm 1 carries from one
 * step to the next is the cached Key and Value states and the previous step's
 * sets (M_{t-1} for Eq. 4, D_{t-1} for the window rule of Sec. 3.4); together
 * with the step / refresh counters, the provenance stamps and the statistics
 * that is the whole state of a handle between two dkv_step calls.
 * dkv_cache_export copies it into `state_host` (HOST memory, at least
 * dkv_cache_state_bytes() bytes: a fixed header, then the K/V slots of every
 * layer and the stored sets); dkv_cache_import loads such a blob into a live
 * handle of the SAME model geometry, batch, seq_len, prompt_len, max_k and
 * policy (on any device, with its own arena), after which dkv_step continues
 * exactly where the exporting handle stood: same active rows, refresh
 * schedule and results.  The caller's tokens / masked arrays are not part of
 * the state.  Both calls synchronise `stream` (and the stream of the handle's
 * last step) before they return.  The blob is valid for this library version
 * only.  Errors: INVALID_ARG (NULL, not an exported state, counters out of
 * range), NOMEM (export: state_bytes too small), SHAPE (import: geometry or
 * policy differ, truncated blob), STATE, CUDA. */
size_t dkv_cache_state_bytes(const dkv_cache* cache);
int dkv_cache_export(dkv_cache* cache, void* state_host, size_t state_bytes, void* stream);
int dkv_cache_import(dkv_cache* cache, const void* state_host, size_t state_bytes, void* stream);

/* Per-kernel-class timing: when enabled, every launch is bracketed by CUDA
 * events on the launching stream (this slows a step slightly; not for timed
 * throughput runs).  dkv_profile_read synchronises and returns, per class, the
 * launch count, total milliseconds, and the algorithmic bytes and flops the
 * library counted for those launches; n = number of classes written. */
#define DKV_PROF_CLASSES 16
typedef struct dkv_profile_entry {
  char name[32];
  int64_t launches;
  double ms;
  double bytes;
  double flops;
} dkv_profile_entry;
int dkv_profile_enable(dkv_cache* cache, int on);
int dkv_profile_read(dkv_cache* cache, dkv_profile_entry* out, int* n);

/* Timeline trace (diagnostics).  records: device buffer of `capacity` entries of
 * 24 bytes {uint64 t_enter_ns, uint64 t_ready_ns, int32 kernel_id, int32 pad};
 * while set, block 0 of every kernel appends one entry: when it started and
 * when its stream predecessor's results were visible to it.  kernel ids: 1
 * compact, 2 embed_norm, 3 tensor-core GEMM, 4 qkv_rope_scatter, 5 attention,
 * 7 resid_norm, 9 swiglu, 11 head_gather, 12 head_stats, 13 select_unmask.
 * records = NULL switches the trace off.  Synchronises the device. */
int dkv_trace_set(void* records, int capacity);

/* Test hook for the error path of the bounded waits (failure detection
 * without a GPU fault): in a fused projection launch the thread blocks of a
 * weight tile wait for each other, at most `wait_cycles` SM clocks (default:
 * about two seconds).  With never_complete != 0 they expect one arrival more
 * than will ever come, so that every such wait runs out after wait_cycles:
 * the kernels skip the row work that depended on it, finish normally and set
 * bit 3 (value 8) of the status word; the step's results are then meaningless
 * and the arrival counters are left non-zero, so the handle must be destroyed
 * and a new one initialised (dkv_init_cache clears them) before the arena is
 * used again.  Nothing traps and no kernel is left waiting.  Errors:
 * INVALID_ARG (wait_cycles outside [1000, default]), STATE. */
int dkv_debug_tail_wait(dkv_cache* cache, long long wait_cycles, int never_complete);

/* ---- kernel-level entry points (single-layer sweeps and unit parity) ---- */

/* out[r, n] = sum_k x[r, k] * w[n, k] for r < rows: the projection GEMM used
 * by every linear layer of Algorithm 1's transformer.  dtype DKV_F32: x and w
 * float.  DKV_BF16 / DKV_F16: x and w of that 16-bit type.  x [rows, K],
 * w [N, K]; out float [rows, N].  `workspace` holds split-K partials:
 * dkv_gemm_workspace_bytes(rows, N) bytes.  splits = 0 lets the library choose.
 * With a 16-bit dtype `out` may be NULL: the partials then stay in the
 * workspace, [splits][rows][N] (for timing the GEMM kernel alone). */
size_t dkv_gemm_workspace_bytes(int rows, int n);
int dkv_op_gemm(const void* x, const void* w, float* out, int rows, int n, int k, int dtype, int splits,
                void* workspace, size_t workspace_bytes, void* stream);

/* Eq. 4's attention: o[r, h, :] = softmax(q[r, h, :] K[b, h/g]^T / sqrt(d_h)) V[b, h/g]
 * over all seq_len slots, no mask.  q, o [rows, n_q_heads, head_dim];
 * k_slots, v_slots [batch][n_kv_heads][seq_len][head_dim]; row_off [batch+1]
 * (device) gives each sequence's rows; rows_per_seq_bound bounds the rows of any one
 * sequence and sizes the grid; q and o must hold batch * rows_per_seq_bound rows
 * (rows that belong to no sequence are neither read for results nor written). */
int dkv_op_attention(const void* q, const void* k_slots, const void* v_slots, void* o, const int32_t* row_off,
                     int batch, int rows_per_seq_bound, int seq_len, int n_q_heads, int n_kv_heads, int head_dim,
                     int dtype, void* stream);

/* The same projection GEMM as dkv_op_gemm for callers that cannot allocate
 * device memory.  (The paper has no counterpart: this entry point exists for
 * integration only.)  Some hosts of this library may not call cudaMalloc or
 * any allocator at the point where they need a projection: a callback on a
 * latency-critical serving thread whose memory pool is fixed at start-up, a
 * plug-in inside a process whose device memory is fully handed to another
 * framework, code that runs after the process has been told to stop
 * allocating.  For them the split-K partial sums, which dkv_op_gemm keeps in a
 * caller-provided workspace, live in an array compiled into the library image:
 * DKV_STATIC_SCRATCH_BYTES (16 MiB) of device memory on every GPU that loads
 * the library, held until the process exits.
 *   x [rows, K], w [N, K] of the 16-bit `dtype` (DKV_F16 or DKV_BF16), out
 *   float [rows, N], all caller-owned device memory; splits = 0 lets the
 *   library choose.
 * Limits: rows * N * 4 bytes (one fp32 slab) must fit in the array, and so
 * must `splits` slabs when splits is given; otherwise DKV_E_NOMEM and nothing
 * is launched.  With splits = 0 the library picks a count that fits.
 * The first call on each device looks up the array's device address (no
 * allocation) and keeps it in a per-device table indexed by the device
 * ordinal of the current (primary) context; make that first call before any
 * stream capture, and not from two host threads at once (the table is filled
 * without a lock).  The function calls no allocator.
 * Every call on a device uses the SAME array and leaves its partial sums
 * there.  Nothing has to be cleared between calls: each call writes every
 * element it later reads.  Two calls whose kernels can overlap on the GPU
 * (different streams) race on the array and give wrong results: serialise them.
 * Errors: INVALID_ARG (NULL), UNSUPPORTED (dtype), SHAPE, NOMEM, CUDA. */
#define DKV_STATIC_SCRATCH_BYTES (16u << 20)
size_t dkv_static_scratch_bytes(void);
int dkv_op_gemm_static(const void* x, const void* w, float* out, int rows, int n, int k, int dtype, int splits,
                       void* stream);

/* Measurement aid (no counterpart in the paper): the memory side of a
 * weight-streaming projection launch without its arithmetic.  `ctas` thread
 * blocks (one per SM) each stream their own slice of `streamed` (unique
 * bytes, meant to come from HBM: make the buffer larger than L2) and, per
 * chunk, reread_chunk_bytes of the small buffer `reread` that every block
 * re-reads (L2 hits, like the activation rows of a projection; 0 = none),
 * through a ring of `stages` shared-memory stages filled by bulk copies; a
 * stage is freed the moment it is full.  Every block moves
 * floor(streamed_bytes / ctas / chunk_bytes) chunks.  The launch's duration
 * (time it with events on `stream`) is the ceiling of that access pattern.
 * Both buffers 16-byte aligned device memory, the chunk sizes multiples of 16,
 * stages * (chunk_bytes + reread_chunk_bytes) at most about 226 KB.  `status`
 * (device int32, may be NULL): bit 3 is set if a bounded wait ran out.
 * Errors: INVALID_ARG, SHAPE, NOMEM (shared memory), CUDA. */
int dkv_op_stream_probe(const void* streamed, long long streamed_bytes, const void* reread, long long reread_bytes,
                        int ctas, int chunk_bytes, int reread_chunk_bytes, int stages, int32_t* status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DKV_H_ */
