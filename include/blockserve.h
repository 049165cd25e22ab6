/*
 * blockserve.h - C ABI of the B200 (sm_100a) mixed-state block-denoising engine.
 *
 * The calls follow the paper's problem formulation (Section 2.1: requests r_i
 * with prompt length p_i, generation length g_i, K_i = ceil(g_i / L) blocks of
 * length L, block index b_i) and its scheduling loop (Algorithm 1).  A user
 * drives it the way Algorithm 1 reads:
 *
 *     bs_admit() x N
 *     loop { bs_evict_refill(&ev, &ad, &n_active); if (n_active == 0) break;
 *            do { bs_denoise_step(); bs_block_done(&done, 0); } while (!done); }
 *     bs_read_tokens()
 *
 * Conventions
 *   - Every call returns BS_OK (0) or a negative bs_status; nothing throws.
 *   - "device" pointers are CUDA device memory owned by the caller (the Python
 *     binding takes them from torch tensors); the library borrows them until
 *     bs_destroy and never allocates device memory itself.  "host" pointers are
 *     ordinary host memory; host inputs are consumed before the call returns.
 *   - All kernels are enqueued on the stream given to bs_init_model.
 *     bs_evict_refill, bs_block_done, bs_read_tokens and bs_debug_read
 *     synchronise that stream; bs_denoise_step does so only when it has to
 *     report n_committed.
 *   - One engine is used from one host thread at a time.
 *   - Every step of the path runs in CUDA kernels; there is no CPU fallback.
 */
#ifndef BLOCKSERVE_H_
#define BLOCKSERVE_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct bs_engine bs_engine; /* opaque */

typedef enum {
  BS_OK = 0,
  BS_E_ARG = -1,         /* bad argument or unsupported shape */
  BS_E_STATE = -2,       /* call out of order (e.g. step with no unfinished block) */
  BS_E_BUDGET = -3,      /* request alone is wider than the token budget (it could never be admitted) */
  BS_E_KV_FULL = -4,     /* request longer than the KV arena, or request table full */
  BS_E_CUDA = -5,        /* a CUDA runtime call failed; see bs_last_error */
  BS_E_TIMEOUT = -6,     /* a bounded device-side wait ran out; the step's results are invalid */
  BS_E_UNKNOWN_REQ = -7  /* request id not known to the engine */
} bs_status;

enum { BS_SUFFIX_FULL = 0, BS_SUFFIX_NONE = 1 };
enum { BS_REQ_QUEUED = 0, BS_REQ_ACTIVE = 1, BS_REQ_FINISHED = 2 };
enum { BS_REFRESH_EVERY_BLOCK = 0, BS_REFRESH_AT_ADMISSION = 1 };

typedef struct {
  /* model: pre-norm bidirectional transformer, RMSNorm, rotate-half RoPE, GQA, SwiGLU, no biases */
  int n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab, mask_id;
  float rms_eps, rope_theta;
  /* method (Section 2.1, 2.4): block length L (<= 64), confidence threshold tau,
     token budget beta of Eq. 1 (<= 0: unlimited), fixed batch cap */
  int block_len;
  float tau;
  long long token_budget;
  int max_batch;                 /* <= 1024 */
  int max_requests;              /* size of the request table: a lifetime cap - every bs_admit takes a slot for good
                                    (finished requests stay readable until bs_destroy), slots are not recycled */
  int max_row_tokens;            /* max p_i + g_i */
  long long kv_capacity_tokens;  /* rows of the KV arena = max packed tokens of one step */
  int suffix_mode;               /* BS_SUFFIX_FULL: a row sees prompt + all g_i positions (future blocks as mask
                                    tokens); BS_SUFFIX_NONE: a row ends with its current block (row width of Eq. 1) */
  int sort_queue;                /* 1: pending queue ascending in p_i, ties by submission (Section 2.4); 0: arrival order */
  int steps_per_block;           /* S of Section 2.5: the block's L masked tokens are spread uniformly over S steps
                                    (step s of a block commits the positions above tau united with its
                                    floor(L/S) + [s < L mod S] most confident ones); 0 or L: one per step */
  int eos_id;                    /* CheckEOS of Algorithm 1: at a block boundary a request whose finished blocks hold
                                    this token id leaves the active set (its later positions stay masked, its state
                                    becomes BS_REQ_FINISHED); < 0: off, every request generates exactly g_i tokens */
  int static_groups;             /* 1: the comparison policy of Section 3.1 (fixed groups: nothing is admitted until
                                    every request of the current group has finished); 0: block-boundary refill */
  int async_advance;             /* 1: per-row block advance - the straggler stall of Section 2.3 (a row whose block is
                                    done idles until the slowest row of the cycle is) relaxed: every bs_denoise_step
                                    ends with the block boundary of Algorithm 1 applied to the rows whose block is
                                    complete (advance or evict, stable compaction, refill under Eq. 1), so a row starts
                                    its next block in the following step.  bs_block_done then reports all_done only
                                    when the active set is empty; bs_evict_refill is the first fill and any later fill
                                    of an empty active set.  0: batch-synchronous block cycles (Algorithm 1) */
  int refresh_policy;            /* when a row's prefix / suffix cache is rebuilt by a whole-row forward (Section 2.5
                                    leaves it open: "frozen prefix cache" vs a block-wise approximate cache).
                                    BS_REFRESH_EVERY_BLOCK (default): at the first step of every block.
                                    BS_REFRESH_AT_ADMISSION: only at the first step after admission; later blocks
                                    start with a cached block step and the cache keeps what earlier steps wrote
                                    (throughput ablation; snapshots are then refused while rows are active) */
  int keep_logits;               /* parity hook: 1 = the LM head also stores the fp32 logits [M_m, vocab] of every step
                                    (4 * max_batch * L * vocab more workspace bytes) so that bs_debug_read can return
                                    them; 0 = the logits never reach device memory, only the confidence partials of
                                    the LM-head epilogue do (a twelfth of their bytes) */
} bs_config;

/* All weights are bf16, row-major [out_features, in_features], device memory.
 * wqkv rows: all q heads, then k heads, then v heads.  The per-layer members
 * are HOST arrays of n_layers DEVICE pointers. */
typedef struct {
  const void* embed;       /* [vocab, d_model] */
  const void* lm_head;     /* [vocab, d_model] */
  const void* final_norm;  /* [d_model] */
  const void* const* wqkv;    /* [(Hq + 2 Hkv) * head_dim, d_model] */
  const void* const* wo;      /* [d_model, Hq * head_dim] */
  const void* const* w_gate;  /* [d_ffn, d_model] */
  const void* const* w_up;    /* [d_ffn, d_model] */
  const void* const* w_down;  /* [d_model, d_ffn] */
  const void* const* norm1;   /* [d_model] */
  const void* const* norm2;   /* [d_model] */
} bs_weights;

typedef struct {
  size_t kv_bytes, workspace_bytes, state_bytes;
} bs_sizes;

typedef struct {
  long long steps;            /* denoise steps run */
  long long cycles;           /* block-cycles started (bs_evict_refill calls that left rows active) */
  long long sum_active;       /* sum over cycles of |A| (numerator of the effective compute ratio, Eq. 2) */
  long long committed;        /* tokens committed by the engine (prompt and pre-committed blocks excluded) */
  long long packed_tokens;    /* sum over steps of the packed query tokens M */
  long long lm_rows;          /* sum over steps of the masked rows M_m */
  long long kernel_launches;  /* kernels this engine has enqueued */
  long long row_steps;        /* sum over steps of the rows that ran a forward (unfinished blocks) */
  long long active_row_steps; /* sum over steps of |A|; row_steps / active_row_steps is the share of active rows
                                 that do work in a step (1 with async_advance) */
} bs_stats;

/* Sizes of the three device buffers the caller must provide for this config
 * (each 256-byte aligned).  Host pointers. */
int bs_query_sizes(const bs_config* cfg, bs_sizes* out);

/* Create an engine over caller-owned device buffers `kv`, `workspace`, `state`
 * (sizes from bs_query_sizes; `state` is cleared by this call) and the caller's
 * CUDA stream (a cudaStream_t passed as void*, NULL = default stream).  The
 * weights struct and its pointer arrays are host memory and are copied. */
int bs_init_model(const bs_config* cfg, const bs_weights* w, void* kv, void* workspace, void* state,
                  void* cuda_stream, bs_engine** out);

/* Section 2.1 / Algorithm 1 input: enqueue request r_i into the pending queue P.
 * prompt: host int32[p]; g: generation length; alpha: logit scale applied to
 * this request's logits; start_block k > 0 means blocks 0..k-1 arrive already
 * committed with the ids in gen_prefix (host int32[k * L], else NULL).
 * Token ids must lie in [0, vocab) and differ from mask_id. */
int bs_admit(bs_engine* e, long long req_id, const int* prompt, int p, int g, float alpha,
             int start_block, const int* gen_prefix);

/* Algorithm 1, block boundary (also the first fill): b_i += 1 for every active
 * row, evict rows with b_i >= K_i, stable compaction, then admit the head of P
 * while Eq. 1's cost stays <= beta, |A| < max_batch and the KV arena has a
 * hole (lowest-address first fit); start every row's next block fully masked
 * and build the next step's gather / scatter indices.  Outputs are host ints
 * (nullable).  BS_E_STATE if a block of the current cycle is unfinished. */
int bs_evict_refill(bs_engine* e, int* n_evicted, int* n_admitted, int* n_active);

/* Section 2.5: one denoise step for all unfinished rows of A - gather by
 * explicit position ids, transformer forward against the dual KV cache (whole
 * row on a block's first step, which rebuilds the cache; the active block
 * afterwards), confidence / argmax per masked position, commit conf > tau plus
 * the top-confidence position, scatter tokens, update done flags, build the
 * next step's indices.  n_committed: host int, nullable (non-NULL forces a
 * stream synchronisation). */
int bs_denoise_step(bs_engine* e, int* n_committed);

/* Block-boundary completion check (Section 2.3): all_done = every active row's
 * block is complete.  per_row_done: host bytes [max_batch], nullable. */
int bs_block_done(bs_engine* e, int* all_done, unsigned char* per_row_done);

/* Copy request req_id's token row (prompt, then generated positions; still
 * masked positions hold mask_id) into host int32 out[cap]; n_valid = p + g;
 * state = BS_REQ_*.  out may be NULL to query n_valid / state only. */
int bs_read_tokens(bs_engine* e, long long req_id, int* out, int cap, int* n_valid, int* state);

int bs_get_stats(bs_engine* e, bs_stats* out);

/* Per-kernel-family device timing (CUDA events on the engine's stream around each family's launches).
 * Off by default; switching it on adds two event records per family per layer.  bs_get_profile fills
 * host arrays of BS_FAM_COUNT entries (any may be NULL): milliseconds, kernel launches, algorithmic
 * flops and algorithmic bytes accumulated since profiling was switched on (or last reset by enabling again).
 * Algorithmic bytes: GEMMs count weights + input + output once; attention counts K and V of every
 * unfinished row once per layer plus q and the output; the epilogue counts the logits once. */
enum {
  BS_FAM_INDEX = 0,      /* fill_tokens, commit + next index build, scheduler */
  BS_FAM_EMBED_NORM = 1, /* embedding gather and RMSNorm launches */
  BS_FAM_GEMM_QKV = 2,
  BS_FAM_ROPE_KV = 3,
  BS_FAM_ATTENTION = 4,
  BS_FAM_GEMM_O = 5,
  BS_FAM_GEMM_GATE_UP = 6,
  BS_FAM_GEMM_DOWN = 7,
  BS_FAM_GEMM_LM_HEAD = 8,
  BS_FAM_CONFIDENCE = 9,        /* merge of the LM-head epilogue's confidence partials */
  BS_FAM_ATTENTION_REFRESH = 10, /* attention of steps that hold whole-row refreshes (compute-bound; BS_FAM_ATTENTION
                                    then counts pure block steps only: cache streaming) */
  BS_FAM_COUNT = 11
};
int bs_set_profiling(bs_engine* e, int on);
int bs_get_profile(bs_engine* e, double* ms, long long* launches, double* flops, double* bytes);
void bs_destroy(bs_engine* e);
const char* bs_last_error(const bs_engine* e); /* NULL engine: error of the last failed bs_init_model */

/* How the library was built.  BS_BUILD_BOUNDS_CHECK: the debugging build whose gather / scatter and index kernels
 * check every data-dependent index before use; a bad index is recorded (its access skipped) and the next call that
 * reads the step header returns BS_E_STATE with the site in bs_last_error.  The paper has no counterpart. */
enum { BS_BUILD_BOUNDS_CHECK = 1 };
int bs_build_flags(void);

/* ---- parity hooks (not on the timed path) ------------------------------ */
enum {
  BS_DBG_HEADER = 0,   /* int32[32]: n_active, M, M_m, all_done, n_committed_step, n_evicted, n_admitted, ... */
  BS_DBG_ROW_SLOT = 1, BS_DBG_ROW_S = 3, BS_DBG_ROW_KV_BASE = 4, /* int32[n_active] */
  BS_DBG_ROW_MASK = 2, /* uint64[n_active]: bit j set = block position j still masked */
  BS_DBG_CU_Q = 5,     /* int32[n_active + 1]  (indices of the step about to run) */
  BS_DBG_TOK_ROW = 6, BS_DBG_TOK_POS = 7, BS_DBG_TOK_KV = 8,   /* int32[M]; filled by the last bs_denoise_step */
  BS_DBG_LM_TOK = 9, BS_DBG_LM_ROW = 10, BS_DBG_LM_SLOT = 11,  /* int32[M_m] of the step about to run */
  BS_DBG_PREV_LM_ROW = 12, BS_DBG_PREV_LM_SLOT = 13,           /* int32[M_m] of the step that just ran */
  BS_DBG_PREV_TOK = 14, BS_DBG_PREV_CONF = 15, BS_DBG_PREV_COMMIT = 16, /* int32 / float / int32 [M_m], last step */
  BS_DBG_PREV_LOGITS = 17, /* float[rows * vocab] of the last step: rows arg0 .. arg0 + arg1 (arg1 = 0: to the end);
                              BS_E_STATE unless the engine was created with keep_logits */
  BS_DBG_REQ_ID_OF_ROW = 18, /* int64[n_active] */
  BS_DBG_KV_ROW = 19   /* bf16 K then V of (layer = arg0, physical row = arg1): 2 * Hkv * head_dim values */
};
/* Copies the named array into host_buf (cap bytes); n = bytes written. */
int bs_debug_read(bs_engine* e, int what, int arg0, int arg1, void* host_buf, size_t cap, size_t* n);

/* Dictated commit (debugging): for the active row `row` (batch order), every block position j with bit j of
 * mask_bits set and still masked takes tokens[j] (host array of 64 ints indexed by block position; entries of other positions
 * are not read) and counts as committed.  The row's step counter does not move, so a row still waiting for the
 * refresh step of its block (Section 2.5) gets it; the index of the pending step is rebuilt.  The paper has no
 * counterpart.  Errors: BS_E_ARG (row not active, bit beyond L, token id out of range or the mask id). */
int bs_debug_force_commit(bs_engine* e, int row, unsigned long long mask_bits, const int* tokens);

/* Snapshot / restore of the engine state between block cycles (host buffers).  Because the block KV cache is rebuilt
 * from the tokens at the first step of every block (Section 2.5, refresh), the state between cycles is the token rows
 * plus the scheduler state; the KV arena is not saved.  bs_debug_snapshot with host_buf = NULL only reports the size
 * in *n; otherwise it writes *n <= cap bytes.  BS_E_STATE while a block cycle is unfinished.  bs_debug_restore takes
 * a snapshot of an engine with the identical bs_config (else BS_E_ARG) and replaces requests, queue, statistics and
 * device state; the weights and buffers stay the caller's.  A restored engine continues bit-identically. */
int bs_debug_snapshot(bs_engine* e, void* host_buf, size_t cap, size_t* n);
int bs_debug_restore(bs_engine* e, const void* host_buf, size_t n_bytes);

/* Failure-path hook: enqueues a kernel whose mbarrier wait can never be satisfied and gives up after about a
 * millisecond, raising the engine's error word exactly as a timed-out pipeline wait would.  The next call that
 * reads the step header returns BS_E_TIMEOUT; the CUDA context stays usable. */
int bs_debug_inject_timeout(bs_engine* e);

/* ---- single operations (parity tests and per-kernel measurement) ------- *
 * All pointers are device memory; `stream` is a cudaStream_t as void*.     */

/* C[M,N] = A[M,K] * W[N,K]^T, bf16 operands, fp32 accumulate (the projections of the transformer block).
 * mode 0: C bf16 store;  1: C fp32 += result (residual);  2: C fp32 = row_scale[m] * result (LM head, alpha_i);
 * mode 3: C bf16 [M,N] = silu(A W^T) * (A W2^T)  (SwiGLU gate/up).  K % 8 == 0.  lda/ldc in elements. */
int bs_op_gemm(const void* A, int lda, const void* W, const void* W2, void* C, int ldc, int M, int N, int K,
               int mode, const float* row_scale, float* scratch /* nullable: k-split partial sums */,
               size_t scratch_bytes, int* error_flag /* nullable device int, set when a bounded wait runs out */,
               void* stream);

/* Plan query (host only, no launch): over how many CTA pairs bs_op_gemm splits the K range of every output tile of
 * this projection INSIDE one thread-block cluster on the current device (the pairs then add their partial accumulators
 * over distributed shared memory and the direct epilogue follows in the same kernel); 0 when the launch takes another
 * plan.  Applies to modes 0 and 1 with a dense, 16-byte aligned C (ldc = N).  The paper has no counterpart. */
int bs_op_gemm_cluster_splits(int M, int N, int K, int mode);

/* y[m,:] = bf16(w * x[idx ? idx[m] : m, :] / sqrt(mean(x^2) + eps)); x fp32 [*, d], y bf16 [M, d]. */
int bs_op_rmsnorm(const float* x, const int* idx, const void* w, void* y, int M, int d, float eps, void* stream);

/* Rotate q and k of packed tokens at their position ids (rotate-half pairing,
 * angle pos * theta^(-2j/dh)) and scatter k, v to KV rows tok_kv[t] (Section 2.5:
 * in-place update at the current query rows only).  qkv bf16 [M, (Hq+2Hkv)*dh] (q rotated in place);
 * kcache / vcache bf16 [kv_rows, Hkv, dh]. */
int bs_op_rope_kv(void* qkv, const int* tok_pos, const int* tok_kv, void* kcache, void* vcache, int M,
                  int n_q_heads, int n_kv_heads, int head_dim, float theta, int max_pos,
                  float* table_scratch /* device float[max_pos * head_dim], overwritten */, void* stream);

/* No counterpart in the paper: bs_op_rope_kv for callers that cannot allocate device memory (a host whose
 * memory pool is fixed at start-up, a plugin whose runtime owns all allocations).  Same arguments and results
 * as bs_op_rope_kv without the scratch buffer: the cos/sin table lives in a fixed array inside the library,
 * BS_ROPE_STATIC_MAX_FLOATS floats (2 MiB) that every GPU loading the library holds until the process exits.
 * Returns BS_E_ARG when max_pos * head_dim exceeds that size.  The call allocates nothing, on the device or
 * through any library.  The first call on each device looks up the array's device address (one-time set-up,
 * with that device current): make it before any stream capture.  All calls share the one table, which keeps
 * the previous call's contents and is rewritten for [0, max_pos) by each call: two calls whose kernels can
 * overlap on the GPU (different streams, no ordering between them) race on it.  Every tok_pos[t] must lie in
 * [0, max_pos): the kernel does not check it, and a larger position would read entries an earlier call left
 * (or, beyond BS_ROPE_STATIC_MAX_FLOATS / head_dim, memory outside the table). */
#define BS_ROPE_STATIC_MAX_FLOATS (512 * 1024)
int bs_op_rope_kv_static(void* qkv, const int* tok_pos, const int* tok_kv, void* kcache, void* vcache, int M,
                         int n_q_heads, int n_kv_heads, int head_dim, float theta, int max_pos, void* stream);

/* Ragged bidirectional attention of packed queries against per-row cache spans:
 * row i owns packed tokens [cu_q[i], cu_q[i+1]) and attends over cache rows
 * [kv_base[i], kv_base[i] + vis[i]) (prefix, fresh block and suffix alike; no causal or padding mask).
 * q: the qkv buffer of bs_op_rope_kv; out bf16 [M, Hq*dh].  Work items are q-tiles of
 * bs_op_attention_q_tile(Hq, Hkv, dh) tokens: cu_tile[i] = sum_{r<i} ceil(n_q(r) / q_tile), n_tiles = cu_tile[n_rows]. */
int bs_op_attention_q_tile(int n_q_heads, int n_kv_heads, int head_dim);
int bs_op_attention(const void* qkv, const void* kcache, const void* vcache, void* out, const int* cu_q,
                    const int* cu_tile, const int* kv_base, const int* vis, int n_rows, int n_tiles,
                    int M /* packed tokens */, int max_vis /* largest vis[i] */,
                    int max_nq /* largest number of query tokens of a row; 0 = unknown */,
                    long long kv_rows /* rows of kcache / vcache; every value in them must be finite */,
                    int n_q_heads, int n_kv_heads, int head_dim,
                    float* scratch /* nullable: lets few work items split their keys over CTAs */,
                    size_t scratch_bytes, int* error_flag /* nullable device int, set on a wait timeout */,
                    void* stream);

/* Per row of fp32 logits [n_rows, vocab]: mask id excluded, tok = argmax (lowest id on ties),
 * conf = exp(max - logsumexp). */
int bs_op_confidence(const float* logits, int n_rows, int vocab, int mask_id, int* tok, float* conf, void* stream);

/* The LM head fused with the confidence pass (the related-work description of confidence-aware parallel decoding:
 * token = argmax, confidence = its softmax probability): logits z[m, v] = row_scale[m] * (hf[m, :] . W[v, :]) are
 * formed in the GEMM's accumulators and reduced there, per row, to tok = argmax over v != mask_id (lowest id on ties)
 * and conf = exp(max - logsumexp); they are written to `logits` (fp32 [M, vocab], nullable) only on request.
 * hf bf16 [M, K] with row stride lda, W bf16 [vocab, K].  `scratch` holds the partials:
 * bs_op_lm_head_confidence_scratch_bytes(M, vocab) bytes, 256-byte aligned. */
size_t bs_op_lm_head_confidence_scratch_bytes(int M, int vocab);
int bs_op_lm_head_confidence(const void* hf, int lda, const void* W, int M, int vocab, int K, const float* row_scale,
                             int mask_id, void* scratch, size_t scratch_bytes, int* tok, float* conf,
                             float* logits /* nullable */, int* error_flag /* nullable */, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BLOCKSERVE_H_ */
