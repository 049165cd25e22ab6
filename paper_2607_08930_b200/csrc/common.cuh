// Shared declarations of the CUDA side: device state layout, launch wrappers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>

#include <utility>

namespace bs {

typedef __nv_bfloat16 bf16;

// Programmatic dependent launch: every kernel of a step is launched with the stream-serialisation attribute, calls
// pdl_wait() before it touches global memory (the grid before it has then completed and its writes are visible) and
// pdl_trigger() right after, so that the next kernel's launch latency and set-up overlap this kernel's run.
// Every CTA of every kernel executes pdl_wait(): completion of a grid then implies completion of all earlier ones.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  static const bool disabled = getenv("BS_NO_PDL") != nullptr;
  cfg.numAttrs = disabled ? 0 : 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

typedef unsigned long long MaskWord;      // one bit per position of a block
constexpr int kMaxBlockLen = 64;
// Largest r in [0, n) with prefix[r] <= item, for a non-decreasing prefix with prefix[0] = 0 <= item; every lane of
// the calling warp takes part and gets the result.  One round trip to memory per 32 rows instead of a dependent
// load per bisection step (the callers are short kernels whose set-up time counts).
__device__ __forceinline__ int warp_find_row(const int* __restrict__ prefix, int n, int item) {
  const int lane = threadIdx.x & 31;
  int below = 0;
  for (int base = 0; base < n; base += 32) {
    const int r = base + lane;
    const bool le = r < n && __ldg(prefix + r) <= item;
    const int c = __popc(__ballot_sync(0xffffffffu, le));
    below += c;
    if (c < 32) break;
  }
  return below - 1;
}

// Bounds-checked build (-DBS_BOUNDS_CHECK, `build(debug=True)`): the data-dependent indices of the gather / scatter
// and index kernels are checked before use; a bad one records its site (100 + site number) in the engine's error word
// and the access is skipped, so the run continues and the host reports BS_E_STATE with the site.  The regular build
// compiles the checks away.
#ifdef BS_BOUNDS_CHECK
#define BS_INDEX_OK(cond, errword, site) ((cond) ? true : (atomicMax((errword), 100 + (site)), false))
constexpr int kBoundsCheck = 1;
#else
#define BS_INDEX_OK(cond, errword, site) (true)
constexpr int kBoundsCheck = 0;
#endif
enum BoundsSite {
  SITE_EMBED = 1, SITE_FILL_TOKENS = 2, SITE_ROPE_KV = 3, SITE_FINISH_QKV = 4, SITE_COMMIT = 5, SITE_INDEX = 6,
  SITE_SCHED = 7, SITE_NORM_GATHER = 8
};

constexpr int kHdrInts = 32;
// header words (device int32[kHdrInts], mirrored to pinned host memory once per step)
enum Hdr {
  H_N_ACTIVE = 0, H_M = 1, H_MM = 2, H_ALL_DONE = 3, H_COMMITTED_STEP = 4, H_EVICTED = 5, H_ADMITTED = 6,
  H_QUEUE_HEAD = 7, H_QUEUE_LEN = 8, H_ERROR = 9, H_PARITY = 10, H_QTILES = 11, H_MAX_VIS = 12, H_WIDTH = 13,
  H_TOTAL_LO = 14, H_TOTAL_HI = 15, H_UNFINISHED = 16, H_STEP_REFRESH = 17,
  H_SUM_KV = 18,  // sum over unfinished rows of the cache rows they attend over
  H_PREV_MM = 19  // masked rows of the step that just ran (its lists stay readable in the other index buffer)
};


// Everything the scheduling / index kernels touch.  Plain pointers into the caller's `state` buffer.
struct DevState {
  int L, max_batch, max_requests, max_row_tokens, suffix_mode, mask_id, vocab;
  int q_tile;           // query tokens per attention work item
  int S;                // diffusion steps per block (transfer quota of Section 2.5); S = L: one forced token per step
  int eos_id;           // CheckEOS of Algorithm 1 (< 0: off)
  int static_groups;    // 1: no admission while any row of the current group is active (comparison policy)
  int async_advance;    // 1: rows advance / leave and the queue refills after every denoise step
  int refresh_policy;   // 0: every block starts with a whole-row forward; 1: only the first block after admission
  long long beta, kv_capacity;
  float tau;
  int* hdr;             // [kHdrInts] followed directly by row_mask[max_batch]
  MaskWord* row_mask;   // bit j set <=> block position j still masked (L <= 64)
  int* req_p; int* req_g; int* req_b; int* req_state; int* req_committed; float* req_alpha;
  int* tokens;          // [max_requests, max_row_tokens]
  int* queue;           // pending slots in admission order
  int* row_slot; int* row_s; int* row_kv_base; int* row_vis;
  int* row_refresh;     // 1: the first step of the row's current block forwards the whole row
  int* cu_q[2]; int* lm_base[2]; int* cu_tile[2];
  int* lm_tok[2]; int* lm_row[2]; int* lm_slot[2];
  int* out_tok[2]; float* out_conf[2]; int* out_commit[2];
  float* lm_scale[2];   // alpha of the row each lm entry belongs to
  const float2* slice_ms;   // [kConfSlices][M_m]: slice partials of the fused LM-head confidence pass
  const int* slice_am;
  int* tok_row; int* tok_pos; int* tok_kv;
};

// ---- launch wrappers (each returns the cudaError_t of the launch) ----------
cudaError_t launch_sched(const DevState& st, cudaStream_t s);
cudaError_t launch_commit_index(const DevState& st, cudaStream_t s);
cudaError_t launch_fill_tokens(const DevState& st, int parity, int M, cudaStream_t s);
// tokens[j] (kMaxBlockLen entries) is read for every bit j of `bits`; positions the row has already committed are skipped.
cudaError_t launch_force_commit(const DevState& st, int row, MaskWord bits, const int* tokens, cudaStream_t s);

cudaError_t launch_embed(const DevState& st, const bf16* embed, float* x, int M, int d, cudaStream_t s);
// `limits` (nullable): what the bounds-checked build compares gather / scatter indices with.
struct IndexLimits {
  int max_pos;          // rows of the RoPE table / largest position id + 1
  long long kv_rows;    // rows of the K and V caches
  int x_rows;           // rows of the gathered activation buffer
  int* error_word;
};
cudaError_t launch_rmsnorm(const float* x, const int* idx, const bf16* w, bf16* y, int M, int d, float eps,
                           cudaStream_t s, const IndexLimits* limits = nullptr);
cudaError_t launch_rope_kv(bf16* qkv, const int* tok_pos, const int* tok_kv, bf16* kc, bf16* vc, int M, int hq,
                           int hkv, int dh, const float* cos_sin, cudaStream_t s, const IndexLimits* limits = nullptr);
// scratch (nullable): fp32 partial results when the keys of a work item are split over several CTAs.
cudaError_t launch_attention(const bf16* qkv, const bf16* kc, const bf16* vc, bf16* out, const int* cu_q,
                             const int* cu_tile, const int* kv_base, const int* vis, int n_rows, int n_tiles, int M,
                             int max_vis, int max_nq, long long kv_rows, int hq, int hkv, int dh, float* scratch,
                             size_t scratch_floats, int* error_flag, cudaStream_t s);
cudaError_t launch_confidence(const float* logits, int n_rows, int vocab, int mask_id, int* tok, float* conf,
                              cudaStream_t s);

// Scratch a GEMM launch may use: fp32 partial sums of a k split, and the word it raises when a bounded wait runs out.
struct GemmScratch {
  float* partial = nullptr;
  size_t partial_floats = 0;
  int* error_flag = nullptr;
};

// Output of the LM head fused with the confidence pass (GEMM mode 5): per (group of 32 output features, token) the
// maximum of the row-scaled outputs, the sum of exp(z - max) and the feature index of the maximum.
struct GemmConf {
  float2* ms;      // [ceil(N / 32)][M]
  int* am;         // [ceil(N / 32)][M]
  int skip;        // output feature that never takes part (the mask id), or -1
};
constexpr int kConfSlices = 16;      // the group partials of a token are merged in this many slices, then once more

// C[M,N] = A[M,K] W[N,K]^T.  mode: 0 bf16 store, 1 fp32 +=, 2 fp32 row-scaled store, 3 SwiGLU (W and W2).
cudaError_t launch_gemm(const bf16* A, int lda, const bf16* W, const bf16* W2, void* C, int ldc, int M, int N, int K,
                        int mode, const float* row_scale, const GemmScratch& scratch, cudaStream_t s);
cudaError_t launch_gemm_tc(const bf16* A, int lda, const bf16* W, const bf16* W2, void* C, int ldc, int M, int N,
                           int K, int mode, const float* row_scale, const GemmScratch& scratch, cudaStream_t s,
                           int* splits_out, const GemmConf* conf = nullptr);
// LM head fused with the confidence pass: group partials by the GEMM epilogue (logits, if not null, receives the scaled
// fp32 outputs as well), then the partials of each token merged into kConfSlices slice partials
// slice_ms / slice_am [kConfSlices][M] (merge_conf_slices() in conf_merge.cuh finishes the job).
cudaError_t launch_lm_head_conf(const bf16* hf, int lda, const bf16* W, int M, int V, int K, const float* row_scale,
                                int mask_id, const GemmConf& groups, float2* slice_ms, int* slice_am, float* logits,
                                const GemmScratch& scratch, cudaStream_t s);
cudaError_t launch_conf_merge(const GemmConf& groups, int M, int V, float2* slice_ms, int* slice_am, cudaStream_t s);
// tok / conf [M] from the slice partials (stand-alone use; the engine's commit kernel does this inline).
cudaError_t launch_conf_final(const float2* slice_ms, const int* slice_am, int M, int* tok, float* conf,
                              cudaStream_t s);
// Why the last launch_gemm* of this thread returned cudaErrorNotSupported (a shape or alignment the tensor-core
// kernels do not take; there is no other GEMM behind them).
const char* gemm_decline_reason();
// Over how many CTA pairs launch_gemm* would split the K range of each output tile of this direct projection (mode 0
// or 1) inside one thread-block cluster, the partial accumulators being reduced over distributed shared memory;
// 0 when the launch takes another plan.
int gemm_cluster_splits(int M, int N, int K, int mode, int ldc, const void* C);
// mode 4: only the k-split partial sums [splits][M][N] are written to scratch.partial; a fused finishing kernel
// (below) adds them in split order and applies what follows the projection.
cudaError_t launch_gemm_partial(const bf16* A, int lda, const bf16* W, int M, int N, int K, const GemmScratch& scratch,
                                cudaStream_t s, int* splits_out);
// q/k/v = bf16(sum of partials); RoPE on q, k at the token's position id; q -> qkv buffer, k / v -> cache rows.
cudaError_t launch_finish_qkv_rope(const float* partial, int splits, int M, bf16* qkv, const int* tok_pos,
                                   const int* tok_kv, bf16* kc, bf16* vc, int hq, int hkv, int dh,
                                   const float* cos_sin, cudaStream_t s, const IndexLimits* limits = nullptr);
// x += sum of partials; if w: h = bf16(RMSNorm(x) * w).
cudaError_t launch_finish_residual_norm(const float* partial, int splits, int M, int d, float* x, const bf16* w,
                                        bf16* h, float eps, cudaStream_t s);

int attention_q_tile(int hq, int hkv, int dh);
void build_rope_table(float* host_cos_sin, int max_pos, int dh, float theta);   // [max_pos, dh/2, 2]

}  // namespace bs
