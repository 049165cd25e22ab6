// Host controller and C ABI of the mixed-state block-denoising engine: argument checks, request table and
// pending queue (sorted insert), per-step kernel sequencing, one small read-back per step.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <string>
#include <unordered_map>
#include <vector>

#include "../../include/blockserve.h"
#include "common.cuh"

using namespace bs;

namespace {

std::string g_init_error;

inline size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

struct Carver {     // hands out 256-byte aligned sub-buffers; with base == nullptr it only counts
  char* base;
  size_t off = 0;
  explicit Carver(void* b) : base(static_cast<char*>(b)) {}
  template <typename T>
  T* take(size_t n) {
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off = align_up(off + n * sizeof(T));
    return p;
  }
};

constexpr long long kMlpChunk = 16384;    // tokens per MLP pass (bounds the gate/up activation buffer)

struct Workspace {
  float* rope;      // [max_row_tokens, dh/2, 2]
  float* x;         // [T, d] residual stream, fp32
  bf16* h;          // [T, d]
  bf16* qkv;        // [T, (Hq + 2 Hkv) dh]
  bf16* attn;       // [T, Hq dh]
  bf16* act;        // [min(T, chunk), ffn]
  bf16* hf;         // [max_batch L, d]
  float* logits;    // [max_batch L, V], only with bs_config.keep_logits
  float2* group_ms; // [ceil(V / 32)][max_batch L]: confidence partials of the LM-head epilogue
  int* group_am;
  float2* slice_ms; // [kConfSlices][max_batch L]
  int* slice_am;
  float* partial;   // k-split partial sums of the projection GEMMs
};

constexpr size_t kPartialFloats = 16u << 20;
constexpr int kSmallStepTokens = 640;     // packed tokens up to which a step takes the fused block-step path

size_t carve_workspace(const bs_config& c, void* base, Workspace* w) {
  Carver cv(base);
  const size_t T = (size_t)c.kv_capacity_tokens, mm = (size_t)c.max_batch * c.block_len;
  Workspace t;
  t.rope = cv.take<float>((size_t)c.max_row_tokens * c.head_dim);
  t.x = cv.take<float>(T * c.d_model);
  t.h = cv.take<bf16>(T * c.d_model);
  t.qkv = cv.take<bf16>(T * (size_t)(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim);
  t.attn = cv.take<bf16>(T * (size_t)c.n_q_heads * c.head_dim);
  t.act = cv.take<bf16>(std::min<size_t>(T, kMlpChunk) * c.d_ffn);
  t.hf = cv.take<bf16>(mm * c.d_model);
  t.logits = c.keep_logits ? cv.take<float>(mm * c.vocab) : nullptr;
  const size_t n_groups = ((size_t)c.vocab + 31) / 32;
  t.group_ms = cv.take<float2>(n_groups * mm);
  t.group_am = cv.take<int>(n_groups * mm);
  t.slice_ms = cv.take<float2>((size_t)kConfSlices * mm);
  t.slice_am = cv.take<int>((size_t)kConfSlices * mm);
  t.partial = cv.take<float>(kPartialFloats);
  if (w) *w = t;
  return cv.off;
}

size_t carve_state(const bs_config& c, void* base, DevState* out) {
  Carver cv(base);
  DevState st;
  memset(&st, 0, sizeof(st));
  const size_t R = c.max_requests, B = c.max_batch, T = (size_t)c.kv_capacity_tokens, mm = B * c.block_len;
  // header and row masks are contiguous: one copy mirrors both to the host
  st.hdr = cv.take<int>(kHdrInts + 2 * B);      // 64-bit mask words: two ints per row
  st.row_mask = base ? reinterpret_cast<MaskWord*>(st.hdr + kHdrInts) : nullptr;
  st.req_p = cv.take<int>(R); st.req_g = cv.take<int>(R); st.req_b = cv.take<int>(R);
  st.req_state = cv.take<int>(R); st.req_committed = cv.take<int>(R); st.req_alpha = cv.take<float>(R);
  st.tokens = cv.take<int>(R * c.max_row_tokens);
  st.queue = cv.take<int>(R);
  st.row_slot = cv.take<int>(B); st.row_s = cv.take<int>(B); st.row_kv_base = cv.take<int>(B);
  st.row_vis = cv.take<int>(B);
  st.row_refresh = cv.take<int>(B);
  for (int k = 0; k < 2; ++k) {
    st.cu_q[k] = cv.take<int>(B + 1); st.lm_base[k] = cv.take<int>(B + 1); st.cu_tile[k] = cv.take<int>(B + 1);
    st.lm_tok[k] = cv.take<int>(mm); st.lm_row[k] = cv.take<int>(mm); st.lm_slot[k] = cv.take<int>(mm);
    st.out_tok[k] = cv.take<int>(mm); st.out_conf[k] = cv.take<float>(mm); st.out_commit[k] = cv.take<int>(mm);
    st.lm_scale[k] = cv.take<float>(mm);
  }
  st.tok_row = cv.take<int>(T); st.tok_pos = cv.take<int>(T); st.tok_kv = cv.take<int>(T);
  if (out) *out = st;
  return cv.off;
}

const char* check_config(const bs_config& c) {
  if (c.n_layers < 1 || c.d_model < 8 || c.d_model % 8 || c.d_model > 8192)
    return "d_model must be a positive multiple of 8, at most 8192";
  if (c.head_dim != 64 && c.head_dim != 128) return "head_dim must be 64 or 128";
  if (c.n_kv_heads < 1 || c.n_q_heads % c.n_kv_heads) return "n_q_heads must be a multiple of n_kv_heads";
  if (c.n_q_heads / c.n_kv_heads > 8) return "at most 8 query heads per kv head";
  if (c.d_ffn < 8 || c.d_ffn % 8) return "d_ffn must be a positive multiple of 8";
  if (c.vocab < 2 || c.vocab % 2) return "vocab must be even";
  if (c.mask_id < 0 || c.mask_id >= c.vocab) return "mask_id outside the vocabulary";
  if (c.block_len < 1 || c.block_len > kMaxBlockLen) return "block_len must be in [1, 64]";
  if (c.max_batch < 1 || c.max_batch > 1024) return "max_batch must be in [1, 1024]";
  if (c.max_requests < 1 || c.max_row_tokens < 2) return "max_requests / max_row_tokens too small";
  if (c.kv_capacity_tokens < c.max_row_tokens) return "kv_capacity_tokens smaller than one row";
  if (c.kv_capacity_tokens > (1ll << 30)) return "kv_capacity_tokens too large";
  if (c.suffix_mode != BS_SUFFIX_FULL && c.suffix_mode != BS_SUFFIX_NONE) return "bad suffix_mode";
  if (!(c.tau >= 0.f)) return "tau must be >= 0";
  if (c.steps_per_block < 0 || c.steps_per_block > c.block_len) return "steps_per_block must be in [0, block_len]";
  if (c.eos_id >= c.vocab || c.eos_id == c.mask_id) return "eos_id must be a token id other than the mask id, or negative";
  if (c.keep_logits != 0 && c.keep_logits != 1) return "keep_logits must be 0 or 1";
  if (c.async_advance != 0 && c.async_advance != 1) return "async_advance must be 0 or 1";
  if (c.refresh_policy != BS_REFRESH_EVERY_BLOCK && c.refresh_policy != BS_REFRESH_AT_ADMISSION)
    return "bad refresh_policy";
  if (c.async_advance && c.static_groups) return "async_advance and static_groups exclude each other";
  return nullptr;
}

}  // namespace

struct bs_engine {
  bs_config cfg;
  DevState st;
  Workspace ws;
  cudaStream_t stream;
  bf16* kv;
  void* state_base = nullptr;   // the caller's state buffer, for snapshots
  size_t state_bytes = 0;
  size_t kv_layer_stride;   // elements between layers: 2 * rows * Hkv * dh
  size_t kv_half;           // elements between K and V of one layer
  const bf16 *embed, *lm_head, *final_norm;
  std::vector<const bf16*> wqkv, wo, w_gate, w_up, w_down, norm1, norm2;
  int* pinned = nullptr;    // hdr + row masks
  cudaEvent_t ev = nullptr;
  bool hdr_pending = false;
  bool hdr_from_step = false;   // the header in flight was written by a denoise step (per-row advance: it may admit)
  bool queue_dirty = false;     // requests were submitted since the queue was last uploaded
  int hdr[kHdrInts];
  std::unordered_map<long long, int> slot_of;
  std::vector<long long> id_of_slot;
  std::vector<int> h_p, h_g, h_b, h_state0;
  std::vector<float> h_alpha;
  std::vector<int> pending;
  int uploaded_slots = 0;
  bs_stats stats;
  std::string err;
  GemmScratch gemm_scratch;
  // per-family device timing
  bool profiling = false;
  std::vector<cudaEvent_t> ev_pool;
  size_t ev_used = 0;
  struct Span { int fam; size_t a, b; };
  std::vector<Span> spans;
  double prof_ms[BS_FAM_COUNT], prof_flops[BS_FAM_COUNT], prof_bytes[BS_FAM_COUNT];
  long long prof_launches[BS_FAM_COUNT];
  int cur_fam = -1;
  size_t cur_a = 0;
};

namespace {

int fail(bs_engine* e, int code, const std::string& msg) {
  if (e) e->err = msg; else g_init_error = msg;
  return code;
}
int cuda_fail(bs_engine* e, cudaError_t r, const char* what) {
  if (r == cudaErrorNotSupported)     // a plan the kernels declined: a property of the arguments, not of the device
    return fail(e, BS_E_ARG, std::string("unsupported shape: ") + bs::gemm_decline_reason() + " (" + what + ")");
  return fail(e, BS_E_CUDA, std::string(what) + ": " + cudaGetErrorString(r));
}
#define CU(e, call)                                         \
  do {                                                      \
    cudaError_t r_ = (call);                                \
    if (r_ != cudaSuccess) return cuda_fail(e, r_, #call);  \
  } while (0)
#define KL(e, call)                                         \
  do {                                                      \
    cudaError_t r_ = (call);                                \
    (e)->stats.kernel_launches++;                           \
    if (r_ != cudaSuccess) return cuda_fail(e, r_, #call);  \
  } while (0)

void prof_collect(bs_engine* e) {     // all recorded events have completed when this runs
  for (const bs_engine::Span& sp : e->spans) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, e->ev_pool[sp.a], e->ev_pool[sp.b]) == cudaSuccess) e->prof_ms[sp.fam] += ms;
  }
  e->spans.clear();
  e->ev_used = 0;
}

cudaEvent_t prof_event(bs_engine* e, size_t* idx) {
  if (e->ev_used == e->ev_pool.size()) {
    cudaEvent_t ev;
    cudaEventCreate(&ev);
    e->ev_pool.push_back(ev);
  }
  *idx = e->ev_used++;
  return e->ev_pool[*idx];
}

// Opens a timed span for `fam` (closing the one in flight); fam < 0 only closes.
void prof_mark(bs_engine* e, int fam) {
  if (!e->profiling) return;
  size_t idx;
  cudaEvent_t ev = prof_event(e, &idx);
  cudaEventRecord(ev, e->stream);
  if (e->cur_fam >= 0) e->spans.push_back({e->cur_fam, e->cur_a, idx});
  e->cur_fam = fam;
  e->cur_a = idx;
}

void prof_work(bs_engine* e, int fam, int launches, double flops, double bytes) {
  if (!e->profiling) return;
  e->prof_launches[fam] += launches;
  e->prof_flops[fam] += flops;
  e->prof_bytes[fam] += bytes;
}

int sync_header(bs_engine* e) {
  if (e->hdr_pending) {
    CU(e, cudaEventSynchronize(e->ev));
    if (e->profiling) prof_collect(e);
    memcpy(e->hdr, e->pinned, sizeof(e->hdr));
    e->hdr_pending = false;
    if (e->hdr_from_step && e->cfg.async_advance) {
      // per-row advance: the step's own boundary may have admitted the head of the queue and evicted rows
      const int adm = e->hdr[H_ADMITTED];
      e->pending.erase(e->pending.begin(), e->pending.begin() + std::min<size_t>(adm, e->pending.size()));
    }
    e->hdr_from_step = false;
    if (e->hdr[H_ERROR] >= 100)
      return fail(e, BS_E_STATE, "bounds-checked build: index out of range at site " + std::to_string(e->hdr[H_ERROR] - 100));
    if (e->hdr[H_ERROR] != 0) return fail(e, BS_E_TIMEOUT, "a bounded device-side wait ran out");
  }
  return BS_OK;
}

int post_header(bs_engine* e, bool from_step = false) {
  CU(e, cudaMemcpyAsync(e->pinned, e->st.hdr, (kHdrInts + 2 * e->cfg.max_batch) * sizeof(int),
                        cudaMemcpyDeviceToHost, e->stream));
  CU(e, cudaEventRecord(e->ev, e->stream));
  e->hdr_pending = true;
  e->hdr_from_step = from_step;
  return BS_OK;
}

// Request table entries of newly submitted requests and the pending queue P go to the device; the queue head restarts
// at zero.  The header must be in sync (the device may have consumed queue entries since the last upload).
int upload_queue(bs_engine* e) {
  DevState& st = e->st;
  const int n_slots = (int)e->id_of_slot.size(), first = e->uploaded_slots;
  if (n_slots > first) {
    const size_t n = n_slots - first;
    std::vector<int> zeros(n, 0);
    CU(e, cudaMemcpyAsync(st.req_p + first, e->h_p.data() + first, n * 4, cudaMemcpyHostToDevice, e->stream));
    CU(e, cudaMemcpyAsync(st.req_g + first, e->h_g.data() + first, n * 4, cudaMemcpyHostToDevice, e->stream));
    CU(e, cudaMemcpyAsync(st.req_b + first, e->h_b.data() + first, n * 4, cudaMemcpyHostToDevice, e->stream));
    CU(e, cudaMemcpyAsync(st.req_alpha + first, e->h_alpha.data() + first, n * 4, cudaMemcpyHostToDevice, e->stream));
    CU(e, cudaMemcpyAsync(st.req_state + first, zeros.data(), n * 4, cudaMemcpyHostToDevice, e->stream));
    CU(e, cudaMemcpyAsync(st.req_committed + first, zeros.data(), n * 4, cudaMemcpyHostToDevice, e->stream));
    e->uploaded_slots = n_slots;
  }
  if (!e->pending.empty())
    CU(e, cudaMemcpyAsync(st.queue, e->pending.data(), e->pending.size() * 4, cudaMemcpyHostToDevice, e->stream));
  const int qh[2] = {0, (int)e->pending.size()};
  CU(e, cudaMemcpyAsync(st.hdr + H_QUEUE_HEAD, qh, sizeof(qh), cudaMemcpyHostToDevice, e->stream));
  e->queue_dirty = false;
  return BS_OK;
}

}  // namespace

namespace bs {
cudaError_t launch_gemm(const bf16* A, int lda, const bf16* W, const bf16* W2, void* C, int ldc, int M, int N, int K,
                        int mode, const float* row_scale, const GemmScratch& scratch, cudaStream_t s) {
  return launch_gemm_tc(A, lda, W, W2, C, ldc, M, N, K, mode, row_scale, scratch, s, nullptr);
}

cudaError_t launch_gemm_partial(const bf16* A, int lda, const bf16* W, int M, int N, int K, const GemmScratch& scratch,
                                cudaStream_t s, int* splits_out) {
  return launch_gemm_tc(A, lda, W, nullptr, nullptr, 0, M, N, K, 4, nullptr, scratch, s, splits_out);
}
}  // namespace bs

extern "C" {

int bs_query_sizes(const bs_config* cfg, bs_sizes* out) {
  if (!cfg || !out) return fail(nullptr, BS_E_ARG, "null argument");
  if (const char* m = check_config(*cfg)) return fail(nullptr, BS_E_ARG, m);
  out->kv_bytes = align_up((size_t)cfg->n_layers * 2 * (size_t)cfg->kv_capacity_tokens * cfg->n_kv_heads *
                           cfg->head_dim * sizeof(bf16));
  out->workspace_bytes = carve_workspace(*cfg, nullptr, nullptr);
  out->state_bytes = carve_state(*cfg, nullptr, nullptr);
  return BS_OK;
}

int bs_init_model(const bs_config* cfg, const bs_weights* w, void* kv, void* workspace, void* state,
                  void* cuda_stream, bs_engine** out) {
  if (!cfg || !w || !kv || !workspace || !state || !out) return fail(nullptr, BS_E_ARG, "null argument");
  if (const char* m = check_config(*cfg)) return fail(nullptr, BS_E_ARG, m);
  if (!w->embed || !w->lm_head || !w->final_norm || !w->wqkv || !w->wo || !w->w_gate || !w->w_up || !w->w_down ||
      !w->norm1 || !w->norm2)
    return fail(nullptr, BS_E_ARG, "null weight pointer");
  if (((uintptr_t)kv | (uintptr_t)workspace | (uintptr_t)state) & 255)
    return fail(nullptr, BS_E_ARG, "device buffers must be 256-byte aligned");
  int dev_count = 0;
  if (cudaGetDeviceCount(&dev_count) != cudaSuccess || dev_count == 0)
    return fail(nullptr, BS_E_CUDA, "no CUDA device: this library has no CPU path");
  bs_engine* e = new bs_engine();
  e->cfg = *cfg;
  e->stream = static_cast<cudaStream_t>(cuda_stream);
  e->kv = static_cast<bf16*>(kv);
  e->kv_half = (size_t)cfg->kv_capacity_tokens * cfg->n_kv_heads * cfg->head_dim;
  e->kv_layer_stride = 2 * e->kv_half;
  carve_workspace(*cfg, workspace, &e->ws);
  const size_t state_bytes = carve_state(*cfg, state, &e->st);
  e->state_base = state;
  e->state_bytes = state_bytes;
  DevState& st = e->st;
  st.L = cfg->block_len; st.max_batch = cfg->max_batch; st.max_requests = cfg->max_requests;
  st.max_row_tokens = cfg->max_row_tokens; st.suffix_mode = cfg->suffix_mode; st.mask_id = cfg->mask_id;
  st.vocab = cfg->vocab; st.beta = cfg->token_budget; st.kv_capacity = cfg->kv_capacity_tokens; st.tau = cfg->tau;
  st.S = cfg->steps_per_block > 0 ? cfg->steps_per_block : cfg->block_len;
  st.eos_id = cfg->eos_id;
  st.static_groups = cfg->static_groups ? 1 : 0;
  st.async_advance = cfg->async_advance ? 1 : 0;
  st.refresh_policy = cfg->refresh_policy;
  st.q_tile = attention_q_tile(cfg->n_q_heads, cfg->n_kv_heads, cfg->head_dim);
  st.slice_ms = e->ws.slice_ms;
  st.slice_am = e->ws.slice_am;
  e->gemm_scratch.partial = e->ws.partial;
  e->gemm_scratch.partial_floats = kPartialFloats;
  e->gemm_scratch.error_flag = st.hdr + H_ERROR;
  e->embed = static_cast<const bf16*>(w->embed);
  e->lm_head = static_cast<const bf16*>(w->lm_head);
  e->final_norm = static_cast<const bf16*>(w->final_norm);
  for (int l = 0; l < cfg->n_layers; ++l) {
    const void* ptrs[7] = {w->wqkv[l], w->wo[l], w->w_gate[l], w->w_up[l], w->w_down[l], w->norm1[l], w->norm2[l]};
    for (const void* p : ptrs)
      if (!p || ((uintptr_t)p & 15)) { delete e; return fail(nullptr, BS_E_ARG, "layer weight null or not 16-byte aligned"); }
    e->wqkv.push_back((const bf16*)ptrs[0]); e->wo.push_back((const bf16*)ptrs[1]);
    e->w_gate.push_back((const bf16*)ptrs[2]); e->w_up.push_back((const bf16*)ptrs[3]);
    e->w_down.push_back((const bf16*)ptrs[4]); e->norm1.push_back((const bf16*)ptrs[5]);
    e->norm2.push_back((const bf16*)ptrs[6]);
  }
  memset(&e->stats, 0, sizeof(e->stats));
  for (int i = 0; i < BS_FAM_COUNT; ++i) e->prof_ms[i] = e->prof_flops[i] = e->prof_bytes[i] = 0.0, e->prof_launches[i] = 0;
  memset(e->hdr, 0, sizeof(e->hdr));
  cudaError_t r = cudaMemsetAsync(state, 0, state_bytes, e->stream);
  // cache rows are read in whole tiles: rows no request has written yet must hold finite values (they meet a
  // probability of exactly zero, and 0 * NaN would poison the row)
  if (r == cudaSuccess)
    r = cudaMemsetAsync(kv, 0, (size_t)cfg->n_layers * 2 * e->kv_half * sizeof(bf16), e->stream);
  if (r == cudaSuccess) r = cudaHostAlloc((void**)&e->pinned, (kHdrInts + 2 * cfg->max_batch) * sizeof(int), cudaHostAllocDefault);
  if (r == cudaSuccess) r = cudaEventCreateWithFlags(&e->ev, cudaEventDisableTiming);
  if (r == cudaSuccess) {
    std::vector<float> tab((size_t)cfg->max_row_tokens * cfg->head_dim);
    build_rope_table(tab.data(), cfg->max_row_tokens, cfg->head_dim, cfg->rope_theta);
    r = cudaMemcpyAsync(e->ws.rope, tab.data(), tab.size() * sizeof(float), cudaMemcpyHostToDevice, e->stream);
    if (r == cudaSuccess) r = cudaStreamSynchronize(e->stream);
  }
  if (r != cudaSuccess) {
    std::string msg = std::string("bs_init_model: ") + cudaGetErrorString(r);
    bs_destroy(e);
    return fail(nullptr, BS_E_CUDA, msg);
  }
  e->h_p.reserve(cfg->max_requests);
  *out = e;
  return BS_OK;
}

int bs_admit(bs_engine* e, long long req_id, const int* prompt, int p, int g, float alpha, int start_block,
             const int* gen_prefix) {
  if (!e) return BS_E_ARG;
  const bs_config& c = e->cfg;
  const int L = c.block_len;
  // per-row advance: a step in flight may still take entries off the front of the queue; account for them before
  // the sorted insert moves positions
  if (c.async_advance)
    if (int rc = sync_header(e)) return rc;
  if (!prompt || p < 1 || g < 1 || start_block < 0) return fail(e, BS_E_ARG, "bad request geometry");
  const int K = (g + L - 1) / L;
  if (start_block >= K) return fail(e, BS_E_ARG, "start_block must be below K_i");
  if (start_block > 0 && !gen_prefix) return fail(e, BS_E_ARG, "gen_prefix required when start_block > 0");
  if (e->slot_of.count(req_id)) return fail(e, BS_E_ARG, "duplicate request id");
  if ((long long)p + g > c.max_row_tokens) return fail(e, BS_E_KV_FULL, "request longer than max_row_tokens");
  if ((int)e->id_of_slot.size() >= c.max_requests) return fail(e, BS_E_KV_FULL, "request table full");
  if (c.token_budget > 0 && (long long)p + (long long)(start_block + 1) * L > c.token_budget)
    return fail(e, BS_E_BUDGET, "request alone is wider than the token budget");
  std::vector<int> row((size_t)p + g, c.mask_id);
  for (int i = 0; i < p; ++i) row[i] = prompt[i];
  for (int i = 0; i < start_block * L; ++i) row[p + i] = gen_prefix[i];
  for (int i = 0; i < p + start_block * L; ++i)
    if (row[i] < 0 || row[i] >= c.vocab || row[i] == c.mask_id) return fail(e, BS_E_ARG, "token id out of range");
  const int slot = (int)e->id_of_slot.size();
  // pageable source: the copy has left `row` when the call returns
  CU(e, cudaMemcpyAsync(e->st.tokens + (size_t)slot * c.max_row_tokens, row.data(), row.size() * sizeof(int),
                        cudaMemcpyHostToDevice, e->stream));
  e->slot_of[req_id] = slot;
  e->id_of_slot.push_back(req_id);
  e->h_p.push_back(p); e->h_g.push_back(g); e->h_b.push_back(start_block); e->h_alpha.push_back(alpha);
  // pending queue P: ascending prompt length, ties by submission order (Section 2.4)
  auto pos = e->pending.end();
  if (c.sort_queue)
    pos = std::upper_bound(e->pending.begin(), e->pending.end(), slot,
                           [&](int a, int b) { return e->h_p[a] < e->h_p[b]; });
  e->pending.insert(pos, slot);
  e->queue_dirty = true;
  return BS_OK;
}

int bs_evict_refill(bs_engine* e, int* n_evicted, int* n_admitted, int* n_active) {
  if (!e) return BS_E_ARG;
  if (int rc = sync_header(e)) return rc;
  if (e->hdr[H_N_ACTIVE] > 0 && !e->hdr[H_ALL_DONE]) return fail(e, BS_E_STATE, "a block of this cycle is unfinished");
  DevState& st = e->st;
  if (int rc = upload_queue(e)) return rc;
  KL(e, launch_sched(st, e->stream));
  if (int rc = post_header(e)) return rc;
  if (int rc = sync_header(e)) return rc;
  const int adm = e->hdr[H_ADMITTED];
  e->pending.erase(e->pending.begin(), e->pending.begin() + adm);
  if (e->hdr[H_N_ACTIVE] > 0) {
    e->stats.cycles++;
    e->stats.sum_active += e->hdr[H_N_ACTIVE];
  }
  if (n_evicted) *n_evicted = e->hdr[H_EVICTED];
  if (n_admitted) *n_admitted = adm;
  if (n_active) *n_active = e->hdr[H_N_ACTIVE];
  return BS_OK;
}

int bs_denoise_step(bs_engine* e, int* n_committed) {
  if (!e) return BS_E_ARG;
  if (int rc = sync_header(e)) return rc;
  const int M = e->hdr[H_M], Mm = e->hdr[H_MM], parity = e->hdr[H_PARITY], n_rows = e->hdr[H_N_ACTIVE];
  if (n_rows == 0 || M == 0 || Mm == 0) return fail(e, BS_E_STATE, "no unfinished block to denoise");
  const bs_config& c = e->cfg;
  DevState& st = e->st;
  Workspace& ws = e->ws;
  cudaStream_t s = e->stream;
  // per-row advance: this step's boundary admits from the queue, so requests submitted meanwhile must be on the device
  if (c.async_advance && e->queue_dirty)
    if (int rc = upload_queue(e)) return rc;
  e->stats.row_steps += e->hdr[H_UNFINISHED];
  e->stats.active_row_steps += n_rows;
  const int d = c.d_model, hq = c.n_q_heads, hkv = c.n_kv_heads, dh = c.head_dim;
  const int qkv_n = (hq + 2 * hkv) * dh;
  const IndexLimits lim{c.max_row_tokens, c.kv_capacity_tokens, M, st.hdr + H_ERROR};     // read by the checked build

  const double dM = (double)M, dd = (double)d, dq = (double)qkv_n, dhq = (double)hq * dh, df = (double)c.d_ffn;
  const double kv_rows = (double)e->hdr[H_SUM_KV];
  prof_mark(e, BS_FAM_INDEX);
  KL(e, launch_fill_tokens(st, parity, M, s));
  prof_work(e, BS_FAM_INDEX, 1, 0, 12.0 * dM);
  prof_mark(e, BS_FAM_EMBED_NORM);
  KL(e, launch_embed(st, e->embed, ws.x, M, d, s));
  prof_work(e, BS_FAM_EMBED_NORM, 1, 0, 6.0 * dM * dd);
  // A block step (few packed tokens) runs the projections that feed a row-wise operator as k-split partial sums
  // and lets one finishing kernel per projection add them and apply that operator (RoPE + KV scatter after QKV,
  // residual + the next RMSNorm after O and down).  A refresh step (many tokens) uses the direct epilogues.
  const int max_nq = e->hdr[H_STEP_REFRESH] > 0 ? 0 : c.block_len;    // 0: rows may bring their whole span
  const bool small = M <= kSmallStepTokens && (size_t)M * (size_t)std::max(qkv_n, d) <= kPartialFloats;
  if (small) {
    prof_mark(e, BS_FAM_EMBED_NORM);
    KL(e, launch_rmsnorm(ws.x, nullptr, e->norm1[0], ws.h, M, d, c.rms_eps, s));
    prof_work(e, BS_FAM_EMBED_NORM, 1, 0, 6.0 * dM * dd);
    for (int l = 0; l < c.n_layers; ++l) {
      bf16* kc = e->kv + (size_t)l * e->kv_layer_stride;
      bf16* vc = kc + e->kv_half;
      int sp = 1;
      prof_mark(e, BS_FAM_GEMM_QKV);
      KL(e, launch_gemm_partial(ws.h, d, e->wqkv[l], M, qkv_n, d, e->gemm_scratch, s, &sp));
      prof_work(e, BS_FAM_GEMM_QKV, 1, 2.0 * dM * dq * dd, 2.0 * (dq * dd + dM * dd) + 4.0 * sp * dM * dq);
      prof_mark(e, BS_FAM_ROPE_KV);
      KL(e, launch_finish_qkv_rope(ws.partial, sp, M, ws.qkv, st.tok_pos, st.tok_kv, kc, vc, hq, hkv, dh, ws.rope, s,
                                   &lim));
      prof_work(e, BS_FAM_ROPE_KV, 1, 0, 4.0 * sp * dM * dq + 2.0 * dM * dq);
      prof_mark(e, BS_FAM_ATTENTION);
      KL(e, launch_attention(ws.qkv, kc, vc, ws.attn, st.cu_q[parity], st.cu_tile[parity], st.row_kv_base,
                             st.row_vis, n_rows, e->hdr[H_QTILES], M, e->hdr[H_MAX_VIS], max_nq,
                             c.kv_capacity_tokens, hq, hkv, dh, ws.partial, kPartialFloats, st.hdr + H_ERROR, s));
      prof_work(e, BS_FAM_ATTENTION, 1, 0, 2.0 * (2.0 * kv_rows * hkv * dh + 2.0 * dM * dhq));
      prof_mark(e, BS_FAM_GEMM_O);
      KL(e, launch_gemm_partial(ws.attn, hq * dh, e->wo[l], M, d, hq * dh, e->gemm_scratch, s, &sp));
      prof_work(e, BS_FAM_GEMM_O, 1, 2.0 * dM * dd * dhq, 2.0 * (dd * dhq + dM * dhq) + 4.0 * sp * dM * dd);
      prof_mark(e, BS_FAM_EMBED_NORM);
      KL(e, launch_finish_residual_norm(ws.partial, sp, M, d, ws.x, e->norm2[l], ws.h, c.rms_eps, s));
      prof_work(e, BS_FAM_EMBED_NORM, 1, 0, (4.0 * sp + 10.0) * dM * dd);
      prof_mark(e, BS_FAM_GEMM_GATE_UP);
      KL(e, launch_gemm(ws.h, d, e->w_gate[l], e->w_up[l], ws.act, c.d_ffn, M, c.d_ffn, d, 3, nullptr,
                        e->gemm_scratch, s));
      prof_work(e, BS_FAM_GEMM_GATE_UP, 1, 4.0 * dM * df * dd, 2.0 * (2.0 * df * dd + dM * dd + dM * df));
      prof_mark(e, BS_FAM_GEMM_DOWN);
      KL(e, launch_gemm_partial(ws.act, c.d_ffn, e->w_down[l], M, d, c.d_ffn, e->gemm_scratch, s, &sp));
      prof_work(e, BS_FAM_GEMM_DOWN, 1, 2.0 * dM * dd * df, 2.0 * (dd * df + dM * df) + 4.0 * sp * dM * dd);
      prof_mark(e, BS_FAM_EMBED_NORM);
      const bf16* next_norm = l + 1 < c.n_layers ? e->norm1[l + 1] : nullptr;
      KL(e, launch_finish_residual_norm(ws.partial, sp, M, d, ws.x, next_norm, ws.h, c.rms_eps, s));
      prof_work(e, BS_FAM_EMBED_NORM, 1, 0, (4.0 * sp + 10.0) * dM * dd);
    }
  } else
  for (int l = 0; l < c.n_layers; ++l) {
    bf16* kc = e->kv + (size_t)l * e->kv_layer_stride;
    bf16* vc = kc + e->kv_half;
    prof_mark(e, BS_FAM_EMBED_NORM);
    KL(e, launch_rmsnorm(ws.x, nullptr, e->norm1[l], ws.h, M, d, c.rms_eps, s));
    prof_work(e, BS_FAM_EMBED_NORM, 1, 0, 6.0 * dM * dd);
    prof_mark(e, BS_FAM_GEMM_QKV);
    KL(e, launch_gemm(ws.h, d, e->wqkv[l], nullptr, ws.qkv, qkv_n, M, qkv_n, d, 0, nullptr, e->gemm_scratch, s));
    prof_work(e, BS_FAM_GEMM_QKV, 1, 2.0 * dM * dq * dd, 2.0 * (dq * dd + dM * dd + dM * dq));
    prof_mark(e, BS_FAM_ROPE_KV);
    KL(e, launch_rope_kv(ws.qkv, st.tok_pos, st.tok_kv, kc, vc, M, hq, hkv, dh, ws.rope, s, &lim));
    prof_work(e, BS_FAM_ROPE_KV, 1, 0, 2.0 * dM * (dq + (double)(hq + 2 * hkv) * dh));
    const int attn_fam = e->hdr[H_STEP_REFRESH] > 0 ? BS_FAM_ATTENTION_REFRESH : BS_FAM_ATTENTION;
    prof_mark(e, attn_fam);
    KL(e, launch_attention(ws.qkv, kc, vc, ws.attn, st.cu_q[parity], st.cu_tile[parity], st.row_kv_base, st.row_vis,
                           n_rows, e->hdr[H_QTILES], M, e->hdr[H_MAX_VIS], max_nq, c.kv_capacity_tokens, hq, hkv, dh,
                           nullptr, 0, st.hdr + H_ERROR, s));
    // every query token of a row meets every cache row of that row: flops = 4 * dh * Hq * sum_rows(n_q * vis);
    // the host knows the sums only for pure block steps and pure refresh steps, else it reports bytes alone
    prof_work(e, attn_fam, 1, 0, 2.0 * (2.0 * kv_rows * hkv * dh + 2.0 * dM * dhq));
    prof_mark(e, BS_FAM_GEMM_O);
    KL(e, launch_gemm(ws.attn, hq * dh, e->wo[l], nullptr, ws.x, d, M, d, hq * dh, 1, nullptr, e->gemm_scratch, s));
    prof_work(e, BS_FAM_GEMM_O, 1, 2.0 * dM * dd * dhq, 2.0 * (dd * dhq + dM * dhq) + 8.0 * dM * dd);
    for (long long c0 = 0; c0 < M; c0 += kMlpChunk) {
      const int mc = (int)std::min<long long>(kMlpChunk, M - c0);
      const double dmc = (double)mc;
      float* xc = ws.x + (size_t)c0 * d;
      prof_mark(e, BS_FAM_EMBED_NORM);
      KL(e, launch_rmsnorm(xc, nullptr, e->norm2[l], ws.h, mc, d, c.rms_eps, s));
      prof_work(e, BS_FAM_EMBED_NORM, 1, 0, 6.0 * dmc * dd);
      prof_mark(e, BS_FAM_GEMM_GATE_UP);
      KL(e, launch_gemm(ws.h, d, e->w_gate[l], e->w_up[l], ws.act, c.d_ffn, mc, c.d_ffn, d, 3, nullptr, e->gemm_scratch, s));
      prof_work(e, BS_FAM_GEMM_GATE_UP, 1, 4.0 * dmc * df * dd, 2.0 * (2.0 * df * dd + dmc * dd + dmc * df));
      prof_mark(e, BS_FAM_GEMM_DOWN);
      KL(e, launch_gemm(ws.act, c.d_ffn, e->w_down[l], nullptr, xc, d, mc, d, c.d_ffn, 1, nullptr, e->gemm_scratch, s));
      prof_work(e, BS_FAM_GEMM_DOWN, 1, 2.0 * dmc * dd * df, 2.0 * (dd * df + dmc * df) + 8.0 * dmc * dd);
    }
  }
  // final norm on the still-masked rows only, LM head scaled by alpha_i, confidence / argmax, commit
  const double dMm = (double)Mm, dV = (double)c.vocab;
  prof_mark(e, BS_FAM_EMBED_NORM);
  KL(e, launch_rmsnorm(ws.x, st.lm_tok[parity], e->final_norm, ws.hf, Mm, d, c.rms_eps, s, &lim));
  prof_work(e, BS_FAM_EMBED_NORM, 1, 0, 6.0 * dMm * dd);
  // LM head with the confidence pass in its epilogue: per (32 vocabulary entries, row) maximum / sum of exponentials
  // / argmax of the alpha-scaled logits, merged per row in two small stages (the second one inside the commit
  // kernel); the fp32 logits reach HBM only when the engine was configured to keep them for the parity hooks.
  prof_mark(e, BS_FAM_GEMM_LM_HEAD);
  GemmConf groups{ws.group_ms, ws.group_am, c.mask_id};
  KL(e, launch_gemm_tc(ws.hf, d, e->lm_head, nullptr, ws.logits, c.vocab, Mm, c.vocab, d, 5, st.lm_scale[parity],
                       e->gemm_scratch, s, nullptr, &groups));
  prof_work(e, BS_FAM_GEMM_LM_HEAD, 1, 2.0 * dMm * dV * dd,
            2.0 * (dV * dd + dMm * dd) + 12.0 * dMm * (dV / 32.0) + (ws.logits ? 4.0 * dMm * dV : 0.0));
  prof_mark(e, BS_FAM_CONFIDENCE);
  KL(e, launch_conf_merge(groups, Mm, c.vocab, ws.slice_ms, ws.slice_am, s));
  prof_work(e, BS_FAM_CONFIDENCE, 1, 0, 12.0 * dMm * (dV / 32.0));
  prof_mark(e, BS_FAM_INDEX);
  KL(e, launch_commit_index(st, s));
  prof_work(e, BS_FAM_INDEX, 1, 0, 0);
  prof_mark(e, -1);
  if (int rc = post_header(e, true)) return rc;
  e->stats.steps++;
  e->stats.packed_tokens += M;
  e->stats.lm_rows += Mm;
  if (n_committed) {
    if (int rc = sync_header(e)) return rc;
    *n_committed = e->hdr[H_COMMITTED_STEP];
  }
  return BS_OK;
}

int bs_block_done(bs_engine* e, int* all_done, unsigned char* per_row_done) {
  if (!e) return BS_E_ARG;
  if (int rc = sync_header(e)) return rc;
  if (all_done) *all_done = e->hdr[H_ALL_DONE] ? 1 : 0;
  if (per_row_done) {
    const MaskWord* masks = reinterpret_cast<const MaskWord*>(e->pinned + kHdrInts);
    for (int i = 0; i < e->cfg.max_batch; ++i) per_row_done[i] = (i < e->hdr[H_N_ACTIVE]) ? (masks[i] == 0ull) : 1;
  }
  return BS_OK;
}

int bs_read_tokens(bs_engine* e, long long req_id, int* out, int cap, int* n_valid, int* state) {
  if (!e) return BS_E_ARG;
  auto it = e->slot_of.find(req_id);
  if (it == e->slot_of.end()) return fail(e, BS_E_UNKNOWN_REQ, "unknown request id");
  const int slot = it->second, n = e->h_p[slot] + e->h_g[slot];
  if (n_valid) *n_valid = n;
  if (out && cap < n) return fail(e, BS_E_ARG, "output buffer too small");
  if (int rc = sync_header(e)) return rc;
  if (out)
    CU(e, cudaMemcpyAsync(out, e->st.tokens + (size_t)slot * e->cfg.max_row_tokens, (size_t)n * 4,
                          cudaMemcpyDeviceToHost, e->stream));
  int stt = BS_REQ_QUEUED;
  if (slot < e->uploaded_slots)
    CU(e, cudaMemcpyAsync(&stt, e->st.req_state + slot, 4, cudaMemcpyDeviceToHost, e->stream));
  CU(e, cudaStreamSynchronize(e->stream));
  if (state) *state = stt;
  return BS_OK;
}

int bs_get_stats(bs_engine* e, bs_stats* out) {
  if (!e || !out) return BS_E_ARG;
  if (int rc = sync_header(e)) return rc;
  e->stats.committed = ((long long)(unsigned)e->hdr[H_TOTAL_HI] << 32) | (unsigned)e->hdr[H_TOTAL_LO];
  *out = e->stats;
  return BS_OK;
}

int bs_set_profiling(bs_engine* e, int on) {
  if (!e) return BS_E_ARG;
  if (int rc = sync_header(e)) return rc;
  CU(e, cudaStreamSynchronize(e->stream));
  e->profiling = on != 0;
  e->spans.clear();
  e->ev_used = 0;
  e->cur_fam = -1;
  if (on)
    for (int i = 0; i < BS_FAM_COUNT; ++i) e->prof_ms[i] = e->prof_flops[i] = e->prof_bytes[i] = 0.0, e->prof_launches[i] = 0;
  return BS_OK;
}

int bs_get_profile(bs_engine* e, double* ms, long long* launches, double* flops, double* bytes) {
  if (!e) return BS_E_ARG;
  if (int rc = sync_header(e)) return rc;
  for (int i = 0; i < BS_FAM_COUNT; ++i) {
    if (ms) ms[i] = e->prof_ms[i];
    if (launches) launches[i] = e->prof_launches[i];
    if (flops) flops[i] = e->prof_flops[i];
    if (bytes) bytes[i] = e->prof_bytes[i];
  }
  return BS_OK;
}

void bs_destroy(bs_engine* e) {
  if (!e) return;
  cudaStreamSynchronize(e->stream);
  for (cudaEvent_t ev : e->ev_pool) cudaEventDestroy(ev);
  if (e->pinned) cudaFreeHost(e->pinned);
  if (e->ev) cudaEventDestroy(e->ev);
  delete e;
}

const char* bs_last_error(const bs_engine* e) { return e ? e->err.c_str() : g_init_error.c_str(); }

int bs_build_flags(void) { return kBoundsCheck ? BS_BUILD_BOUNDS_CHECK : 0; }

int bs_debug_read(bs_engine* e, int what, int arg0, int arg1, void* host_buf, size_t cap, size_t* n_out) {
  if (!e || !host_buf) return BS_E_ARG;
  if (int rc = sync_header(e)) return rc;
  CU(e, cudaStreamSynchronize(e->stream));
  DevState& st = e->st;
  const int n = e->hdr[H_N_ACTIVE], par = e->hdr[H_PARITY], prev = par ^ 1;
  const void* src = nullptr;
  size_t bytes = 0;
  std::vector<long long> ids;
  const int prev_mm = e->hdr[H_PREV_MM];     // length of the lists of the step that just ran
  switch (what) {
    case BS_DBG_HEADER: src = st.hdr; bytes = kHdrInts * 4; break;
    case BS_DBG_ROW_SLOT: src = st.row_slot; bytes = n * 4; break;
    case BS_DBG_ROW_MASK: src = st.row_mask; bytes = n * sizeof(MaskWord); break;
    case BS_DBG_ROW_S: src = st.row_s; bytes = n * 4; break;
    case BS_DBG_ROW_KV_BASE: src = st.row_kv_base; bytes = n * 4; break;
    case BS_DBG_CU_Q: src = st.cu_q[par]; bytes = (n + 1) * 4; break;
    case BS_DBG_TOK_ROW: src = st.tok_row; bytes = (size_t)arg0 * 4; break;
    case BS_DBG_TOK_POS: src = st.tok_pos; bytes = (size_t)arg0 * 4; break;
    case BS_DBG_TOK_KV: src = st.tok_kv; bytes = (size_t)arg0 * 4; break;
    case BS_DBG_LM_TOK: src = st.lm_tok[par]; bytes = (size_t)e->hdr[H_MM] * 4; break;
    case BS_DBG_LM_ROW: src = st.lm_row[par]; bytes = (size_t)e->hdr[H_MM] * 4; break;
    case BS_DBG_LM_SLOT: src = st.lm_slot[par]; bytes = (size_t)e->hdr[H_MM] * 4; break;
    case BS_DBG_PREV_LM_ROW: src = st.lm_row[prev]; bytes = (size_t)prev_mm * 4; break;
    case BS_DBG_PREV_LM_SLOT: src = st.lm_slot[prev]; bytes = (size_t)prev_mm * 4; break;
    case BS_DBG_PREV_TOK: src = st.out_tok[prev]; bytes = (size_t)prev_mm * 4; break;
    case BS_DBG_PREV_CONF: src = st.out_conf[prev]; bytes = (size_t)prev_mm * 4; break;
    case BS_DBG_PREV_COMMIT: src = st.out_commit[prev]; bytes = (size_t)prev_mm * 4; break;
    case BS_DBG_PREV_LOGITS: {   // arg0 = first masked row, arg1 = number of rows (0: all rows from arg0)
      if (!e->ws.logits) return fail(e, BS_E_STATE, "the engine was created without keep_logits");
      if (arg0 < 0 || arg0 > prev_mm || arg1 < 0 || arg0 + arg1 > prev_mm) return fail(e, BS_E_ARG, "bad logit rows");
      const int rows = arg1 > 0 ? arg1 : prev_mm - arg0;
      src = e->ws.logits + (size_t)arg0 * e->cfg.vocab;
      bytes = (size_t)rows * e->cfg.vocab * 4;
      break;
    }
    case BS_DBG_REQ_ID_OF_ROW: {
      std::vector<int> slots(n);
      if (n) CU(e, cudaMemcpy(slots.data(), st.row_slot, n * 4, cudaMemcpyDeviceToHost));
      ids.resize(n);
      for (int i = 0; i < n; ++i) ids[i] = e->id_of_slot[slots[i]];
      bytes = (size_t)n * 8;
      if (bytes > cap) return fail(e, BS_E_ARG, "debug buffer too small");
      memcpy(host_buf, ids.data(), bytes);
      if (n_out) *n_out = bytes;
      return BS_OK;
    }
    case BS_DBG_KV_ROW: {
      if (arg0 < 0 || arg0 >= e->cfg.n_layers || arg1 < 0 || arg1 >= e->cfg.kv_capacity_tokens)
        return fail(e, BS_E_ARG, "bad layer / row");
      const size_t rowe = (size_t)e->cfg.n_kv_heads * e->cfg.head_dim;
      bytes = 2 * rowe * sizeof(bf16);
      if (bytes > cap) return fail(e, BS_E_ARG, "debug buffer too small");
      const bf16* kc = e->kv + (size_t)arg0 * e->kv_layer_stride + (size_t)arg1 * rowe;
      CU(e, cudaMemcpy(host_buf, kc, rowe * sizeof(bf16), cudaMemcpyDeviceToHost));
      CU(e, cudaMemcpy((char*)host_buf + rowe * sizeof(bf16), kc + e->kv_half, rowe * sizeof(bf16), cudaMemcpyDeviceToHost));
      if (n_out) *n_out = bytes;
      return BS_OK;
    }
    default: return fail(e, BS_E_ARG, "unknown debug selector");
  }
  if (bytes > cap) return fail(e, BS_E_ARG, "debug buffer too small");
  if (bytes) CU(e, cudaMemcpy(host_buf, src, bytes, cudaMemcpyDeviceToHost));
  if (n_out) *n_out = bytes;
  return BS_OK;
}

int bs_debug_force_commit(bs_engine* e, int row, unsigned long long mask_bits, const int* tokens) {
  if (!e || !tokens) return BS_E_ARG;
  if (int rc = sync_header(e)) return rc;
  if (row < 0 || row >= e->hdr[H_N_ACTIVE]) return fail(e, BS_E_ARG, "row is not an active row");
  const int L = e->cfg.block_len;
  if (L < kMaxBlockLen && (mask_bits >> L) != 0ull) return fail(e, BS_E_ARG, "bit beyond the block length");
  int toks[kMaxBlockLen] = {0};
  for (int j = 0; j < kMaxBlockLen; ++j)
    if ((mask_bits >> j) & 1ull) {
      if (tokens[j] < 0 || tokens[j] >= e->cfg.vocab || tokens[j] == e->cfg.mask_id)
        return fail(e, BS_E_ARG, "token id out of range");
      toks[j] = tokens[j];
    }
  KL(e, launch_force_commit(e->st, row, mask_bits, toks, e->stream));
  return post_header(e);
}

namespace {
struct SnapHeader {
  unsigned long long magic;
  unsigned long long total_bytes, state_bytes;
  unsigned long long n_slots, n_pending, uploaded_slots;
  bs_config cfg;
  bs_stats stats;
  int hdr[kHdrInts];
};
constexpr unsigned long long kSnapMagic = 0x31304e5353424c42ull;   // "BLBSSN01"
size_t snapshot_bytes(const bs_engine* e) {
  const size_t n = e->id_of_slot.size();
  return sizeof(SnapHeader) + n * (sizeof(long long) + 3 * sizeof(int) + sizeof(float)) +
         e->pending.size() * sizeof(int) + e->state_bytes;
}
}  // namespace

int bs_debug_snapshot(bs_engine* e, void* host_buf, size_t cap, size_t* n_out) {
  if (!e || !n_out) return BS_E_ARG;
  if (int rc = sync_header(e)) return rc;
  const size_t need = snapshot_bytes(e);
  *n_out = need;
  if (!host_buf) return BS_OK;                      // size query
  if (cap < need) return fail(e, BS_E_ARG, "snapshot buffer too small");
  // The KV cache is not saved: it is rebuilt from the tokens at the first step of every block, so the state is
  // complete only between block cycles.
  if (e->hdr[H_N_ACTIVE] > 0 && !e->hdr[H_ALL_DONE])
    return fail(e, BS_E_STATE, "snapshots are taken between block cycles");
  if (e->cfg.refresh_policy != BS_REFRESH_EVERY_BLOCK && e->hdr[H_N_ACTIVE] > 0)
    return fail(e, BS_E_STATE, "without a refresh at every block start the KV cache is part of the state");
  CU(e, cudaStreamSynchronize(e->stream));
  char* out = static_cast<char*>(host_buf);
  SnapHeader h;
  memset(&h, 0, sizeof(h));
  h.magic = kSnapMagic;
  h.total_bytes = need;
  h.state_bytes = e->state_bytes;
  h.n_slots = e->id_of_slot.size();
  h.n_pending = e->pending.size();
  h.uploaded_slots = (unsigned long long)e->uploaded_slots;
  h.cfg = e->cfg;
  h.stats = e->stats;
  memcpy(h.hdr, e->hdr, sizeof(h.hdr));
  memcpy(out, &h, sizeof(h)); out += sizeof(h);
  const size_t n = h.n_slots;
  auto put = [&](const void* src, size_t bytes) { if (bytes) memcpy(out, src, bytes); out += bytes; };
  put(e->id_of_slot.data(), n * sizeof(long long));
  put(e->h_p.data(), n * sizeof(int));
  put(e->h_g.data(), n * sizeof(int));
  put(e->h_b.data(), n * sizeof(int));
  put(e->h_alpha.data(), n * sizeof(float));
  put(e->pending.data(), h.n_pending * sizeof(int));
  CU(e, cudaMemcpy(out, e->state_base, e->state_bytes, cudaMemcpyDeviceToHost));
  return BS_OK;
}

int bs_debug_restore(bs_engine* e, const void* host_buf, size_t n_bytes) {
  if (!e || !host_buf) return BS_E_ARG;
  if (int rc = sync_header(e)) return rc;
  if (n_bytes < sizeof(SnapHeader)) return fail(e, BS_E_ARG, "not a snapshot");
  const char* in = static_cast<const char*>(host_buf);
  SnapHeader h;
  memcpy(&h, in, sizeof(h)); in += sizeof(h);
  if (h.magic != kSnapMagic || h.total_bytes != n_bytes) return fail(e, BS_E_ARG, "not a snapshot");
  if (memcmp(&h.cfg, &e->cfg, sizeof(bs_config)) != 0 || h.state_bytes != e->state_bytes)
    return fail(e, BS_E_ARG, "snapshot of an engine with another configuration");
  const size_t n = h.n_slots;
  if (n > (size_t)e->cfg.max_requests || h.n_pending > n || h.uploaded_slots > n ||
      sizeof(SnapHeader) + n * (sizeof(long long) + 3 * sizeof(int) + sizeof(float)) + h.n_pending * sizeof(int) +
              h.state_bytes != n_bytes)
    return fail(e, BS_E_ARG, "snapshot sizes are inconsistent");
  CU(e, cudaStreamSynchronize(e->stream));
  auto get = [&](void* dst, size_t bytes) { if (bytes) memcpy(dst, in, bytes); in += bytes; };
  e->id_of_slot.resize(n); e->h_p.resize(n); e->h_g.resize(n); e->h_b.resize(n); e->h_alpha.resize(n);
  e->pending.resize(h.n_pending);
  get(e->id_of_slot.data(), n * sizeof(long long));
  get(e->h_p.data(), n * sizeof(int));
  get(e->h_g.data(), n * sizeof(int));
  get(e->h_b.data(), n * sizeof(int));
  get(e->h_alpha.data(), n * sizeof(float));
  get(e->pending.data(), h.n_pending * sizeof(int));
  e->slot_of.clear();
  for (size_t i = 0; i < n; ++i) e->slot_of[e->id_of_slot[i]] = (int)i;
  e->uploaded_slots = (int)h.uploaded_slots;
  e->stats = h.stats;
  memcpy(e->hdr, h.hdr, sizeof(e->hdr));
  e->hdr_pending = false;
  CU(e, cudaMemcpy(e->state_base, in, e->state_bytes, cudaMemcpyHostToDevice));
  return BS_OK;
}

// A wait that nothing ever satisfies, with a short limit: the same bounded-wait helper pattern the tensor-core
// kernels use.  It runs out after about a millisecond, raises the engine's error word and returns.
__global__ void k_wait_that_runs_out(int* error_word, long long limit_cycles) {
  __shared__ __align__(8) unsigned long long bar;
  const unsigned addr = (unsigned)__cvta_generic_to_shared(&bar);
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(addr));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const long long t0 = clock64();
    bool done = false;
    while (!done) {
      unsigned ok;
      asm volatile(
          "{\n\t.reg .pred p;\n\t"
          "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
          "selp.u32 %0, 1, 0, p;\n\t}"
          : "=r"(ok) : "r"(addr), "r"(0u) : "memory");
      if (ok) done = true;
      else if (clock64() - t0 > limit_cycles) {
        atomicExch(error_word, 1);
        done = true;
      }
    }
  }
}

int bs_debug_inject_timeout(bs_engine* e) {
  if (!e) return BS_E_ARG;
  k_wait_that_runs_out<<<1, 32, 0, e->stream>>>(e->st.hdr + H_ERROR, 2000000ll);
  e->stats.kernel_launches++;
  return cudaGetLastError() == cudaSuccess ? BS_OK : BS_E_CUDA;
}

// ---- single operations ----------------------------------------------------------------------------------

int bs_op_gemm(const void* A, int lda, const void* W, const void* W2, void* C, int ldc, int M, int N, int K, int mode,
               const float* row_scale, float* scratch, size_t scratch_bytes, int* error_flag, void* stream) {
  if (M == 0) return BS_OK;
  if (!A || !W || !C || M < 0 || N < 1 || K < 8 || K % 8 || N % 2 || mode < 0 || mode > 3) return BS_E_ARG;
  if (mode == 3 && !W2) return BS_E_ARG;
  if (mode == 2 && !row_scale) return BS_E_ARG;
  if (lda % 8 || (((uintptr_t)A | (uintptr_t)W | (uintptr_t)W2) & 15)) return BS_E_ARG;
  GemmScratch sc;
  sc.partial = scratch;
  sc.partial_floats = scratch ? scratch_bytes / sizeof(float) : 0;
  sc.error_flag = error_flag;
  cudaError_t r = launch_gemm((const bf16*)A, lda, (const bf16*)W, (const bf16*)W2, C, ldc, M, N, K, mode, row_scale,
                              sc, (cudaStream_t)stream);
  return r == cudaSuccess ? BS_OK : (r == cudaErrorNotSupported ? BS_E_ARG : BS_E_CUDA);
}

int bs_op_gemm_cluster_splits(int M, int N, int K, int mode) {
  if (M < 0 || N < 1 || K < 8) return 0;
  return gemm_cluster_splits(M, N, K, mode, N, nullptr);
}

int bs_op_rmsnorm(const float* x, const int* idx, const void* w, void* y, int M, int d, float eps, void* stream) {
  if (!x || !w || !y || M < 0 || d < 8 || d % 8) return BS_E_ARG;
  return launch_rmsnorm(x, idx, (const bf16*)w, (bf16*)y, M, d, eps, (cudaStream_t)stream) == cudaSuccess ? BS_OK
                                                                                                          : BS_E_CUDA;
}

int bs_op_rope_kv(void* qkv, const int* tok_pos, const int* tok_kv, void* kcache, void* vcache, int M, int n_q_heads,
                  int n_kv_heads, int head_dim, float theta, int max_pos, float* table_scratch, void* stream) {
  if (!qkv || !tok_pos || !tok_kv || !kcache || !vcache || !table_scratch || M < 0 || head_dim % 8 || max_pos < 1)
    return BS_E_ARG;
  std::vector<float> tab((size_t)max_pos * head_dim);
  build_rope_table(tab.data(), max_pos, head_dim, theta);
  cudaStream_t s = (cudaStream_t)stream;
  if (cudaMemcpyAsync(table_scratch, tab.data(), tab.size() * 4, cudaMemcpyHostToDevice, s) != cudaSuccess)
    return BS_E_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return BS_E_CUDA;
  return launch_rope_kv((bf16*)qkv, tok_pos, tok_kv, (bf16*)kcache, (bf16*)vcache, M, n_q_heads, n_kv_heads, head_dim,
                        table_scratch, s) == cudaSuccess ? BS_OK : BS_E_CUDA;
}

int bs_op_attention_q_tile(int n_q_heads, int n_kv_heads, int head_dim) {
  if (n_kv_heads < 1 || n_q_heads % n_kv_heads) return BS_E_ARG;
  return attention_q_tile(n_q_heads, n_kv_heads, head_dim);
}

int bs_op_attention(const void* qkv, const void* kcache, const void* vcache, void* out, const int* cu_q,
                    const int* cu_tile, const int* kv_base, const int* vis, int n_rows, int n_tiles, int M,
                    int max_vis, int max_nq, long long kv_rows, int n_q_heads, int n_kv_heads, int head_dim,
                    float* scratch, size_t scratch_bytes, int* error_flag, void* stream) {
  if (!qkv || !kcache || !vcache || !out || !cu_q || !cu_tile || !kv_base || !vis || kv_rows < 1) return BS_E_ARG;
  return launch_attention((const bf16*)qkv, (const bf16*)kcache, (const bf16*)vcache, (bf16*)out, cu_q, cu_tile,
                          kv_base, vis, n_rows, n_tiles, M, max_vis, max_nq, kv_rows, n_q_heads, n_kv_heads, head_dim,
                          scratch, scratch ? scratch_bytes / sizeof(float) : 0, error_flag,
                          (cudaStream_t)stream) == cudaSuccess
             ? BS_OK : BS_E_CUDA;
}

size_t bs_op_lm_head_confidence_scratch_bytes(int M, int vocab) {
  if (M < 0 || vocab < 1) return 0;
  const size_t parts = ((size_t)vocab + 31) / 32 + kConfSlices;
  return align_up(parts * (size_t)M * sizeof(float2)) + align_up(parts * (size_t)M * sizeof(int));
}

int bs_op_lm_head_confidence(const void* hf, int lda, const void* W, int M, int vocab, int K, const float* row_scale,
                             int mask_id, void* scratch, size_t scratch_bytes, int* tok, float* conf, float* logits,
                             int* error_flag, void* stream) {
  if (M == 0) return BS_OK;
  if (!hf || !W || !row_scale || !scratch || !tok || !conf || M < 0 || vocab < 2 || K < 8 || K % 8 || lda % 8)
    return BS_E_ARG;
  if ((((uintptr_t)hf | (uintptr_t)W) & 15) || ((uintptr_t)scratch & 255)) return BS_E_ARG;
  if (scratch_bytes < bs_op_lm_head_confidence_scratch_bytes(M, vocab)) return BS_E_ARG;
  const size_t n_groups = ((size_t)vocab + 31) / 32, parts = n_groups + kConfSlices;
  float2* ms = static_cast<float2*>(scratch);
  int* am = reinterpret_cast<int*>(static_cast<char*>(scratch) + align_up(parts * (size_t)M * sizeof(float2)));
  GemmConf groups{ms, am, mask_id};
  float2* slice_ms = ms + n_groups * (size_t)M;
  int* slice_am = am + n_groups * (size_t)M;
  GemmScratch sc;
  sc.error_flag = error_flag;
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t r = launch_lm_head_conf((const bf16*)hf, lda, (const bf16*)W, M, vocab, K, row_scale, mask_id, groups,
                                      slice_ms, slice_am, logits, sc, s);
  if (r == cudaSuccess) r = launch_conf_final(slice_ms, slice_am, M, tok, conf, s);
  return r == cudaSuccess ? BS_OK : (r == cudaErrorNotSupported ? BS_E_ARG : BS_E_CUDA);
}

int bs_op_confidence(const float* logits, int n_rows, int vocab, int mask_id, int* tok, float* conf, void* stream) {
  if (!logits || !tok || !conf || n_rows < 0 || vocab < 2) return BS_E_ARG;
  return launch_confidence(logits, n_rows, vocab, mask_id, tok, conf, (cudaStream_t)stream) == cudaSuccess ? BS_OK
                                                                                                           : BS_E_CUDA;
}

}  // extern "C"
