// Scheduling and gather/scatter index kernels (integer work, single CTA):
//   k_sched        - Algorithm 1's block boundary: advance, evict, stable compaction, refill under Eq. 1
//   k_commit_index - confidence-thresholded commit per request + block-done flags + next step's indices
//   k_fill_tokens  - per packed token: row, logical position id, physical KV row (Section 2.5)
#include "conf_merge.cuh"

namespace bs {

constexpr int kSchedThreads = 1024;

__device__ __forceinline__ int warp_incl_scan(int v) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += t;
  }
  return v;
}

// Exclusive prefix sum over the block (blockDim.x == 1024).  sm: int[33].
__device__ int block_excl_scan(int v, int* total, int* sm) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  int inc = warp_incl_scan(v);
  if (lane == 31) sm[w] = inc;
  __syncthreads();
  if (w == 0) {
    int x = sm[lane];
    int xi = warp_incl_scan(x);
    sm[lane] = xi - x;
    if (lane == 31) sm[32] = xi;
  }
  __syncthreads();
  int r = inc - v + sm[w];
  *total = sm[32];
  __syncthreads();
  return r;
}

__device__ long long block_max_ll(long long v, long long* sm) {   // sm: long long[33]
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    long long t = __shfl_xor_sync(0xffffffffu, v, o);
    v = t > v ? t : v;
  }
  if (lane == 0) sm[w] = v;
  __syncthreads();
  if (w == 0) {
    long long x = sm[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      long long t = __shfl_xor_sync(0xffffffffu, x, o);
      x = t > x ? t : x;
    }
    if (lane == 0) sm[32] = x;
  }
  __syncthreads();
  long long r = sm[32];
  __syncthreads();
  return r;
}

// Index header of the step about to run, for the rows of A in order (all threads of the CTA call this).
__device__ void build_index(const DevState& st, int parity, int n, int* smi) {
  const int i = threadIdx.x;
  int nq = 0, nm = 0, vis = 0, unfinished = 0, refresh = 0;
  if (i < n) {
    const int slot = st.row_slot[i];
    const int p = st.req_p[slot], g = st.req_g[slot], b = st.req_b[slot];
    const int s = st.row_s[i];
    const MaskWord mask = st.row_mask[i];
    const int lo = p + b * st.L;
    const int hi = min(lo + st.L, p + g);
    vis = st.suffix_mode == 0 ? p + g : hi;
    st.row_vis[i] = vis;
    if (mask != 0ull) {
      refresh = (s == 0 && st.row_refresh[i] != 0);
      nq = refresh ? vis : hi - lo;
      unfinished = 1;
    }
    nm = __popcll(mask);
  }
  int tot_q, tot_m, tot_t, tot_u, tot_r;
  const int eq = block_excl_scan(nq, &tot_q, smi);
  const int em = block_excl_scan(nm, &tot_m, smi);
  const int et = block_excl_scan((nq + st.q_tile - 1) / st.q_tile, &tot_t, smi);
  block_excl_scan(unfinished, &tot_u, smi);
  block_excl_scan(refresh, &tot_r, smi);
  int tot_kv;
  block_excl_scan(unfinished ? vis : 0, &tot_kv, smi);
  __shared__ long long sm_max[33];
  const int max_vis = (int)block_max_ll(unfinished ? vis : 0, sm_max);
  if (i < n) {
    st.cu_q[parity][i] = eq;
    st.lm_base[parity][i] = em;
    st.cu_tile[parity][i] = et;
  }
  if (i == 0) {
    (void)BS_INDEX_OK(tot_q <= st.kv_capacity && tot_m <= st.max_batch * st.L && n <= st.max_batch, st.hdr + H_ERROR,
                      SITE_INDEX);
    st.cu_q[parity][n] = tot_q;
    st.lm_base[parity][n] = tot_m;
    st.cu_tile[parity][n] = tot_t;
    st.hdr[H_M] = tot_q;
    st.hdr[H_MM] = tot_m;
    st.hdr[H_QTILES] = tot_t;
    st.hdr[H_ALL_DONE] = (tot_m == 0);
    st.hdr[H_UNFINISHED] = tot_u;
    st.hdr[H_STEP_REFRESH] = tot_r;
    st.hdr[H_SUM_KV] = tot_kv;
    st.hdr[H_MAX_VIS] = max_vis;
    st.hdr[H_PARITY] = parity;
  }
  __syncthreads();
  // still-masked block positions, row order then position order
  const int lane = threadIdx.x & 31;
  for (int r = threadIdx.x >> 5; r < n; r += kSchedThreads / 32) {
    const MaskWord mask = st.row_mask[r];
    if (mask == 0ull) continue;
#pragma unroll
    for (int j = lane; j < kMaxBlockLen; j += 32) {     // a lane looks after block positions lane and lane + 32
      if ((mask >> j) & 1ull) {
        const int slot = st.row_slot[r];
        const int lo = st.req_p[slot] + st.req_b[slot] * st.L;
        const int k = st.lm_base[parity][r] + __popcll(mask & ((1ull << j) - 1ull));
        if (!BS_INDEX_OK(k >= 0 && k < st.max_batch * st.L && slot >= 0 && slot < st.max_requests, st.hdr + H_ERROR,
                         SITE_INDEX))
          continue;
        st.lm_tok[parity][k] = st.cu_q[parity][r] + ((st.row_s[r] == 0 && st.row_refresh[r] != 0) ? lo + j : j);
        st.lm_row[parity][k] = r;
        st.lm_slot[parity][k] = j;
        st.lm_scale[parity][k] = st.req_alpha[slot];
      }
    }
  }
}

// Algorithm 1's block boundary for the rows of A (all threads of the CTA call this): advance, evict, stable
// compaction, refill under Eq. 1, new blocks fully masked, index of the next step.
//   only_done = false: the synchronous cycle - every active row advances by one block.
//   only_done = true:  per-row advance (the straggler stall of Section 2.3 relaxed), run after every denoise step -
//                      only rows whose block is complete advance or leave; the others keep their block, step counter
//                      and mask word and merely move up when rows before them leave.
__device__ void sched_body(const DevState& st, bool only_done) {
  __shared__ int smi[33];
  __shared__ long long sml[33];
  __shared__ int s_n, s_head, s_stop;
  __shared__ long long s_w;
  const int i = threadIdx.x;
  const int n0 = st.hdr[H_N_ACTIVE];
  const int L = st.L;

  // ---- advance, evict finished rows (b_i >= K_i or CheckEOS), compact (order preserved) ----
  int keep = 0, slot = -1, kvb = 0, srow = 0, rfr = 0;
  MaskWord mask = 0ull;
  if (i < n0) {
    slot = st.row_slot[i];
    kvb = st.row_kv_base[i];
    mask = st.row_mask[i];
    srow = st.row_s[i];
    rfr = st.row_refresh[i];
    if (only_done && mask != 0ull) {
      keep = 1;                                            // mid-block: nothing changes for this row
    } else {
      const int b = st.req_b[slot] + 1;
      st.req_b[slot] = b;
      const int K = (st.req_g[slot] + L - 1) / L;          // K_i = ceil(g_i / L)
      keep = b < K;
      if (keep && st.eos_id >= 0) {                        // CheckEOS over the blocks finished so far
        const int p = st.req_p[slot];
        const int* row = st.tokens + (size_t)slot * st.max_row_tokens;
        const int upto = min(p + b * L, p + st.req_g[slot]);
        for (int t = p; t < upto; ++t)
          if (row[t] == st.eos_id) { keep = 0; break; }
      }
      if (!keep) st.req_state[slot] = 2;
      srow = -1;                                           // marks "starts a block now"
      rfr = st.refresh_policy == 0;                        // later blocks are refreshed only under the default policy
    }
  }
  int n_keep;
  const int dst = block_excl_scan(keep, &n_keep, smi);
  if (keep) {
    st.row_slot[dst] = slot;
    st.row_kv_base[dst] = kvb;
    st.row_mask[dst] = mask;
    st.row_s[dst] = srow;
    st.row_refresh[dst] = rfr;
  }
  __syncthreads();

  // ---- width of the bounding box over survivors: max_i p_i + (b_i + 1) L ----
  long long w = 0;
  if (i < n_keep) {
    const int sl = st.row_slot[i];
    w = (long long)st.req_p[sl] + (long long)(st.req_b[sl] + 1) * L;
  }
  w = block_max_ll(w, sml);
  if (i == 0) {
    s_n = n_keep;
    s_head = st.hdr[H_QUEUE_HEAD];
    s_w = w;
    s_stop = (st.static_groups && n_keep > 0) ? 1 : 0;    // static groups refill only an empty batch
  }
  __syncthreads();

  // ---- refill: admit the head of P while Eq. 1 holds, the cap holds and the arena has a hole ----
  const int qlen = st.hdr[H_QUEUE_LEN];
  while (true) {
    const int n = s_n, head = s_head;
    if (s_stop || head >= qlen || n >= st.max_batch) break;
    const int c = st.queue[head];
    if (!BS_INDEX_OK(c >= 0 && c < st.max_requests, st.hdr + H_ERROR, SITE_SCHED)) break;     // (uniform: all threads read c)
    const long long wc = (long long)st.req_p[c] + (long long)(st.req_b[c] + 1) * L;
    const long long w2 = wc > s_w ? wc : s_w;
    const long long need = (long long)st.req_p[c] + st.req_g[c];
    bool ok = !(st.beta > 0 && (long long)(n + 1) * w2 > st.beta);
    long long start = 0;
    if (ok) {   // lowest-address first fit: jump past the furthest slab that overlaps [start, start + need)
      long long my_b = -1, my_e = -1;
      if (i < n) {
        const int sl = st.row_slot[i];
        my_b = st.row_kv_base[i];
        my_e = my_b + st.req_p[sl] + st.req_g[sl];
      }
      for (int it = 0; it <= n; ++it) {
        long long e = (i < n && my_b < start + need && my_e > start) ? my_e : -1;
        e = block_max_ll(e, sml);
        if (e < 0) break;
        start = e;
      }
      ok = start + need <= st.kv_capacity;
    }
    __syncthreads();
    if (i == 0) {
      if (ok) {
        st.row_slot[n] = c;
        st.row_kv_base[n] = (int)start;
        st.row_s[n] = -1;
        st.row_refresh[n] = 1;                             // a newly admitted row has no cache yet
        st.req_state[c] = 1;
        s_n = n + 1;
        s_head = head + 1;
        s_w = w2;
      } else {
        s_stop = 1;
      }
    }
    __syncthreads();
  }
  const int n = s_n;
  // ---- rows that start a block (advanced or admitted) begin it fully masked ----
  if (i < n && st.row_s[i] < 0) {
    const int sl = st.row_slot[i];
    const int lo = st.req_p[sl] + st.req_b[sl] * L;
    const int len = min(L, st.req_p[sl] + st.req_g[sl] - lo);
    st.row_mask[i] = len >= 64 ? ~0ull : ((1ull << len) - 1ull);
    st.row_s[i] = 0;
  }
  if (i == 0) {
    st.hdr[H_N_ACTIVE] = n;
    st.hdr[H_EVICTED] = n0 - n_keep;
    st.hdr[H_ADMITTED] = n - n_keep;
    st.hdr[H_QUEUE_HEAD] = s_head;
    st.hdr[H_WIDTH] = (int)s_w;
    if (!only_done) st.hdr[H_COMMITTED_STEP] = 0;
  }
  __syncthreads();
  build_index(st, st.hdr[H_PARITY] ^ 1, n, smi);
}

__global__ void __launch_bounds__(kSchedThreads) k_sched(DevState st) {
  pdl_wait();
  pdl_trigger();
  sched_body(st, false);
}

// Commit rule per request (one warp per row): positions with conf > tau, plus the step's quota of most confident
// positions (lower position first on ties), so that every step commits at least its quota (one when S = L).
__global__ void __launch_bounds__(kSchedThreads) k_commit_index(DevState st) {
  __shared__ int smi[33];
  __shared__ int s_count;
  pdl_wait();
  pdl_trigger();
  const int parity = st.hdr[H_PARITY];
  const int n = st.hdr[H_N_ACTIVE];
  const int lane = threadIdx.x & 31;
  if (threadIdx.x == 0) s_count = 0;
  __syncthreads();
  for (int r = threadIdx.x >> 5; r < n; r += kSchedThreads / 32) {
    const int base = st.lm_base[parity][r];
    const int nm = st.lm_base[parity][r + 1] - base;      // still-masked positions of the row: at most L <= 64
    if (nm == 0) continue;
    // a lane looks after list entries lane and lane + 32
    float conf[2] = {-1.0f, -1.0f};
    int tok[2] = {0, 0}, bit[2] = {0, 0};
    bool picked[2] = {false, false};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int k = lane + 32 * h;
      if (k < nm) {
        // last stage of the confidence pass: the slice partials of this masked position -> token id and confidence
        merge_conf_slices(st.slice_ms, st.slice_am, st.lm_base[parity][n], base + k, &tok[h], &conf[h]);
        st.out_conf[parity][base + k] = conf[h];
        st.out_tok[parity][base + k] = tok[h];
        bit[h] = st.lm_slot[parity][base + k];
      }
    }
    // transfer quota of this step (Section 2.5): the block's L masked tokens spread uniformly over S steps
    const int s_in_block = st.row_s[r];
    const int quota = s_in_block >= st.S ? 1 : st.L / st.S + (s_in_block < st.L % st.S ? 1 : 0);
    for (int it = 0; it < quota; ++it) {          // warp-uniform trip count
      // this lane's better unpicked entry (the lower entry on ties), then the warp's
      float bc = -2.0f;
      int bj = 64;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int k = lane + 32 * h;
        if (k < nm && !picked[h] && conf[h] > bc) { bc = conf[h]; bj = k; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float oc = __shfl_xor_sync(0xffffffffu, bc, o);
        const int oj = __shfl_xor_sync(0xffffffffu, bj, o);
        if (oc > bc || (oc == bc && oj < bj)) { bc = oc; bj = oj; }
      }
      if (bc < -1.5f) break;                      // nothing left to pick (warp-uniform)
      if ((bj & 31) == lane) picked[bj >> 5] = true;
    }
    const int slot = st.row_slot[r];
    unsigned lo_bits = 0u, hi_bits = 0u;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int k = lane + 32 * h;
      const bool sel = k < nm && (conf[h] > st.tau || picked[h]);
      if (sel) {
        const int lo = st.req_p[slot] + st.req_b[slot] * st.L;
        if (!BS_INDEX_OK(lo + bit[h] < st.req_p[slot] + st.req_g[slot] && lo + bit[h] < st.max_row_tokens &&
                             tok[h] >= 0 && tok[h] < st.vocab && tok[h] != st.mask_id, st.hdr + H_ERROR, SITE_COMMIT))
          continue;
        st.tokens[(size_t)slot * st.max_row_tokens + lo + bit[h]] = tok[h];
        if (bit[h] < 32) lo_bits |= 1u << bit[h]; else hi_bits |= 1u << (bit[h] - 32);
      }
      if (k < nm) st.out_commit[parity][base + k] = sel ? 1 : 0;
    }
    lo_bits = __reduce_or_sync(0xffffffffu, lo_bits);
    hi_bits = __reduce_or_sync(0xffffffffu, hi_bits);
    if (lane == 0) {
      const MaskWord bits = ((MaskWord)hi_bits << 32) | lo_bits;
      st.row_mask[r] &= ~bits;
      st.row_s[r] += 1;
      st.req_committed[slot] += __popcll(bits);
      atomicAdd(&s_count, __popcll(bits));
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    st.hdr[H_PREV_MM] = st.lm_base[parity][n];
    st.hdr[H_COMMITTED_STEP] = s_count;
    unsigned long long tot = ((unsigned long long)(unsigned)st.hdr[H_TOTAL_HI] << 32) | (unsigned)st.hdr[H_TOTAL_LO];
    tot += (unsigned long long)s_count;
    st.hdr[H_TOTAL_LO] = (int)(unsigned)(tot & 0xffffffffull);
    st.hdr[H_TOTAL_HI] = (int)(unsigned)(tot >> 32);
  }
  __syncthreads();
  if (st.async_advance) sched_body(st, true);     // finished rows move on or leave now, the queue refills
  else build_index(st, parity ^ 1, n, smi);
}

// Debug aid: commits the given block positions of one active row with the given tokens, as if a step had chosen
// them, and rebuilds the index of the pending step.  The row's step counter is left alone, so a row that has not
// had its refresh step yet still gets one.
struct ForcedTokens { int t[kMaxBlockLen]; };
__global__ void __launch_bounds__(kSchedThreads) k_force_commit(DevState st, int row, MaskWord bits, ForcedTokens ft) {
  __shared__ int smi[33];
  const int parity = st.hdr[H_PARITY];
  const int n = st.hdr[H_N_ACTIVE];
  if (row < n) {
    const MaskWord take = bits & st.row_mask[row];
    const int slot = st.row_slot[row];
    const int lo = st.req_p[slot] + st.req_b[slot] * st.L;
    if (threadIdx.x < kMaxBlockLen && ((take >> threadIdx.x) & 1ull))
      st.tokens[(size_t)slot * st.max_row_tokens + lo + threadIdx.x] = ft.t[threadIdx.x];
    __syncthreads();
    if (threadIdx.x == 0) {
      st.row_mask[row] &= ~take;
      st.req_committed[slot] += __popcll(take);
      unsigned long long tot = ((unsigned long long)(unsigned)st.hdr[H_TOTAL_HI] << 32) | (unsigned)st.hdr[H_TOTAL_LO];
      tot += (unsigned long long)__popcll(take);
      st.hdr[H_TOTAL_LO] = (int)(unsigned)(tot & 0xffffffffull);
      st.hdr[H_TOTAL_HI] = (int)(unsigned)(tot >> 32);
    }
  }
  __syncthreads();
  build_index(st, parity, n, smi);
}

__global__ void k_fill_tokens(DevState st, int parity, int M) {
  pdl_wait();
  pdl_trigger();
  const int n = st.hdr[H_N_ACTIVE];
  const int* cu = st.cu_q[parity];
  for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < M; t += gridDim.x * blockDim.x) {
    int lo = 0, hi = n;                  // largest r with cu[r] <= t
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (cu[mid] <= t) lo = mid; else hi = mid;
    }
    const int r = lo;
    const int slot = st.row_slot[r];
    if (!BS_INDEX_OK(slot >= 0 && slot < st.max_requests, st.hdr + H_ERROR, SITE_FILL_TOKENS)) continue;
    const int first = (st.row_s[r] == 0 && st.row_refresh[r] != 0) ? 0 : st.req_p[slot] + st.req_b[slot] * st.L;
    const int pos = first + (t - cu[r]);
    if (!BS_INDEX_OK(pos >= 0 && pos < st.req_p[slot] + st.req_g[slot] && pos < st.max_row_tokens &&
                         (long long)st.row_kv_base[r] + pos < st.kv_capacity && t < st.kv_capacity, st.hdr + H_ERROR,
                     SITE_FILL_TOKENS))
      continue;
    st.tok_row[t] = r;
    st.tok_pos[t] = pos;                 // logical position id: 0 = first prompt token of the request
    st.tok_kv[t] = st.row_kv_base[r] + pos;
  }
}

cudaError_t launch_sched(const DevState& st, cudaStream_t s) {
  return launch_pdl(k_sched, dim3(1), dim3(kSchedThreads), 0, s, st);
}
cudaError_t launch_commit_index(const DevState& st, cudaStream_t s) {
  return launch_pdl(k_commit_index, dim3(1), dim3(kSchedThreads), 0, s, st);
}
cudaError_t launch_force_commit(const DevState& st, int row, MaskWord bits, const int* tokens, cudaStream_t s) {
  ForcedTokens ft;
  for (int i = 0; i < kMaxBlockLen; ++i) ft.t[i] = tokens[i];
  k_force_commit<<<1, kSchedThreads, 0, s>>>(st, row, bits, ft);
  return cudaGetLastError();
}
cudaError_t launch_fill_tokens(const DevState& st, int parity, int M, cudaStream_t s) {
  if (M <= 0) return cudaSuccess;
  const int threads = 256;
  const int blocks = min((M + threads - 1) / threads, 148 * 8);
  return launch_pdl(k_fill_tokens, dim3(blocks), dim3(threads), 0, s, st, parity, M);
}

}  // namespace bs
