// Ragged bidirectional attention against the dual KV cache on the 5th-generation tensor cores (head_dim 128).
//
// Work item = (row i, a span of the row's packed tokens, kv head).  Its query rows are the flattened
// (token, head-in-group) pairs, so all query heads of a kv head share each K/V tile; they form up to two Q tiles of
// at most 128 rows (one UMMA M tile each), and both Q tiles use every K/V tile the CTA loads.
// Keys are the row's cache span [kv_base_i, kv_base_i + vis_i) - prefix, fresh block and suffix alike; no causal
// or padding mask.  One CTA per SM, warp-specialised:
//   warp 0      TMA producer: the Q tiles once (3-D boxes: 64 dims x group heads x tokens), then 64-key K and V
//               tiles (3-D boxes over the cache [row][kv head][dim]) through a four-stage ring
//   warp 1      MMA issuer: per Q tile S = Q K^T into one of two TMEM buffers (the next key tile's scores are
//               computed while this tile's softmax runs), then O += P V with P as the A operand from tensor memory
//               and V as an MN-major operand straight from the cache layout
//   warps 2..9  softmax, four warps per Q tile: thread r owns query row r (TMEM lane r), so row maxima and sums
//               need no shuffles; p = 2^(s - m) goes back to tensor memory as bf16 pairs, into the first 32 columns
//               of the scores buffer it came from (one tcgen05.st per row, no shared-memory round trip);
//               the output accumulates in TMEM over all key tiles and is rescaled lazily (only when a row's
//               maximum has grown by more than 2^8), the running sum follows the same scale
// Instantiations: two Q tiles per CTA (a work item's Q tiles share every K/V tile the CTA loads) for steps with many
// work items; one Q tile per CTA (half the tensor memory) for steps with few, with a four-stage K/V ring and one
// CTA per SM, or a two-stage ring and two CTAs per SM.  A launch with few work items may also cut every row's keys
// into chunks (grid z): each chunk leaves an unnormalised fp32 partial (output, scale, sum) and a small kernel
// merges them.
// Every wait is bounded; on a timeout the flag is raised, all roles drain, TMEM is freed.
#include <math.h>
#include <stdlib.h>

#include <algorithm>
#include <mutex>
#include <unordered_map>

#include "tc_common.cuh"

namespace bs {

namespace {

using namespace tc;

constexpr int DH = 128;
__host__ __device__ constexpr int threads_for(int nq) { return 64 + 128 * nq; }     // producer warp, MMA warp, 4 softmax warps per Q tile
constexpr int kHalfBytes = 128 * 128;      // 128 rows x 64 bf16: one swizzled sub-tile of Q or P
constexpr int kQBytes = 2 * kHalfBytes;

__device__ __forceinline__ void tma_load_3d(unsigned dst, const CUtensorMap* map, int c0, int c1, int c2, unsigned bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}
// fp32 accumulator, bf16 operands, A K-major, M = 128; B K-major (scores) or MN-major (values).
__device__ __forceinline__ unsigned umma_idesc(int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) | ((unsigned)(n >> 3) << 17) |
         ((128u >> 4) << 24);
}
// tcgen05.mma from descriptor low words (see tc_common.cuh); K-major and MN-major tiles share the 1024-byte group stride.
__device__ __forceinline__ void umma_lo(unsigned d_tmem, unsigned a_lo, unsigned b_lo, unsigned idesc,
                                        unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "mov.b64 da, {%1, %5};\n\t"
      "mov.b64 db, {%2, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi) : "memory");
}
// A operand from tensor memory (lane = row, one 32-bit column = two adjacent bf16 of the row), B from shared memory.
__device__ __forceinline__ void umma_ts(unsigned d_tmem, unsigned a_tmem, unsigned b_lo, unsigned idesc,
                                        unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "mov.b64 db, {%2, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi) : "memory");
}

__device__ __forceinline__ void tmem_st32(unsigned taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
        "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
        "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])),
        "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])), "r"(__float_as_uint(v[16])),
        "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
        "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])),
        "r"(__float_as_uint(v[23])), "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])),
        "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])), "r"(__float_as_uint(v[28])),
        "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st32_words(unsigned taddr, const unsigned* w) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]), "r"(w[8]),
        "r"(w[9]), "r"(w[10]), "r"(w[11]), "r"(w[12]), "r"(w[13]), "r"(w[14]), "r"(w[15]), "r"(w[16]), "r"(w[17]),
        "r"(w[18]), "r"(w[19]), "r"(w[20]), "r"(w[21]), "r"(w[22]), "r"(w[23]), "r"(w[24]), "r"(w[25]), "r"(w[26]),
        "r"(w[27]), "r"(w[28]), "r"(w[29]), "r"(w[30]), "r"(w[31])
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// A row's output accumulator is rescaled only when its running maximum has grown by more than this (log2
// units); until then probabilities are formed against the older maximum and stay below 2^kLazy.
constexpr float kLazy = 8.0f;

struct AttnTcParams {
  const int* cu_q;
  const int* cu_tile;
  const int* kv_base;
  const int* vis;
  bf16* out;
  int n_rows, hq, hkv;
  int tq;            // tokens per Q tile (a work item holds two Q tiles)
  int chunks;        // key chunks per row (grid z); > 1: partials below instead of the output
  float* part_o;     // [chunks][M][Hq * 128] unnormalised outputs
  float2* part_ml;   // [chunks][M][Hq] (scale in log2 units, sum); sum = 0 marks an empty chunk
  int M;
  int* error_flag;
};

constexpr int KT = 64;                                   // keys per tile
constexpr int kKvHalf = KT * 128;                        // KT rows x 64 bf16
constexpr int kStageBytes = 4 * kKvHalf;                 // K halves, V halves
__host__ __device__ constexpr int smem_for(int q_tiles, int stages) {
  return q_tiles * kQBytes + stages * kStageBytes + 1024;
}

// NG: softmax warp groups (each with its own scores buffers and output accumulator in tensor memory).
//   KS = false: group x serves Q tile x of the CTA (NG Q tiles in shared memory, every K/V tile used by all of them).
//   KS = true (NG = 2): one Q tile; the two groups are two independent streams over the row's key tiles - group x
//        takes tiles x, x + 2, x + 4, ... with its own running maximum, sum and accumulator - and the streams are
//        merged once at the end.  A single stream is a dependent chain per key tile (scores -> softmax -> P V ->
//        next softmax); two of them keep the tensor pipe and the exponent unit busy through each other's waits.
template <int NG, int STAGES, bool KS>
__global__ void __launch_bounds__(threads_for(NG), smem_for(KS ? 1 : NG, STAGES) <= 112 * 1024 ? 2 : 1)
k_attention_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const AttnTcParams p) {
  static_assert(!KS || NG == 2, "two streams need two softmax groups");
  constexpr int kStages = STAGES;
  constexpr int kQTiles = KS ? 1 : NG;                      // Q tiles of this CTA
  constexpr unsigned kTmemCols = NG == 2 ? 512u : 256u;
  // Barrier slots
  enum { B_QFULL = 0, B_KVFULL = 1, B_KVEMPTY = B_KVFULL + kStages, B_SFULL = B_KVEMPTY + kStages,   // [group][2]
         B_PFULL = B_SFULL + 4, B_OFULL = B_PFULL + 2, B_COUNT = B_OFULL + 2 };
  extern __shared__ unsigned char smem_dyn[];
  __shared__ __align__(8) unsigned long long bars[B_COUNT];
  __shared__ unsigned tmem_base_slot;
  __shared__ int s_abort;
  __shared__ float2 s_ml[KS ? 128 : 1];                     // (scale, sum) of stream 1, per query row

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned smem0 = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  const unsigned sQ = smem0;                              // [Q tile][dim half][128 rows x 128 B]
  const unsigned sKV = sQ + kQTiles * kQBytes;
  const unsigned bar0 = smem_u32(&bars[0]);
  auto bar = [&](int i) { return bar0 + 8u * (unsigned)i; };

  if (threadIdx.x == 0) {
    s_abort = 0;
    mbar_init(bar(B_QFULL), 1);
    for (int i = 0; i < kStages; ++i) {
      mbar_init(bar(B_KVFULL + i), 1);
      mbar_init(bar(B_KVEMPTY + i), 1);
    }
    for (int i = 0; i < 4; ++i) {
      mbar_init(bar(B_SFULL + i), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(B_PFULL + i), 4);      // one arrival per softmax warp of the group
      mbar_init(bar(B_OFULL + i), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&tmem_base_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const unsigned tmem_base = tmem_base_slot;
  volatile int* abort_flag = &s_abort;
  pdl_trigger();
  // The index arrays were written by the commit / scheduler kernel of the previous step, many kernels ago (the
  // kernel before this one wrote q and the cache rows): they are read before the wait, so that the row search and
  // its dependent loads overlap the previous kernel's tail.
  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
  }

  // ---- which row owns this work item: largest r with cu_tile[r] <= item ----
  const int G = p.hq / p.hkv;
  const int kh = blockIdx.y;
  constexpr bool kSplit = kQTiles == 1;                     // one CTA per Q tile: two CTAs share a work item
  const int item = kSplit ? (int)blockIdx.x >> 1 : (int)blockIdx.x;
  const int row = warp_find_row(p.cu_tile, p.n_rows, item);
  const int per_cta = kQTiles * p.tq;
  const int cq0 = __ldg(p.cu_q + row), cq1 = __ldg(p.cu_q + row + 1), ct0 = __ldg(p.cu_tile + row);
  const int vis = __ldg(p.vis + row);
  const int kvb = __ldg(p.kv_base + row);
  const int t0 = cq0 + (item - ct0) * 2 * p.tq + (kSplit ? ((int)blockIdx.x & 1) * p.tq : 0);
  const int nt = min(per_cta, cq1 - t0);                    // query tokens of this CTA (CTA-uniform)
  const int n_qt = nt <= 0 ? 0 : (nt > p.tq ? 2 : 1);       // Q tiles in use
  // key tiles of this CTA's chunk: [kt0, kt0 + n_tiles) of the row's ceil(vis / KT)
  const int tiles_all = (vis + KT - 1) / KT;
  const int per_chunk = (tiles_all + p.chunks - 1) / p.chunks;
  const int kt0 = (int)blockIdx.z * per_chunk;
  const int n_tiles = nt > 0 ? max(0, min(tiles_all, kt0 + per_chunk) - kt0) : 0;
  pdl_wait();       // q and the cache rows of this step come from the kernel before this one
  const int n_groups = KS ? min(2, n_tiles) : n_qt;         // softmax groups with work

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && n_tiles > 0) {
      mbar_expect_tx(bar(B_QFULL), (unsigned)(n_qt * 2 * p.tq * G * 128));
      for (int x = 0; x < n_qt; ++x) {
        tma_load_3d(sQ + x * kQBytes, &map_q, 0, kh * G, t0 + x * p.tq, bar(B_QFULL));
        tma_load_3d(sQ + x * kQBytes + kHalfBytes, &map_q, 64, kh * G, t0 + x * p.tq, bar(B_QFULL));
      }
      for (int t = 0; t < n_tiles; ++t) {
        const int s = t % kStages;
        if (!mbar_wait(bar(B_KVEMPTY + s), (unsigned)((t / kStages) & 1) ^ 1u, abort_flag)) break;
        const unsigned st = sKV + s * kStageBytes;
        mbar_expect_tx(bar(B_KVFULL + s), (unsigned)kStageBytes);
        const int key0 = kvb + (kt0 + t) * KT;
        tma_load_3d(st, &map_k, 0, kh, key0, bar(B_KVFULL + s));
        tma_load_3d(st + kKvHalf, &map_k, 64, kh, key0, bar(B_KVFULL + s));
        tma_load_3d(st + 2 * kKvHalf, &map_v, 0, kh, key0, bar(B_KVFULL + s));
        tma_load_3d(st + 3 * kKvHalf, &map_v, 64, kh, key0, bar(B_KVFULL + s));
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && n_tiles > 0) {
      const unsigned idesc_s = umma_idesc(KT, false);
      const unsigned idesc_o = umma_idesc(DH, true);
      bool ok = mbar_wait(bar(B_QFULL), 0, abort_flag);
      // S = Q K^T of key tile t into scores buffer b of group x.
      // The buffer is free: the softmax warps finished with the scores it held two of the group's tiles ago before
      // they published the probabilities (same columns), and the P V product that read those was issued by this
      // thread after that and before this product; the tensor pipe runs one thread's instructions in order.
      auto scores = [&](unsigned st, int x, int q_tile, int b) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const unsigned q_lo = desc_lo(sQ + q_tile * kQBytes), k_lo = desc_lo(st), d_s = tmem_base + x * 256 + b * 64;
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_lo(d_s, q_lo + h * (kHalfBytes >> 4) + 2 * k, k_lo + h * (kKvHalf >> 4) + 2 * k, idesc_s,
                    (h | k) ? 1u : 0u);
        umma_commit(bar(B_SFULL + 2 * x + b));
      };
      // O_x += P V: P from tensor memory (the first 32 columns of scores buffer b of group x: 64 bf16 per row);
      // V is an MN-major operand whose two 64-wide dim halves are kKvHalf bytes apart (leading byte offset)
      auto pv = [&](unsigned st, int x, int b, bool first) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const unsigned p_tm = tmem_base + x * 256 + b * 64, v_lo = desc_lo(st + 2 * kKvHalf, kKvHalf);
        const unsigned d_o = tmem_base + x * 256 + 128;
#pragma unroll
        for (int j = 0; j < KT / 16; ++j)           // 16 keys per step; the output accumulates over the group's tiles
          umma_ts(d_o, p_tm + j * 8, v_lo + j * (2048 >> 4), idesc_o, (!first || j) ? 1u : 0u);
        umma_commit(bar(B_OFULL + x));
      };
      auto stage_of = [&](int t) { return sKV + (unsigned)(t % kStages) * kStageBytes; };
      auto wait_kv = [&](int t) { return mbar_wait(bar(B_KVFULL + t % kStages), (unsigned)(t / kStages) & 1u, abort_flag); };
      if (KS) {
        // key tile t belongs to stream x = t & 1 as its i-th tile, i = t >> 1; the scores of tiles t + 1 and t + 2
        // are in flight while tile t's softmax runs
        auto issue_scores = [&](int t) -> bool {
          if (!wait_kv(t)) return false;
          scores(stage_of(t), t & 1, 0, (t >> 1) & 1);
          return true;
        };
        if (ok) ok = issue_scores(0);
        if (ok && n_tiles > 1) ok = issue_scores(1);
        for (int t = 0; t < n_tiles && ok; ++t) {
          if (t + 2 < n_tiles) ok = issue_scores(t + 2);
          if (!ok) break;
          const int x = t & 1, i = t >> 1;
          if (!mbar_wait(bar(B_PFULL + x), (unsigned)i & 1u, abort_flag)) { ok = false; break; }
          pv(stage_of(t), x, i & 1, i == 0);
          umma_commit(bar(B_KVEMPTY + (t % kStages)));
        }
      } else {
        // The scores run TWO tiles ahead of the P V products, one per scores buffer: S(t + 2) goes into the buffer
        // whose probabilities P V(t) has just been issued to read (the tensor pipe runs this thread's instructions
        // in order).  A group's softmax then finds its next scores finished when it publishes a tile, and this
        // thread waits for probabilities only.  Traced with cycle stamps, the earlier order - S(t + 1) for both groups,
        // then the two P V(t) - left both sides idle for a third of a tile: the scores a softmax group waited for
        // were issued only after the other group's P V, and back-pressured issue kept this thread from looking at
        // probabilities that had been ready for 1800 clk.
        for (int t0s = 0; t0s < 2 && t0s < n_tiles && ok; ++t0s) {
          ok = wait_kv(t0s);
          for (int x = 0; x < n_qt && ok; ++x) scores(stage_of(t0s), x, x, t0s & 1);
        }
        for (int t = 0; t < n_tiles && ok; ++t) {
          for (int x = 0; x < n_qt && ok; ++x) {
            if (!mbar_wait(bar(B_PFULL + x), (unsigned)t & 1u, abort_flag)) { ok = false; break; }
            pv(stage_of(t), x, t & 1, t == 0);
            if (t + 2 < n_tiles) {
              if (x == 0 && !wait_kv(t + 2)) { ok = false; break; }
              scores(stage_of(t + 2), x, x, t & 1);
            }
          }
          if (ok) umma_commit(bar(B_KVEMPTY + (t % kStages)));
        }
      }
    }
  } else if (nt > 0) {
    // ------------------------------------------------------------------ softmax warps: one query row per thread
    // warps 2..5 are group 0, warps 6..9 group 1; within a group, warp w reads TMEM lanes 32 (w % 4) ..
    const int x = (warp - 2) >> 2;
    const int q = warp & 3;
    const int r = q * 32 + lane;                        // query row of the Q tile = TMEM lane
    const int q_tile = KS ? 0 : x;                      // the Q tile this group serves
    const int nrows = (q_tile == 0 ? min(nt, p.tq) : nt - p.tq) * G;      // valid rows of that Q tile
    const int my_tiles = x < n_groups ? (KS ? (n_tiles - x + 1) / 2 : n_tiles) : 0;
    const unsigned t_lane = tmem_base + ((unsigned)(q * 32) << 16) + x * 256;
    const unsigned t_out = t_lane + 128;
    const float sc = 1.4426950408889634f * rsqrtf((float)DH);
    const bool warp_has_rows = q * 32 < nrows;          // warps without valid rows only keep the barriers moving
    float m = -INFINITY, l = 0.f;                       // m: the maximum the accumulator is currently scaled by
    bool ok = true;
    for (int i = 0; i < my_tiles && ok; ++i) {
      const int t = KS ? 2 * i + x : i;                 // key tile inside the chunk
      const int b = i & 1;
      if (!mbar_wait(bar(B_SFULL + 2 * x + b), (unsigned)(i >> 1) & 1u, abort_flag)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      float v[KT];
      float f = 1.0f;
      bool rescale = false;
      if (warp_has_rows) {
        // scores -> probabilities in registers; this part overlaps the group's previous P V product
        const int key0 = (kt0 + t) * KT;
        {   // both halves of the tile's scores in flight before the one wait
          unsigned raw[KT];
          tmem_ld32_nowait(t_lane + b * 64, raw);
          tmem_ld32_nowait(t_lane + b * 64 + 32, raw + 32);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < KT; ++j) v[j] = __uint_as_float(raw[j]);
        }
        // eight independent chains for the row maximum and the row sum: one warp per scheduler has no other
        // warp to hide a 64-long dependent chain behind.  The maximum is taken over the raw scores (the scale
        // is positive) and the scale folded into the exponent's fma.
        float mx8[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) mx8[k] = -INFINITY;
        if (key0 + KT <= vis) {
#pragma unroll
          for (int j = 0; j < KT; ++j) mx8[j & 7] = fmaxf(mx8[j & 7], v[j]);
        } else {
#pragma unroll
          for (int j = 0; j < KT; ++j) {
            v[j] = (key0 + j < vis) ? v[j] : -INFINITY;
            mx8[j & 7] = fmaxf(mx8[j & 7], v[j]);
          }
        }
        const float mx = sc * fmaxf(fmaxf(fmaxf(mx8[0], mx8[1]), fmaxf(mx8[2], mx8[3])),
                                    fmaxf(fmaxf(mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])));   // finite: a valid key exists
        // lazy rescale (warp-uniform decision: TMEM loads and stores are warp-wide)
        const bool grow = mx > m + kLazy;               // always true on the first tile (m = -inf)
        rescale = __any_sync(0xffffffffu, grow);
        if (grow) {
          f = ex2(m - mx);                              // first tile: 2^-inf = 0, and the accumulator is empty
          m = mx;
        }
        float rs8[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) rs8[k] = 0.f;
        const float neg_m = -m;
#pragma unroll
        for (int j = 0; j < KT; ++j) {
          v[j] = ex2(fmaf(v[j], sc, neg_m));            // 2^(-inf) = 0 for masked keys
          rs8[j & 7] += v[j];
        }
        l = l * f + (((rs8[0] + rs8[1]) + (rs8[2] + rs8[3])) + ((rs8[4] + rs8[5]) + (rs8[6] + rs8[7])));
      }
      // the group's previous P V product must have finished before its accumulator is touched
      if (i > 0 && !mbar_wait(bar(B_OFULL + x), (unsigned)(i - 1) & 1u, abort_flag)) { ok = false; break; }
      if (rescale && i > 0) {                       // warp-uniform
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          float o[32];
          tmem_ld32(t_out + c * 32, o);
#pragma unroll
          for (int j = 0; j < 32; ++j) o[j] *= f;
          tmem_st32(t_out + c * 32, o);
        }
      }
      if (warp_has_rows) {
        // P as bf16 pairs into the first 32 columns of this tile's scores buffer: the A operand of the P V product
        unsigned w[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          const __nv_bfloat162 pr = __floats2bfloat162_rn(v[2 * c], v[2 * c + 1]);
          w[c] = *reinterpret_cast<const unsigned*>(&pr);
        }
        tmem_st32_words(t_lane + b * 64, w);
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_PFULL + x));
    }
    // the group's last P V product
    const bool have = ok && my_tiles > 0 && mbar_wait(bar(B_OFULL + x), (unsigned)(my_tiles - 1) & 1u, abort_flag);
    if (!have) l = 0.f;                                 // no keys (or a wait ran out): this group contributes nothing
    const int tok = r / G, hg = r % G;
    const bool valid = r < nrows;
    const size_t out_at = (size_t)(t0 + q_tile * p.tq + (valid ? tok : 0)) * (p.hq * DH) + (size_t)(kh * G + hg) * DH;
    const size_t ml_at = ((size_t)blockIdx.z * p.M + t0 + q_tile * p.tq + (valid ? tok : 0)) * p.hq + kh * G + hg;
    float w_own = 1.0f, w_other = 0.f;                  // weights of this group's and the other stream's accumulator
    bool writer = x < n_qt;                             // KS = false: every group with a Q tile writes its own rows
    if (KS) {
      // merge the two streams: stream 1 publishes its (scale, sum); stream 0 reads them and both accumulators
      if (x == 1) s_ml[r] = make_float2(m, l);
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      asm volatile("bar.sync 1, 256;" ::: "memory");    // the eight softmax warps
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      writer = x == 0;
      if (writer) {
        const float2 o1 = s_ml[r];
        const float mm = fmaxf(l > 0.f ? m : -INFINITY, o1.y > 0.f ? o1.x : -INFINITY);
        w_own = l > 0.f ? ex2(m - mm) : 0.f;
        w_other = o1.y > 0.f ? ex2(o1.x - mm) : 0.f;
        l = w_own * l + w_other * o1.y;
        m = mm;
      }
    }
    if (writer && warp_has_rows) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (p.chunks > 1) {
        // unnormalised partial of this key chunk (sum 0 marks a chunk without keys); the merge kernel finishes
        if (valid) p.part_ml[ml_at] = make_float2(l > 0.f ? m : 0.f, l);
        float* pdst = p.part_o + (size_t)blockIdx.z * p.M * (p.hq * DH) + out_at;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          float o[32];
          tmem_ld32(t_out + c * 32, o);        // (every lane takes part in the load; unused values are masked below)
          if (KS) {
            float o2[32];
            tmem_ld32(t_out + 256 + c * 32, o2);
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = (w_own > 0.f ? w_own * o[j] : 0.f) + (w_other > 0.f ? w_other * o2[j] : 0.f);
          }
          if (valid && l > 0.f) {
#pragma unroll
            for (int g = 0; g < 8; ++g)
              *reinterpret_cast<float4*>(pdst + c * 32 + g * 4) =
                  make_float4(o[g * 4], o[g * 4 + 1], o[g * 4 + 2], o[g * 4 + 3]);
          }
        }
      } else {
        const float inv = 1.0f / l;
        bf16* dst = p.out + out_at;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          float o[32];
          tmem_ld32(t_out + c * 32, o);
          if (KS) {
            float o2[32];
            tmem_ld32(t_out + 256 + c * 32, o2);
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = (w_own > 0.f ? w_own * o[j] : 0.f) + (w_other > 0.f ? w_other * o2[j] : 0.f);
          }
          if (valid && l > 0.f) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              uint4 w;
              __nv_bfloat162 h0 = __floats2bfloat162_rn(o[g * 8 + 0] * inv, o[g * 8 + 1] * inv);
              __nv_bfloat162 h1 = __floats2bfloat162_rn(o[g * 8 + 2] * inv, o[g * 8 + 3] * inv);
              __nv_bfloat162 h2 = __floats2bfloat162_rn(o[g * 8 + 4] * inv, o[g * 8 + 5] * inv);
              __nv_bfloat162 h3 = __floats2bfloat162_rn(o[g * 8 + 6] * inv, o[g * 8 + 7] * inv);
              w.x = *reinterpret_cast<unsigned*>(&h0);
              w.y = *reinterpret_cast<unsigned*>(&h1);
              w.z = *reinterpret_cast<unsigned*>(&h2);
              w.w = *reinterpret_cast<unsigned*>(&h3);
              *reinterpret_cast<uint4*>(dst + c * 32 + g * 8) = w;
            }
          }
        }
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (s_abort && threadIdx.x == 0 && p.error_flag) atomicExch(p.error_flag, 1);
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// Merges the key chunks of every (token, head): out = sum_c w_c o_c / sum_c w_c l_c with w_c = 2^(m_c - max m).
constexpr int kMaxChunks = 4;
__global__ void __launch_bounds__(256) k_attention_tc_combine(const float* __restrict__ part_o,
                                                              const float2* __restrict__ part_ml, int chunks, int M,
                                                              bf16* __restrict__ out, int hq) {
  pdl_wait();
  pdl_trigger();
  const int t = blockIdx.x;
  const int out_ld = hq * DH;
  for (int u = threadIdx.x; u < out_ld / 4; u += 256) {
    const int h = (4 * u) / DH;
    // every load of this element first (independent), then the arithmetic
    float2 ml[kMaxChunks];
    float4 ov[kMaxChunks];
#pragma unroll
    for (int c = 0; c < kMaxChunks; ++c)
      if (c < chunks) {
        ml[c] = part_ml[((size_t)c * M + t) * hq + h];
        ov[c] = *reinterpret_cast<const float4*>(part_o + ((size_t)c * M + t) * out_ld + 4 * u);
      }
    float mmax = -INFINITY;
#pragma unroll
    for (int c = 0; c < kMaxChunks; ++c)
      if (c < chunks && ml[c].y > 0.f) mmax = fmaxf(mmax, ml[c].x);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float L = 0.f;
#pragma unroll
    for (int c = 0; c < kMaxChunks; ++c)
      if (c < chunks && ml[c].y > 0.f) {      // (a chunk without keys left its output slots unwritten: never used)
        const float w = exp2f(ml[c].x - mmax);
        acc.x += w * ov[c].x; acc.y += w * ov[c].y; acc.z += w * ov[c].z; acc.w += w * ov[c].w;
        L += w * ml[c].y;
      }
    const float inv = 1.0f / L;
    __nv_bfloat162 a = __floats2bfloat162_rn(acc.x * inv, acc.y * inv), b = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
    uint2 o;
    o.x = *reinterpret_cast<unsigned*>(&a);
    o.y = *reinterpret_cast<unsigned*>(&b);
    *reinterpret_cast<uint2*>(out + (size_t)t * out_ld + 4 * u) = o;
  }
}

// ---- host side ---------------------------------------------------------------------------------------------

std::mutex g_mutex;
struct Key3 {
  const void* ptr; long long d1, d2, s1, s2; int b1, b2;
  bool operator==(const Key3& o) const {
    return ptr == o.ptr && d1 == o.d1 && d2 == o.d2 && s1 == o.s1 && s2 == o.s2 && b1 == o.b1 && b2 == o.b2;
  }
};
struct Hash3 {
  size_t operator()(const Key3& k) const {
    size_t h = std::hash<const void*>()(k.ptr);
    h = h * 1000003u ^ std::hash<long long>()(k.d1 * 131 + k.d2);
    h = h * 1000003u ^ std::hash<long long>()(k.s1 * 257 + k.s2 * 7 + k.b1 * 3 + k.b2);
    return h;
  }
};
std::unordered_map<Key3, CUtensorMap, Hash3> g_maps;

// bf16 tensor [d2][d1][128] with byte strides s1 (dim 1) and s2 (dim 2); box 64 x b1 x b2, 128-byte swizzle.
bool get_map3(const bf16* ptr, long long d1, long long d2, long long s1, long long s2, int b1, int b2, CUtensorMap* out) {
  PFN_cuTensorMapEncodeTiled_v12000 encode = tensor_map_encoder();
  if (!encode) return false;
  std::lock_guard<std::mutex> lock(g_mutex);
  const Key3 key{ptr, d1, d2, s1, s2, b1, b2};
  auto it = g_maps.find(key);
  if (it != g_maps.end()) { *out = it->second; return true; }
  if (g_maps.size() > 8192) g_maps.clear();
  CUtensorMap m;
  const cuuint64_t dims[3] = {(cuuint64_t)DH, (cuuint64_t)d1, (cuuint64_t)d2};
  const cuuint64_t strides[2] = {(cuuint64_t)s1, (cuuint64_t)s2};
  const cuuint32_t box[3] = {64, (cuuint32_t)b1, (cuuint32_t)b2};
  const cuuint32_t estr[3] = {1, 1, 1};
  if (encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<bf16*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  g_maps.emplace(key, m);
  *out = m;
  return true;
}

}  // namespace

// Tokens per Q tile: as many as fit 128 flattened (token, head-in-group) rows, in multiples of 16.
static int tokens_per_q_tile(int hq, int hkv) {
  const int G = hq / hkv;
  return G == 1 ? 128 : (G == 2 ? 64 : (G <= 4 ? 32 : 16));
}

// Query tokens per work item (two Q tiles share every K/V tile a CTA loads).
int attention_tc_q_tile(int hq, int hkv) { return 2 * tokens_per_q_tile(hq, hkv); }

// Returns cudaSuccess with *handled = false when the shape is left to the streaming kernel.
cudaError_t launch_attention_tc(const bf16* qkv, const bf16* kc, const bf16* vc, bf16* out, const int* cu_q,
                                const int* cu_tile, const int* kv_base, const int* vis, int n_rows, int n_tiles,
                                int M, long long kv_rows, int max_nq, int max_vis, int hq, int hkv, int dh,
                                float* scratch, size_t scratch_floats, int* error_flag, cudaStream_t s,
                                bool* handled) {
  *handled = false;
  if (dh != DH || hq % hkv || hq / hkv > 8 || kv_rows <= 0) return cudaSuccess;
  if (((uintptr_t)qkv | (uintptr_t)kc | (uintptr_t)vc) & 15) return cudaSuccess;
  const int G = hq / hkv;
  const int tq = tokens_per_q_tile(hq, hkv);
  static int num_sms_of[kMaxDevices];      // per device; non-zero once the kernel attributes are set there
  int* sms = device_slot(num_sms_of);
  if (!sms) return cudaErrorInvalidDevice;
  if (!*sms) {
    std::lock_guard<std::mutex> lock(g_mutex);
    int dev = 0, n = 0;
    cudaGetDevice(&dev);
    if (cudaFuncSetAttribute(k_attention_tc<1, 2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_for(1, 2)) != cudaSuccess ||
        cudaFuncSetAttribute(k_attention_tc<1, 4, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_for(1, 4)) != cudaSuccess ||
        cudaFuncSetAttribute(k_attention_tc<2, 4, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_for(2, 4)) != cudaSuccess ||
        cudaFuncSetAttribute(k_attention_tc<2, 4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_for(1, 4)) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
      return cudaErrorInvalidDevice;
    *sms = n;
  }
  const int num_sms = *sms;
  CUtensorMap mq, mk, mv;
  const long long qkv_heads = hq + 2 * hkv;
  if (!get_map3(qkv, qkv_heads, M, DH * 2, qkv_heads * DH * 2, G, tq, &mq)) return cudaSuccess;
  if (!get_map3(kc, hkv, kv_rows, DH * 2, (long long)hkv * DH * 2, 1, KT, &mk)) return cudaSuccess;
  if (!get_map3(vc, hkv, kv_rows, DH * 2, (long long)hkv * DH * 2, 1, KT, &mv)) return cudaSuccess;
  *handled = true;
  AttnTcParams p;
  p.cu_q = cu_q; p.cu_tile = cu_tile; p.kv_base = kv_base; p.vis = vis; p.out = out;
  p.n_rows = n_rows; p.hq = hq; p.hkv = hkv; p.tq = tq; p.error_flag = error_flag; p.M = M;
  // Few work items (a block step): each CTA is one long dependent chain over the row's key tiles.  Every Q tile gets
  // its own small CTA, two of them share an SM, and the rows' keys are cut into chunks until about two CTAs per SM
  // are in flight.  Many work items (a refresh step): the two Q tiles of an item share each K/V tile they load.
  static const int env_chunks = getenv("BS_ATTN_TC_CHUNKS") ? atoi(getenv("BS_ATTN_TC_CHUNKS")) : 0;
  static const int env_plan = getenv("BS_ATTN_TC_PLAN") ? atoi(getenv("BS_ATTN_TC_PLAN")) : 0;   // 1 .. 4 below
  const long long items = (long long)n_tiles * hkv;
  // plan 1: two Q tiles per CTA sharing every K/V tile (refresh steps, and block steps with many rows);
  // plan 2: one Q tile per CTA, four-stage K/V ring, optionally key chunks (block steps with few rows);
  // plans 3 and 4 (measurement only, BS_ATTN_TC_PLAN): one Q tile per CTA with a two-stage ring and two CTAs per SM,
  //         or with the row's key tiles in two interleaved streams merged at the end.
  // Plan choice by a small cost model fitted to measurements on B200 (microseconds): a CTA costs a fixed ~8 (launch,
  // tensor-memory allocation, Q load, first K/V tile, output) plus ~1.3 per 64-key tile with two Q tiles or ~0.7 with
  // one (softmax arithmetic and the scores products bound a tile, not the dependent chain: the two-stream plan 4
  // measured the same as plan 2); CTAs beyond one per SM run in further waves; key chunks add a merge kernel (~8).
  const int key_tiles = max_vis > 0 ? (max_vis + KT - 1) / KT : 1;
  const bool block_step = max_nq > 0 && max_nq <= 2 * tq;          // every row has one work item of up to two Q tiles
  auto waves = [&](long long ctas) { return (double)((ctas + num_sms - 1) / num_sms); };
  int plan = 1, chunks = 1;
  if (block_step && max_vis > 0) {
    double best = waves(items) * (8.0 + 1.3 * key_tiles);
    const int max_chunks = scratch ? kMaxChunks : 1;
    for (int c = 1; c <= max_chunks; ++c) {
      if (c > 1 && ((size_t)c * M * ((size_t)hq * DH + 2 * hq) > scratch_floats || key_tiles / c < 4)) break;
      const double cost = waves(2 * items * c) * (8.0 + 0.7 * ((key_tiles + c - 1) / c)) + (c > 1 ? 8.0 : 0.0);
      if (cost < best) { best = cost; plan = 2; chunks = c; }
    }
  }
  if (env_plan >= 1 && env_plan <= 4) { plan = env_plan; if (plan == 1) chunks = 1; }
  if (env_chunks >= 1 && env_chunks <= kMaxChunks && plan != 1 && scratch &&
      (size_t)env_chunks * M * ((size_t)hq * DH + 2 * hq) <= scratch_floats)
    chunks = env_chunks;
  p.chunks = chunks;
  p.part_o = scratch;
  p.part_ml = reinterpret_cast<float2*>(scratch + (size_t)chunks * M * hq * DH);
  cudaError_t r;
  const dim3 grid1(2 * n_tiles, hkv, chunks);
  if (plan == 4)
    r = launch_pdl(k_attention_tc<2, 4, true>, grid1, dim3(threads_for(2)), (size_t)smem_for(1, 4), s, mq, mk, mv, p);
  else if (plan == 3)
    r = launch_pdl(k_attention_tc<1, 2, false>, grid1, dim3(threads_for(1)), (size_t)smem_for(1, 2), s, mq, mk, mv, p);
  else if (plan == 2)
    r = launch_pdl(k_attention_tc<1, 4, false>, grid1, dim3(threads_for(1)), (size_t)smem_for(1, 4), s, mq, mk, mv, p);
  else
    r = launch_pdl(k_attention_tc<2, 4, false>, dim3(n_tiles, hkv, 1), dim3(threads_for(2)), (size_t)smem_for(2, 4), s,
                   mq, mk, mv, p);
  if (r != cudaSuccess || chunks == 1) return r;
  return launch_pdl(k_attention_tc_combine, dim3(M), dim3(256), 0, s, (const float*)p.part_o,
                    (const float2*)p.part_ml, chunks, M, out, hq);
}

}  // namespace bs
