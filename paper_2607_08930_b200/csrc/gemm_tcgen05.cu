// Projection GEMM on the 5th-generation tensor cores: C[M,N] = A[M,K] W[N,K]^T, bf16 operands, fp32 accumulate.
//
// Orientation: the weight rows sit on the 128-row side of the UMMA tile and the packed tokens on its N side
// (N = 32 .. 256), so that a block step with a few dozen tokens wastes no tensor-core rows and every CTA streams a
// disjoint slab of the weights.  One persistent CTA per SM, warp-specialised:
//   warp 0      TMA producer   (cp.async.bulk.tensor.2d, 128B-swizzled K-major tiles of 64 bf16, mbarrier tx counts)
//   warp 1      MMA issuer     (tcgen05.mma cta_group::1 kind::f16, accumulators in TMEM, tcgen05.commit)
//   warps 2..5  epilogue       (tcgen05.ld -> registers -> fused epilogue -> global), double-buffered against the
//                              next tile's main loop through two TMEM accumulator buffers
// Work items are (n tile, token tile, k split); split partial sums go to an fp32 scratch buffer and a small
// kernel adds them in a fixed order and applies the epilogue (deterministic, no atomics).
// Every wait is bounded: when one runs out the kernel raises a flag, all roles drain, TMEM is freed and the
// host reports BS_E_TIMEOUT.
#include <stdio.h>
#include <stdlib.h>

#include <mutex>
#include <string>
#include <unordered_map>

#include "tc_common.cuh"

namespace bs {

namespace {

using namespace tc;

constexpr int BK = 64;                 // K elements per pipeline stage (128 bytes: one swizzle span)
constexpr int TILE_N = 128;            // weight rows per tile (UMMA M)
constexpr int kThreads = 192;
constexpr int kPairThreads = 320;       // the pair kernel runs two groups of four epilogue warps (alternate token chunks)
constexpr int kSmemBudget = 200 * 1024;
constexpr int kSmemBudgetConf = 176 * 1024;   // pair kernel, mode 5 on all eight epilogue warps: eight 4 KB tiles are static

struct GemmParams {
  int M, N, K;
  int tn;            // tokens per tile (UMMA N)
  int n_tiles, m_tiles, splits, kblocks;
  int stages;
  int ksub;          // 64-wide k sub-blocks per pipeline stage
  int mode;          // 0 bf16 store, 1 fp32 +=, 2 fp32 row-scaled store, 3 SwiGLU, 4 fp32 partial sums only,
                     // 5 row-scaled confidence partials (max, sum exp, argmax per token and 32 output features)
  int dual;
  int wide;          // two 128-row tiles of the same weight matrix share every token tile (256 weight rows per item)
  int rows;          // weight rows per work item: 128 or 256
  int nbuf;          // TMEM accumulator buffers: 2, or 1 when two accumulators need more than 256 columns
  int acc1_off;      // column offset of the second accumulator
  void* C;
  int ldc;
  const float* row_scale;
  float* partial;    // [splits][M][N] fp32 when splits > 1
  int* error_flag;
  // mode 5: per (group of 32 output features, token) the running maximum and sum of exponentials of the row-scaled
  // outputs and the feature index of the maximum; feature `skip` never takes part (the mask id)
  float2* conf_ms;   // [ceil(N / 32)][M]
  int* conf_am;      // [ceil(N / 32)][M]
  int skip;
  int vec_store;     // bf16 output rows take 16-byte stores (ldc and N multiples of 8, C 16-byte aligned)
  int mgroup;        // token tiles per group of the work-item order (0: token tile fastest over all of them)
};

__device__ __forceinline__ void tma_load_2d(unsigned dst, const CUtensorMap* map, int c0, int c1, unsigned bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

// Work-item order.  Output tiles are numbered token tile fastest, so that the CTAs of one round share a weight tile;
// with `mgroup` > 0 the token tiles are taken in groups of that many, all weight tiles within a group before the
// next group: the group's activations then stay in L2 while the weights stream past them (many tokens: without it
// every weight tile re-reads the whole activation matrix, which no longer fits L2 beyond ~8 k tokens).
__device__ __forceinline__ void tile_of(const GemmParams& p, int tile, int* mt, int* nt) {
  if (p.mgroup <= 0) {
    *mt = tile % p.m_tiles;
    *nt = tile / p.m_tiles;
    return;
  }
  const int per_group = p.mgroup * p.n_tiles;
  const int g = tile / per_group, r = tile - g * per_group;
  const int g_size = min(p.mgroup, p.m_tiles - g * p.mgroup);
  *nt = r / g_size;
  *mt = g * p.mgroup + r % g_size;
}

// kind::f16 instruction descriptor: fp32 accumulator, bf16 x bf16, both K-major, shape 128 x n x 16.
__device__ __forceinline__ unsigned umma_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((unsigned)(n >> 3) << 17) | ((unsigned)(TILE_N >> 4) << 24);
}
// tcgen05.mma from descriptor low words (see tc_common.cuh), for one CTA or a CTA pair.
template <int CG>
__device__ __forceinline__ void umma_lo(unsigned d_tmem, unsigned a_lo, unsigned b_lo, unsigned idesc,
                                        unsigned accumulate) {
  if (CG == 1) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "mov.b64 da, {%1, %5};\n\t"
        "mov.b64 db, {%2, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi) : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "mov.b64 da, {%1, %5};\n\t"
        "mov.b64 db, {%2, %5};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi) : "memory");
  }
}
// One pipeline stage: 64 k elements = four K=16 steps (descriptor low word + 2 per step) for one or two accumulators.
template <int CG, bool TWO>
__device__ __forceinline__ void issue_stage(unsigned d0, unsigned d1, unsigned a0_lo, unsigned a1_lo, unsigned b_lo,
                                            unsigned idesc, unsigned first_accum) {
  umma_lo<CG>(d0, a0_lo, b_lo, idesc, first_accum);
  if (TWO) umma_lo<CG>(d1, a1_lo, b_lo, idesc, first_accum);
#pragma unroll
  for (int k = 1; k < BK / 16; ++k) {
    umma_lo<CG>(d0, a0_lo + 2 * k, b_lo + 2 * k, idesc, 1u);
    if (TWO) umma_lo<CG>(d1, a1_lo + 2 * k, b_lo + 2 * k, idesc, 1u);
  }
}
// x·sigmoid(x) from the two special-function approximations (2^x, 1/x; relative error ~2^-21, far below the bf16
// rounding that follows).  The IEEE division it replaces carries a slow-path branch per element, which kept the
// compiler from interleaving the columns of a chunk and made the SwiGLU epilogue latency-bound.
__device__ __forceinline__ float silu_f(float x) {
  float e, r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * -1.4426950408889634f));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));      // e = +inf (x << 0) gives r = 0
  return x * r;
}

// Epilogue of one accumulator row: this thread holds output feature n for the tn tokens of token tile mt, whose
// fp32 sums sit in TMEM at t_row (lane already selected) in columns 0 .. tn-1.  EPI: 0 bf16 store, 1 fp32 +=,
// 2 fp32 row-scaled store, 3 SwiGLU, 4 fp32 partial sums of a k split.  The four epilogue warps each own one
// scheduler, so their instruction count is what an epilogue costs: one pointer and one stride per chunk, and the
// per-token predicate only in the ragged last chunk.
template <int EPI, bool FULL>
__device__ __forceinline__ void epilogue_chunk(const float* v, const float* u, char* ptr, size_t stride, int jmax,
                                               const float* scale) {
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    if (!FULL && j >= jmax) break;
    char* q = ptr + (size_t)j * stride;
    if (EPI == 0) *reinterpret_cast<bf16*>(q) = __float2bfloat16_rn(v[j]);
    else if (EPI == 1) *reinterpret_cast<float*>(q) = u[j] + v[j];
    else if (EPI == 2) *reinterpret_cast<float*>(q) = v[j] * __ldg(scale + j);
    else if (EPI == 3) *reinterpret_cast<bf16*>(q) = __float2bfloat16_rn(v[j]);      // v already holds silu(gate)·up
    else *reinterpret_cast<float*>(q) = v[j];
  }
}
// Stores one chunk: v[j] is the finished value of (feature n, token t0 + j), j < jmax.
template <int EPI>
__device__ __forceinline__ void epilogue_store(const GemmParams& p, float* v, float* u, char* base, int ld, int n,
                                               bool n_ok, int t0, int jmax, bf16* tile) {
  constexpr int esize = (EPI == 0 || EPI == 3) ? 2 : 4;
  const size_t stride = (size_t)ld * esize;
  const int lane = threadIdx.x & 31;
  if ((EPI == 0 || EPI == 3) && tile != nullptr) {
    __syncwarp();                             // the previous chunk's reads of the tile are done
#pragma unroll
    for (int j = 0; j < 32; ++j) tile[j * 32 + lane] = __float2bfloat16_rn(v[j]);
    __syncwarp();
    const int piece = lane & 3;               // eight features = 16 bytes
    const int nb = n - lane + piece * 8;
    if (nb < p.N) {                           // N is a multiple of 8 on this path
      char* dst = base + ((size_t)t0 * ld + nb) * esize;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int tok = i * 8 + (lane >> 2);
        if (tok < jmax)
          *reinterpret_cast<uint4*>(dst + (size_t)tok * stride) =
              *reinterpret_cast<const uint4*>(tile + tok * 32 + piece * 8);
      }
    }
    return;
  }
  if (!n_ok) return;                          // (TMEM loads are warp-collective; the stores are not)
  char* ptr = base + ((size_t)t0 * ld + n) * esize;
  if (EPI == 1) {
    // all loads first, then the stores: interleaving them would serialise on the load latency
#pragma unroll
    for (int j = 0; j < 32; ++j) u[j] = j < jmax ? *reinterpret_cast<const float*>(ptr + (size_t)j * stride) : 0.f;
  }
  const float* scale = EPI == 2 ? p.row_scale + t0 : nullptr;
  if (jmax == 32) epilogue_chunk<EPI, true>(v, u, ptr, stride, jmax, scale);
  else epilogue_chunk<EPI, false>(v, u, ptr, stride, jmax, scale);
}

// bf16 outputs (modes 0 and 3) leave through a per-warp shared-memory tile [32 tokens][32 features] when the output
// rows allow 16-byte stores: a thread that stored one 2-byte element per token (32 store instructions per chunk, each
// a 64-byte segment) instead writes four 16-byte vectors, eight token rows per warp instruction.  It matters for the
// SwiGLU GEMM, whose epilogue is exposed (its two 256-column accumulators fill TMEM, so the tensor core waits for it).
// `release` (may be empty) runs once, as soon as the item's last TMEM load of this warp has completed: the
// accumulator is handed back to the MMA issuer before the last chunk's arithmetic and stores.  Returns whether it ran.
template <int EPI, typename Release>
__device__ __forceinline__ bool epilogue_row(const GemmParams& p, int split, int mt, int n, bool n_ok, unsigned t_row,
                                             Release release, bf16* tile = nullptr, int c_first = 0, int c_step = 32) {
  const int ld = EPI == 4 ? p.N : p.ldc;
  char* base = EPI == 4 ? reinterpret_cast<char*>(p.partial + ((size_t)split * p.M) * p.N)
                        : reinterpret_cast<char*>(p.C);
  // SwiGLU: the TMEM loads of the next chunk are issued before this chunk's stores, so that they are complete when
  // the next iteration waits (tcgen05.wait::ld covers every outstanding load of the thread).
  unsigned rv[EPI == 3 ? 32 : 1], ru[EPI == 3 ? 32 : 1];
  bool released = false;
  if (EPI == 3 && c_first < p.tn && mt * p.tn + c_first < p.M) {
    tmem_ld32_nowait(t_row + c_first, rv);
    tmem_ld32_nowait(t_row + p.acc1_off + c_first, ru);
  }
  for (int c0 = c_first; c0 < p.tn; c0 += c_step) {
    const int t0 = mt * p.tn + c0;
    if (t0 >= p.M) break;                     // warp-uniform
    // columns of this chunk that hold tokens of this tile (the tile width is a multiple of 16, not of 32)
    const int jmax = min(min(32, p.tn - c0), p.M - t0);
    const int cn = c0 + c_step;
    const bool more = cn < p.tn && mt * p.tn + cn < p.M;       // this warp has another chunk of the item
    float v[32], u[32];
    if (EPI == 3) {
      tmem_ld_wait();
      // all 32 products before any store, and no branch in silu_f: an epilogue warp's latency hiding is the
      // independence of the 32 columns (and the one other warp on its scheduler)
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = silu_f(__uint_as_float(rv[j])) * __uint_as_float(ru[j]);
      if (more) {
        tmem_ld32_nowait(t_row + cn, rv);
        tmem_ld32_nowait(t_row + p.acc1_off + cn, ru);
      }
    } else {
      tmem_ld32(t_row + c0, v);
    }
    if (!more) { release(); released = true; }
    epilogue_store<EPI>(p, v, u, base, ld, n, n_ok, t0, jmax, tile);
  }
  return released;
}

// Epilogue of the LM head fused with the confidence pass (mode 5).  A warp holds 32 output features (vocabulary
// entries n0 .. n0 + 31, one per lane = TMEM lane) for the tn tokens of the tile.  Per chunk of 32 tokens the
// 32 x 32 block goes through a padded shared-memory tile, after which lane j owns token j with its 32 features:
// it scales them by the token's row scale, and keeps their maximum, the sum of exp(z - max) and the lowest feature
// index of the maximum - one partial per (feature group, token), a twelfth of the bytes of the logits.  When p.C
// is set the scaled fp32 logits are stored as well (parity hooks read them; the timed path passes nullptr).
__device__ __forceinline__ void epilogue_conf(const GemmParams& p, int mt, int n0, int lane, unsigned t_row,
                                              float* tile /* [32][33] of this warp */, int c_first = 0,
                                              int c_step = 32) {
  const int group = n0 >> 5;
  const int n_valid = min(32, p.N - n0);                 // features of this group that exist (warp-uniform)
  const int i_skip = p.skip - n0;                         // index of the excluded feature inside the group, if any
  for (int c0 = c_first; c0 < p.tn; c0 += c_step) {
    const int t0 = mt * p.tn + c0;
    if (t0 >= p.M) break;                                 // warp-uniform
    const int jmax = min(min(32, p.tn - c0), p.M - t0);
    float v[32];
    tmem_ld32(t_row + c0, v);
    __syncwarp();                                         // the previous chunk's reads of the tile are done
#pragma unroll
    for (int j = 0; j < 32; ++j) tile[lane * 33 + j] = v[j];
    __syncwarp();
    if (lane < jmax && n_valid > 0) {
      const int t = t0 + lane;
      const float a = __ldg(p.row_scale + t);
      float z[32];
      float m = -INFINITY;
      int am = 0;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        z[i] = tile[i * 33 + lane] * a;
        const bool use = i < n_valid && i != i_skip;
        if (use && z[i] > m) { m = z[i]; am = i; }       // ascending index, strict: the lowest index wins ties
      }
      float sum = 0.f;
      if (m > -INFINITY) {
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (i < n_valid && i != i_skip) sum += __expf(z[i] - m);
      }
      const size_t at = (size_t)group * p.M + t;
      p.conf_ms[at] = make_float2(m, sum);
      p.conf_am[at] = n0 + am;
      if (p.C) {
        float* dst = reinterpret_cast<float*>(p.C) + (size_t)t * p.ldc + n0;
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (i < n_valid) dst[i] = z[i];
      }
    }
  }
}

template <int EPI>
__global__ void __launch_bounds__(kThreads, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_w2,
          const __grid_constant__ CUtensorMap map_x, const GemmParams p) {
  extern __shared__ unsigned char smem_dyn[];
  __shared__ __align__(8) unsigned long long bars[2 * 16 + 4];     // full[16], empty[16], tmem_full[2], tmem_empty[2]
  __shared__ unsigned tmem_base_slot;
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned smem0 = (smem_u32(smem_dyn) + 1023u) & ~1023u;     // 1024-byte alignment for the swizzle atoms
  const int w_bytes = TILE_N * BK * 2;
  const int x_bytes = p.tn * BK * 2;
  const bool two_a = p.dual || p.wide;
  const int sub_bytes = (two_a ? 2 : 1) * w_bytes + x_bytes;
  const int stage_bytes = p.ksub * sub_bytes;
  const unsigned full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[16]);
  const unsigned tfull0 = smem_u32(&bars[32]), tempty0 = smem_u32(&bars[34]);

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int i = 0; i < p.stages; ++i) {
      mbar_init(full0 + 8 * i, 1);
      mbar_init(empty0 + 8 * i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(tfull0 + 8 * i, 1);
      mbar_init(tempty0 + 8 * i, 4);       // one arrival per epilogue warp
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {                          // TMEM: the whole 512 columns (one CTA per SM)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&tmem_base_slot))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const unsigned tmem_base = tmem_base_slot;
  volatile int* abort_flag = &s_abort;
  // Barriers, TMEM and descriptors are set up.  Each role waits for the previous kernel of the stream only where
  // it first touches something that kernel may have written.
  pdl_trigger();

  const int items = p.n_tiles * p.m_tiles * p.splits;
  const int acc_cols = 256;                 // columns per accumulator buffer (dual: gate at +0, up at +128)

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      unsigned phase = 0;
      bool ok = true;
      // Weights are constants of the model: the first stages of the first item fetch their weight tiles while
      // the previous kernel is still running; the token tiles follow once it has completed.
      int npre = 0;
      {
        const int it = blockIdx.x;
        const int split = it % p.splits;
        int mt_, nt;
        tile_of(p, it / p.splits, &mt_, &nt);
        (void)mt_;
        const int kb0 = (int)((long long)p.kblocks * split / p.splits);
        const int kb1 = (int)((long long)p.kblocks * (split + 1) / p.splits);
        npre = min(p.stages, kb1 - kb0);
        for (int i = 0; i < npre; ++i) {
          mbar_expect_tx(full0 + 8 * i, (unsigned)stage_bytes);
          for (int sub = 0; sub < p.ksub; ++sub) {
            const unsigned sw = smem0 + i * stage_bytes + sub * sub_bytes;
            const int k0 = ((kb0 + i) * p.ksub + sub) * BK;
            tma_load_2d(sw, &map_w, k0, nt * p.rows, full0 + 8 * i);
            if (p.dual) tma_load_2d(sw + w_bytes, &map_w2, k0, nt * p.rows, full0 + 8 * i);
            if (p.wide) tma_load_2d(sw + w_bytes, &map_w, k0, nt * p.rows + TILE_N, full0 + 8 * i);
          }
        }
      }
      pdl_wait();
      for (int it = blockIdx.x; it < items && ok; it += gridDim.x) {
        const int split = it % p.splits;
        const int tile = it / p.splits;
        int mt, nt;
        tile_of(p, tile, &mt, &nt);
        const int kb0 = (int)((long long)p.kblocks * split / p.splits);
        const int kb1 = (int)((long long)p.kblocks * (split + 1) / p.splits);
        for (int kb = kb0; kb < kb1; ++kb) {
          const bool prefetched = it == (int)blockIdx.x && kb - kb0 < npre;
          if (!prefetched) {
            if (!mbar_wait(empty0 + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
            mbar_expect_tx(full0 + 8 * stage, (unsigned)stage_bytes);
          }
          for (int sub = 0; sub < p.ksub; ++sub) {
            const unsigned sw = smem0 + stage * stage_bytes + sub * sub_bytes;
            const int k0 = (kb * p.ksub + sub) * BK;       // beyond K the box is filled with zeros
            if (!prefetched) {
              tma_load_2d(sw, &map_w, k0, nt * p.rows, full0 + 8 * stage);
              if (p.dual) tma_load_2d(sw + w_bytes, &map_w2, k0, nt * p.rows, full0 + 8 * stage);
              if (p.wide) tma_load_2d(sw + w_bytes, &map_w, k0, nt * p.rows + TILE_N, full0 + 8 * stage);
            }
            tma_load_2d(sw + (two_a ? 2 : 1) * w_bytes, &map_x, k0, mt * p.tn, full0 + 8 * stage);
          }
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0;
      unsigned phase = 0;
      int local = 0;
      const unsigned idesc = umma_idesc(p.tn);
      bool ok = true;
      const unsigned lo0 = desc_lo(smem0);
      const unsigned stage_step = (unsigned)stage_bytes >> 4, sub_step = (unsigned)sub_bytes >> 4;
      const unsigned w_step = (unsigned)w_bytes >> 4, x_off = (two_a ? 2u : 1u) * w_step;
      unsigned lo_stage = lo0;
      for (int it = blockIdx.x; it < items && ok; it += gridDim.x, ++local) {
        const int split = it % p.splits;
        const int kb0 = (int)((long long)p.kblocks * split / p.splits);
        const int kb1 = (int)((long long)p.kblocks * (split + 1) / p.splits);
        const int acc = local % p.nbuf;
        const unsigned acc_phase = (unsigned)(local / p.nbuf) & 1u;
        if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, abort_flag)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const unsigned d_gate = tmem_base + acc * acc_cols;
        const unsigned d_up = d_gate + p.acc1_off;
        unsigned accum = 0u;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full0 + 8 * stage, phase, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          unsigned lo = lo_stage;
          for (int sub = 0; sub < p.ksub; ++sub, lo += sub_step) {
            if (two_a) issue_stage<1, true>(d_gate, d_up, lo, lo + w_step, lo + x_off, idesc, accum);
            else issue_stage<1, false>(d_gate, d_up, lo, lo, lo + x_off, idesc, accum);
            accum = 1u;
          }
          umma_commit(empty0 + 8 * stage);        // the stage is free once these MMAs have read it
          lo_stage += stage_step;
          if (++stage == p.stages) { stage = 0; phase ^= 1u; lo_stage = lo0; }
        }
        if (ok) umma_commit(tfull0 + 8 * acc);    // accumulator complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int q = warp & 3;                       // TMEM lane quarter this warp may read
    int local = 0;
    pdl_wait();                                   // the output (and the residual it may add to) is shared state
    for (int it = blockIdx.x; it < items; it += gridDim.x, ++local) {
      const int split = it % p.splits;
      const int tile = it / p.splits;
      int mt, nt;
      tile_of(p, tile, &mt, &nt);
      const int acc = local % p.nbuf;
      const unsigned acc_phase = (unsigned)(local / p.nbuf) & 1u;
      if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag)) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      bool released = false;
      const int n_acc = p.wide ? 2 : 1;                   // a wide item holds two 128-row accumulators
      for (int a = 0; a < n_acc; ++a) {
        const int n = nt * p.rows + a * TILE_N + q * 32 + lane;
        const bool n_ok = n < p.N;
        const unsigned t_row = tmem_base + ((unsigned)(q * 32) << 16) + acc * acc_cols + a * p.acc1_off;
        const bool last_acc = a == n_acc - 1;
        auto release = [&]() {
          if (!last_acc) return;
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
        };
        if constexpr (EPI == 5) {
          __shared__ float conf_tile[4][32 * 33];
          epilogue_conf(p, mt, n - lane, lane, t_row, conf_tile[q]);
        } else if constexpr (EPI == 0 || EPI == 3) {
          __shared__ __align__(16) bf16 out_tile[4][32 * 32];
          released = epilogue_row<EPI>(p, split, mt, n, n_ok, t_row, release, p.vec_store ? out_tile[q] : nullptr) && last_acc;
        } else {
          released = epilogue_row<EPI>(p, split, mt, n, n_ok, t_row, release) && last_acc;
        }
      }
      if (!released) {
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (s_abort && threadIdx.x == 0 && p.error_flag) atomicExch(p.error_flag, 1);
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
  }
}

// ---- CTA-pair variant ---------------------------------------------------------------------------------------
// Two CTAs of a cluster share every tensor-core instruction (tcgen05.mma cta_group::2, UMMA M = 256): each CTA
// stages 128 weight rows and HALF of the token tile, and the hardware reads the other half from the partner's
// shared memory.  A CTA therefore streams 128 + tn/2 operand rows per k step for a 128 x tn accumulator instead of
// 128 + tn, which is what the L2-to-SM path limits at large M.  Roles per CTA are those of k_gemm_tc; the MMA issuer
// runs in the leader CTA (cluster rank 0) only:
//   full[s]    leader's barrier; both CTAs' TMA loads complete their bytes on it
//   empty[s]   one per CTA, released for both by the leader's multicast tcgen05.commit
//   tfull[a]   one per CTA, same mechanism;  tempty[a]  leader's barrier, 4 epilogue warps of each CTA arrive on it
__device__ __forceinline__ unsigned cluster_ctarank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ unsigned map_to_cta(unsigned addr, unsigned rank) {
  unsigned r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(unsigned dst, const CUtensorMap* map, int c0, int c1,
                                                 unsigned bar_in_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar_in_cluster) : "memory");
}
__device__ __forceinline__ unsigned umma_idesc_pair(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((unsigned)(n >> 3) << 17) | ((unsigned)(256 >> 4) << 24);
}
// arrives on the barrier at this shared-memory offset in both CTAs of the pair
__device__ __forceinline__ void umma_commit_pair(unsigned bar) {
  const unsigned short mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void mbar_arrive_in_cluster(unsigned bar_in_cluster) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_in_cluster) : "memory");
}
__device__ __forceinline__ void store_in_cluster(unsigned addr_in_cluster, int v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr_in_cluster), "r"(v) : "memory");
}

template <int EPI>
__global__ void __launch_bounds__(kPairThreads, 1)
k_gemm_pair(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_w2,
            const __grid_constant__ CUtensorMap map_x, const GemmParams p) {
  extern __shared__ unsigned char smem_dyn[];
  __shared__ __align__(8) unsigned long long bars[2 * 16 + 4];     // full[16], empty[16], tmem_full[2], tmem_empty[2]
  __shared__ unsigned tmem_base_slot;
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const unsigned smem0 = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  const int w_bytes = TILE_N * BK * 2;
  const int half_tn = p.tn >> 1;                                    // token rows this CTA stages
  const bool two_w = p.dual || p.wide;                              // two weight tiles share each token tile
  const int n_w = two_w ? 2 : 1;
  const int stage_bytes = n_w * w_bytes + half_tn * BK * 2;
  const unsigned full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[16]);
  const unsigned tfull0 = smem_u32(&bars[32]), tempty0 = smem_u32(&bars[34]);
  const unsigned full_leader0 = map_to_cta(full0, 0), tempty_leader0 = map_to_cta(tempty0, 0);
  const unsigned peer_abort = map_to_cta(smem_u32(&s_abort), rank ^ 1u);

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int i = 0; i < p.stages; ++i) {
      mbar_init(full0 + 8 * i, 1);
      mbar_init(empty0 + 8 * i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(tfull0 + 8 * i, 1);
      mbar_init(tempty0 + 8 * i, 16);      // one arrival per epilogue warp of either CTA
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {                          // both CTAs of the pair allocate their 512 columns
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&tmem_base_slot))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();                       // the partner's barriers exist before anything signals them
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const unsigned tmem_base = tmem_base_slot;
  volatile int* abort_flag = &s_abort;
  pdl_trigger();

  const int items = p.n_tiles * p.m_tiles * p.splits;
  const int acc_cols = 256;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      unsigned phase = 0;
      bool ok = true;
      int npre = 0;
      if (pair < items) {                   // weight tiles of the first stages: constants, fetched before the wait
        const int it = pair;
        const int split = it % p.splits;
        int mt_, nt;
        tile_of(p, it / p.splits, &mt_, &nt);
        (void)mt_;
        const int kb0 = (int)((long long)p.kblocks * split / p.splits);
        const int kb1 = (int)((long long)p.kblocks * (split + 1) / p.splits);
        npre = min(p.stages, kb1 - kb0);
        const int wrow = nt * p.rows + (int)rank * TILE_N;
        for (int i = 0; i < npre; ++i) {
          if (leader) mbar_expect_tx(full0 + 8 * i, 2u * (unsigned)stage_bytes);
          const unsigned sw = smem0 + i * stage_bytes;
          const int k0 = (kb0 + i) * BK;
          tma_load_2d_pair(sw, &map_w, k0, wrow, full_leader0 + 8 * i);
          if (p.dual) tma_load_2d_pair(sw + w_bytes, &map_w2, k0, wrow, full_leader0 + 8 * i);
          if (p.wide) tma_load_2d_pair(sw + w_bytes, &map_w, k0, wrow + 256, full_leader0 + 8 * i);
        }
      }
      pdl_wait();
      for (int it = pair; it < items && ok; it += n_pairs) {
        const int split = it % p.splits;
        const int tile = it / p.splits;
        int mt, nt;
        tile_of(p, tile, &mt, &nt);
        const int kb0 = (int)((long long)p.kblocks * split / p.splits);
        const int kb1 = (int)((long long)p.kblocks * (split + 1) / p.splits);
        const int wrow = nt * p.rows + (int)rank * TILE_N;
        const int xrow = mt * p.tn + (int)rank * half_tn;
        for (int kb = kb0; kb < kb1; ++kb) {
          const bool prefetched = it == pair && kb - kb0 < npre;
          const unsigned sw = smem0 + stage * stage_bytes;
          const int k0 = kb * BK;
          if (!prefetched) {
            if (!mbar_wait(empty0 + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
            if (leader) mbar_expect_tx(full0 + 8 * stage, 2u * (unsigned)stage_bytes);
            tma_load_2d_pair(sw, &map_w, k0, wrow, full_leader0 + 8 * stage);
            if (p.dual) tma_load_2d_pair(sw + w_bytes, &map_w2, k0, wrow, full_leader0 + 8 * stage);
            if (p.wide) tma_load_2d_pair(sw + w_bytes, &map_w, k0, wrow + 256, full_leader0 + 8 * stage);
          }
          tma_load_2d_pair(sw + n_w * w_bytes, &map_x, k0, xrow, full_leader0 + 8 * stage);
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) store_in_cluster(peer_abort, 1);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && leader) {
      int stage = 0;
      unsigned phase = 0;
      int local = 0;
      const unsigned idesc = umma_idesc_pair(p.tn);
      bool ok = true;
      const unsigned lo0 = desc_lo(smem0);
      const unsigned stage_step = (unsigned)stage_bytes >> 4;
      const unsigned w_step = (unsigned)w_bytes >> 4, x_off = (unsigned)n_w * w_step;
      unsigned lo_stage = lo0;
      for (int it = pair; it < items && ok; it += n_pairs, ++local) {
        const int split = it % p.splits;
        const int kb0 = (int)((long long)p.kblocks * split / p.splits);
        const int kb1 = (int)((long long)p.kblocks * (split + 1) / p.splits);
        const int acc = local % p.nbuf;
        const unsigned acc_phase = (unsigned)(local / p.nbuf) & 1u;
        if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const unsigned d_gate = tmem_base + acc * acc_cols;
        const unsigned d_up = d_gate + p.acc1_off;
        unsigned accum = 0u;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full0 + 8 * stage, phase, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          if (two_w) issue_stage<2, true>(d_gate, d_up, lo_stage, lo_stage + w_step, lo_stage + x_off, idesc, accum);
          else issue_stage<2, false>(d_gate, d_up, lo_stage, lo_stage, lo_stage + x_off, idesc, accum);
          accum = 1u;
          umma_commit_pair(empty0 + 8 * stage);
          lo_stage += stage_step;
          if (++stage == p.stages) { stage = 0; phase ^= 1u; lo_stage = lo0; }
        }
        if (ok) umma_commit_pair(tfull0 + 8 * acc);
      }
      if (!ok) store_in_cluster(peer_abort, 1);
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (both CTAs)
    // Warps 2-5 and 6-9: warp w reads TMEM lanes 32·(w mod 4) .. +31; the two groups take alternate 32-token chunks,
    // which halves the time an accumulator that is not double-buffered keeps the tensor core waiting.
    const int q = warp & 3;
    const int group = (warp - 2) >> 2;
    int local = 0;
    bool ok = true;
    pdl_wait();
    for (int it = pair; it < items; it += n_pairs, ++local) {
      const int split = it % p.splits;
      const int tile = it / p.splits;
      int mt, nt;
      tile_of(p, tile, &mt, &nt);
      const int acc = local % p.nbuf;
      const unsigned acc_phase = (unsigned)(local / p.nbuf) & 1u;
      if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      bool released = false;
      const int n_acc = p.wide ? 2 : 1;                   // a wide item holds two 256-row accumulators
      for (int a = 0; a < n_acc; ++a) {
        const int n = nt * p.rows + a * 256 + (int)rank * TILE_N + q * 32 + lane;
        const unsigned t_row = tmem_base + ((unsigned)(q * 32) << 16) + acc * acc_cols + a * p.acc1_off;
        const bool last_acc = a == n_acc - 1;
        auto release = [&]() {
          if (!last_acc) return;
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive_in_cluster(tempty_leader0 + 8 * acc);
        };
        if constexpr (EPI == 5) {
          __shared__ float conf_tile[4][32 * 33];         // one transposition tile per lane quarter: group 0 only
          if (group == 0) epilogue_conf(p, mt, n - lane, lane, t_row, conf_tile[q]);
        } else if constexpr (EPI == 6) {
          // mode 5 with token tiles wider than 128: the confidence pass of a tile would outlast the next tile's main
          // loop on four warps, so all eight take part (eight tiles of static shared memory, a shorter operand ring)
          __shared__ float conf_tile[8][32 * 33];
          epilogue_conf(p, mt, n - lane, lane, t_row, conf_tile[group * 4 + q], group * 32, 64);
        } else if constexpr (EPI == 0 || EPI == 3) {
          __shared__ __align__(16) bf16 out_tile[8][32 * 32];
          released = epilogue_row<EPI>(p, split, mt, n, n < p.N, t_row, release,
                                       p.vec_store ? out_tile[group * 4 + q] : nullptr, group * 32, 64) && last_acc;
        } else {
          released = epilogue_row<EPI>(p, split, mt, n, n < p.N, t_row, release, nullptr, group * 32, 64) && last_acc;
        }
      }
      if (!released) {
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive_in_cluster(tempty_leader0 + 8 * acc);
      }
    }
    if (!ok && lane == 0) store_in_cluster(peer_abort, 1);
  }

  // Neither CTA may leave (or free its TMEM) while the partner can still read its shared memory, write its
  // accumulators or signal its barriers.
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();
  if (s_abort && threadIdx.x == 0 && p.error_flag) atomicExch(p.error_flag, 1);
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
  }
}

// ---- CTA-pair variant with the k split inside a cluster -----------------------------------------------------------
// A block step has fewer output tiles than CTA pairs, so the K range of a tile is split over S pairs.  Here the S
// pairs of a tile form ONE cluster of 2 S CTAs (pair = cluster ranks 2 s, 2 s + 1) and exchange their partial
// accumulators through distributed shared memory instead of an fp32 round trip through L2 and a finishing kernel:
//   1. every pair runs its K range into its own TMEM accumulator (as k_gemm_pair, one work item per cluster);
//   2. cluster barrier: all accumulators complete, every operand ring idle;
//   3. reduce-scatter: the 32-token chunk c of the tile is owned by split c mod S; a CTA sends every chunk it does not
//      own to the owner with the same half of the weight rows (st.shared::cluster into the owner's idle operand ring);
//   4. cluster barrier;
//   5. each CTA adds, in split order, its own and the received partials of the chunks it owns and applies the direct
//      epilogue (0: bf16 store, 1: fp32 +=).  The order is fixed, so the result is deterministic.
// Every thread of the cluster reaches both barriers whatever happened before (a wait that ran out only marks the
// result as failed), so no CTA can be left waiting.
__device__ __forceinline__ void st_cluster_v4(unsigned addr_in_cluster, float a, float b, float c, float d) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr_in_cluster), "f"(a), "f"(b), "f"(c), "f"(d)
               : "memory");
}
__device__ __forceinline__ float4 ld_shared_v4(unsigned addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}

template <int EPI>
__global__ void __launch_bounds__(kPairThreads, 1)
k_gemm_pair_ks(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, const GemmParams p) {
  extern __shared__ unsigned char smem_dyn[];
  __shared__ __align__(8) unsigned long long bars[2 * 16 + 1];     // full[16], empty[16], tmem_full
  __shared__ unsigned tmem_base_slot;
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int S = p.splits;
  const unsigned rank = cluster_ctarank();
  const int split = (int)(rank >> 1);
  const unsigned half = rank & 1u;
  const bool leader = half == 0;
  const unsigned leader_rank = rank & ~1u;
  const int tile_id = (int)blockIdx.x / (2 * S);
  const int mt = tile_id % p.m_tiles, nt = tile_id / p.m_tiles;
  const unsigned smem0 = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  const int w_bytes = TILE_N * BK * 2;
  const int half_tn = p.tn >> 1;
  const int stage_bytes = w_bytes + half_tn * BK * 2;
  const unsigned full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[16]), tfull = smem_u32(&bars[32]);
  const unsigned full_leader0 = map_to_cta(full0, leader_rank);
  const unsigned peer_abort = map_to_cta(smem_u32(&s_abort), rank ^ 1u);
  const int kb0 = (int)((long long)p.kblocks * split / S);
  const int kb1 = (int)((long long)p.kblocks * (split + 1) / S);

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int i = 0; i < p.stages; ++i) {
      mbar_init(full0 + 8 * i, 1);
      mbar_init(empty0 + 8 * i, 1);
    }
    mbar_init(tfull, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(smem_u32(&tmem_base_slot))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const unsigned tmem_base = tmem_base_slot;
  volatile int* abort_flag = &s_abort;
  pdl_trigger();

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs of every pair)
    if (lane == 0) {
      const int wrow = nt * 256 + (int)half * TILE_N;
      const int xrow = mt * p.tn + (int)half * half_tn;
      const int npre = min(p.stages, kb1 - kb0);
      for (int i = 0; i < npre; ++i) {      // weights are constants: fetched before the previous kernel has completed
        if (leader) mbar_expect_tx(full0 + 8 * i, 2u * (unsigned)stage_bytes);
        tma_load_2d_pair(smem0 + i * stage_bytes, &map_w, (kb0 + i) * BK, wrow, full_leader0 + 8 * i);
      }
      pdl_wait();
      int stage = 0;
      unsigned phase = 0;
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb) {
        const unsigned sw = smem0 + stage * stage_bytes;
        if (kb - kb0 >= npre) {
          if (!mbar_wait(empty0 + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
          if (leader) mbar_expect_tx(full0 + 8 * stage, 2u * (unsigned)stage_bytes);
          tma_load_2d_pair(sw, &map_w, kb * BK, wrow, full_leader0 + 8 * stage);
        }
        tma_load_2d_pair(sw + w_bytes, &map_x, kb * BK, xrow, full_leader0 + 8 * stage);
        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
      }
      if (!ok) store_in_cluster(peer_abort, 1);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA of every pair)
    if (lane == 0 && leader) {
      const unsigned idesc = umma_idesc_pair(p.tn);
      const unsigned short mask = (unsigned short)(3u << (2 * split));      // the two CTAs of this pair
      auto commit = [&](unsigned bar) {
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                     ::"r"(bar), "h"(mask) : "memory");
      };
      const unsigned lo0 = desc_lo(smem0);
      const unsigned stage_step = (unsigned)stage_bytes >> 4, x_off = (unsigned)w_bytes >> 4;
      unsigned lo_stage = lo0;
      int stage = 0;
      unsigned phase = 0, accum = 0u;
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!mbar_wait(full0 + 8 * stage, phase, abort_flag)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        issue_stage<2, false>(tmem_base, tmem_base, lo_stage, lo_stage, lo_stage + x_off, idesc, accum);
        accum = 1u;
        commit(empty0 + 8 * stage);
        lo_stage += stage_step;
        if (++stage == p.stages) { stage = 0; phase ^= 1u; lo_stage = lo0; }
      }
      if (ok) commit(tfull);
      else store_in_cluster(peer_abort, 1);
    }
  }

  // ---- epilogue warps 2..9: wait for this pair's accumulator ----
  const int q = warp & 3;                       // TMEM lane quarter of this warp
  const int group = (warp - 2) >> 2;            // the two groups take alternate chunks
  const bool epi = warp >= 2;
  if (epi) {
    pdl_wait();
    if (!mbar_wait(tfull, 0, abort_flag) && lane == 0) store_in_cluster(peer_abort, 1);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  cluster_sync_all();                           // every accumulator of the tile is complete, every operand ring idle
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

  // received partials: [sender split][owned chunk index][lane quarter][4-column group][lane][4 floats]
  const int nch = (min(p.tn, p.M - mt * p.tn) + 31) >> 5;        // chunks of this tile that hold tokens
  const int kmax = (((p.tn + 31) >> 5) + S - 1) / S;              // owned chunks per CTA at most
  const unsigned t_row = tmem_base + ((unsigned)(q * 32) << 16);
  auto slot = [&](int sender, int k) { return smem0 + (unsigned)(((sender * kmax + k) * 4 + q) * 4096 + lane * 16); };
  if (epi) {
    for (int c = 0; c < nch; ++c) {
      const int owner = c % S, k = c / S;
      if (owner == split || (k & 1) != group) continue;         // warp-uniform
      float v[32];
      tmem_ld32(t_row + c * 32, v);
      const unsigned dst = map_to_cta(slot(split, k), (unsigned)(2 * owner) + half);
#pragma unroll
      for (int g = 0; g < 8; ++g) st_cluster_v4(dst + g * 512, v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
    }
  }
  cluster_sync_all();                           // the partials have arrived
  if (epi) {
    const int n = nt * 256 + (int)half * TILE_N + q * 32 + lane;
    const bool n_ok = n < p.N;
    char* base = reinterpret_cast<char*>(p.C);
    __shared__ __align__(16) bf16 out_tile[EPI == 0 ? 8 : 1][32 * 32];
    bf16* tile = (EPI == 0 && p.vec_store) ? out_tile[group * 4 + q] : nullptr;
    for (int c = split; c < nch; c += S) {
      const int k = c / S;
      if ((k & 1) != group) continue;                           // warp-uniform
      const int t0 = mt * p.tn + c * 32;
      const int jmax = min(min(32, p.tn - c * 32), p.M - t0);
      float own[32], v[32], u[32];
      tmem_ld32(t_row + c * 32, own);
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = 0.f;
      for (int sdr = 0; sdr < S; ++sdr) {                       // split order
        if (sdr == split) {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] += own[j];
        } else {
          const unsigned src = slot(sdr, k);
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            const float4 r = ld_shared_v4(src + g * 512);
            v[4 * g] += r.x; v[4 * g + 1] += r.y; v[4 * g + 2] += r.z; v[4 * g + 3] += r.w;
          }
        }
      }
      epilogue_store<EPI>(p, v, u, base, p.ldc, n, n_ok, t0, jmax, tile);
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();                           // nobody leaves while a partner may still signal or read it
  if (s_abort && threadIdx.x == 0 && p.error_flag) atomicExch(p.error_flag, 1);
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 256;" ::"r"(tmem_base) : "memory");
  }
}

// Adds the k-split partial sums in split order and applies the epilogue.
__global__ void k_gemm_finish(const float* __restrict__ partial, int splits, int M, int N, int mode, void* Cv, int ldc,
                              const float* __restrict__ row_scale) {
  pdl_wait();
  pdl_trigger();
  const size_t total = (size_t)M * N;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int t = (int)(i / N), n = (int)(i % N);
    float g = 0.f;
    for (int s = 0; s < splits; ++s) g += partial[(size_t)s * total + i];
    if (mode == 0) {
      reinterpret_cast<bf16*>(Cv)[(size_t)t * ldc + n] = __float2bfloat16_rn(g);
    } else if (mode == 1) {
      reinterpret_cast<float*>(Cv)[(size_t)t * ldc + n] += g;
    } else if (mode == 2) {
      reinterpret_cast<float*>(Cv)[(size_t)t * ldc + n] = g * row_scale[t];
    } else {
      float u = 0.f;
      for (int s = 0; s < splits; ++s) u += partial[(size_t)(splits + s) * total + i];
      reinterpret_cast<bf16*>(Cv)[(size_t)t * ldc + n] = __float2bfloat16_rn(silu_f(g) * u);
    }
  }
}

// ---- host side ---------------------------------------------------------------------------------------------

std::mutex g_mutex;

struct MapKey {
  const void* ptr; long long rows, cols, ld; int box_rows;
  bool operator==(const MapKey& o) const {
    return ptr == o.ptr && rows == o.rows && cols == o.cols && ld == o.ld && box_rows == o.box_rows;
  }
};
struct MapHash {
  size_t operator()(const MapKey& k) const {
    size_t h = std::hash<const void*>()(k.ptr);
    h = h * 1000003u ^ std::hash<long long>()(k.rows * 131 + k.cols);
    h = h * 1000003u ^ std::hash<long long>()(k.ld * 257 + k.box_rows);
    return h;
  }
};
std::unordered_map<MapKey, CUtensorMap, MapHash> g_maps;

bool get_map(const bf16* ptr, long long rows, long long cols, long long ld, int box_rows, CUtensorMap* out) {
  PFN_cuTensorMapEncodeTiled_v12000 encode = tensor_map_encoder();
  if (!encode) return false;
  std::lock_guard<std::mutex> lock(g_mutex);
  const MapKey key{ptr, rows, cols, ld, box_rows};
  auto it = g_maps.find(key);
  if (it != g_maps.end()) { *out = it->second; return true; }
  if (g_maps.size() > 8192) g_maps.clear();
  CUtensorMap m;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(bf16)};
  const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<bf16*>(ptr), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  g_maps.emplace(key, m);
  *out = m;
  return true;
}

// Plan overrides for measurements (environment, read once per process; the defaults are the measured best).
struct Tuning {
  int pair;         // BS_GEMM_PAIR: -1 automatic, 0 single-CTA kernel only, n > 0 CTA pairs from n tokens
  int pair_wide;    // BS_GEMM_PAIR_WIDE: 512-row pair items: -1 automatic, 0 never, 1 wherever they fit
  int pair_splits;  // BS_GEMM_PAIR_SPLITS: cap of the pair kernel's k split
  int wide_off;     // BS_GEMM_WIDE=0: no 256-row items in the single-CTA kernel
  int ksub;         // BS_GEMM_KSUB: 0 automatic, 1 or 2 k sub-blocks per stage
  int splits;       // BS_GEMM_SPLITS: 0 automatic, 1..8
  int stages;       // BS_GEMM_STAGES: 0 automatic
  int debug;        // BS_GEMM_DEBUG: print every plan
  int no_pdl;       // BS_NO_PDL
  int ks;           // BS_GEMM_KS: -1 automatic, 0 never split K inside a cluster, 2 or 4 that many splits where they fit
  int wide_fill;    // BS_GEMM_WIDE_FILL: per-item constant of the last-round fill cost for 512-row items (0: no fill)
  int mgroup;       // BS_GEMM_MGROUP: token tiles per group of the work-item order: -1 automatic, 0 off
};
int env_int(const char* name, int dflt) {
  const char* v = getenv(name);
  return v ? atoi(v) : dflt;
}
const Tuning& tuning() {
  static const Tuning t = {env_int("BS_GEMM_PAIR", -1), env_int("BS_GEMM_PAIR_WIDE", -1),
                           env_int("BS_GEMM_PAIR_SPLITS", 8), getenv("BS_GEMM_WIDE") && env_int("BS_GEMM_WIDE", 1) == 0,
                           env_int("BS_GEMM_KSUB", 0), env_int("BS_GEMM_SPLITS", 0), env_int("BS_GEMM_STAGES", 0),
                           getenv("BS_GEMM_DEBUG") != nullptr, getenv("BS_NO_PDL") != nullptr, env_int("BS_GEMM_KS", -1),
                           env_int("BS_GEMM_WIDE_FILL", 8), env_int("BS_GEMM_MGROUP", -1)};
  return t;
}

using GemmKernel = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const GemmParams);
GemmKernel kernel_tc(int epi) {
  switch (epi) {
    case 0: return k_gemm_tc<0>;
    case 1: return k_gemm_tc<1>;
    case 2: return k_gemm_tc<2>;
    case 3: return k_gemm_tc<3>;
    case 5: return k_gemm_tc<5>;
    default: return k_gemm_tc<4>;
  }
}
GemmKernel kernel_pair(int epi) {
  switch (epi) {
    case 0: return k_gemm_pair<0>;
    case 1: return k_gemm_pair<1>;
    case 2: return k_gemm_pair<2>;
    case 3: return k_gemm_pair<3>;
    case 5: return k_gemm_pair<5>;
    case 6: return k_gemm_pair<6>;
    default: return k_gemm_pair<4>;
  }
}
bool allow_big_smem(GemmKernel (*table)(int), int variants) {
  for (int e = 0; e < variants; ++e)
    if (cudaFuncSetAttribute(table(e), cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (e == 6 ? kSmemBudgetConf : kSmemBudget) + 1024) != cudaSuccess)
      return false;
  return true;
}

// One-time set-up per device: SM count, kernel attributes, resident CTA pairs.
struct DevInfo {
  int num_sms;      // 0: not initialised
  int tc_ok;        // the single-CTA kernels may use their shared-memory budget
  int max_pairs;    // 0: not queried; < 0: the pair kernel cannot be used; else resident clusters of two CTAs
  int max_ks[2];    // resident clusters of 4 and of 8 CTAs of the cluster k-split kernel (0: it cannot be used)
};
DevInfo g_dev[kMaxDevices];

DevInfo* dev_info() {
  DevInfo* d = device_slot(g_dev);
  if (!d) return nullptr;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!d->num_sms) {
    int dev = 0, n = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return nullptr;
    d->tc_ok = allow_big_smem(kernel_tc, 6) ? 1 : 0;
    if (!d->tc_ok) cudaGetLastError();
    d->num_sms = n;
  }
  if (!d->max_pairs) {
    if (!allow_big_smem(kernel_pair, 7)) {
      cudaGetLastError();
      d->max_pairs = -1;
    } else {
      cudaLaunchConfig_t qc = {};
      qc.gridDim = dim3(2 * d->num_sms);
      qc.blockDim = dim3(kPairThreads);
      qc.dynamicSmemBytes = (size_t)kSmemBudget + 1024;
      cudaLaunchAttribute qa[1];
      qa[0].id = cudaLaunchAttributeClusterDimension;
      qa[0].val.clusterDim.x = 2; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
      qc.attrs = qa; qc.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, k_gemm_pair<0>, &qc) != cudaSuccess || n < 1) { cudaGetLastError(); n = -1; }
      d->max_pairs = n;
    }
    d->max_ks[0] = d->max_ks[1] = 0;
    if (d->max_pairs > 0 &&
        cudaFuncSetAttribute(k_gemm_pair_ks<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 1024) == cudaSuccess &&
        cudaFuncSetAttribute(k_gemm_pair_ks<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 1024) == cudaSuccess) {
      for (int i = 0; i < 2; ++i) {
        const int cs = i == 0 ? 4 : 8;
        cudaLaunchConfig_t qc = {};
        qc.gridDim = dim3((unsigned)(d->num_sms / cs * cs));
        qc.blockDim = dim3(kPairThreads);
        qc.dynamicSmemBytes = (size_t)kSmemBudget + 1024;
        cudaLaunchAttribute qa[1];
        qa[0].id = cudaLaunchAttributeClusterDimension;
        qa[0].val.clusterDim.x = (unsigned)cs; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
        qc.attrs = qa; qc.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, k_gemm_pair_ks<0>, &qc) != cudaSuccess || n < 1) { cudaGetLastError(); n = 0; }
        d->max_ks[i] = n;
      }
    } else {
      cudaGetLastError();
    }
    if (tuning().debug)
      fprintf(stderr, "gemm pair kernel: %d resident CTA pairs; cluster k-split: %d clusters of 4, %d of 8\n", d->max_pairs,
              d->max_ks[0], d->max_ks[1]);
  }
  return d;
}

thread_local std::string g_decline;     // why the last launch on this thread was refused
cudaError_t decline(const char* why) {
  g_decline = why;
  return cudaErrorNotSupported;
}

// Fraction of the persistent grid that has work, averaged over its rounds.
double grid_busy(long long items, int workers) {
  const long long rounds = (items + workers - 1) / workers;
  return rounds > 0 ? (double)items / (double)(rounds * workers) : 0.0;
}
int split_for(long long base_items, int workers, int kblocks, size_t out_floats, const GemmScratch& scratch, bool dual) {
  if (dual || !scratch.partial || base_items * 4 >= (long long)workers * 3) return 1;
  int sp = (int)(workers / base_items);
  if (sp > 8) sp = 8;
  while (sp > 1 && (kblocks / sp < 4 || (size_t)sp * out_floats > scratch.partial_floats)) --sp;
  return sp < 1 ? 1 : sp;
}

cudaError_t launch_finish(const GemmParams& p, int mode, int num_sms, cudaStream_t s) {
  const size_t total = (size_t)p.M * p.N;
  const size_t want = (total + 255) / 256, cap = (size_t)num_sms * 8;
  return launch_pdl(k_gemm_finish, dim3((unsigned)(want < cap ? want : cap)), dim3(256), 0, s, (const float*)p.partial,
                    p.splits, p.M, p.N, mode, p.C, p.ldc, p.row_scale);
}

// The down projection of a block step with more than one token tile (k-split partial sums, K = 18944): 512-row items
// of the pair kernel, 7 x 2 x 5 splits = 70 for 74 pairs, instead of 140 256-row items of the single-CTA kernel — a CTA
// then loads half of each token tile (48 instead of 64 bytes per clock from L2 at the full tensor rate).
// Measured on the Dream-7B-shaped job: +0.6 % (the steps with 288-512 packed tokens are a third of it).
static bool pair_wide_partials(int mode, int M, int N, int K) {
  return mode == 4 && K >= 8192 && M > 256 && N >= 1024 && tuning().pair_wide < 0;
}

// Plans and launches the CTA-pair kernel.
cudaError_t launch_gemm_pair(const DevInfo& dv, const bf16* A, int lda, const bf16* W, const bf16* W2, void* C, int ldc,
                             int M, int N, int K, int mode, const float* row_scale, const GemmScratch& scratch,
                             cudaStream_t s, int* splits_out, const GemmConf* conf) {
  const int max_pairs = dv.max_pairs;
  const int dual = mode == 3;
  GemmParams p;
  p.M = M; p.N = N; p.K = K; p.mode = mode; p.dual = dual; p.C = C; p.ldc = ldc; p.row_scale = row_scale;
  p.error_flag = scratch.error_flag;
  p.conf_ms = conf ? conf->ms : nullptr; p.conf_am = conf ? conf->am : nullptr; p.skip = conf ? conf->skip : -1;
  p.vec_store = (ldc % 8 == 0 && N % 8 == 0 && ((uintptr_t)C & 15) == 0) ? 1 : 0;
  // Two 256-row weight tiles per pair and work item halve the token-tile traffic once more (48 instead of 64 bytes
  // per clock and SM from L2, the SwiGLU GEMM's figure) at the price of single-buffered accumulators; with a long K
  // the exposed epilogue is a per cent of the item.  Measured on B200 in seconds-long loops (power-capped, the state
  // a refresh step runs in): the down projection (K = 18944) 2-14 % faster from 2048 tokens on, and 10-15 % with token
  // tiles narrowed to fill the last round of items (7 wide weight tiles leave 74 pairs badly divided); slower below
  // 2048 tokens and for the K = 3584 projections (3-7 %).  BS_GEMM_PAIR_WIDE: -1 automatic, 0 never, 1 wherever it fits.
  const int wide_mode = tuning().pair_wide, wide_fill = tuning().wide_fill;
  p.wide = (!dual && mode != 5 && N >= 1024 &&
            (wide_mode > 0 || (wide_mode < 0 && K >= 8192 && (M >= 2048 || pair_wide_partials(mode, M, N, K))))) ? 1 : 0;
  p.rows = p.wide ? 512 : 256;
  p.ksub = 1;
  p.n_tiles = (N + p.rows - 1) / p.rows;
  // Token tiles of up to 256.  With gate and up accumulators that fills TMEM, so the SwiGLU GEMM runs
  // single-buffered above 128 tokens (the epilogue is not overlapped with the next item's main loop), but a CTA
  // then moves 40 % fewer bytes from L2 per flop: measured faster at every M (1330 vs 1259 TFLOP/s at M = 4096).
  const int tn_cap = 256;
  p.m_tiles = (M + tn_cap - 1) / tn_cap;
  // The tensor-core time of a work item is linear in its token-tile width.  When the number of weight tiles does not
  // divide the grid (the LLaDA-shaped gate/up has 48 for 74 pairs), slightly narrower token tiles that fill the last
  // round of work items finish earlier; measured for the SwiGLU GEMM only (up to -3.5 %), where items are long.
  if ((dual || (p.wide && wide_fill)) && (long long)p.n_tiles * p.m_tiles > max_pairs) {
    const int lo = p.m_tiles;
    long long best_cost = -1;
    for (int mt = lo; mt <= lo + lo / 2 + 1; ++mt) {
      const int tn = (((M + mt - 1) / mt) + 15) / 16 * 16;
      const long long rounds = ((long long)p.n_tiles * mt + max_pairs - 1) / max_pairs;
      const long long cost = rounds * (tn + (dual ? 48 : wide_fill));            // + a fixed per-item cost (ramp, exposed epilogue)
      if (best_cost < 0 || cost < best_cost) { best_cost = cost; p.m_tiles = mt; }
    }
  }
  p.tn = (((M + p.m_tiles - 1) / p.m_tiles) + 15) / 16 * 16;
  // Token tiles in groups once the activation matrix no longer fits L2 beside the weight stream (measured in
  // power-capped loops: neutral or slightly slower up to ~6 k tokens of K = 3584, then QKV / O +5-8 % at 8735 tokens
  // and +27-34 % from 16384 on, gate/up +11 % and down +9 % at 16384; group sizes 4-16 within 2 %, 16 best for gate/up and the LM head, whose weights are the larger stream).
  // BS_GEMM_MGROUP: -1 automatic, 0 off, n that many token tiles per group.
  int mgroup = tuning().mgroup;
  if (mgroup < 0) mgroup = (size_t)M * K * sizeof(bf16) > ((size_t)56 << 20) ? ((dual || N >= 32768) ? 16 : 8) : 0;
  p.mgroup = mgroup > 0 && p.m_tiles > mgroup ? mgroup : 0;
  p.nbuf = ((dual || p.wide) && p.tn > 128) ? 1 : 2;
  p.acc1_off = p.nbuf == 1 ? 256 : 128;
  p.kblocks = (K + BK - 1) / BK;
  const int stage_bytes = ((dual || p.wide) ? 2 : 1) * TILE_N * BK * 2 + (p.tn / 2) * BK * 2;
  const bool conf8 = mode == 5 && p.tn > 128;
  const int smem_budget = conf8 ? kSmemBudgetConf : kSmemBudget;
  p.stages = smem_budget / stage_bytes;
  if (p.stages > 16) p.stages = 16;
  if (const int st = tuning().stages) { if (st >= 2 && st < p.stages) p.stages = st; }
  p.splits = 1;
  const long long base_items = (long long)p.n_tiles * p.m_tiles;
  if (scratch.partial && !dual && mode != 5 && base_items * 4 < (long long)max_pairs * 3) {
    int sp = (int)(max_pairs / base_items);
    if (sp > tuning().pair_splits) sp = tuning().pair_splits;
    if (sp > 8) sp = 8;
    while (sp > 1 && (p.kblocks / sp < 4 || (size_t)sp * (size_t)M * N > scratch.partial_floats)) --sp;
    p.splits = sp < 1 ? 1 : sp;
  }
  if (mode == 4 && (!scratch.partial || (size_t)p.splits * (size_t)M * N > scratch.partial_floats))
    return decline("partial-sum scratch too small for this projection");
  p.partial = scratch.partial;
  if (splits_out) *splits_out = p.splits;
  CUtensorMap mw, mw2, mx;
  if (!get_map(W, N, K, K, TILE_N, &mw)) return decline("tensor map of the weight matrix could not be encoded");
  if (dual) {
    if (!get_map(W2, N, K, K, TILE_N, &mw2)) return decline("tensor map of the second weight matrix could not be encoded");
  } else {
    mw2 = mw;
  }
  if (!get_map(A, M, K, lda, p.tn / 2, &mx)) return decline("tensor map of the activations could not be encoded");
  const long long items = base_items * p.splits;
  if (tuning().debug)
    fprintf(stderr, "pair gemm M=%d N=%d K=%d mode=%d tn=%d m_tiles=%d n_tiles=%d splits=%d stages=%d\n", M, N, K, mode,
            p.tn, p.m_tiles, p.n_tiles, p.splits, p.stages);
  const int pairs = (int)(items < max_pairs ? items : max_pairs);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(kPairThreads);
  cfg.dynamicSmemBytes = (size_t)smem_budget + 1024;
  cfg.stream = s;
  cudaLaunchAttribute attrs[2];
  attrs[0].id = cudaLaunchAttributeClusterDimension;
  attrs[0].val.clusterDim.x = 2; attrs[0].val.clusterDim.y = 1; attrs[0].val.clusterDim.z = 1;
  attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attrs[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attrs;
  cfg.numAttrs = tuning().no_pdl ? 1 : 2;
  cudaError_t r = cudaLaunchKernelEx(&cfg, kernel_pair((p.splits > 1 || mode == 4) ? 4 : (conf8 ? 6 : mode)), mw, mw2, mx, p);
  if (r != cudaSuccess) return r;
  if (p.splits > 1 && mode != 4) r = launch_finish(p, mode, dv.num_sms, s);
  return r;
}

// Plan of the cluster k-split kernel for a direct projection (mode 0 or 1) of a block step: how many pairs share a
// tile's K range, or 0 when the shape is left to the other kernels.  One wave of clusters only (a cluster holds its
// SMs until its slowest pair is done), at least 8 k blocks per pair, and at least 3/8 of the SMs busy.
struct KsPlan { int splits, tn, m_tiles, n_tiles, kblocks; };
KsPlan plan_ks(const DevInfo& dv, int M, int N, int K, int mode, int ldc, const void* C) {
  KsPlan pl = {0, 0, 0, 0, 0};
  const int want = tuning().ks;
  if (want == 0 || (mode != 0 && mode != 1) || M < 128 || M > 1024 || N < 256) return pl;
  if (mode == 0 && !(ldc % 8 == 0 && N % 8 == 0 && ((uintptr_t)C & 15) == 0)) return pl;
  pl.n_tiles = (N + 255) / 256;
  pl.m_tiles = (M + 255) / 256;
  pl.tn = (((M + pl.m_tiles - 1) / pl.m_tiles) + 15) / 16 * 16;
  pl.kblocks = (K + BK - 1) / BK;
  const int tiles = pl.n_tiles * pl.m_tiles;
  for (int i = 1; i >= 0; --i) {
    const int sp = i == 0 ? 2 : 4;
    if (want > 0 && want != sp) continue;
    if (tiles > dv.max_ks[i] || pl.kblocks / sp < 8) continue;
    if (want < 0 && tiles * 2 * sp * 8 < dv.num_sms * 3) continue;
    pl.splits = sp;
    break;
  }
  return pl;
}

cudaError_t launch_gemm_pair_ks(const KsPlan& pl, const bf16* A, int lda, const bf16* W, void* C, int ldc, int M, int N,
                                int K, int mode, const GemmScratch& scratch, cudaStream_t s) {
  GemmParams p = {};
  p.M = M; p.N = N; p.K = K; p.mode = mode; p.C = C; p.ldc = ldc;
  p.error_flag = scratch.error_flag;
  p.skip = -1;
  p.vec_store = (ldc % 8 == 0 && N % 8 == 0 && ((uintptr_t)C & 15) == 0) ? 1 : 0;
  p.rows = 256; p.ksub = 1; p.nbuf = 1; p.acc1_off = 0;
  p.n_tiles = pl.n_tiles; p.m_tiles = pl.m_tiles; p.tn = pl.tn; p.kblocks = pl.kblocks; p.splits = pl.splits;
  const int stage_bytes = TILE_N * BK * 2 + (p.tn / 2) * BK * 2;
  p.stages = kSmemBudget / stage_bytes;
  if (p.stages > 16) p.stages = 16;
  if (const int st = tuning().stages) { if (st >= 2 && st < p.stages) p.stages = st; }
  CUtensorMap mw, mx;
  if (!get_map(W, N, K, K, TILE_N, &mw)) return decline("tensor map of the weight matrix could not be encoded");
  if (!get_map(A, M, K, lda, p.tn / 2, &mx)) return decline("tensor map of the activations could not be encoded");
  if (tuning().debug)
    fprintf(stderr, "cluster k-split gemm M=%d N=%d K=%d mode=%d tn=%d m_tiles=%d n_tiles=%d splits=%d stages=%d\n", M, N, K,
            mode, p.tn, p.m_tiles, p.n_tiles, p.splits, p.stages);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(p.n_tiles * p.m_tiles * 2 * p.splits));
  cfg.blockDim = dim3(kPairThreads);
  cfg.dynamicSmemBytes = (size_t)kSmemBudget + 1024;
  cfg.stream = s;
  cudaLaunchAttribute attrs[2];
  attrs[0].id = cudaLaunchAttributeClusterDimension;
  attrs[0].val.clusterDim.x = (unsigned)(2 * p.splits); attrs[0].val.clusterDim.y = 1; attrs[0].val.clusterDim.z = 1;
  attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attrs[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attrs;
  cfg.numAttrs = tuning().no_pdl ? 1 : 2;
  return mode == 0 ? cudaLaunchKernelEx(&cfg, k_gemm_pair_ks<0>, mw, mx, p) : cudaLaunchKernelEx(&cfg, k_gemm_pair_ks<1>, mw, mx, p);
}

}  // namespace

const char* gemm_decline_reason() { return g_decline.c_str(); }

int gemm_cluster_splits(int M, int N, int K, int mode, int ldc, const void* C) {
  const DevInfo* dv = dev_info();
  return dv && dv->tc_ok ? plan_ks(*dv, M, N, K, mode, ldc, C).splits : 0;
}

// Plans and launches one projection.  A shape the tensor-core kernels cannot take is an error
// (cudaErrorNotSupported, reason in gemm_decline_reason()): there is no second GEMM implementation behind this one.
cudaError_t launch_gemm_tc(const bf16* A, int lda, const bf16* W, const bf16* W2, void* C, int ldc, int M, int N,
                           int K, int mode, const float* row_scale, const GemmScratch& scratch, cudaStream_t s,
                           int* splits_out, const GemmConf* conf) {
  if (mode == 5 && (!conf || !conf->ms || !conf->am || !row_scale)) return decline("confidence partial buffers missing");
  float* const g_partial = scratch.partial;
  const size_t g_partial_floats = scratch.partial_floats;
  if (M <= 0 || N <= 0) return cudaSuccess;
  if (K % 8 || lda % 8 || ((uintptr_t)A & 15) || ((uintptr_t)W & 15) || (W2 && ((uintptr_t)W2 & 15)))
    return decline("operand rows must be 16-byte aligned (K and lda multiples of 8)");
  const DevInfo* dvp = dev_info();
  if (!dvp || !dvp->tc_ok) return decline("the device does not grant the kernels' shared-memory budget");
  const DevInfo& dv = *dvp;
  const int num_sms = dv.num_sms;
  if (mode == 0 || mode == 1) {
    const KsPlan pl = plan_ks(dv, M, N, K, mode, ldc, C);
    if (pl.splits > 0) {
      if (splits_out) *splits_out = 1;
      return launch_gemm_pair_ks(pl, A, lda, W, C, ldc, M, N, K, mode, scratch, s);
    }
  }
  // CTA pairs that share each token tile move fewer bytes per flop and are faster per work item (measured on B200:
  // +8 to +20 %), but their grid has half as many workers.  From 128 tokens on, the pair plan is taken unless it
  // would leave clearly more of its grid idle than the single-CTA plan (few 256-row tiles and no k split, or a last
  // round that is mostly empty).
  bool use_pair = false;
  if (dv.max_pairs > 0) {
    if (tuning().pair >= 0) use_pair = tuning().pair > 0 && M >= tuning().pair;
    else if (M >= ((mode == 2 || mode == 5) ? 64 : 128)) {     // the LM head (many weight tiles, no k split) gains from 64 on
      const bool dual_ = mode == 3 || mode == 5;      // no k split for these
      const int kb = (K + BK - 1) / BK;
      const int rows_p = pair_wide_partials(mode, M, N, K) ? 512 : 256;
      const long long items_p = (long long)((N + rows_p - 1) / rows_p) * ((M + 255) / 256);
      const double busy_p =
          grid_busy(items_p * split_for(items_p, dv.max_pairs, kb, (size_t)M * N, scratch, dual_), dv.max_pairs);
      const bool wide_s = mode != 3 && N >= 512 && K >= 8192;
      const int tn_cap_s = (mode == 3 && (M <= 128 || M > 256)) ? 128 : 256;
      const long long items_s = (long long)((N + (wide_s ? 255 : 127)) / (wide_s ? 256 : 128)) * ((M + tn_cap_s - 1) / tn_cap_s);
      const double busy_s = grid_busy(items_s * split_for(items_s, num_sms, kb, (size_t)M * N, scratch, dual_), num_sms);
      use_pair = busy_p * 1.1 >= busy_s;
    }
  }
  if (use_pair)
    return launch_gemm_pair(dv, A, lda, W, W2, C, ldc, M, N, K, mode, row_scale, scratch, s, splits_out, conf);
  const int dual = mode == 3;
  GemmParams p;
  p.M = M; p.N = N; p.K = K; p.mode = mode; p.dual = dual; p.C = C; p.ldc = ldc; p.row_scale = row_scale;
  p.n_tiles = (N + TILE_N - 1) / TILE_N;
  p.mgroup = 0;
  p.error_flag = scratch.error_flag;
  p.conf_ms = conf ? conf->ms : nullptr; p.conf_am = conf ? conf->am : nullptr; p.skip = conf ? conf->skip : -1;
  p.vec_store = (ldc % 8 == 0 && N % 8 == 0 && ((uintptr_t)C & 15) == 0) ? 1 : 0;
  // ---- token tile and k split ----
  // Few tokens (a block step): one or two token tiles that cover M exactly (UMMA N is any multiple of 16), and a
  // k split that spreads the weight stream over all SMs when there are fewer weight tiles than SMs.
  // Many tokens (a refresh step): the widest tile, no split.
  // Two 128-row weight tiles per work item (gate and up, or 256 rows of one matrix) share each token tile:
  // the same tensor-core work then needs a third fewer bytes through L2.  Their two accumulators fit TMEM
  // twice over only up to 128 tokens; wider token tiles run single-buffered (the epilogue is then not overlapped),
  // which pays only when the main loop is long: measured on B200, 256-row items win for K >= 8192 (the down
  // projection: -25 % at M >= 512) and lose or tie for K = 3584.
  const bool wide_off = tuning().wide_off;
  p.wide = (!dual && !wide_off && M >= 128 && N >= 512 && K >= 8192) ? 1 : 0;
  p.rows = p.wide ? 2 * TILE_N : TILE_N;
  p.n_tiles = (N + p.rows - 1) / p.rows;
  const bool two_a = dual || p.wide;
  int tn_cap = 256;
  if (dual && (wide_off || M <= 128 || M > 256)) tn_cap = 128;   // several token tiles: keep the epilogue overlapped
  p.m_tiles = (M + tn_cap - 1) / tn_cap;
  p.tn = (((M + p.m_tiles - 1) / p.m_tiles) + 15) / 16 * 16;     // tiles of equal width that cover M
  p.nbuf = (two_a && p.tn > 128) ? 1 : 2;
  p.acc1_off = p.nbuf == 1 ? 256 : 128;
  // narrow token tiles are weight-streaming bound: 128-wide k stages halve the per-stage barrier round trips
  p.ksub = p.tn <= 64 ? 2 : 1;
  if (tuning().ksub) p.ksub = tuning().ksub == 2 ? 2 : 1;
  p.kblocks = (K + BK * p.ksub - 1) / (BK * p.ksub);
  p.splits = 1;
  const long long base_items = (long long)p.n_tiles * p.m_tiles;
  if (g_partial && mode != 5 && base_items * 4 < (long long)num_sms * 3) {
    int sp = (int)(num_sms / base_items);
    if (sp > 8) sp = 8;
    while (sp > 1 && (p.kblocks / sp < 4 || (size_t)sp * (size_t)M * N > g_partial_floats)) --sp;
    p.splits = sp < 1 ? 1 : sp;
  }
  if (const int sp = tuning().splits)
    if (sp >= 1 && sp <= 8 && (sp == 1 || (g_partial && (size_t)sp * (size_t)M * N <= g_partial_floats))) p.splits = sp;
  if (mode == 4 && (!g_partial || (size_t)p.splits * (size_t)M * N > g_partial_floats))
    return decline("partial-sum scratch too small for this projection");
  if (dual || mode == 5) p.splits = 1;
  p.partial = g_partial;
  if (splits_out) *splits_out = p.splits;
  const int stage_bytes = p.ksub * ((two_a ? 2 : 1) * TILE_N * BK * 2 + p.tn * BK * 2);
  p.stages = kSmemBudget / stage_bytes;
  if (const int st = tuning().stages) { if (st >= 2 && st < p.stages) p.stages = st; }
  if (p.stages > 16) p.stages = 16;
  if (p.stages < 2) return decline("operand stages do not fit shared memory");

  CUtensorMap mw, mw2, mx;
  if (!get_map(W, N, K, K, TILE_N, &mw)) return decline("tensor map of the weight matrix could not be encoded");
  if (dual) {
    if (!get_map(W2, N, K, K, TILE_N, &mw2)) return decline("tensor map of the second weight matrix could not be encoded");
  } else {
    mw2 = mw;
  }
  if (!get_map(A, M, K, lda, p.tn, &mx)) return decline("tensor map of the activations could not be encoded");

  const long long items = (long long)p.n_tiles * p.m_tiles * p.splits;
  if (tuning().debug)
    fprintf(stderr, "gemm M=%d N=%d K=%d mode=%d tn=%d m_tiles=%d n_tiles=%d splits=%d stages=%d wide=%d nbuf=%d\n", M,
            N, K, mode, p.tn, p.m_tiles, p.n_tiles, p.splits, p.stages, p.wide, p.nbuf);
  const int grid = (int)(items < num_sms ? items : num_sms);
  cudaError_t r = launch_pdl(kernel_tc((p.splits > 1 || mode == 4) ? 4 : mode), dim3(grid), dim3(kThreads),
                             (size_t)kSmemBudget + 1024, s, mw, mw2, mx, p);
  if (r != cudaSuccess) return r;
  if (p.splits > 1 && mode != 4) r = launch_finish(p, mode, num_sms, s);
  return r;
}

}  // namespace bs
