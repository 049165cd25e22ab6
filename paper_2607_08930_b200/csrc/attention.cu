// Ragged bidirectional attention against the dual KV cache (Section 2.5).
// Work item = (row i, q-tile of the row's packed tokens, kv head).  All query heads of the kv head's group
// share each K/V tile (GQA): the flattened "query rows" of a CTA are (token, head-in-group) pairs.
// Keys are the row's cache span [kv_base_i, kv_base_i + vis_i): prefix, fresh block and suffix alike;
// there is no causal mask and no padding mask.  Online softmax with warp shuffles, mma.sync m16n8k16.
#include <math.h>
#include <stdlib.h>

#include <mutex>

#include "tc_common.cuh"

namespace bs {

namespace {

__device__ __forceinline__ void cp_async16(void* dst, const void* src, int bytes) {
  const unsigned d = (unsigned)__cvta_generic_to_shared(dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(d), "l"(src), "r"(bytes));
}
__device__ __forceinline__ void ldsm_x4(unsigned& r0, unsigned& r1, unsigned& r2, unsigned& r3, const void* p) {
  const unsigned a = (unsigned)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(a));
}
__device__ __forceinline__ void ldsm_x4_t(unsigned& r0, unsigned& r1, unsigned& r2, unsigned& r3, const void* p) {
  const unsigned a = (unsigned)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(a));
}
__device__ __forceinline__ void mma16816(float* c, const unsigned* a, unsigned b0, unsigned b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned pack_bf16(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<unsigned*>(&h);
}

// Partial result of one KV chunk of a work item: unnormalised output (fp32) plus (running max in log2 units, sum).
struct AttnPartial {
  float* o;        // [chunks][M][Hq * dh]
  float2* ml;      // [chunks][M][Hq]
  int chunks;
  int M;
};

template <int DH, int KT, int NSTAGE, int MINB>
__global__ void __launch_bounds__(256, MINB) k_attention(const bf16* __restrict__ qkv, const bf16* __restrict__ kc,
                                                         const bf16* __restrict__ vc, bf16* __restrict__ out,
                                                         const int* __restrict__ cu_q, const int* __restrict__ cu_tile,
                                                         const int* __restrict__ kv_base,
                                                         const int* __restrict__ vis_arr, int n_rows, int hq, int hkv,
                                                         int q_tile, AttnPartial part) {
  constexpr int LD = DH + 8;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  bf16* smem = reinterpret_cast<bf16*>(smem_raw);      // [NSTAGE][K tile, V tile][KT][LD]
  const int G = hq / hkv;
  const int kh = blockIdx.y;
  pdl_trigger();
  // which row owns this q-tile: largest r with cu_tile[r] <= blockIdx.x.  (The index arrays were written by the
  // commit / scheduler kernel of the previous step: they are read before the wait for the kernel before this one.)
  const int row = warp_find_row(cu_tile, n_rows, (int)blockIdx.x);
  const int t0 = cu_q[row] + ((int)blockIdx.x - cu_tile[row]) * q_tile;
  const int nt = min(q_tile, cu_q[row + 1] - t0);
  const int vis = vis_arr[row];
  const size_t kvb = (size_t)kv_base[row];
  pdl_wait();
  if (nt <= 0) return;
  const int qkv_ld = (hq + 2 * hkv) * DH;
  // key tiles of this CTA's chunk
  const int nkt_all = (vis + KT - 1) / KT;
  const int per = (nkt_all + part.chunks - 1) / part.chunks;
  const int kt0 = (int)blockIdx.z * per;
  const int kt1 = min(nkt_all, kt0 + per);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nthreads = blockDim.x;
  const bool warp_active = warp * 16 < nt * G;
  // the two flattened query rows this thread owns inside its warp's 16
  const int f0 = warp * 16 + (lane >> 2), f1 = f0 + 8;
  const int tk0 = f0 / G, tk1 = f1 / G;
  const bool v0 = tk0 < nt, v1 = tk1 < nt;
  const int hd0 = kh * G + f0 % G, hd1 = kh * G + f1 % G;

  unsigned qf[DH / 16][4];
  {
    const bf16* q0 = qkv + (size_t)(t0 + (v0 ? tk0 : 0)) * qkv_ld + hd0 * DH + (lane & 3) * 2;
    const bf16* q1 = qkv + (size_t)(t0 + (v1 ? tk1 : 0)) * qkv_ld + hd1 * DH + (lane & 3) * 2;
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks) {
      qf[ks][0] = v0 ? *reinterpret_cast<const unsigned*>(q0 + ks * 16) : 0u;
      qf[ks][1] = v1 ? *reinterpret_cast<const unsigned*>(q1 + ks * 16) : 0u;
      qf[ks][2] = v0 ? *reinterpret_cast<const unsigned*>(q0 + ks * 16 + 8) : 0u;
      qf[ks][3] = v1 ? *reinterpret_cast<const unsigned*>(q1 + ks * 16 + 8) : 0u;
    }
  }

  auto load_tile = [&](int stage, int kt) {
    bf16* sK = smem + stage * 2 * KT * LD;
    bf16* sV = sK + KT * LD;
    constexpr int CH = DH / 8;
    for (int c = tid; c < KT * CH; c += nthreads) {
      const int r = c / CH, cc = (c % CH) * 8;
      const int key = kt * KT + r;
      const bool ok = key < vis;
      const size_t off = ((kvb + (ok ? key : 0)) * hkv + kh) * DH + cc;
      cp_async16(sK + r * LD + cc, kc + off, ok ? 16 : 0);
      cp_async16(sV + r * LD + cc, vc + off, ok ? 16 : 0);
    }
  };

  float o[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  const float sc = 1.4426950408889634f / sqrtf((float)DH);    // log2(e) / sqrt(dh)

#pragma unroll
  for (int i = 0; i < NSTAGE - 1; ++i) {
    if (kt0 + i < kt1) load_tile(i, kt0 + i);
    asm volatile("cp.async.commit_group;\n" ::);
  }
  for (int kt = kt0; kt < kt1; ++kt) {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(NSTAGE - 2));
    __syncthreads();
    if (kt + NSTAGE - 1 < kt1) load_tile((kt - kt0 + NSTAGE - 1) % NSTAGE, kt + NSTAGE - 1);
    asm volatile("cp.async.commit_group;\n" ::);
    if (warp_active) {
      const bf16* sK = smem + ((kt - kt0) % NSTAGE) * 2 * KT * LD;
      const bf16* sV = sK + KT * LD;
      float s[KT / 8][4];
#pragma unroll
      for (int i = 0; i < KT / 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < DH / 16; ++ks) {
#pragma unroll
        for (int np = 0; np < KT / 16; ++np) {
          unsigned b0, b1, b2, b3;
          ldsm_x4(b0, b1, b2, b3,
                  sK + (np * 16 + (lane & 7) + ((lane >> 4) << 3)) * LD + ks * 16 + ((lane >> 3) & 1) * 8);
          mma16816(s[2 * np], qf[ks], b0, b1);
          mma16816(s[2 * np + 1], qf[ks], b2, b3);
        }
      }
      // scale, mask keys beyond the row's span, running max
      float mx0 = -INFINITY, mx1 = -INFINITY;
      const int kbase = kt * KT + (lane & 3) * 2;
#pragma unroll
      for (int i = 0; i < KT / 8; ++i) {
        const int key = kbase + i * 8;
        s[i][0] = key < vis ? s[i][0] * sc : -INFINITY;
        s[i][1] = key + 1 < vis ? s[i][1] * sc : -INFINITY;
        s[i][2] = key < vis ? s[i][2] * sc : -INFINITY;
        s[i][3] = key + 1 < vis ? s[i][3] * sc : -INFINITY;
        mx0 = fmaxf(mx0, fmaxf(s[i][0], s[i][1]));
        mx1 = fmaxf(mx1, fmaxf(s[i][2], s[i][3]));
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float nm0 = fmaxf(m0, mx0), nm1 = fmaxf(m1, mx1);     // finite: every tile holds >= 1 valid key
      const float a0 = exp2f(m0 - nm0), a1 = exp2f(m1 - nm1);
      m0 = nm0;
      m1 = nm1;
      float rs0 = 0.f, rs1 = 0.f;
#pragma unroll
      for (int i = 0; i < KT / 8; ++i) {
        s[i][0] = exp2f(s[i][0] - nm0);
        s[i][1] = exp2f(s[i][1] - nm0);
        s[i][2] = exp2f(s[i][2] - nm1);
        s[i][3] = exp2f(s[i][3] - nm1);
        rs0 += s[i][0] + s[i][1];
        rs1 += s[i][2] + s[i][3];
      }
      l0 = l0 * a0 + rs0;
      l1 = l1 * a1 + rs1;
#pragma unroll
      for (int i = 0; i < DH / 8; ++i) {
        o[i][0] *= a0;
        o[i][1] *= a0;
        o[i][2] *= a1;
        o[i][3] *= a1;
      }
#pragma unroll
      for (int kk = 0; kk < KT / 16; ++kk) {
        unsigned pa[4];
        pa[0] = pack_bf16(s[2 * kk][0], s[2 * kk][1]);
        pa[1] = pack_bf16(s[2 * kk][2], s[2 * kk][3]);
        pa[2] = pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]);
        pa[3] = pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
        for (int nd = 0; nd < DH / 16; ++nd) {
          unsigned b0, b1, b2, b3;
          ldsm_x4_t(b0, b1, b2, b3,
                    sV + (kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LD + nd * 16 + (lane >> 4) * 8);
          mma16816(o[2 * nd], pa, b0, b1);
          mma16816(o[2 * nd + 1], pa, b2, b3);
        }
      }
    }
  }
  asm volatile("cp.async.wait_group 0;\n" ::);
  if (!warp_active) return;
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const int out_ld = hq * DH;
  if (part.chunks > 1) {
    // unnormalised partial of this KV chunk; the combine kernel merges the chunks
    const size_t zoff = (size_t)blockIdx.z * part.M;
    if (v0) {
      float* dst = part.o + (zoff + t0 + tk0) * out_ld + hd0 * DH + (lane & 3) * 2;
      if (l0 > 0.f) {
#pragma unroll
        for (int i = 0; i < DH / 8; ++i) *reinterpret_cast<float2*>(dst + i * 8) = make_float2(o[i][0], o[i][1]);
      }
      if ((lane & 3) == 0) part.ml[(zoff + t0 + tk0) * hq + hd0] = make_float2(m0, l0);
    }
    if (v1) {
      float* dst = part.o + (zoff + t0 + tk1) * out_ld + hd1 * DH + (lane & 3) * 2;
      if (l1 > 0.f) {
#pragma unroll
        for (int i = 0; i < DH / 8; ++i) *reinterpret_cast<float2*>(dst + i * 8) = make_float2(o[i][2], o[i][3]);
      }
      if ((lane & 3) == 0) part.ml[(zoff + t0 + tk1) * hq + hd1] = make_float2(m1, l1);
    }
    return;
  }
  const float i0 = 1.0f / l0, i1 = 1.0f / l1;
  if (v0) {
    bf16* dst = out + (size_t)(t0 + tk0) * out_ld + hd0 * DH + (lane & 3) * 2;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i)
      *reinterpret_cast<__nv_bfloat162*>(dst + i * 8) = __floats2bfloat162_rn(o[i][0] * i0, o[i][1] * i0);
  }
  if (v1) {
    bf16* dst = out + (size_t)(t0 + tk1) * out_ld + hd1 * DH + (lane & 3) * 2;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i)
      *reinterpret_cast<__nv_bfloat162*>(dst + i * 8) = __floats2bfloat162_rn(o[i][2] * i1, o[i][3] * i1);
  }
}

// Merges the KV chunks of every (token, head): out = sum_c w_c o_c / sum_c w_c l_c with w_c = 2^(m_c - max m).
__global__ void __launch_bounds__(256) k_attention_combine(AttnPartial part, bf16* __restrict__ out, int hq, int dh) {
  pdl_wait();
  pdl_trigger();
  const int t = blockIdx.x;
  const int out_ld = hq * dh;
  const int pairs = out_ld / 2;
  for (int u = threadIdx.x; u < pairs; u += 256) {
    const int h = (2 * u) / dh;
    float mmax = -INFINITY;
    for (int c = 0; c < part.chunks; ++c) {
      const float2 ml = part.ml[((size_t)c * part.M + t) * hq + h];
      if (ml.y > 0.f) mmax = fmaxf(mmax, ml.x);
    }
    float2 acc = make_float2(0.f, 0.f);
    float L = 0.f;
    for (int c = 0; c < part.chunks; ++c) {
      const float2 ml = part.ml[((size_t)c * part.M + t) * hq + h];
      if (ml.y > 0.f) {
        const float w = exp2f(ml.x - mmax);
        const float2 ov = *reinterpret_cast<const float2*>(part.o + ((size_t)c * part.M + t) * out_ld + 2 * u);
        acc.x += w * ov.x;
        acc.y += w * ov.y;
        L += w * ml.y;
      }
    }
    const float inv = 1.0f / L;
    *reinterpret_cast<__nv_bfloat162*>(out + (size_t)t * out_ld + 2 * u) = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
  }
}
}  // namespace

int attention_tc_q_tile(int hq, int hkv);
cudaError_t launch_attention_tc(const bf16* qkv, const bf16* kc, const bf16* vc, bf16* out, const int* cu_q,
                                const int* cu_tile, const int* kv_base, const int* vis, int n_rows, int n_tiles,
                                int M, long long kv_rows, int max_nq, int max_vis, int hq, int hkv, int dh,
                                float* scratch, size_t scratch_floats, int* error_flag, cudaStream_t s,
                                bool* handled);

static bool use_tc_attention(int hq, int hkv, int dh) {
  static const bool legacy = getenv("BS_ATTN_LEGACY") != nullptr;
  return !legacy && dh == 128 && hkv > 0 && hq % hkv == 0 && hq / hkv <= 8;
}

// Query tokens per attention work item; the index kernels build their work-item prefix with it.
int attention_q_tile(int hq, int hkv, int dh) {
  if (use_tc_attention(hq, hkv, dh)) return attention_tc_q_tile(hq, hkv);
  const int G = hq / hkv;
  return G >= 5 ? 16 : (G == 1 ? 64 : 32);     // the legacy kernel's tile
}

namespace {
template <int DH, int KT, int NSTAGE, int MINB>
cudaError_t launch_variant(dim3 grid, int threads, cudaStream_t s, const bf16* qkv, const bf16* kc, const bf16* vc,
                           bf16* out, const int* cu_q, const int* cu_tile, const int* kv_base, const int* vis,
                           int n_rows, int hq, int hkv, int qt, AttnPartial part) {
  constexpr size_t smem = (size_t)NSTAGE * 2 * KT * (DH + 8) * sizeof(bf16);
  static int done_on[kMaxDevices];         // per device: the attribute belongs to the device's copy of the kernel
  static std::mutex mu;
  int* done = device_slot(done_on);
  if (!done) return cudaErrorInvalidDevice;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!*done) {
      if (cudaFuncSetAttribute(k_attention<DH, KT, NSTAGE, MINB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)smem) != cudaSuccess)
        return cudaErrorInvalidDevice;
      *done = 1;
    }
  }
  return launch_pdl(k_attention<DH, KT, NSTAGE, MINB>, grid, dim3(threads), smem, s, qkv, kc, vc, out, cu_q, cu_tile,
                    kv_base, vis, n_rows, hq, hkv, qt, part);
}
}  // namespace

cudaError_t launch_attention(const bf16* qkv, const bf16* kc, const bf16* vc, bf16* out, const int* cu_q,
                             const int* cu_tile, const int* kv_base, const int* vis, int n_rows, int n_tiles, int M,
                             int max_vis, int max_nq, long long kv_rows, int hq, int hkv, int dh, float* scratch,
                             size_t scratch_floats, int* error_flag, cudaStream_t s) {
  if (n_tiles <= 0 || n_rows <= 0) return cudaSuccess;
  // Block steps of a model with one or two query heads per kv head are pure cache streaming with a few dozen
  // query rows: several small CTAs per SM hide the load latency better than one tensor-core CTA.  Every row has
  // at most one work item there, so the work-item prefix is the same for either kernel's q-tile.
  // (BS_ATTN_STREAM, read once: 0 sends these steps to the tensor-core kernel as well, 1 is the default)
  static const int env_stream = getenv("BS_ATTN_STREAM") ? atoi(getenv("BS_ATTN_STREAM")) : 1;
  const bool stream_small = env_stream != 0 && max_nq > 0 && max_nq <= 32 && hq / hkv <= 2;
  if (use_tc_attention(hq, hkv, dh) && !stream_small) {
    bool handled = false;
    cudaError_t r = launch_attention_tc(qkv, kc, vc, out, cu_q, cu_tile, kv_base, vis, n_rows, n_tiles, M, kv_rows,
                                        max_nq, max_vis, hq, hkv, dh, scratch, scratch_floats, error_flag, s, &handled);
    return handled ? r : cudaErrorNotSupported;     // the work-item prefix was built for this kernel's q-tile
  }
  const int G = hq / hkv;
  const int qt = G >= 5 ? 16 : (G == 1 ? 64 : 32);
  // 16 flattened (token, head) rows per warp; a block step has at most L <= 32 query tokens per row, so a
  // 64-token q-tile (MHA) needs only the warps that hold tokens
  int qt_used = qt;
  if (max_nq > 0 && max_nq < qt) qt_used = (max_nq + 15) / 16 * 16;
  const int threads = ((qt_used * G + 15) / 16) * 32;
  if (threads > 256 || (dh != 64 && dh != 128) || hq % hkv != 0) return cudaErrorInvalidValue;
  // KV chunks: a block step has few (row, kv head, q tile) items, each a long serial walk over the row's keys;
  // splitting the walk fills the SMs.  A refresh step has plenty of items already.
  static int num_sms_of[kMaxDevices];
  int* sms = device_slot(num_sms_of);
  if (!sms) return cudaErrorInvalidDevice;
  if (!*sms) {
    int dev = 0, n = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
      return cudaErrorInvalidDevice;
    *sms = n;
  }
  const int num_sms = *sms;
  // (measured on B200: with fewer work items than a quarter / a half of the SMs, 4 / 2 chunks shorten the
  // serial walk enough to pay for the merge; beyond that the legacy-path MMAs are the limit and chunks only add work)
  const long long base = (long long)n_tiles * hkv;
  int chunks = 1;
  if (scratch && max_vis >= 256) {
    chunks = base * 4 <= num_sms + 12 ? 4 : (base * 2 <= num_sms ? 2 : 1);
    while (chunks > 1 && (size_t)chunks * M * ((size_t)hq * dh + 2 * hq) > scratch_floats) chunks >>= 1;
  }
  // measurement overrides, read once per process
  static const int env_chunks = getenv("BS_ATTN_CHUNKS") ? atoi(getenv("BS_ATTN_CHUNKS")) : 0;
  static const int variant = getenv("BS_ATTN_VARIANT") ? atoi(getenv("BS_ATTN_VARIANT")) : 1;
  if (env_chunks >= 1 && (env_chunks == 1 || scratch)) chunks = env_chunks;
  AttnPartial part;
  part.chunks = chunks;
  part.M = M;
  part.o = scratch;
  part.ml = reinterpret_cast<float2*>(scratch + (size_t)chunks * M * hq * dh);
  dim3 grid(n_tiles, hkv, chunks);
  cudaError_t r;
  if (dh == 128) {
    if (variant == 0)
      r = launch_variant<128, 32, 3, 2>(grid, threads, s, qkv, kc, vc, out, cu_q, cu_tile, kv_base, vis, n_rows, hq,
                                        hkv, qt, part);
    else if (variant == 2)
      r = launch_variant<128, 64, 3, 1>(grid, threads, s, qkv, kc, vc, out, cu_q, cu_tile, kv_base, vis, n_rows, hq,
                                        hkv, qt, part);
    else
      r = launch_variant<128, 64, 2, 1>(grid, threads, s, qkv, kc, vc, out, cu_q, cu_tile, kv_base, vis, n_rows, hq,
                                        hkv, qt, part);
  } else {
    r = launch_variant<64, 64, 2, 2>(grid, threads, s, qkv, kc, vc, out, cu_q, cu_tile, kv_base, vis, n_rows, hq, hkv,
                                     qt, part);
  }
  if (r != cudaSuccess) return r;
  if (chunks > 1) {
    r = launch_pdl(k_attention_combine, dim3(M), dim3(256), 0, s, part, out, hq, dh);
  }
  return r;
}

}  // namespace bs
