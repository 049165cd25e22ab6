// HBM-bound row kernels: embedding gather, RMSNorm, RoPE at gathered positions + KV scatter,
// and the per-row vocabulary pass of the confidence epilogue.
#include <math.h>

#include "conf_merge.cuh"

namespace bs {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// x[t, :] = E[token at (row, position) of packed token t]   (gather of the active regions, Section 2.5)
__global__ void k_embed(DevState st, const bf16* __restrict__ embed, float* __restrict__ x, int M, int d) {
  pdl_wait();
  pdl_trigger();
  const int t = blockIdx.x;
  if (t >= M) return;
  const int trow = st.tok_row[t], tpos = st.tok_pos[t];
  if (!BS_INDEX_OK(trow >= 0 && trow < st.max_batch && tpos >= 0 && tpos < st.max_row_tokens, st.hdr + H_ERROR, SITE_EMBED))
    return;
  const int slot = st.row_slot[trow];
  if (!BS_INDEX_OK(slot >= 0 && slot < st.max_requests, st.hdr + H_ERROR, SITE_EMBED)) return;
  const int id = st.tokens[(size_t)slot * st.max_row_tokens + tpos];
  if (!BS_INDEX_OK(id >= 0 && id < st.vocab, st.hdr + H_ERROR, SITE_EMBED)) return;
  const uint4* src = reinterpret_cast<const uint4*>(embed + (size_t)id * d);
  float4* dst = reinterpret_cast<float4*>(x + (size_t)t * d);
  for (int c = threadIdx.x; c < d / 8; c += blockDim.x) {
    const uint4 v = src[c];
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
    const float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
    const float2 e = __bfloat1622float2(h[2]), f = __bfloat1622float2(h[3]);
    dst[2 * c] = make_float4(a.x, a.y, b.x, b.y);
    dst[2 * c + 1] = make_float4(e.x, e.y, f.x, f.y);
  }
}

// y[m, :] = bf16(w * x[row, :] * rsqrt(mean(x^2) + eps)); one CTA per output row.
__global__ void __launch_bounds__(256) k_rmsnorm(const float* __restrict__ x, const int* __restrict__ idx,
                                                 const bf16* __restrict__ w, bf16* __restrict__ y, int d, float eps,
                                                 IndexLimits lim) {
  __shared__ float red[8];
  pdl_wait();
  pdl_trigger();
  const int m = blockIdx.x;
  const int row = idx ? idx[m] : m;
  if (lim.error_word && !BS_INDEX_OK(row >= 0 && row < lim.x_rows, lim.error_word, SITE_NORM_GATHER)) return;
  const float4* src = reinterpret_cast<const float4*>(x + (size_t)row * d);
  float ss = 0.f;
  for (int c = threadIdx.x; c < d / 4; c += 256) {
    const float4 v = src[c];
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) tot += red[i];
  const float r = rsqrtf(tot / (float)d + eps);
  const uint2* wp = reinterpret_cast<const uint2*>(w);
  uint2* dst = reinterpret_cast<uint2*>(y + (size_t)m * d);
  for (int c = threadIdx.x; c < d / 4; c += 256) {
    const float4 v = src[c];
    const uint2 wv = wp[c];
    const __nv_bfloat162* wh = reinterpret_cast<const __nv_bfloat162*>(&wv);
    const float2 w0 = __bfloat1622float2(wh[0]), w1 = __bfloat1622float2(wh[1]);
    __nv_bfloat162 o0 = __floats2bfloat162_rn(v.x * r * w0.x, v.y * r * w0.y);
    __nv_bfloat162 o1 = __floats2bfloat162_rn(v.z * r * w1.x, v.w * r * w1.y);
    uint2 o;
    o.x = *reinterpret_cast<unsigned*>(&o0);
    o.y = *reinterpret_cast<unsigned*>(&o1);
    dst[c] = o;
  }
}

// One CTA per packed token: rotate q (in place) and k by the token's position id, scatter k and v to the
// token's physical cache row.  cos_sin: [max_pos, dh/2] float2 (cos, sin).
__global__ void __launch_bounds__(256) k_rope_kv(bf16* __restrict__ qkv, const int* __restrict__ tok_pos,
                                                 const int* __restrict__ tok_kv, bf16* __restrict__ kc,
                                                 bf16* __restrict__ vc, int hq, int hkv, int dh,
                                                 const float2* __restrict__ cos_sin, IndexLimits lim) {
  pdl_wait();
  pdl_trigger();
  const int t = blockIdx.x;
  const int pos = tok_pos[t];
  if (lim.error_word && !BS_INDEX_OK(pos >= 0 && pos < lim.max_pos && tok_kv[t] >= 0 && tok_kv[t] < lim.kv_rows,
                                     lim.error_word, SITE_ROPE_KV))
    return;
  const size_t kvrow = (size_t)tok_kv[t];
  const int half = dh / 2;
  bf16* base = qkv + (size_t)t * (hq + 2 * hkv) * dh;
  const float2* cs = cos_sin + (size_t)pos * half;
  const int pairs_per_head = half / 2;                  // bf16x2 granules per half head
  const int n_rot = (hq + hkv) * pairs_per_head;
  for (int u = threadIdx.x; u < n_rot; u += 256) {
    const int h = u / pairs_per_head, j = (u % pairs_per_head) * 2;
    __nv_bfloat162* p1 = reinterpret_cast<__nv_bfloat162*>(base + h * dh + j);
    __nv_bfloat162* p2 = reinterpret_cast<__nv_bfloat162*>(base + h * dh + half + j);
    const float2 a = __bfloat1622float2(*p1), b = __bfloat1622float2(*p2);
    const float2 c0 = cs[j], c1 = cs[j + 1];
    const __nv_bfloat162 o1 = __floats2bfloat162_rn(a.x * c0.x - b.x * c0.y, a.y * c1.x - b.y * c1.y);
    const __nv_bfloat162 o2 = __floats2bfloat162_rn(b.x * c0.x + a.x * c0.y, b.y * c1.x + a.y * c1.y);
    if (h < hq) {
      *p1 = o1;
      *p2 = o2;
    } else {
      bf16* dstk = kc + (kvrow * hkv + (h - hq)) * dh;
      *reinterpret_cast<__nv_bfloat162*>(dstk + j) = o1;
      *reinterpret_cast<__nv_bfloat162*>(dstk + half + j) = o2;
    }
  }
  const uint4* vsrc = reinterpret_cast<const uint4*>(base + (hq + hkv) * dh);
  uint4* vdst = reinterpret_cast<uint4*>(vc + kvrow * hkv * dh);
  for (int u = threadIdx.x; u < hkv * dh / 8; u += 256) vdst[u] = vsrc[u];
}

// Per row of fp32 logits: online (max, sum exp, argmax) in one pass, mask id excluded,
// lowest id on ties; conf = 1 / sum exp(z - max) = exp(max - logsumexp).
constexpr int kConfThreads = 512;
__global__ void __launch_bounds__(kConfThreads) k_confidence(const float* __restrict__ logits, int vocab, int mask_id,
                                                             int* __restrict__ tok, float* __restrict__ conf) {
  __shared__ float s_m[kConfThreads / 32], s_s[kConfThreads / 32];
  __shared__ int s_i[kConfThreads / 32];
  pdl_wait();
  pdl_trigger();
  const int row = blockIdx.x;
  const float* z = logits + (size_t)row * vocab;
  float m = -INFINITY, s = 0.f;
  int am = 0x7fffffff;
  const int nv = (vocab % 4 == 0) ? vocab / 4 : 0;      // vector part (rows are 16-byte aligned iff vocab % 4 == 0)
  const float4* z4 = reinterpret_cast<const float4*>(z);
  for (int c = threadIdx.x; c < nv; c += kConfThreads) {
    float4 v = __ldcs(z4 + c);
    const int i0 = c * 4;
    if (mask_id >= i0 && mask_id < i0 + 4) {
      if (mask_id == i0) v.x = -INFINITY;
      else if (mask_id == i0 + 1) v.y = -INFINITY;
      else if (mask_id == i0 + 2) v.z = -INFINITY;
      else v.w = -INFINITY;
    }
    float lm = v.x;
    int li = i0;
    if (v.y > lm) { lm = v.y; li = i0 + 1; }
    if (v.z > lm) { lm = v.z; li = i0 + 2; }
    if (v.w > lm) { lm = v.w; li = i0 + 3; }
    if (lm > m) {
      s *= __expf(m - lm);
      m = lm;
      am = li;
    }
    if (m > -INFINITY) s += __expf(v.x - m) + __expf(v.y - m) + __expf(v.z - m) + __expf(v.w - m);
  }
  for (int i = nv * 4 + threadIdx.x; i < vocab; i += kConfThreads) {
    const float v = (i == mask_id) ? -INFINITY : z[i];
    if (v > m) {
      s *= __expf(m - v);
      m = v;
      am = i;
    }
    if (m > -INFINITY) s += __expf(v - m);
  }
  // merge (m, s, am): larger max wins, ties keep the lower id
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, o);
    const float os = __shfl_xor_sync(0xffffffffu, s, o);
    const int oi = __shfl_xor_sync(0xffffffffu, am, o);
    const float nm = fmaxf(m, om);
    const float a = (m > -INFINITY) ? s * __expf(m - nm) : 0.f;
    const float b = (om > -INFINITY) ? os * __expf(om - nm) : 0.f;
    if (om > m || (om == m && oi < am)) am = oi;
    m = nm;
    s = a + b;
  }
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) { s_m[w] = m; s_s[w] = s; s_i[w] = am; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float M = s_m[0], S = s_s[0];
    int A = s_i[0];
    for (int k = 1; k < kConfThreads / 32; ++k) {
      const float om = s_m[k], os = s_s[k];
      const int oi = s_i[k];
      const float nm = fmaxf(M, om);
      const float a = (M > -INFINITY) ? S * __expf(M - nm) : 0.f;
      const float b = (om > -INFINITY) ? os * __expf(om - nm) : 0.f;
      if (om > M || (om == M && oi < A)) A = oi;
      M = nm;
      S = a + b;
    }
    tok[row] = A;
    conf[row] = 1.0f / S;
  }
}

// Second stage of the fused LM-head confidence pass: the GEMM epilogue left one partial per (group of 32 vocabulary
// entries, token).  CTA (x, y): 32 consecutive tokens (lane = token, so every load is one coalesced 256-byte row of
// the [group][token] arrays) and slice y of the groups, its eight warps striding over the slice; one slice partial
// per token comes out.  The commit kernel merges the kConfSlices slices.
constexpr int kMergeWarps = 8;
__global__ void __launch_bounds__(kMergeWarps * 32) k_conf_merge(const float2* __restrict__ group_ms,
                                                                 const int* __restrict__ group_am, int M, int n_groups,
                                                                 float2* __restrict__ slice_ms,
                                                                 int* __restrict__ slice_am) {
  __shared__ float s_m[kMergeWarps][32], s_s[kMergeWarps][32];
  __shared__ int s_i[kMergeWarps][32];
  pdl_wait();
  pdl_trigger();
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int t = blockIdx.x * 32 + lane;
  const int per = (n_groups + kConfSlices - 1) / kConfSlices;
  const int g0 = blockIdx.y * per, g1 = min(n_groups, g0 + per);
  ConfPart acc = conf_empty();
  if (t < M) {
    int g = g0 + w;
    for (; g + 3 * kMergeWarps < g1; g += 4 * kMergeWarps) {       // four loads in flight per thread
      float2 ms[4];
      int am[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const size_t at = (size_t)(g + u * kMergeWarps) * M + t;
        ms[u] = __ldcs(group_ms + at);
        am[u] = __ldcs(group_am + at);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) conf_merge(acc, ms[u].x, ms[u].y, am[u]);
    }
    for (; g < g1; g += kMergeWarps) {
      const size_t at = (size_t)g * M + t;
      const float2 ms = __ldcs(group_ms + at);
      conf_merge(acc, ms.x, ms.y, __ldcs(group_am + at));
    }
  }
  s_m[w][lane] = acc.m; s_s[w][lane] = acc.s; s_i[w][lane] = acc.am;
  __syncthreads();
  if (w == 0 && t < M) {
    for (int k = 1; k < kMergeWarps; ++k) conf_merge(acc, s_m[k][lane], s_s[k][lane], s_i[k][lane]);
    slice_ms[(size_t)blockIdx.y * M + t] = make_float2(acc.m, acc.s);
    slice_am[(size_t)blockIdx.y * M + t] = acc.am;
  }
}

__global__ void k_conf_final(const float2* __restrict__ slice_ms, const int* __restrict__ slice_am, int M,
                             int* __restrict__ tok, float* __restrict__ conf) {
  pdl_wait();
  pdl_trigger();
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < M) merge_conf_slices(slice_ms, slice_am, M, t, tok + t, conf + t);
}

constexpr int kMaxSplits = 8;

// Finishing kernel of the QKV projection on block steps: adds the k-split partial sums in split order, rounds q / k / v
// to bf16, rotates q and k at the token's position id and scatters k, v to the token's cache row.
// grid (tokens, head groups of kHeadsPerBlock); all partial loads of an element are issued before they are summed.
// Eight heads of 128 dims give each of the 128 threads exactly one unit of 4 rotation pairs (four heads left half of
// the CTA idle and doubled the number of CTAs: the job measured 0.45 % slower).
constexpr int kHeadsPerBlock = 8;
__global__ void __launch_bounds__(128) k_finish_qkv_rope(const float* __restrict__ partial, int splits, int M,
                                                         bf16* __restrict__ qkv, const int* __restrict__ tok_pos,
                                                         const int* __restrict__ tok_kv, bf16* __restrict__ kc,
                                                         bf16* __restrict__ vc, int hq, int hkv, int dh,
                                                         const float2* __restrict__ cos_sin, IndexLimits lim) {
  pdl_wait();
  pdl_trigger();
  const int t = blockIdx.x;
  if (lim.error_word && !BS_INDEX_OK(tok_pos[t] >= 0 && tok_pos[t] < lim.max_pos && tok_kv[t] >= 0 &&
                                         tok_kv[t] < lim.kv_rows, lim.error_word, SITE_FINISH_QKV))
    return;
  const int n_heads = hq + 2 * hkv;
  const int N = n_heads * dh, half = dh / 2;
  const size_t slice = (size_t)M * N;
  const float* row = partial + (size_t)t * N;
  const int pos = tok_pos[t];
  const size_t kvrow = (size_t)tok_kv[t];
  const float2* cs = cos_sin + (size_t)pos * half;
  bf16* qrow = qkv + (size_t)t * N;
  const int quads_per_head = half / 4;                 // a thread rotates 4 adjacent pairs (j..j+3, j+half..)
  const int h0 = blockIdx.y * kHeadsPerBlock;
  for (int u = threadIdx.x; u < kHeadsPerBlock * quads_per_head; u += 128) {
    const int h = h0 + u / quads_per_head, j = (u % quads_per_head) * 4;
    if (h >= n_heads) break;
    float4 pa[kMaxSplits], pb[kMaxSplits];
#pragma unroll
    for (int s = 0; s < kMaxSplits; ++s)
      if (s < splits) {
        pa[s] = *reinterpret_cast<const float4*>(row + s * slice + h * dh + j);
        if (h < hq + hkv) pb[s] = *reinterpret_cast<const float4*>(row + s * slice + h * dh + half + j);
      }
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
#pragma unroll
    for (int s = 0; s < kMaxSplits; ++s)
      if (s < splits) {
        a.x += pa[s].x; a.y += pa[s].y; a.z += pa[s].z; a.w += pa[s].w;
        if (h < hq + hkv) { b.x += pb[s].x; b.y += pb[s].y; b.z += pb[s].z; b.w += pb[s].w; }
      }
    if (h < hq + hkv) {
      // the projection's output is a bf16 tensor: round, rotate in fp32, round again
      const float2 a01 = __bfloat1622float2(__floats2bfloat162_rn(a.x, a.y));
      const float2 a23 = __bfloat1622float2(__floats2bfloat162_rn(a.z, a.w));
      const float2 b01 = __bfloat1622float2(__floats2bfloat162_rn(b.x, b.y));
      const float2 b23 = __bfloat1622float2(__floats2bfloat162_rn(b.z, b.w));
      const float2 c0 = cs[j], c1 = cs[j + 1], c2 = cs[j + 2], c3 = cs[j + 3];
      __nv_bfloat162 lo01 = __floats2bfloat162_rn(a01.x * c0.x - b01.x * c0.y, a01.y * c1.x - b01.y * c1.y);
      __nv_bfloat162 lo23 = __floats2bfloat162_rn(a23.x * c2.x - b23.x * c2.y, a23.y * c3.x - b23.y * c3.y);
      __nv_bfloat162 hi01 = __floats2bfloat162_rn(b01.x * c0.x + a01.x * c0.y, b01.y * c1.x + a01.y * c1.y);
      __nv_bfloat162 hi23 = __floats2bfloat162_rn(b23.x * c2.x + a23.x * c2.y, b23.y * c3.x + a23.y * c3.y);
      bf16* dst = h < hq ? qrow + h * dh : kc + (kvrow * hkv + (h - hq)) * dh;
      uint2 lo, hi;
      lo.x = *reinterpret_cast<unsigned*>(&lo01); lo.y = *reinterpret_cast<unsigned*>(&lo23);
      hi.x = *reinterpret_cast<unsigned*>(&hi01); hi.y = *reinterpret_cast<unsigned*>(&hi23);
      *reinterpret_cast<uint2*>(dst + j) = lo;
      *reinterpret_cast<uint2*>(dst + half + j) = hi;
    } else {
      // a v head: this thread owns 4 values of the first half; the second half is handled below
      bf16* dst = vc + (kvrow * hkv + (h - hq - hkv)) * dh;
      __nv_bfloat162 v01 = __floats2bfloat162_rn(a.x, a.y), v23 = __floats2bfloat162_rn(a.z, a.w);
      uint2 o;
      o.x = *reinterpret_cast<unsigned*>(&v01); o.y = *reinterpret_cast<unsigned*>(&v23);
      *reinterpret_cast<uint2*>(dst + j) = o;
      float4 c = make_float4(0.f, 0.f, 0.f, 0.f);
      float4 pc[kMaxSplits];
#pragma unroll
      for (int s = 0; s < kMaxSplits; ++s)
        if (s < splits) pc[s] = *reinterpret_cast<const float4*>(row + s * slice + h * dh + half + j);
#pragma unroll
      for (int s = 0; s < kMaxSplits; ++s)
        if (s < splits) { c.x += pc[s].x; c.y += pc[s].y; c.z += pc[s].z; c.w += pc[s].w; }
      v01 = __floats2bfloat162_rn(c.x, c.y);
      v23 = __floats2bfloat162_rn(c.z, c.w);
      o.x = *reinterpret_cast<unsigned*>(&v01); o.y = *reinterpret_cast<unsigned*>(&v23);
      *reinterpret_cast<uint2*>(dst + half + j) = o;
    }
  }
}

// Finishing kernel of the O and down projections on block steps: x += sum of the k-split partial sums (split order),
// then, if a gain vector is given, the RMSNorm that feeds the next projection.  One CTA per token.
__global__ void __launch_bounds__(256) k_finish_residual_norm(const float* __restrict__ partial, int splits, int M,
                                                              int d, float* __restrict__ x,
                                                              const bf16* __restrict__ w, bf16* __restrict__ h,
                                                              float eps) {
  __shared__ float red[8];
  pdl_wait();
  pdl_trigger();
  const int t = blockIdx.x;
  const size_t slice = (size_t)M * d;
  float4* xr = reinterpret_cast<float4*>(x + (size_t)t * d);
  const float* prow = partial + (size_t)t * d;
  float4 vals[8];
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int c = threadIdx.x + i * 256;
    if (c < d / 4) {
      float4 v = xr[c];
      float4 pv[kMaxSplits];
#pragma unroll
      for (int s = 0; s < kMaxSplits; ++s)
        if (s < splits) pv[s] = *reinterpret_cast<const float4*>(prow + s * slice + 4 * c);
#pragma unroll
      for (int s = 0; s < kMaxSplits; ++s)
        if (s < splits) { v.x += pv[s].x; v.y += pv[s].y; v.z += pv[s].z; v.w += pv[s].w; }
      xr[c] = v;
      vals[i] = v;
      ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
  }
  if (w == nullptr) return;
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) tot += red[i];
  const float r = rsqrtf(tot / (float)d + eps);
  const uint2* wp = reinterpret_cast<const uint2*>(w);
  uint2* dst = reinterpret_cast<uint2*>(h + (size_t)t * d);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int c = threadIdx.x + i * 256;
    if (c < d / 4) {
      const float4 v = vals[i];
      const uint2 wv = wp[c];
      const __nv_bfloat162* wh = reinterpret_cast<const __nv_bfloat162*>(&wv);
      const float2 w0 = __bfloat1622float2(wh[0]), w1 = __bfloat1622float2(wh[1]);
      __nv_bfloat162 o0 = __floats2bfloat162_rn(v.x * r * w0.x, v.y * r * w0.y);
      __nv_bfloat162 o1 = __floats2bfloat162_rn(v.z * r * w1.x, v.w * r * w1.y);
      uint2 o;
      o.x = *reinterpret_cast<unsigned*>(&o0);
      o.y = *reinterpret_cast<unsigned*>(&o1);
      dst[c] = o;
    }
  }
}

static IndexLimits limits_or_none(const IndexLimits* limits) {
  return (limits && kBoundsCheck) ? *limits : IndexLimits{0, 0, 0, nullptr};
}
cudaError_t launch_finish_qkv_rope(const float* partial, int splits, int M, bf16* qkv, const int* tok_pos,
                                   const int* tok_kv, bf16* kc, bf16* vc, int hq, int hkv, int dh,
                                   const float* cos_sin, cudaStream_t s, const IndexLimits* limits) {
  if (M <= 0) return cudaSuccess;
  if (splits > kMaxSplits || dh % 8) return cudaErrorInvalidValue;
  dim3 grid(M, (hq + 2 * hkv + kHeadsPerBlock - 1) / kHeadsPerBlock);
  return launch_pdl(k_finish_qkv_rope, grid, dim3(128), 0, s, partial, splits, M, qkv, tok_pos, tok_kv, kc, vc, hq, hkv,
                    dh, reinterpret_cast<const float2*>(cos_sin), limits_or_none(limits));
}
cudaError_t launch_finish_residual_norm(const float* partial, int splits, int M, int d, float* x, const bf16* w,
                                        bf16* h, float eps, cudaStream_t s) {
  if (M <= 0) return cudaSuccess;
  if (d > 8192 || splits > kMaxSplits) return cudaErrorInvalidValue;
  return launch_pdl(k_finish_residual_norm, dim3(M), dim3(256), 0, s, partial, splits, M, d, x, w, h, eps);
}

cudaError_t launch_embed(const DevState& st, const bf16* embed, float* x, int M, int d, cudaStream_t s) {
  if (M <= 0) return cudaSuccess;
  return launch_pdl(k_embed, dim3(M), dim3(128), 0, s, st, embed, x, M, d);
}
cudaError_t launch_rmsnorm(const float* x, const int* idx, const bf16* w, bf16* y, int M, int d, float eps,
                           cudaStream_t s, const IndexLimits* limits) {
  if (M <= 0) return cudaSuccess;
  return launch_pdl(k_rmsnorm, dim3(M), dim3(256), 0, s, x, idx, w, y, d, eps, limits_or_none(limits));
}
cudaError_t launch_rope_kv(bf16* qkv, const int* tok_pos, const int* tok_kv, bf16* kc, bf16* vc, int M, int hq,
                           int hkv, int dh, const float* cos_sin, cudaStream_t s, const IndexLimits* limits) {
  if (M <= 0) return cudaSuccess;
  return launch_pdl(k_rope_kv, dim3(M), dim3(256), 0, s, qkv, tok_pos, tok_kv, kc, vc, hq, hkv, dh,
                    reinterpret_cast<const float2*>(cos_sin), limits_or_none(limits));
}
cudaError_t launch_confidence(const float* logits, int n_rows, int vocab, int mask_id, int* tok, float* conf,
                              cudaStream_t s) {
  if (n_rows <= 0) return cudaSuccess;
  return launch_pdl(k_confidence, dim3(n_rows), dim3(kConfThreads), 0, s, logits, vocab, mask_id, tok, conf);
}

cudaError_t launch_lm_head_conf(const bf16* hf, int lda, const bf16* W, int M, int V, int K, const float* row_scale,
                                int mask_id, const GemmConf& groups, float2* slice_ms, int* slice_am, float* logits,
                                const GemmScratch& scratch, cudaStream_t s) {
  if (M <= 0) return cudaSuccess;
  GemmConf gc = groups;
  gc.skip = mask_id;
  cudaError_t r = launch_gemm_tc(hf, lda, W, nullptr, logits, V, M, V, K, 5, row_scale, scratch, s, nullptr, &gc);
  if (r != cudaSuccess) return r;
  return launch_conf_merge(gc, M, V, slice_ms, slice_am, s);
}
cudaError_t launch_conf_merge(const GemmConf& groups, int M, int V, float2* slice_ms, int* slice_am, cudaStream_t s) {
  if (M <= 0) return cudaSuccess;
  return launch_pdl(k_conf_merge, dim3((M + 31) / 32, kConfSlices), dim3(kMergeWarps * 32), 0, s,
                    (const float2*)groups.ms, (const int*)groups.am, M, (V + 31) / 32, slice_ms, slice_am);
}
cudaError_t launch_conf_final(const float2* slice_ms, const int* slice_am, int M, int* tok, float* conf,
                              cudaStream_t s) {
  if (M <= 0) return cudaSuccess;
  return launch_pdl(k_conf_final, dim3((M + 127) / 128), dim3(128), 0, s, slice_ms, slice_am, M, tok, conf);
}

void build_rope_table(float* out, int max_pos, int dh, float theta) {
  const int half = dh / 2;
  for (int j = 0; j < half; ++j) {
    const double inv = pow((double)theta, -2.0 * (double)j / (double)dh);
    for (int p = 0; p < max_pos; ++p) {
      const double a = (double)p * inv;
      out[((size_t)p * half + j) * 2 + 0] = (float)cos(a);
      out[((size_t)p * half + j) * 2 + 1] = (float)sin(a);
    }
  }
}

}  // namespace bs
