// Merging confidence partials (maximum m, sum s of exp(z - m), index am of the maximum) of disjoint parts of a
// vocabulary row: the larger maximum wins, equal maxima keep the lower index, sums are rescaled to the common maximum.
#pragma once
#include <math.h>

#include "common.cuh"

namespace bs {

struct ConfPart {
  float m, s;
  int am;
};
__device__ __forceinline__ ConfPart conf_empty() { return ConfPart{-INFINITY, 0.f, 0x7fffffff}; }
__device__ __forceinline__ void conf_merge(ConfPart& a, float m, float s, int am) {
  if (!(m > -INFINITY)) return;                       // an empty part
  if (m > a.m) {
    a.s = a.s * __expf(a.m - m) + s;                  // exp(-inf) = 0 for an empty accumulator
    a.m = m;
    a.am = am;
  } else {
    a.s += s * __expf(m - a.m);
    if (m == a.m && am < a.am) a.am = am;
  }
}
// Final merge of the kConfSlices slice partials of lm row t; confidence = exp(max - logsumexp) = 1 / s.
__device__ __forceinline__ void merge_conf_slices(const float2* __restrict__ slice_ms, const int* __restrict__ slice_am,
                                                  int M, int t, int* tok, float* conf) {
  ConfPart acc = conf_empty();
#pragma unroll
  for (int sl = 0; sl < kConfSlices; ++sl) {
    const float2 ms = slice_ms[(size_t)sl * M + t];
    conf_merge(acc, ms.x, ms.y, slice_am[(size_t)sl * M + t]);
  }
  *tok = acc.am;
  *conf = 1.0f / acc.s;
}

}  // namespace bs
