// Legacy-path GEMM (mma.sync m16n8k16, cp.async pipeline): C[M,N] = A[M,K] W[N,K]^T with fused epilogues.
// Kept for shapes the tcgen05 kernel does not take (K not a multiple of 64 elements, tiny problems).
#include "common.cuh"

namespace bs {

namespace {
constexpr int BM = 128, BNS = 128, BK = 32, STAGES = 3, PAD = 8, LDS = BK + PAD;
constexpr int kGemmThreads = 256;
constexpr int kStageElems = (BM + BNS) * LDS;
constexpr int kSmemBytes = STAGES * kStageElems * 2;

__device__ __forceinline__ void cp_async16(void* dst, const void* src, int bytes) {
  const unsigned d = (unsigned)__cvta_generic_to_shared(dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(d), "l"(src), "r"(bytes));
}
__device__ __forceinline__ void ldmatrix_x4(unsigned& r0, unsigned& r1, unsigned& r2, unsigned& r3, const void* p) {
  const unsigned a = (unsigned)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(a));
}
__device__ __forceinline__ void mma16816(float* c, const unsigned* a, unsigned b0, unsigned b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float silu_f(float x) { return x / (1.0f + __expf(-x)); }

template <bool DUAL>
__global__ void __launch_bounds__(kGemmThreads) k_gemm_mma(const bf16* __restrict__ A, int lda,
                                                           const bf16* __restrict__ W, const bf16* __restrict__ W2,
                                                           void* __restrict__ Cv, int ldc, int M, int N, int K,
                                                           int mode, const float* __restrict__ row_scale) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  bf16* smem = reinterpret_cast<bf16*>(smem_raw);
  constexpr int BN_OUT = DUAL ? 64 : 128;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN_OUT;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = warp >> 2, wn = warp & 3;
  const int nk = (K + BK - 1) / BK;
  pdl_wait();
  pdl_trigger();

  auto load_stage = [&](int stage, int kt) {
    bf16* sA = smem + stage * kStageElems;
    bf16* sB = sA + BM * LDS;
    const int k0 = kt * BK;
#pragma unroll
    for (int it = 0; it < 2; ++it) {
      const int ch = tid + it * kGemmThreads;      // 0..511
      const int r = ch >> 2, cc = (ch & 3) * 8;
      const bool kin = (k0 + cc) < K;
      {
        const bool ok = kin && (m0 + r) < M;
        const bf16* src = ok ? A + (size_t)(m0 + r) * lda + k0 + cc : A;
        cp_async16(sA + r * LDS + cc, src, ok ? 16 : 0);
      }
      {
        const bf16* base = W;
        int nr = n0 + r;
        if (DUAL) {
          if (r >= 64) { base = W2; nr = n0 + r - 64; }
        }
        const bool ok = kin && nr < N;
        const bf16* src = ok ? base + (size_t)nr * K + k0 + cc : base;
        cp_async16(sB + r * LDS + cc, src, ok ? 16 : 0);
      }
    }
  };

  float acc[4][4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int k = 0; k < 4; ++k) acc[i][j][k] = 0.f;

#pragma unroll
  for (int s = 0; s < STAGES - 1; ++s) {
    if (s < nk) load_stage(s, s);
    asm volatile("cp.async.commit_group;\n" ::);
  }
  const int brow0 = DUAL ? wn * 16 : wn * 32;
  const int brow1 = DUAL ? 64 + wn * 16 : wn * 32 + 16;
  for (int kt = 0; kt < nk; ++kt) {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(STAGES - 2));
    __syncthreads();
    if (kt + STAGES - 1 < nk) load_stage((kt + STAGES - 1) % STAGES, kt + STAGES - 1);
    asm volatile("cp.async.commit_group;\n" ::);
    const bf16* sA = smem + (kt % STAGES) * kStageElems;
    const bf16* sB = sA + BM * LDS;
#pragma unroll
    for (int ks = 0; ks < BK; ks += 16) {
      unsigned af[4][4], bfr[4][2];
#pragma unroll
      for (int mt = 0; mt < 4; ++mt)
        ldmatrix_x4(af[mt][0], af[mt][1], af[mt][2], af[mt][3],
                    sA + (wm * 64 + mt * 16 + (lane & 15)) * LDS + ks + (lane >> 4) * 8);
      {
        const int rr = (lane & 7) + ((lane >> 4) << 3), cc = ks + ((lane >> 3) & 1) * 8;
        ldmatrix_x4(bfr[0][0], bfr[0][1], bfr[1][0], bfr[1][1], sB + (brow0 + rr) * LDS + cc);
        ldmatrix_x4(bfr[2][0], bfr[2][1], bfr[3][0], bfr[3][1], sB + (brow1 + rr) * LDS + cc);
      }
#pragma unroll
      for (int mt = 0; mt < 4; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) mma16816(acc[mt][nt], af[mt], bfr[nt][0], bfr[nt][1]);
    }
  }
  asm volatile("cp.async.wait_group 0;\n" ::);

  // ---- epilogue ----
#pragma unroll
  for (int mt = 0; mt < 4; ++mt) {
#pragma unroll
    for (int hrow = 0; hrow < 2; ++hrow) {
      const int m = m0 + wm * 64 + mt * 16 + (lane >> 2) + hrow * 8;
      if (m >= M) continue;
      if (DUAL) {
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const int n = n0 + wn * 16 + nt * 8 + (lane & 3) * 2;
          if (n >= N) continue;
          const float g0 = acc[mt][nt][hrow * 2], g1 = acc[mt][nt][hrow * 2 + 1];
          const float u0 = acc[mt][nt + 2][hrow * 2], u1 = acc[mt][nt + 2][hrow * 2 + 1];
          bf16* C = reinterpret_cast<bf16*>(Cv);
          *reinterpret_cast<__nv_bfloat162*>(C + (size_t)m * ldc + n) =
              __floats2bfloat162_rn(silu_f(g0) * u0, silu_f(g1) * u1);
        }
      } else {
        const float sc = (mode == 2) ? row_scale[m] : 1.0f;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          const int n = n0 + wn * 32 + nt * 8 + (lane & 3) * 2;
          if (n >= N) continue;
          const float v0 = acc[mt][nt][hrow * 2], v1 = acc[mt][nt][hrow * 2 + 1];
          if (mode == 0) {
            bf16* C = reinterpret_cast<bf16*>(Cv);
            *reinterpret_cast<__nv_bfloat162*>(C + (size_t)m * ldc + n) = __floats2bfloat162_rn(v0, v1);
          } else {
            float2* p = reinterpret_cast<float2*>(reinterpret_cast<float*>(Cv) + (size_t)m * ldc + n);
            if (mode == 1) {
              float2 o = *p;
              o.x += v0;
              o.y += v1;
              *p = o;
            } else {
              *p = make_float2(v0 * sc, v1 * sc);
            }
          }
        }
      }
    }
  }
}
}  // namespace

cudaError_t launch_gemm_mma(const bf16* A, int lda, const bf16* W, const bf16* W2, void* C, int ldc, int M, int N,
                            int K, int mode, const float* row_scale, cudaStream_t s) {
  if (M <= 0 || N <= 0) return cudaSuccess;
  static bool attr_done = false;
  if (!attr_done) {
    cudaFuncSetAttribute(k_gemm_mma<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    cudaFuncSetAttribute(k_gemm_mma<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    attr_done = true;
  }
  if (mode == 3) {
    dim3 grid((N + 63) / 64, (M + BM - 1) / BM);
    return launch_pdl(k_gemm_mma<true>, grid, dim3(kGemmThreads), kSmemBytes, s, A, lda, W, W2, C, ldc, M, N, K, mode,
                      row_scale);
  } else {
    dim3 grid((N + 127) / 128, (M + BM - 1) / BM);
    return launch_pdl(k_gemm_mma<false>, grid, dim3(kGemmThreads), kSmemBytes, s, A, lda, W, W2, C, ldc, M, N, K, mode,
                      row_scale);
  }
  return cudaGetLastError();
}

}  // namespace bs
