// RoPE + KV scatter for callers that cannot allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a memory pool that was sized once at
// start-up, inside a plugin whose embedding runtime owns every allocation, or on a path that must not touch the
// allocator because it would serialise with other streams.  bs_op_rope_kv needs a scratch buffer for its cos/sin
// table; this variant keeps that table in a fixed array that is part of the loaded module instead.
#include <mutex>

#include "../../include/blockserve.h"
#include "common.cuh"

namespace {

// cos/sin table, [max_pos, head_dim / 2] pairs.  Every GPU that loads the library holds these 2 MiB until exit.
constexpr int kStaticTableFloats = BS_ROPE_STATIC_MAX_FLOATS;
static __device__ __align__(256) float g_rope_table[kStaticTableFloats];

constexpr int kMaxDevices = 64;
float* g_table_ptr[kMaxDevices] = {};     // device address of g_rope_table, per device, filled on first use
std::mutex g_table_mutex;

// tab[p, j] = (cos, sin)(p * theta^(-2j/dh)), evaluated in double and rounded once.
__global__ void k_fill_rope_table(float* __restrict__ tab, int max_pos, int dh, double theta) {
  const int half = dh / 2;
  const int n = max_pos * half;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const int p = i / half, j = i % half;
    const double a = (double)p * pow(theta, -2.0 * (double)j / (double)dh);
    tab[2 * i] = (float)cos(a);
    tab[2 * i + 1] = (float)sin(a);
  }
}

// The array's name is only a host-side handle; kernels need its device address, which differs per device.
int table_address(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BS_E_CUDA;
  std::lock_guard<std::mutex> lock(g_table_mutex);
  if (!g_table_ptr[dev]) {
    float* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_rope_table) != cudaSuccess || !p) return BS_E_CUDA;
    g_table_ptr[dev] = p;
  }
  *out = g_table_ptr[dev];
  return BS_OK;
}

}  // namespace

extern "C" int bs_op_rope_kv_static(void* qkv, const int* tok_pos, const int* tok_kv, void* kcache, void* vcache,
                                    int M, int n_q_heads, int n_kv_heads, int head_dim, float theta, int max_pos,
                                    void* stream) {
  if (!qkv || !tok_pos || !tok_kv || !kcache || !vcache || M < 0 || n_q_heads < 1 || n_kv_heads < 1 ||
      head_dim < 8 || head_dim % 8 || max_pos < 1 || !(theta > 0.f))
    return BS_E_ARG;
  if ((long long)max_pos * head_dim > (long long)kStaticTableFloats) return BS_E_ARG;   // table would not fit
  float* table = nullptr;
  if (int rc = table_address(&table)) return rc;
  cudaStream_t s = (cudaStream_t)stream;
  // The table keeps whatever the previous call left; every entry this call can read is rewritten first.
  const int n = max_pos * (head_dim / 2);
  k_fill_rope_table<<<(n + 255) / 256 < 592 ? (n + 255) / 256 : 592, 256, 0, s>>>(table, max_pos, head_dim,
                                                                                  (double)theta);
  if (cudaGetLastError() != cudaSuccess) return BS_E_CUDA;
  return bs::launch_rope_kv((bs::bf16*)qkv, tok_pos, tok_kv, (bs::bf16*)kcache, (bs::bf16*)vcache, M, n_q_heads,
                            n_kv_heads, head_dim, table, s) == cudaSuccess ? BS_OK : BS_E_CUDA;
}
