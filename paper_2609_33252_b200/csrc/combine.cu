// Top-k weighted combine + unpermute (Appendix "Output return and combine"): every routed
// contribution is weighted by its routing coefficient exactly once and accumulated at its
// token; results are written in token order.  Slots are accumulated in ascending slot
// order in fp32 and rounded to bf16 once.  Tokens with no local expert get exact zeros.  An optional addend
// row (the shared expert's output for the token, which the paper sums with the routed result) is added
// in fp32 after the routed contributions, before the single rounding.
#include <cuda_bf16.h>

#include "cep_common.h"

namespace cep {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ void fma_bf16x8(float (&acc)[8], const uint4& v, float w) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __bfloat1622float2(h[i]);
    acc[2 * i] = fmaf(w, f.x, acc[2 * i]);
    acc[2 * i + 1] = fmaf(w, f.y, acc[2 * i + 1]);
  }
}

__global__ void __launch_bounds__(kThreads)
combine_kernel(const __grid_constant__ BatchDesc batch, int k, int H, const int32_t* __restrict__ row_of_pair,
               const __nv_bfloat16* __restrict__ y, const __nv_bfloat16* __restrict__ addend,
               __nv_bfloat16* __restrict__ out) {
  __shared__ int32_t s_rows[32];
  __shared__ float s_w[32];
  pdl_enter();
  const int t = blockIdx.x;
  int c = 0;
  while (c + 1 < batch.n_chunks && t >= batch.chunk[c + 1].token_base) ++c;
  const int tl = t - batch.chunk[c].token_base;
  if (threadIdx.x < k) {
    s_rows[threadIdx.x] = row_of_pair[(size_t)t * k + threadIdx.x];
    s_w[threadIdx.x] = __ldg(batch.chunk[c].weights + (size_t)tl * k + threadIdx.x);
  }
  __syncthreads();
  const int n_vec = H >> 3;
  uint4* dst = reinterpret_cast<uint4*>(out + (size_t)(batch.chunk[c].token_offset + tl) * H);
  const uint4* add = addend ? reinterpret_cast<const uint4*>(addend + (size_t)(batch.chunk[c].token_offset + tl) * H) : nullptr;
  for (int v = threadIdx.x; v < n_vec; v += kThreads) {
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    int j = 0;
    for (; j + 4 <= k; j += 4) {                 // four independent row loads in flight
      uint4 val[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int row = s_rows[j + u];
        val[u] = (row >= 0) ? __ldcs(reinterpret_cast<const uint4*>(y + (size_t)row * H) + v)
                            : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (s_rows[j + u] >= 0) fma_bf16x8(acc, val[u], s_w[j + u]);
    }
    for (; j < k; ++j) {
      const int row = s_rows[j];
      if (row >= 0) fma_bf16x8(acc, __ldcs(reinterpret_cast<const uint4*>(y + (size_t)row * H) + v), s_w[j]);
    }
    if (add) fma_bf16x8(acc, __ldg(add + v), 1.0f);
    uint4 o;
    __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
    for (int i = 0; i < 4; ++i) oh[i] = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
    dst[v] = o;
  }
}

}  // namespace

cudaError_t launch_combine(const BatchDesc& batch, const cep_config& cfg, const LayoutPtrs& lp, const void* y,
                           const void* addend, void* out, cudaStream_t s, int64_t* launches) {
  if (batch.n_tokens == 0) return cudaSuccess;
  *launches += 1;
  return launch_pdl(combine_kernel, dim3(batch.n_tokens), dim3(kThreads), 0, s, 1, batch, cfg.top_k, cfg.hidden,
                    (const int32_t*)lp.row_of_pair, static_cast<const __nv_bfloat16*>(y),
                    static_cast<const __nv_bfloat16*>(addend), static_cast<__nv_bfloat16*>(out));
}

}  // namespace cep
