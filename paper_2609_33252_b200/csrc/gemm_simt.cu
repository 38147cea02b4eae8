// Slow grouped expert GEMM on CUDA cores.  Not the product path: it exists so that tests can
// tell a fault in the tensor-core kernels from a fault anywhere else in the library (select
// it with cep_config.gemm_impl = CEP_GEMM_SIMT).  Same operands, same fused SiLU(gate)*up
// epilogue, fp32 accumulation in ascending K order, one rounding to bf16.
#include <cuda_bf16.h>

#include "cep_common.h"

namespace cep {
namespace {

constexpr int kTM = 64, kTN = 64, kTK = 16;

// grid: (m-tiles of 128 rows (upper bound), out-column tiles of 64, 2 halves of the m-tile)
__global__ void __launch_bounds__(256)
gemm_simt_kernel(GemmProblem p, const __nv_bfloat16* __restrict__ a, const __nv_bfloat16* __restrict__ b,
                 __nv_bfloat16* __restrict__ out, const int32_t* __restrict__ tile_prefix,
                 const int32_t* __restrict__ counts, const int32_t* __restrict__ padded_offsets) {
  const int mt = blockIdx.x;
  if (mt >= tile_prefix[p.n_experts]) return;
  int e = 0;
  while (tile_prefix[e + 1] <= mt) ++e;
  const int m_in_e = (mt - tile_prefix[e]) * kRowAlign + blockIdx.z * kTM;   // first row inside the group
  if (m_in_e >= counts[e]) return;
  const int row0 = padded_offsets[e] + m_in_e;
  const int rows_valid = min(kTM, counts[e] - m_in_e);
  const int oc0 = blockIdx.y * kTN;                                         // first output column
  // packed weight rows holding the operands of output columns oc0..oc0+63
  const int n0 = p.swiglu ? (oc0 >> 7) * 256 + (oc0 & 127) : oc0;
  const __nv_bfloat16* bw = b + (size_t)e * p.N * p.K;

  __shared__ float As[kTK][kTM + 1], Bs[kTK][kTN + 1], Bu[kTK][kTN + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;                    // 16 x 16 threads, 4x4 outputs each
  float accg[4][4] = {}, accu[4][4] = {};
  for (int k0 = 0; k0 < p.K; k0 += kTK) {
    for (int i = threadIdx.x; i < kTM * kTK; i += 256) {
      const int r = i / kTK, kk = i % kTK;
      As[kk][r] = (r < rows_valid) ? __bfloat162float(a[(size_t)(row0 + r) * p.K + k0 + kk]) : 0.f;
      Bs[kk][r] = __bfloat162float(bw[(size_t)(n0 + r) * p.K + k0 + kk]);
      if (p.swiglu) Bu[kk][r] = __bfloat162float(bw[(size_t)(n0 + 128 + r) * p.K + k0 + kk]);
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kTK; ++kk) {
      float av[4], bv[4], uv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { av[i] = As[kk][ty * 4 + i]; bv[i] = Bs[kk][tx * 4 + i]; uv[i] = p.swiglu ? Bu[kk][tx * 4 + i] : 0.f; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { accg[i][j] = fmaf(av[i], bv[j], accg[i][j]); accu[i][j] = fmaf(av[i], uv[j], accu[i][j]); }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = ty * 4 + i;
    if (r >= rows_valid) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float v = accg[i][j];
      if (p.swiglu) v = (v / (1.f + __expf(-v))) * accu[i][j];
      out[(size_t)(row0 + r) * p.out_ld + oc0 + tx * 4 + j] = __float2bfloat16_rn(v);
    }
  }
}

}  // namespace

cudaError_t launch_gemm_simt(const GemmProblem& p, const void* a, const void* b, void* out, const LayoutPtrs& lp,
                             cudaStream_t s, int64_t* launches) {
  if (p.is_fp8) return cudaErrorNotSupported;
  const int out_cols = p.swiglu ? p.N / 2 : p.N;
  dim3 grid(p.cap_rows / kRowAlign, out_cols / kTN, 2);
  if (grid.x == 0) return cudaSuccess;
  gemm_simt_kernel<<<grid, 256, 0, s>>>(p, (const __nv_bfloat16*)a, (const __nv_bfloat16*)b, (__nv_bfloat16*)out,
                                        lp.tile_prefix, lp.counts, lp.padded_offsets);
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace cep
