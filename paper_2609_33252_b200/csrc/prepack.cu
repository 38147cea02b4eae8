// One-off weight prepack (off the hot path): the caller's [E,H,I] gate/up and [E,I,H] down
// tensors are transposed to K-major panels the tensor-core kernels consume directly.
//   W13p[e][n][h], n in [0,2I): 256-wide column blocks of [128 gate | 128 up] columns, so one
//                  256-column accumulator tile holds matching gate and up columns and the
//                  SiLU(gate)*up epilogue needs no second pass over memory.
//   W2p[e][h][i]
#include "cep_common.h"

namespace cep {
namespace {

// mode 0: n = c; mode 1 (gate): n = (c/128)*256 + c%128; mode 2 (up): that + 128
__host__ __device__ inline int packed_col(int c, int mode) {
  if (mode == 0) return c;
  return (c >> 7) * 256 + (c & 127) + (mode == 2 ? 128 : 0);
}

template <typename T>
__global__ void __launch_bounds__(256)
transpose_pack_kernel(const T* __restrict__ src, T* __restrict__ dst, int R, int C, int n_dst, int mode) {
  __shared__ T tile[32][33];
  const int e = blockIdx.z;
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  const T* s = src + (size_t)e * R * C;
  T* d = dst + (size_t)e * n_dst * R;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;          // 32 x 8
  for (int i = ty; i < 32; i += 8) {
    const int r = r0 + i, c = c0 + tx;
    if (r < R && c < C) tile[i][tx] = s[(size_t)r * C + c];
  }
  __syncthreads();
  for (int i = ty; i < 32; i += 8) {
    const int c = c0 + i, r = r0 + tx;
    if (r < R && c < C) d[(size_t)packed_col(c, mode) * R + r] = tile[tx][i];
  }
}

template <typename T>
cudaError_t pack_all(const cep_config& cfg, const void* w_gate, const void* w_up, const void* w_down,
                     void* w13p, void* w2p, cudaStream_t s) {
  const int H = cfg.hidden, I = cfg.inter, E = cfg.n_experts_local;
  dim3 g1((I + 31) / 32, (H + 31) / 32, E), g2((H + 31) / 32, (I + 31) / 32, E);
  transpose_pack_kernel<T><<<g1, 256, 0, s>>>((const T*)w_gate, (T*)w13p, H, I, 2 * I, 1);
  transpose_pack_kernel<T><<<g1, 256, 0, s>>>((const T*)w_up, (T*)w13p, H, I, 2 * I, 2);
  transpose_pack_kernel<T><<<g2, 256, 0, s>>>((const T*)w_down, (T*)w2p, I, H, H, 0);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prepack(const cep_config& cfg, const void* w_gate, const void* w_up, const void* w_down,
                           void* w13p, void* w2p, cudaStream_t s, int64_t* launches) {
  *launches += 3;
  if (cfg.dtype == CEP_FP8_E4M3_BLOCK128)
    return pack_all<uint8_t>(cfg, w_gate, w_up, w_down, w13p, w2p, s);
  return pack_all<uint16_t>(cfg, w_gate, w_up, w_down, w13p, w2p, s);
}

}  // namespace cep
