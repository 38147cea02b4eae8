// Router step in front of the routed-expert path (the benchmark's definition: softmax over all experts,
// keep the k most probable, renormalise over those k; the paper itself does not describe its router).
// One warp per token.  Selection is by logit (softmax is monotone), ties go to the lower expert id, slots are
// in descending probability.  The renormalised weights are the softmax over the k selected logits, so the
// full softmax denominator is never needed.  HBM-bound: T*E_g*4 bytes read, T*k*8 written.
#include "cep_common.h"

namespace cep {
namespace {

constexpr int kMaxPerLane = 32;          // E_g <= 1024

__global__ void __launch_bounds__(256)
route_kernel(const float* __restrict__ logits, int T, int E_g, int k, int32_t* __restrict__ ids,
             float* __restrict__ weights) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= T) return;
  const float* row = logits + (size_t)warp * E_g;
  float v[kMaxPerLane];
  const int per_lane = (E_g + 31) >> 5;
#pragma unroll
  for (int i = 0; i < kMaxPerLane; ++i) {
    const int e = i * 32 + lane;                       // coalesced: consecutive lanes, consecutive experts
    v[i] = (i < per_lane && e < E_g) ? __ldg(row + e) : -INFINITY;
  }
  float sel_logit = 0.f, first = 0.f, denom = 0.f;
  int sel_id = 0;
  for (int j = 0; j < k; ++j) {
    // lane-local best (lowest index wins ties because i ascends and the comparison is strict)
    float best = -INFINITY; int best_e = 0x7fffffff;
#pragma unroll
    for (int i = 0; i < kMaxPerLane; ++i) {
      const int e = i * 32 + lane;
      if (i < per_lane && v[i] > best) { best = v[i]; best_e = e; }
    }
    // warp argmax on (value desc, id asc)
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, off);
      const int oe = __shfl_xor_sync(0xffffffffu, best_e, off);
      if (ob > best || (ob == best && oe < best_e)) { best = ob; best_e = oe; }
    }
    if (j == 0) first = best;
    const float p = __expf(best - first);              // best <= first: no overflow
    denom += p;
    if (lane == j) { sel_logit = p; sel_id = best_e; } // lane j keeps slot j (k <= 32)
    if ((best_e & 31) == lane) {                       // owner removes it from further rounds
#pragma unroll
      for (int i = 0; i < kMaxPerLane; ++i) if (i == (best_e >> 5)) v[i] = -INFINITY;
    }
  }
  if (lane < k) {
    ids[(size_t)warp * k + lane] = sel_id;
    weights[(size_t)warp * k + lane] = sel_logit / denom;
  }
}

}  // namespace

// Synthetic routing for the throughput profile: slot j < k_loc of token t goes to local expert (t*k_loc + j) mod E
// (every expert gets the same number of rows), the remaining slots to experts of other ranks; weights 1/k_loc.
__global__ void uniform_routing_kernel(int32_t* __restrict__ ids, float* __restrict__ w, int T, int k, int k_loc, int E) {
  const long long n = (long long)T * k;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const long long t = i / k; const int j = (int)(i % k);
    ids[i] = j < k_loc ? (int32_t)((t * k_loc + j) % E) : E + (j - k_loc);
    w[i] = 1.f / (float)k_loc;
  }
}

cudaError_t launch_uniform_routing(int32_t* ids, float* w, int T, int k, int k_loc, int E, cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  uniform_routing_kernel<<<256, 256, 0, s>>>(ids, w, T, k, k_loc, E);
  return cudaGetLastError();
}

cudaError_t launch_route(const float* logits, int T, int E_g, int k, int32_t* ids, float* weights, cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  const int warps_per_block = 8;
  route_kernel<<<(T + warps_per_block - 1) / warps_per_block, warps_per_block * 32, 0, s>>>(logits, T, E_g, k, ids, weights);
  return cudaGetLastError();
}

}  // namespace cep
