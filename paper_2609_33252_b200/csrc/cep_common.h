// Shared declarations of the streamFFN library's translation units (host + device).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/cascade_ffn.h"

namespace cep {

constexpr int kRowAlign = CEP_ROW_ALIGN;        // rows per GEMM M tile; expert groups start on multiples
constexpr int kMaxChunksPerInv = CEP_MAX_CHUNKS_PER_INVOCATION;
constexpr int kSegPairs = 2048;                 // pairs per block in the histogram / rank kernels
constexpr int kQuantBlock = 128;                // fp8 scale block
constexpr int kMxBlock = 32;                    // microscaling block (elements sharing a ue8m0 scale)
// Microscaling scale factors travel in 512-byte "atoms": the scales of 128 rows x 4 consecutive 32-blocks of K,
// byte (r%32)*16 + (r/32)*4 + kb, which is the order tcgen05.cp (32x128b.warpx4) and the block-scaled MMA
// expect them in.  An operand of R rows and K columns has (R/128) x (K/128) atoms, K fastest.
constexpr int kSfAtomBytes = 512;
__host__ __device__ inline size_t sf_atom_offset(long long row, int kb32, int k128_per_row) {
  return ((size_t)(row >> 7) * k128_per_row + (kb32 >> 2)) * kSfAtomBytes + (size_t)((row & 31) * 16 + ((row >> 5) & 3) * 4 + (kb32 & 3));
}
__host__ __device__ inline bool dtype_is_bytes(int dtype) { return dtype != CEP_BF16; }   // one-byte activation codes

// Device status word layout (int32 each).
enum StatusWord { kStBadRouting = 0, kStTimeout = 1, kStBoundsViolation = 2, kStDetail = 3, kStWords = 8 };

// One chunk of a batch as the kernels see it.
struct ChunkDesc {
  const void* tokens;         // [n,H] bf16 | e4m3
  const void* scales;         // fp8: fp32 [n,H/128]; mxfp4: ue8m0 bytes [n,H/32]
  const int32_t* ids;         // [n,k]
  const float* weights;       // [n,k]
  int32_t n_tokens;
  int32_t token_offset;       // row of `out` of the chunk's first token
  int32_t token_base;         // index of the chunk's first token inside the batch
  int32_t pad_;
};

struct BatchDesc {
  ChunkDesc chunk[kMaxChunksPerInv];
  int32_t n_chunks;
  int32_t n_tokens;           // tokens in the batch
};

// Per-slot integer scratch produced by the layout transform.
struct LayoutPtrs {
  int32_t* counts;            // [E]
  int32_t* offsets;           // [E+1]
  int32_t* padded_offsets;    // [E+1]
  int32_t* tile_prefix;       // [E+1] cumulative number of 128-row tiles
  int32_t* block_base;        // [n_seg_max, E] per (segment, expert): first histogram, then row base
  int32_t* row_of_pair;       // [max_tokens*k] physical row, -1 when not local
  int32_t* pair_of_row;       // [cap_rows] batch pair index, -1 on padding
  int32_t* status;            // [kStWords]
  int32_t* sched;             // [2] tile counters of the two GEMMs of an invocation (zeroed by the scan kernel)
  int32_t* src_row;           // [cap_rows] gather_a plans only: row of the caller's token tensor a physical row holds
};

// ---------------------------------------------------------------- programmatic dependent launch
// Every kernel of an invocation is launched with programmatic stream serialization: it may be scheduled
// while its predecessor in the stream is still draining, so launch latency and block scheduling overlap the
// predecessor's tail.  Each thread first waits for the predecessor grid to complete (its memory is then
// visible), and only then lets the successor be scheduled.  Launched without the attribute both are no-ops.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_enter() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
#endif

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, int cluster_x,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  int n = 0;
  attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster_x; attr[n].val.clusterDim.y = 1; attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cfg.attrs = attr; cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---------------------------------------------------------------- tile scheduling arithmetic
// Linear tile index -> (expert, m_block, n_block).  Tiles are expert-major.  Inside an expert the n
// blocks are taken in chunks of `n_group` (the last chunk may be shorter); a chunk is swept over all
// m blocks of the expert with n as the fast index.  The CTAs running at one time then share the
// chunk's weight panel (sized by the caller to stay L2-resident for the whole sweep) while the
// expert's activation rows stream past it, one pass per chunk.
struct TileCoord { int expert, m_block, n_block; };

__host__ __device__ inline bool decode_tile(const int32_t* __restrict__ tile_prefix, int n_experts,
                                            int n_blocks_n, int n_group, int tile, TileCoord* out) {
  if (tile < 0 || n_blocks_n <= 0 || n_group <= 0) return false;
  int lo = 0, hi = n_experts;            // find e: prefix[e]*NB <= tile < prefix[e+1]*NB
  if ((long long)tile >= (long long)tile_prefix[n_experts] * n_blocks_n) return false;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if ((long long)tile_prefix[mid] * n_blocks_n <= tile) lo = mid; else hi = mid;
  }
  // now prefix[lo] <= tile / NB < prefix[lo+1]: expert lo has tiles and owns this one
  const int mt = tile_prefix[lo + 1] - tile_prefix[lo];
  const int li = tile - tile_prefix[lo] * n_blocks_n;
  const int c = li / (mt * n_group);                 // chunk of n blocks (all but the last are full)
  const int rem = li - c * mt * n_group;
  int gn = n_blocks_n - c * n_group;
  if (gn > n_group) gn = n_group;
  out->expert = lo;
  out->m_block = rem / gn;
  out->n_block = c * n_group + (rem - out->m_block * gn);
  return true;
}

// n blocks per chunk so that one chunk's weight panel (block_cols x K elements each) stays within a
// budget the L2 keeps resident next to the streamed operand.
__host__ inline int n_group_for(int n_blocks_n, int block_cols, int K, int elt_bytes) {
  const long long budget = 32ll << 20;
  long long g = budget / ((long long)block_cols * K * elt_bytes);
  if (g < 1) g = 1;
  if (g > n_blocks_n) g = n_blocks_n;
  return (int)g;
}

// ---------------------------------------------------------------- kernel launchers (defined in the .cu files)
struct GemmProblem {
  // A operand: rows x K, K contiguous (the permuted activations or the intermediate)
  // B operand: per expert N x K, K contiguous (packed weights)
  int K, N;                   // N = columns of the weight panel (2I for GEMM1, H for GEMM2)
  int n_experts;
  int swiglu;                 // 1: output column j = silu(acc[:, pair(j)]) * acc[:, pair(j)+128]
  int out_ld;                 // elements per output row
  int cap_rows;               // rows the A / output buffers hold
  int is_fp8;                 // any one-byte operand format (block-scaled e4m3 or microscaling)
};

// after_index: optional event recorded between the index kernels (hist, scan, rank) and the row scatter
cudaError_t launch_layout(const BatchDesc& batch, const cep_config& cfg, const LayoutPtrs& lp, void* xp,
                          void* xp_scales, int cap_rows, int n_seg, cudaStream_t s, cudaEvent_t after_index,
                          int64_t* launches);
cudaError_t launch_combine(const BatchDesc& batch, const cep_config& cfg, const LayoutPtrs& lp,
                           const void* y, const void* addend, void* out, cudaStream_t s, int64_t* launches);
cudaError_t launch_route(const float* logits, int T, int E_g, int k, int32_t* ids, float* weights, cudaStream_t s);
cudaError_t launch_uniform_routing(int32_t* ids, float* weights, int T, int k, int k_loc, int E, cudaStream_t s);
cudaError_t launch_gemm_simt(const GemmProblem& p, const void* a, const void* b, void* out,
                             const LayoutPtrs& lp, cudaStream_t s, int64_t* launches);
cudaError_t launch_prepack(const cep_config& cfg, const void* w_gate, const void* w_up, const void* w_down,
                           void* w13p, void* w2p, cudaStream_t s, int64_t* launches);

}  // namespace cep
