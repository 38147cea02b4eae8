// Layout transform of one grouped FFN invocation (Appendix "Grouped FFN invocations"):
// selected rows of the ready chunks are gathered into contiguous, tile-aligned groups by
// expert, with per-expert offsets computed from the counts and an inverse map kept for
// the combine.  Four kernels: histogram -> exclusive scan -> stable rank -> row scatter.
//
// Pair order inside a batch is (chunk position, token, slot) lexicographic; the rank of
// a pair inside its expert group is the number of earlier pairs with the same expert
// (a stable counting sort), so every index is uniquely defined and reproducible.
#include "cep_common.h"

namespace cep {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ int load_pair_id(const BatchDesc& b, int k, int p /*batch pair index*/) {
  const int t = p / k;
  int c = 0;
#pragma unroll 1
  while (c + 1 < b.n_chunks && t >= b.chunk[c + 1].token_base) ++c;
  const long long off = (long long)(t - b.chunk[c].token_base) * k + (p - t * k);
  return __ldg(b.chunk[c].ids + off);
}

// ---- 1. histogram: per segment of kSegPairs pairs, per local expert
__global__ void __launch_bounds__(kThreads)
hist_kernel(const __grid_constant__ BatchDesc batch, int k, int E, int E_global, int check_duplicates,
            int32_t* __restrict__ seg_hist, int32_t* __restrict__ status) {
  extern __shared__ int32_t sh[];
  pdl_enter();
  for (int e = threadIdx.x; e < E; e += kThreads) sh[e] = 0;
  __syncthreads();
  const int n_pairs = batch.n_tokens * k;
  const int p0 = blockIdx.x * kSegPairs;
  const int p1 = min(p0 + kSegPairs, n_pairs);
  bool bad = false;
  constexpr int kPerThread = kSegPairs / kThreads;
  int ids[kPerThread];
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {          // independent loads first: one memory latency, not eight
    const int p = p0 + i * kThreads + threadIdx.x;
    ids[i] = p < p1 ? load_pair_id(batch, k, p) : E;   // E: in range, not local, counted nowhere
  }
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    const int e = ids[i];
    if (e < 0 || e >= E_global) { if (p0 + i * kThreads + (int)threadIdx.x < p1) bad = true; }
    else if (e < E) atomicAdd(&sh[e], 1);
  }
  if (bad) atomicOr(&status[kStBadRouting], 1);
  if (check_duplicates) {                         // debug plans only: a token must not name an expert twice
    bool dup = false;
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) {
      const int p = p0 + i * kThreads + threadIdx.x;
      if (p >= p1) continue;
      const int j = p % k;
      for (int j2 = 0; j2 < j; ++j2) dup |= load_pair_id(batch, k, p - j + j2) == ids[i];
    }
    if (dup) atomicOr(&status[kStBadRouting], 2);
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += kThreads) seg_hist[(size_t)blockIdx.x * E + e] = sh[e];
}

// ---- 2. scan: counts, offsets, tile-aligned offsets, tile prefix, and per (segment, expert) row base
__global__ void __launch_bounds__(1024)
scan_kernel(int n_seg, int E, int32_t* __restrict__ seg_hist /*in: hist, out: row base*/,
            int32_t* __restrict__ counts, int32_t* __restrict__ offsets, int32_t* __restrict__ padded_offsets,
            int32_t* __restrict__ tile_prefix, int32_t* __restrict__ sched) {
  __shared__ int32_t s_cnt[1024];
  pdl_enter();
  if (threadIdx.x < 2) sched[threadIdx.x] = 0;   // tile counters of this invocation's two GEMMs
  __shared__ int32_t s_off[1025], s_pad[1025];
  const int e = threadIdx.x;
  int total = 0;
  if (e < E) {                                  // loads only, eight in flight: the stores come in the second pass
    int s = 0;
    for (; s + 8 <= n_seg; s += 8) {
      int c[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) c[u] = seg_hist[(size_t)(s + u) * E + e];
#pragma unroll
      for (int u = 0; u < 8; ++u) total += c[u];
    }
    for (; s < n_seg; ++s) total += seg_hist[(size_t)s * E + e];
  }
  s_cnt[e] = (e < E) ? total : 0;
  __syncthreads();
  if (threadIdx.x == 0) {                       // E <= 1024: a serial scan costs about a microsecond
    int o = 0, po = 0;
    for (int i = 0; i < E; ++i) {
      s_off[i] = o; s_pad[i] = po;
      o += s_cnt[i];
      po += (s_cnt[i] + kRowAlign - 1) / kRowAlign * kRowAlign;
    }
    s_off[E] = o; s_pad[E] = po;
  }
  __syncthreads();
  if (e < E) {
    counts[e] = s_cnt[e];
    offsets[e] = s_off[e];
    padded_offsets[e] = s_pad[e];
    tile_prefix[e] = s_pad[e] / kRowAlign;
    // histogram -> first row of each (segment, expert): exclusive prefix over the segments on top of the group start
    int run = s_pad[e];
    int s = 0;
    for (; s + 8 <= n_seg; s += 8) {
      int c[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) c[u] = seg_hist[(size_t)(s + u) * E + e];
#pragma unroll
      for (int u = 0; u < 8; ++u) { seg_hist[(size_t)(s + u) * E + e] = run; run += c[u]; }
    }
    for (; s < n_seg; ++s) { const int c = seg_hist[(size_t)s * E + e]; seg_hist[(size_t)s * E + e] = run; run += c; }
  }
  if (e == 0) {
    offsets[E] = s_off[E];
    padded_offsets[E] = s_pad[E];
    tile_prefix[E] = s_pad[E] / kRowAlign;
  }
}

// ---- 3. stable rank: physical row of every pair, and the inverse map
__global__ void __launch_bounds__(kThreads)
rank_kernel(const __grid_constant__ BatchDesc batch, int k, int E, const int32_t* __restrict__ seg_base,
            int32_t* __restrict__ row_of_pair, int32_t* __restrict__ pair_of_row, int cap_rows,
            int32_t* __restrict__ status, int32_t* __restrict__ src_row /*NULL unless GEMM1 gathers its rows*/) {
  extern __shared__ int32_t sh[];              // [kWarps][E] running row cursor per warp and expert
  pdl_enter();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = threadIdx.x; i < kWarps * E; i += kThreads) sh[i] = 0;
  __syncthreads();
  const int n_pairs = batch.n_tokens * k;
  constexpr int kPerWarp = kSegPairs / kWarps;
  const int w0 = blockIdx.x * kSegPairs + warp * kPerWarp;
  int32_t* mine = sh + warp * E;
  // this lane's ids for both passes, loaded once with independent loads
  int my_ids[kPerWarp / 32];
#pragma unroll
  for (int i = 0; i < kPerWarp / 32; ++i) {
    const int p = w0 + i * 32 + lane;
    int e = -2;
    if (p < n_pairs) { e = load_pair_id(batch, k, p); if (e < 0 || e >= E) e = -1; }
    my_ids[i] = e;
  }
  // pass 1: this warp's count per expert
#pragma unroll
  for (int it = 0; it < kPerWarp; it += 32) {
    const int e = my_ids[it / 32];
    const unsigned m = __match_any_sync(0xffffffffu, e);
    if (e >= 0 && lane == (__ffs(m) - 1)) mine[e] += __popc(m);
    __syncwarp();
  }
  __syncthreads();
  // exclusive prefix over the warps of this block, on top of the segment's row base
  for (int e = threadIdx.x; e < E; e += kThreads) {
    int run = seg_base[(size_t)blockIdx.x * E + e];
    for (int w = 0; w < kWarps; ++w) { const int c = sh[w * E + e]; sh[w * E + e] = run; run += c; }
  }
  __syncthreads();
  // pass 2: rows in pair order
#pragma unroll
  for (int it = 0; it < kPerWarp; it += 32) {
    const int p = w0 + it + lane;
    const int e = my_ids[it / 32];
    const unsigned m = __match_any_sync(0xffffffffu, e);
    int row = -1;
    if (e >= 0) row = mine[e] + __popc(m & ((1u << lane) - 1u));
    __syncwarp();
    if (e >= 0 && lane == (__ffs(m) - 1)) mine[e] += __popc(m);
    __syncwarp();
    if (p < n_pairs) {
      if (row >= cap_rows) { atomicOr(&status[kStBoundsViolation], 1); row = -1; }
      row_of_pair[p] = row;
      if (row >= 0) pair_of_row[row] = p;
      if (row >= 0 && src_row) {                 // where the pair's token sits in the caller's token tensor
        const int t = p / k;
        int c = 0;
#pragma unroll 1
        while (c + 1 < batch.n_chunks && t >= batch.chunk[c + 1].token_base) ++c;
        src_row[row] = batch.chunk[c].token_offset + (t - batch.chunk[c].token_base);
      }
    }
  }
}

// ---- 4'. gather_a plans: no payload moves; only the padding rows' inverse-map entries are marked
__global__ void __launch_bounds__(128)
mark_padding_kernel(int E, const int32_t* __restrict__ counts, const int32_t* __restrict__ padded_offsets,
                    int32_t* __restrict__ pair_of_row, int cap_rows) {
  pdl_enter();
  const int e = blockIdx.x;
  if (e >= E) return;
  const int r0 = padded_offsets[e] + counts[e], r1 = padded_offsets[e + 1];
  for (int r = r0 + threadIdx.x; r < r1 && r < cap_rows; r += blockDim.x) pair_of_row[r] = -1;
}

// ---- 4. payload: one block per token reads its row once and writes it to each local expert's group;
//         the first E blocks zero the padding rows of each group (first, so that the one block that
//         has up to 127 rows to clear does not run alone at the end).
template <int kVecPerThread>
__global__ void __launch_bounds__(kThreads)
scatter_rows_kernel(const __grid_constant__ BatchDesc batch, int k, int E, int row_bytes, int n_scale,
                    const int32_t* __restrict__ row_of_pair, const int32_t* __restrict__ counts,
                    const int32_t* __restrict__ padded_offsets, int32_t* __restrict__ pair_of_row,
                    uint8_t* __restrict__ xp, uint32_t* __restrict__ xp_scales /*32-bit words: an fp32 scale, or
                    four ue8m0 bytes*/, int sf_atoms /*scale words go to the 512-byte atom order*/, int cap_rows) {
  pdl_enter();
  const int n_vec = row_bytes >> 4;
  if ((int)blockIdx.x < E) {                     // padding rows of expert e
    const int e = blockIdx.x;
    const int r0 = padded_offsets[e] + counts[e], r1 = padded_offsets[e + 1];
    for (int r = r0; r < r1 && r < cap_rows; ++r) {
      uint4* dst = reinterpret_cast<uint4*>(xp + (size_t)r * row_bytes);
      for (int v = threadIdx.x; v < n_vec; v += kThreads) dst[v] = make_uint4(0, 0, 0, 0);
      if (xp_scales)
        for (int v = threadIdx.x; v < n_scale; v += kThreads)
          xp_scales[sf_atoms ? sf_atom_offset(r, 4 * v, n_scale) >> 2 : (size_t)r * n_scale + v] = 0u;
      if (threadIdx.x == 0) pair_of_row[r] = -1;
    }
    return;
  }
  __shared__ int32_t s_rows[32];
  const int t = blockIdx.x - E;
  int c = 0;
  while (c + 1 < batch.n_chunks && t >= batch.chunk[c + 1].token_base) ++c;
  const int tl = t - batch.chunk[c].token_base;
  if (threadIdx.x < k) s_rows[threadIdx.x] = row_of_pair[(size_t)t * k + threadIdx.x];
  __syncthreads();
  const uint4* src = reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(batch.chunk[c].tokens) +
                                                    (size_t)tl * row_bytes);
  for (int v0 = threadIdx.x; v0 < n_vec; v0 += kThreads * kVecPerThread) {
    uint4 val[kVecPerThread];
#pragma unroll
    for (int i = 0; i < kVecPerThread; ++i) {
      const int v = v0 + i * kThreads;
      if (v < n_vec) val[i] = __ldg(src + v);
    }
    for (int j = 0; j < k; ++j) {
      const int row = s_rows[j];
      if (row < 0) continue;
      uint4* dst = reinterpret_cast<uint4*>(xp + (size_t)row * row_bytes);
#pragma unroll
      for (int i = 0; i < kVecPerThread; ++i) {
        const int v = v0 + i * kThreads;
        if (v < n_vec) dst[v] = val[i];
      }
    }
  }
  if (xp_scales) {
    const uint32_t* ss = static_cast<const uint32_t*>(batch.chunk[c].scales) + (size_t)tl * n_scale;
    for (int v = threadIdx.x; v < n_scale; v += kThreads) {
      const uint32_t sv = __ldg(ss + v);
      for (int j = 0; j < k; ++j) {
        const int row = s_rows[j];
        if (row >= 0) xp_scales[sf_atoms ? sf_atom_offset(row, 4 * v, n_scale) >> 2 : (size_t)row * n_scale + v] = sv;
      }
    }
  }
}

}  // namespace

cudaError_t launch_layout(const BatchDesc& batch, const cep_config& cfg, const LayoutPtrs& lp, void* xp,
                          void* xp_scales, int cap_rows, int n_seg, cudaStream_t s, cudaEvent_t after_index,
                          int64_t* launches) {
  const int k = cfg.top_k, E = cfg.n_experts_local;
  if (n_seg < 1) n_seg = 1;
  cudaError_t err;
  err = launch_pdl(hist_kernel, dim3(n_seg), dim3(kThreads), E * sizeof(int32_t), s, 1, batch, k, E, cfg.n_experts_global,
                   cfg.debug_checks != 0 ? 1 : 0, lp.block_base, lp.status);
  if (err != cudaSuccess) return err;
  err = launch_pdl(scan_kernel, dim3(1), dim3(1024), 0, s, 1, n_seg, E, lp.block_base, lp.counts, lp.offsets,
                   lp.padded_offsets, lp.tile_prefix, lp.sched);
  if (err != cudaSuccess) return err;
  err = launch_pdl(rank_kernel, dim3(n_seg), dim3(kThreads), kWarps * E * sizeof(int32_t), s, 1, batch, k, E,
                   (const int32_t*)lp.block_base, lp.row_of_pair, lp.pair_of_row, cap_rows, lp.status,
                   cfg.gather_a ? lp.src_row : (int32_t*)nullptr);
  if (err != cudaSuccess) return err;
  if (after_index) { err = cudaEventRecord(after_index, s); if (err != cudaSuccess) return err; }
  if (cfg.gather_a) {
    err = launch_pdl(mark_padding_kernel, dim3(E), dim3(128), 0, s, 1, E, (const int32_t*)lp.counts,
                     (const int32_t*)lp.padded_offsets, lp.pair_of_row, cap_rows);
    *launches += 4;
    return err;
  }
  const bool fp8 = cfg.dtype == CEP_FP8_E4M3_BLOCK128, mx = cfg.dtype == CEP_MXFP4_E4M3;
  const int row_bytes = cfg.hidden * (dtype_is_bytes(cfg.dtype) ? 1 : 2);
  const int n_scale = (fp8 || mx) ? cfg.hidden / kQuantBlock : 0;       // 32-bit scale words per row
  err = launch_pdl(scatter_rows_kernel<4>, dim3(batch.n_tokens + E), dim3(kThreads), 0, s, 1, batch, k, E, row_bytes, n_scale,
                   (const int32_t*)lp.row_of_pair, (const int32_t*)lp.counts, (const int32_t*)lp.padded_offsets,
                   lp.pair_of_row, static_cast<uint8_t*>(xp), (fp8 || mx) ? static_cast<uint32_t*>(xp_scales) : (uint32_t*)nullptr,
                   mx ? 1 : 0, cap_rows);
  *launches += 4;
  return err;
}

}  // namespace cep

// ---------------------------------------------------------------------------------------------
// Allocation-free variant of the index part of the layout transform (histogram -> scan -> rank).
//
// Some users of this library cannot give it scratch memory at all: a plug-in running inside an
// inference server whose memory pool already owns the whole device (a cudaMalloc there fails, or
// steals from the KV cache), or a caller on a latency-critical path where an allocation would
// synchronise the device.  For them the kernels' integer scratch (per-segment histograms, tile
// prefix, status words) lives in the fixed array below, which every GPU that loads the library
// holds (about 1 MiB) until the process exits.  The array is shared by all calls and keeps the
// previous call's contents: what must start at zero is cleared at the start of each call, and
// two calls whose GPU work overlaps (different streams, no ordering between them) race on it.
namespace {

constexpr int kNoAllocHistInts = 262144;          // room for n_segments * n_experts_local histogram cells
constexpr int kNoAllocHeadInts = 2048;            // tile prefix [E+1 <= 1025] and the status words
static __device__ __align__(256) int32_t g_noalloc_scratch[kNoAllocHeadInts + kNoAllocHistInts];

constexpr int kMaxDevices = 64;
int32_t* g_noalloc_ptr[kMaxDevices] = {};         // device address of the array, per device

// The array's name is only a host-side handle; its device address is looked up once per device.
cudaError_t noalloc_scratch_address(int32_t** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!g_noalloc_ptr[dev]) {
    int32_t* ptr = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    g_noalloc_ptr[dev] = ptr;
  }
  *out = g_noalloc_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int layout_indices_noalloc(const int32_t* topk_ids, int32_t n_tokens, int32_t top_k,
                                      int32_t n_experts_local, int32_t n_experts_global, int32_t* counts,
                                      int32_t* offsets, int32_t* padded_offsets, int32_t* row_of_pair,
                                      int32_t* pair_of_row, int32_t pair_of_row_capacity, int32_t* status,
                                      void* stream) {
  using namespace cep;
  if (!topk_ids || !counts || !offsets || !padded_offsets || !row_of_pair || !pair_of_row) return CEP_ERR_ARG;
  if (n_tokens <= 0 || top_k <= 0 || top_k > 32 || n_experts_local <= 0 || n_experts_local > 1024 ||
      n_experts_global < n_experts_local || pair_of_row_capacity <= 0)
    return CEP_ERR_ARG;
  const long long n_pairs = (long long)n_tokens * top_k;
  if (n_pairs > (1ll << 30)) return CEP_ERR_CAPACITY;
  const long long n_seg = (n_pairs + kSegPairs - 1) / kSegPairs;
  if (n_seg * n_experts_local > kNoAllocHistInts) return CEP_ERR_CAPACITY;   // beyond the fixed scratch
  int32_t* scratch = nullptr;
  if (noalloc_scratch_address(&scratch) != cudaSuccess) return CEP_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t* tile_prefix = scratch;                       // [E+1]
  int32_t* st_words = scratch + 1536;                   // [kStWords]
  int32_t* seg_hist = scratch + kNoAllocHeadInts;       // [n_seg, E]
  if (cudaMemsetAsync(st_words, 0, kStWords * sizeof(int32_t), st) != cudaSuccess) return CEP_ERR_CUDA;
  BatchDesc batch{};
  batch.chunk[0].ids = topk_ids;
  batch.chunk[0].n_tokens = n_tokens;
  batch.n_chunks = 1;
  batch.n_tokens = n_tokens;
  const int E = n_experts_local;
  hist_kernel<<<(int)n_seg, kThreads, E * sizeof(int32_t), st>>>(batch, top_k, E, n_experts_global, 0, seg_hist, st_words);
  scan_kernel<<<1, 1024, 0, st>>>((int)n_seg, E, seg_hist, counts, offsets, padded_offsets, tile_prefix, scratch + 1600);
  rank_kernel<<<(int)n_seg, kThreads, kWarps * E * sizeof(int32_t), st>>>(batch, top_k, E, seg_hist, row_of_pair,
                                                                        pair_of_row, pair_of_row_capacity, st_words,
                                                                        (int32_t*)nullptr);
  if (cudaGetLastError() != cudaSuccess) return CEP_ERR_CUDA;
  if (status) {
    // status[0]: an id was outside [0, n_experts_global); status[1]: a row did not fit pair_of_row
    if (cudaMemcpyAsync(status, st_words + kStBadRouting, sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(status + 1, st_words + kStBoundsViolation, sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
      return CEP_ERR_CUDA;
  }
  return CEP_OK;
}
