// Grouped expert GEMM on the sm_100a tensor cores: the "expert GEMMs" of a grouped FFN
// invocation (Appendix "Grouped FFN invocations"), with the intervening activation fused
// into the first GEMM's epilogue.
//
//   D[rows of expert e, N] = A[rows of expert e, K] * B[e][N, K]^T        (both operands K-major)
//
// Persistent, warp-specialised CTAs (one per SM):
//   warp 0      TMA producer: 128xK-slab of A and 256xK-slab of B per stage, 128-byte swizzle
//   warp 1      MMA issuer:   tcgen05.mma (M=128, N=256) accumulating fp32 in tensor memory
//   warps 2-5   epilogue:     tcgen05.ld -> registers -> (SiLU(gate)*up) -> bf16 -> global
// Tensor memory holds two 128x256 fp32 accumulators, so the epilogue of tile i overlaps the
// main loop of tile i+1.  All mbarrier waits are bounded: on expiry the kernel records
// kStTimeout in the status word and every role drains and exits normally.
#include <cuda.h>
#include <cuda_bf16.h>

#include "cep_common.h"
#include "gemm_tcgen05.h"
#include "tcgen05_ptx.cuh"

namespace cep {
namespace {

constexpr int BM = 128;                 // rows per tile (UMMA M)
constexpr int BN = 256;                 // accumulator columns per tile (UMMA N)
constexpr int BKB = 128;                // bytes of K per stage = one 128-byte swizzle span
constexpr int kStages = 4;
constexpr int A_STAGE = BM * BKB;       // 16 KiB
constexpr int B_STAGE = BN * BKB;       // 32 KiB
constexpr int kThreads = 192;
constexpr int kEpiWarp0 = 2;
constexpr int kTmemCols = 512;

struct __align__(8) Barriers {
  uint64_t full[kStages], empty[kStages], acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};
constexpr int kSmemBytes = kStages * (A_STAGE + B_STAGE) + 1024 /*alignment slack*/ + 256;
static_assert(sizeof(Barriers) <= 256, "barrier block");

using namespace ptx;

// Epilogue of one 128-row x 256-column accumulator: each thread owns one row (one tensor-memory
// lane), reads it 32 columns at a time, applies SiLU(gate)*up when the tile holds [128 gate | 128 up]
// columns, rounds to bf16 once and stores 64 contiguous bytes.  Rows at or beyond the expert's
// count (padding, or the next expert's rows under a pair tile) are not stored.
template <bool kSwiglu>
__device__ __forceinline__ void epilogue_tile(uint32_t t_addr, int r_in_group, int expert, int n_block,
                                              int n_out_cols, int out_ld, __nv_bfloat16* __restrict__ out,
                                              const int32_t* __restrict__ counts,
                                              const int32_t* __restrict__ padded_offsets) {
  const bool row_ok = r_in_group < counts[expert];
  const size_t grow = (size_t)(padded_offsets[expert] + r_in_group);
  if (kSwiglu) {
    __nv_bfloat16* orow = out + grow * out_ld + n_block * (BN / 2);
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
      uint32_t g[32], u[32];
      tc_ld32(t_addr + c * 32, g);
      tc_ld32(t_addr + 128 + c * 32, u);
      tc_wait_ld();
      if (row_ok && n_block * (BN / 2) + c * 32 < n_out_cols) {
        uint4* dst = reinterpret_cast<uint4*>(orow + c * 32);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint4 v;
          v.x = pack_bf16(silu_mul(__uint_as_float(g[8 * q + 0]), __uint_as_float(u[8 * q + 0])),
                          silu_mul(__uint_as_float(g[8 * q + 1]), __uint_as_float(u[8 * q + 1])));
          v.y = pack_bf16(silu_mul(__uint_as_float(g[8 * q + 2]), __uint_as_float(u[8 * q + 2])),
                          silu_mul(__uint_as_float(g[8 * q + 3]), __uint_as_float(u[8 * q + 3])));
          v.z = pack_bf16(silu_mul(__uint_as_float(g[8 * q + 4]), __uint_as_float(u[8 * q + 4])),
                          silu_mul(__uint_as_float(g[8 * q + 5]), __uint_as_float(u[8 * q + 5])));
          v.w = pack_bf16(silu_mul(__uint_as_float(g[8 * q + 6]), __uint_as_float(u[8 * q + 6])),
                          silu_mul(__uint_as_float(g[8 * q + 7]), __uint_as_float(u[8 * q + 7])));
          dst[q] = v;
        }
      }
    }
  } else {
    __nv_bfloat16* orow = out + grow * out_ld + n_block * BN;
#pragma unroll 1
    for (int c = 0; c < 8; ++c) {
      uint32_t d[32];
      tc_ld32(t_addr + c * 32, d);
      tc_wait_ld();
      if (row_ok && n_block * BN + c * 32 < n_out_cols) {
        uint4* dst = reinterpret_cast<uint4*>(orow + c * 32);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint4 v;
          v.x = pack_bf16(__uint_as_float(d[8 * q + 0]), __uint_as_float(d[8 * q + 1]));
          v.y = pack_bf16(__uint_as_float(d[8 * q + 2]), __uint_as_float(d[8 * q + 3]));
          v.z = pack_bf16(__uint_as_float(d[8 * q + 4]), __uint_as_float(d[8 * q + 5]));
          v.w = pack_bf16(__uint_as_float(d[8 * q + 6]), __uint_as_float(d[8 * q + 7]));
          dst[q] = v;
        }
      }
    }
  }
}

// ------------------------------------------------------------------ the kernel (one CTA per tile)
template <bool kSwiglu>
__global__ void __launch_bounds__(kThreads, 1)
grouped_gemm_bf16_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                         int num_kb /*K*2/128*/, int n_blocks_n, int n_group, int n_experts, int n_out_cols, int out_ld,
                         __nv_bfloat16* __restrict__ out, const int32_t* __restrict__ tile_prefix,
                         const int32_t* __restrict__ counts, const int32_t* __restrict__ padded_offsets,
                         int32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  pdl_enter();
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + kStages * A_STAGE;
  Barriers* bars = reinterpret_cast<Barriers*>(smem + kStages * (A_STAGE + B_STAGE));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&bars->full[s]), 1); mbar_init(smem_u32(&bars->empty[s]), 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&bars->acc_full[s]), 1); mbar_init(smem_u32(&bars->acc_empty[s]), 4); }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&bars->tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  const int total_tiles = tile_prefix[n_experts] * n_blocks_n;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
        TileCoord tc;
        if (!decode_tile(tile_prefix, n_experts, n_blocks_n, n_group, tile, &tc)) break;
        const int row0 = padded_offsets[tc.expert] + tc.m_block * BM;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag, status)) { ok = false; break; }
          const uint32_t full = smem_u32(&bars->full[stage]);
          mbar_expect_tx(full, A_STAGE + B_STAGE);
          tma_load_2d(smem_u32(smem_a + stage * A_STAGE), &tm_a, kb * (BKB / 2), row0, full);
          tma_load_3d(smem_u32(smem_b + stage * B_STAGE), &tm_b, kb * (BKB / 2), tc.n_block * BN, tc.expert, full);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(BM, BN);
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
        if (!mbar_wait(smem_u32(&bars->acc_empty[acc]), acc_phase ^ 1u, abort_flag, status)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(smem_u32(&bars->full[stage]), phase, abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t adesc = make_smem_desc(smem_u32(smem_a + stage * A_STAGE));
          const uint64_t bdesc = make_smem_desc(smem_u32(smem_b + stage * B_STAGE));
#pragma unroll
          for (int k4 = 0; k4 < BKB / 32; ++k4)       // 32 bytes of K per MMA (16 bf16)
            tc_mma_f16(d_tmem, adesc + (uint64_t)(k4 * 2), bdesc + (uint64_t)(k4 * 2), idesc, (kb | k4) != 0 ? 1u : 0u);
          tc_commit(smem_u32(&bars->empty[stage]));   // frees the stage once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(smem_u32(&bars->acc_full[acc]));     // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue (warps 2..5)
    const int lane_grp = warp & 3;                     // tensor-memory lanes this warp may read
    int acc = 0; uint32_t acc_phase = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
      TileCoord tc;
      if (!decode_tile(tile_prefix, n_experts, n_blocks_n, n_group, tile, &tc)) break;
      // the lanes may leave the polling loop in different iterations; the tensor-memory loads below are
      // warp-collective (.sync.aligned), so the warp must be converged again before it issues them
      const bool got = mbar_wait_relaxed(smem_u32(&bars->acc_full[acc]), acc_phase, abort_flag, status);
      if (!__all_sync(0xffffffffu, got)) break;
      tc_fence_after();
      epilogue_tile<kSwiglu>(tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(acc * BN),
                             tc.m_block * BM + lane_grp * 32 + lane, tc.expert, tc.n_block, n_out_cols, out_ld, out,
                             counts, padded_offsets);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->acc_empty[acc]));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }
  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}


// ------------------------------------------------------------------ the kernel (a CTA pair per 256x256 tile)
// Two CTAs of a cluster share one tile of 256 rows x 256 accumulator columns (tcgen05 cta_group::2):
// each loads its own 128 activation rows and HALF of the weight tile, the leader (cluster rank 0)
// issues M=256 MMAs that read both CTAs' shared memory, and each CTA keeps the accumulator of its
// own 128 rows in its own tensor memory.  Per k-step an SM takes in 32 KB instead of 48 KB for the
// same number of MMA cycles.  An expert with an odd number of 128-row blocks leaves the second half
// of its last pair tile empty (those rows are computed and not stored).
//
// Barriers: full[s] (leader; its producer's arrival + both CTAs' TMA bytes), empty[s] (one per CTA,
// arrived by the leader's commit), acc_full[a] (one per CTA, leader's commit), acc_empty[a] (leader;
// 4 epilogue warps x 2 CTAs).
#ifndef CEP_PAIR_STAGES
#define CEP_PAIR_STAGES 6
#endif
constexpr int kPairStages = CEP_PAIR_STAGES;
constexpr int PB_STAGE = (BN / 2) * BKB;               // 16 KiB: this CTA's half of the weight tile
#ifndef CEP_PAIR_MAXE
#define CEP_PAIR_MAXE 1024
#endif
constexpr int kMaxExperts = CEP_PAIR_MAXE;
constexpr int kTilePoison = -2;
constexpr int kSchedRing = 4;                          // tile ids in flight between the scheduler and its readers
constexpr int kSchedReaders = 11;                      // leader: producer, MMA, 4 epilogue warps; peer: producer, 4 epilogue warps
constexpr int kPairThreads = 224;                      // warp 6 of the leader CTA hands out tiles
#ifndef CEP_GATHER_WARPS
#define CEP_GATHER_WARPS 8
#endif
constexpr int kGatherWarps = CEP_GATHER_WARPS;         // gathering variant: warps 7.. of both CTAs fetch the activation rows
constexpr int kGatherLanes = 32 / kGatherWarps;        // lanes of each that issue one four-row gather per stage
constexpr int kPairThreadsGather = kPairThreads + 32 * kGatherWarps;
struct __align__(8) PairBarriers {
  uint64_t full[kPairStages], empty[kPairStages], acc_full[2], acc_empty[2];
  uint64_t sched_full[kSchedRing], sched_empty[kSchedRing];
  int32_t sched_tile[kSchedRing];
  uint32_t tmem_base;
  int abort_flag;
};

// Reader side of the tile ring: every reading role (a single thread, or a warp in lock-step) walks
// the ring in order; -1 ends the kernel.  The peer CTA's copy of the ring is written by the leader
// through the cluster, so its readers acquire at cluster scope.
struct TileReader {
  int slot = 0; uint32_t phase = 0;
  // Waits for the next tile id.  The caller must call done() once every thread of the role has the value.
  __device__ __forceinline__ int next(PairBarriers* bars, bool is_peer, volatile int* abort_flag, int32_t* status) {
    const uint32_t bar = smem_u32(&bars->sched_full[slot]);
    const bool ok = is_peer ? mbar_wait_acq_cluster(bar, phase, abort_flag, status) : mbar_wait_relaxed(bar, phase, abort_flag, status);
    if (!ok) return -1;
    const int t = bars->sched_tile[slot];
    if (t < -1) {                              // a slot read before its value arrived: report, never use it
      atomicExch(&status[kStDetail], 0x5C4ED);
      atomicExch(&status[kStTimeout], 1);
      *abort_flag = 1;
      return -1;
    }
    return t;
  }
  // Frees the ring slot for the scheduler (one arrival per reading role) and advances.
  __device__ __forceinline__ void done(PairBarriers* bars, bool signal) {
    if (signal) mbar_arrive_cluster(mapa(smem_u32(&bars->sched_empty[slot]), 0));
    if (++slot == kSchedRing) { slot = 0; phase ^= 1u; }
  }
};
constexpr int kPairSmemBytes = kPairStages * (A_STAGE + PB_STAGE) + (kMaxExperts + 1) * 4 + 1024 + 256;
static_assert(sizeof(PairBarriers) <= 256, "barrier block");

// kGather: the activation operand is not the permuted copy but the caller's token tensor itself; tm_a then
// describes that tensor with one-row boxes, src_row[r] is the tensor row that physical row r holds, and the
// producer warp fetches every 128-row operand stage as 32 four-row gathers (one per lane).
template <bool kSwiglu, bool kGather>
__global__ void __launch_bounds__(kGather ? kPairThreadsGather : kPairThreads, 1)
grouped_gemm_bf16_pair_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                              int num_kb, int n_blocks_n, int n_group, int n_experts, int n_out_cols, int out_ld,
                              __nv_bfloat16* __restrict__ out, const int32_t* __restrict__ tile_prefix,
                              const int32_t* __restrict__ counts, const int32_t* __restrict__ padded_offsets,
                              const int32_t* __restrict__ src_row, int32_t* __restrict__ tile_counter,
                              int32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  pdl_enter();
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + kPairStages * A_STAGE;
  PairBarriers* bars = reinterpret_cast<PairBarriers*>(smem + kPairStages * (A_STAGE + PB_STAGE));
  int32_t* pair_prefix = reinterpret_cast<int32_t*>(smem + kPairStages * (A_STAGE + PB_STAGE) + 256);   // [E+1]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  volatile int* abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kPairStages; ++s) { mbar_init(smem_u32(&bars->full[s]), 1); mbar_init(smem_u32(&bars->empty[s]), 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&bars->acc_full[s]), 1); mbar_init(smem_u32(&bars->acc_empty[s]), 8); }
    for (int s = 0; s < kSchedRing; ++s) {
      mbar_init(smem_u32(&bars->sched_full[s]), 1); mbar_init(smem_u32(&bars->sched_empty[s]), kSchedReaders + (kGather ? 2 * kGatherWarps : 0));
      bars->sched_tile[s] = kTilePoison;     // shared memory keeps what the previous CTA on this SM left
    }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x == 32) {          // cumulative number of pair tiles (two 128-row blocks) per expert
    int run = 0;
    for (int e = 0; e < n_experts; ++e) {
      pair_prefix[e] = run;
      run += (tile_prefix[e + 1] - tile_prefix[e] + 1) >> 1;
    }
    pair_prefix[n_experts] = run;
  }
  __syncthreads();
  if (warp == 1) {                  // executed by the same warp of both CTAs
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&bars->tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();               // both CTAs' barriers are initialised before any remote arrival
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  const int total_tiles = pair_prefix[n_experts] * n_blocks_n;
  const bool is_peer = rank != 0;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      TileReader rd;
      for (;ok;) {
        const int tile = rd.next(bars, is_peer, abort_flag, status);
        rd.done(bars, true);
        if (tile < 0) break;
        TileCoord tc;
        if (!decode_tile(pair_prefix, n_experts, n_blocks_n, n_group, tile, &tc)) break;
        const int row0 = padded_offsets[tc.expert] + tc.m_block * (2 * BM) + (int)rank * BM;
        const int n0 = tc.n_block * BN + (int)rank * (BN / 2);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag, status)) { ok = false; break; }
          const uint32_t full = mapa(smem_u32(&bars->full[stage]), 0);        // the leader's barrier
          // the leader alone arrives, announcing both CTAs' bytes; the peer's bytes can only land in
          // this phase because its loads wait for the stage to be freed by the leader's MMAs
          if (rank == 0) mbar_expect_tx(smem_u32(&bars->full[stage]), 2 * (A_STAGE + PB_STAGE));
          // (the gathering variant's activation rows are fetched by warps 7.., which wait for the stage themselves)
          if constexpr (!kGather) tma_load_2d_pair(smem_u32(smem_a + stage * A_STAGE), &tm_a, kb * (BKB / 2), row0, full);
          tma_load_3d_pair(smem_u32(smem_b + stage * PB_STAGE), &tm_b, kb * (BKB / 2), n0, tc.expert, full);
          if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(2 * BM, BN);
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      TileReader rd;
      for (;ok;) {
        const int tile = rd.next(bars, false, abort_flag, status);
        rd.done(bars, true);
        if (tile < 0) break;
        if (!mbar_wait(smem_u32(&bars->acc_empty[acc]), acc_phase ^ 1u, abort_flag, status)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(smem_u32(&bars->full[stage]), phase, abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t adesc = make_smem_desc(smem_u32(smem_a + stage * A_STAGE));
          const uint64_t bdesc = make_smem_desc(smem_u32(smem_b + stage * PB_STAGE));
#pragma unroll
          for (int k4 = 0; k4 < BKB / 32; ++k4)
            tc_mma_f16_pair(d_tmem, adesc + (uint64_t)(k4 * 2), bdesc + (uint64_t)(k4 * 2), idesc, (kb | k4) != 0 ? 1u : 0u);
          tc_commit_pair_both(smem_u32(&bars->empty[stage]), 3);   // frees the stage in both CTAs
          if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit_pair_both(smem_u32(&bars->acc_full[acc]), 3);  // accumulator complete, both halves
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else if (warp >= 7) {
    // ---------------------------------------------------------------- row gather (kGather only; both CTAs)
    // Warp g fetches rows [g, g+1) * 128/kGatherWarps of this CTA's operand block: its first kGatherLanes lanes
    // issue one four-row gather each per stage.  The warp walks tiles and stages in lock-step behind lane 0,
    // which does the waiting; the stage's byte count is announced by the producer warp of the leader CTA.
    if constexpr (kGather) {
      const int g = warp - 7;
      int stage = 0; uint32_t phase = 0;
      TileReader rd;
      for (;;) {
        int tile = -1;
        if (lane == 0) { tile = rd.next(bars, is_peer, abort_flag, status); rd.done(bars, true); }
        tile = __shfl_sync(0xffffffffu, tile, 0);
        if (tile < 0) break;
        TileCoord tc;
        if (!decode_tile(pair_prefix, n_experts, n_blocks_n, n_group, tile, &tc)) break;
        const int poff = padded_offsets[tc.expert], count = counts[tc.expert];
        const int row_in_block = (g * kGatherLanes + lane) * 4;                       // first of this lane's four rows
        const int r_local = tc.m_block * (2 * BM) + (int)rank * BM + row_in_block;
        // Rows past the expert's count are padding: their products are never stored, so they re-read the
        // expert's first row (always a real row) instead of an index that nothing wrote.
        const int first = __ldg(src_row + poff);
        int4 idx = make_int4(first, first, first, first);
        if (lane < kGatherLanes && r_local < count) {
          const int4 got = __ldg(reinterpret_cast<const int4*>(src_row + poff + r_local));
          idx.x = got.x;
          if (r_local + 1 < count) idx.y = got.y;
          if (r_local + 2 < count) idx.z = got.z;
          if (r_local + 3 < count) idx.w = got.w;
        }
        int ok = 1;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (lane == 0) ok = mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag, status) ? 1 : 0;
          ok = __shfl_sync(0xffffffffu, ok, 0);
          if (!ok) break;
          if (lane < kGatherLanes)
            tma_gather4_pair(smem_u32(smem_a + stage * A_STAGE + row_in_block * BKB), &tm_a, kb * (BKB / 2), idx,
                             mapa(smem_u32(&bars->full[stage]), 0));
          if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
      }
    }
  } else if (warp == 6) {
    // ---------------------------------------------------------------- tile scheduler (leader CTA only)
    // Tiles are handed out in linear order from a global counter, so the CTA pairs running at any time
    // work on neighbouring tiles whatever their individual speeds: the set of operand rows in flight
    // (and so the L2 working set) stays one wave wide instead of spreading as slower pairs fall behind.
    if (lane == 0 && !is_peer) {
      int slot = 0; uint32_t phase = 0;
      for (;;) {
        if (!mbar_wait_relaxed(smem_u32(&bars->sched_empty[slot]), phase ^ 1u, abort_flag, status)) break;
        int t = atomicAdd(tile_counter, 1);
        if (t >= total_tiles) t = -1;
        bars->sched_tile[slot] = t;
        st_shared_cluster_u32(mapa(smem_u32(&bars->sched_tile[slot]), 1), (uint32_t)t);
        mbar_arrive(smem_u32(&bars->sched_full[slot]));
        mbar_arrive_release_cluster(mapa(smem_u32(&bars->sched_full[slot]), 1));
        if (t < 0) break;
        if (++slot == kSchedRing) { slot = 0; phase ^= 1u; }
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue (warps 2..5, both CTAs)
    const int lane_grp = warp & 3;
    int acc = 0; uint32_t acc_phase = 0;
    TileReader rd;
    for (;;) {
      const int tile = rd.next(bars, is_peer, abort_flag, status);
      __syncwarp();                                    // every lane holds the id before the slot is freed
      rd.done(bars, lane == 0);
      if (tile < 0) break;
      TileCoord tc;
      if (!decode_tile(pair_prefix, n_experts, n_blocks_n, n_group, tile, &tc)) break;
      // the lanes may leave the polling loop in different iterations; the tensor-memory loads below are
      // warp-collective (.sync.aligned), so the warp must be converged again before it issues them
      const bool got = mbar_wait_relaxed(smem_u32(&bars->acc_full[acc]), acc_phase, abort_flag, status);
      if (!__all_sync(0xffffffffu, got)) break;
      tc_fence_after();
      epilogue_tile<kSwiglu>(tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(acc * BN),
                             tc.m_block * (2 * BM) + (int)rank * BM + lane_grp * 32 + lane, tc.expert, tc.n_block,
                             n_out_cols, out_ld, out, counts, padded_offsets);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa(smem_u32(&bars->acc_empty[acc]), 0));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }
  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();               // no CTA leaves while its peer may still signal or read it
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// Probe of the bounded-wait path: one CTA waits, with the same wait routine the GEMM kernels use, on a
// barrier that nothing ever arrives on.  The wait gives up after limit_ns, records the timeout in the status
// word and the kernel exits normally (no trap, the context stays usable).
__global__ void wait_probe_kernel(unsigned long long limit_ns, int32_t* __restrict__ status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const bool got = mbar_wait_limit(smem_u32(&bar), 0u, &abort_flag, status, limit_ns);
  if (got && threadIdx.x == 0) atomicExch(&status[kStDetail], 0xBAD);   // cannot happen: nobody arrives
}

}  // namespace

cudaError_t launch_wait_probe(unsigned long long limit_ns, int32_t* status, cudaStream_t s, int64_t* launches) {
  wait_probe_kernel<<<1, 64, 0, s>>>(limit_ns, status);
  *launches += 1;
  return cudaGetLastError();
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// rows x K operand, K contiguous; box = 128 bytes of K x box_rows rows; 128-byte swizzle.
int make_operand_map(GemmTensorMap* out, const void* base, int elt_bytes, int K, long long rows, int n_batch,
                     int box_rows) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return -1;
  static_assert(sizeof(GemmTensorMap) == sizeof(CUtensorMap), "tensor map size");
  CUtensorMap* m = reinterpret_cast<CUtensorMap*>(out);
  const CUtensorMapDataType dt = elt_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8;
  cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, (cuuint64_t)n_batch};
  cuuint64_t strides[2] = {(cuuint64_t)K * elt_bytes, (cuuint64_t)K * elt_bytes * (cuuint64_t)rows};
  cuuint32_t box[3] = {(cuuint32_t)(BKB / elt_bytes), (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  const int rank = n_batch > 0 ? 3 : 2;
  CUresult r = enc(m, dt, rank, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -2;
}

int make_store_map(GemmTensorMap* out, void* base, int elt_bytes, int cols, long long rows) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return -1;
  CUtensorMap* m = reinterpret_cast<CUtensorMap*>(out);
  const CUtensorMapDataType dt = elt_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * elt_bytes};
  cuuint32_t box[2] = {(cuuint32_t)(64 / elt_bytes), 32};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(m, dt, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B,
                   CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -2;
}

int gemm_tile_rows() { return BM; }
int gemm_tile_cols() { return BN; }

// cudaFuncSetAttribute and the occupancy answer hold per device: one slot per device ordinal
constexpr int kMaxDevices = 64;
static int g_pair_clusters[kMaxDevices];   // co-resident CTA pairs on the device + 1 (0: not set up yet)
static bool g_single_ready[kMaxDevices];

static cudaError_t current_device(int* dev) {
  cudaError_t e = cudaGetDevice(dev);
  if (e != cudaSuccess) return e;
  return (*dev < 0 || *dev >= kMaxDevices) ? cudaErrorInvalidDevice : cudaSuccess;
}

static cudaError_t setup_pair_kernels(int dev, int n_sms) {
  if (g_pair_clusters[dev] > 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(grouped_gemm_bf16_pair_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmemBytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(grouped_gemm_bf16_pair_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmemBytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(grouped_gemm_bf16_pair_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmemBytes);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3(n_sms & ~1, 1, 1); cfg.blockDim = dim3(kPairThreads, 1, 1);
  cfg.dynamicSmemBytes = kPairSmemBytes; cfg.attrs = attr; cfg.numAttrs = 1;
  int n = 0;
  e = cudaOccupancyMaxActiveClusters(&n, grouped_gemm_bf16_pair_kernel<true, false>, &cfg);
  if (e != cudaSuccess) return e;
  g_pair_clusters[dev] = n + 1;
  return cudaSuccess;
}

cudaError_t launch_gemm_tcgen05_pair(const GemmProblem& p, const GemmTensorMap& tm_a, const GemmTensorMap& tm_b,
                                     void* out, const LayoutPtrs& lp, const int32_t* src_row, int max_pair_tiles,
                                     int n_sms, cudaStream_t s, int64_t* launches) {
  if (p.is_fp8 || (src_row && !p.swiglu)) return cudaErrorNotSupported;
  int dev = 0;
  cudaError_t e = current_device(&dev);
  if (e != cudaSuccess) return e;
  e = setup_pair_kernels(dev, n_sms);
  if (e != cudaSuccess) return e;
  const int resident = g_pair_clusters[dev] - 1;
  if (resident < 1) return cudaErrorNotSupported;
  const int n_blocks_n = (p.N + BN - 1) / BN;
  const int n_out_cols = p.swiglu ? p.N / 2 : p.N;
  int clusters = max_pair_tiles < resident ? max_pair_tiles : resident;
  if (clusters < 1) return cudaSuccess;
  int num_kb = p.K * 2 / BKB;
  int n_experts = p.n_experts, out_ld = p.out_ld;
  int n_group = n_group_for(n_blocks_n, BN, p.K, 2);
  int32_t* counter = lp.sched + (p.swiglu ? 0 : 1);     // zeroed by this invocation's scan kernel
  __nv_bfloat16* o = (__nv_bfloat16*)out;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = dim3(2 * clusters, 1, 1); cfg.blockDim = dim3(kPairThreads, 1, 1);
  cfg.dynamicSmemBytes = kPairSmemBytes; cfg.stream = s; cfg.attrs = attr; cfg.numAttrs = 2;
  const CUtensorMap& a = reinterpret_cast<const CUtensorMap&>(tm_a);
  const CUtensorMap& b = reinterpret_cast<const CUtensorMap&>(tm_b);
  const int32_t* no_rows = nullptr;
  if (src_row) cfg.blockDim = dim3(kPairThreadsGather, 1, 1);
  if (src_row)
    e = cudaLaunchKernelEx(&cfg, grouped_gemm_bf16_pair_kernel<true, true>, a, b, num_kb, n_blocks_n, n_group, n_experts, n_out_cols, out_ld,
                           o, (const int32_t*)lp.tile_prefix, (const int32_t*)lp.counts, (const int32_t*)lp.padded_offsets, src_row, counter, lp.status);
  else if (p.swiglu)
    e = cudaLaunchKernelEx(&cfg, grouped_gemm_bf16_pair_kernel<true, false>, a, b, num_kb, n_blocks_n, n_group, n_experts, n_out_cols, out_ld,
                           o, (const int32_t*)lp.tile_prefix, (const int32_t*)lp.counts, (const int32_t*)lp.padded_offsets, no_rows, counter, lp.status);
  else
    e = cudaLaunchKernelEx(&cfg, grouped_gemm_bf16_pair_kernel<false, false>, a, b, num_kb, n_blocks_n, n_group, n_experts, n_out_cols, out_ld,
                           o, (const int32_t*)lp.tile_prefix, (const int32_t*)lp.counts, (const int32_t*)lp.padded_offsets, no_rows, counter, lp.status);
  *launches += 1;
  return e;
}

cudaError_t launch_gemm_tcgen05(const GemmProblem& p, const GemmTensorMap& tm_a, const GemmTensorMap& tm_b,
                                void* out, const LayoutPtrs& lp, int max_tiles, int n_sms, cudaStream_t s,
                                int64_t* launches) {
  if (p.is_fp8) return cudaErrorNotSupported;
  int dev = 0;
  cudaError_t e = current_device(&dev);
  if (e != cudaSuccess) return e;
  if (!g_single_ready[dev]) {
    e = cudaFuncSetAttribute(grouped_gemm_bf16_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(grouped_gemm_bf16_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    g_single_ready[dev] = true;
  }
  const int n_blocks_n = (p.N + BN - 1) / BN;
  const int n_out_cols = p.swiglu ? p.N / 2 : p.N;
  int grid = max_tiles < n_sms ? max_tiles : n_sms;
  if (grid < 1) return cudaSuccess;
  const int num_kb = p.K * 2 / BKB;
  const int n_group = n_group_for(n_blocks_n, BN, p.K, 2);
  const CUtensorMap& a = reinterpret_cast<const CUtensorMap&>(tm_a);
  const CUtensorMap& b = reinterpret_cast<const CUtensorMap&>(tm_b);
  if (p.swiglu)
    grouped_gemm_bf16_kernel<true><<<grid, kThreads, kSmemBytes, s>>>(a, b, num_kb, n_blocks_n, n_group, p.n_experts, n_out_cols,
        p.out_ld, (__nv_bfloat16*)out, lp.tile_prefix, lp.counts, lp.padded_offsets, lp.status);
  else
    grouped_gemm_bf16_kernel<false><<<grid, kThreads, kSmemBytes, s>>>(a, b, num_kb, n_blocks_n, n_group, p.n_experts, n_out_cols,
        p.out_ld, (__nv_bfloat16*)out, lp.tile_prefix, lp.counts, lp.padded_offsets, lp.status);
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace cep
