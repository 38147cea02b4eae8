// Grouped expert GEMM for block-scaled e4m3 operands (fp32 scales per 1x128 activation block and per
// 128x128 weight block), CTA pairs on 256x256 tiles:
//
//   D[m, n] = sum over 128-deep K blocks kb of  sa[m, kb] * sw[kb, n/128] * ( A_codes[m, kb] . B_codes[n, kb] )
//
// The scales are plain fp32, so they cannot ride on the tensor core's own (power-of-two, 1x32) block
// scaling.  Each K block is therefore multiplied on its own into a scratch accumulator in tensor memory
// (tcgen05.mma kind::f8f6f4, fp32 accumulate, two scratch buffers in flight), and eight "promotion"
// warps pull every partial product out of tensor memory and add it, scaled, into fp32 accumulators
// they hold in registers (128 per thread).
//
// Two things pace such a loop.  The thread that issues the MMAs: every tcgen05 instruction (mma, commit) and
// every barrier wait costs that one thread 60-100 cycles, and a K block here needs two waits (operands
// landed, scratch buffer free) on top of its four MMAs, against 512 cycles of tensor work.  And the round
// trip of a scratch buffer (MMAs complete -> promotion warps see it -> 128 values per thread read out ->
// buffer handed back -> next MMA), of which only two can be in flight.  So the issue
// is split over TWO threads, one per scratch buffer: K blocks alternate between them, each thread waits,
// issues and commits for its own buffer only, and since every K block goes to its own buffer and the
// promotion warps consume the buffers in K order, the result does not depend on how the two threads'
// MMAs interleave in the tensor pipe.  One commit per K block serves both as "operands consumed" for the
// TMA producer and as "partial product ready" for the promotion warps (barrier done[stage]).
// The promotion warps also run the epilogue:
//   GEMM1: SiLU(gate)*up, per-row amax over the tile's 128 columns, scale = amax/448, e4m3 codes
//          (round-to-nearest-even, saturating) + the scale: the "activation and quantization" step
//          between the two expert GEMMs (Appendix "Grouped FFN invocations")
//   GEMM2: bf16
// Roles (384 threads): warp 0 TMA producer, warps 1 and 3 MMA issuers of even / odd K blocks (leader CTA),
// warp 2 tile scheduler (leader CTA), warps 4-11 promotion + epilogue.  Tiles come from a global
// counter, as in the bf16 kernel.  All waits are bounded.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "cep_common.h"
#include "gemm_tcgen05.h"
#include "tcgen05_ptx.cuh"

namespace cep {
namespace {

using namespace ptx;

constexpr int BM = 128, BN = 256, BKB = 128;          // BKB bytes = 128 e4m3 elements = one scale block
constexpr int A_STAGE = BM * BKB;                      // 16 KiB
// kPair: CTA pairs (256x256 tiles, each CTA loads half of the weight tile, 6 stages of 32 KiB);
// !kPair: one CTA per 128x256 tile (whole weight tile per CTA, 4 stages of 48 KiB): every hand-off
// between the MMA warp and the promotion warps stays inside the SM
constexpr int kBarBytes = 512;
constexpr int kPromoWarp0 = 4, kPromoWarps = 8;
constexpr int kStoreStage = 2048;                      // per promotion warp: 32 rows x 64 bytes of output on their way to global memory
template <bool kPair> struct Geo {
  static constexpr int kStages = kPair ? 6 : 4;
  static constexpr int B_STAGE = (kPair ? BN / 2 : BN) * BKB;
  static constexpr int kRingReaders = kPair ? 20 : 11;    // producer, 2 MMA issuers, 8 promotion warps (+ peer: producer, 8)
  static constexpr int kPartArrivals = kPair ? 16 : 8;
  static constexpr int kSmemBytes = kStages * (A_STAGE + B_STAGE) + kBarBytes + (1024 + 1) * 4 + 12 + 2 * 2 * BM * 4 +
                                    kPromoWarps * kStoreStage + 512 + 1024;
};
constexpr int kMaxStages = 6;
constexpr int kThreads = 384;
constexpr int kTmemCols = 512;
constexpr int kMaxExperts = 1024;
constexpr int kRing = 4;
constexpr int kTilePoison = -2;

struct __align__(8) Bars {
  uint64_t full[kMaxStages];                          // operands of the stage have landed
  uint64_t done[kMaxStages];                          // the stage's MMAs have completed: operands consumed, partial ready
  uint64_t part_empty[2];                             // scratch accumulators in tensor memory read out
  uint64_t sched_full[kRing], sched_empty[kRing];
  uint64_t amax_bar[4];                               // per lane group: the two warps sharing its rows
  int32_t sched_tile[kRing][8];                       // a handed-out tile, decoded: see TileInfo
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(Bars) <= kBarBytes, "barrier block");
static_assert(BKB == 128 && Geo<true>::kStages % 2 == 0 && Geo<false>::kStages % 2 == 0, "a stage always pairs with the same scratch buffer");

// What the scheduler thread publishes per tile, so that no other role has to search the tile table or
// touch global memory at a tile boundary.
struct TileInfo {
  int tile;                    // linear index, -1: no more tiles
  int expert, m_block, n_block;
  int count;                   // rows of the expert
  int poff;                    // first (tile-aligned) row of the expert's group
};

struct Ring {
  int slot = 0; uint32_t phase = 0;
  __device__ __forceinline__ TileInfo next(Bars* b, bool is_peer, volatile int* abort_flag, int32_t* status) {
    TileInfo ti;
    ti.tile = -1; ti.expert = ti.m_block = ti.n_block = ti.count = ti.poff = 0;
    const uint32_t bar = smem_u32(&b->sched_full[slot]);
    const bool ok = is_peer ? mbar_wait_acq_cluster(bar, phase, abort_flag, status) : mbar_wait(bar, phase, abort_flag, status);
    if (!ok) return ti;
    const int4 v = *reinterpret_cast<const int4*>(&b->sched_tile[slot][0]);
    const int2 w = *reinterpret_cast<const int2*>(&b->sched_tile[slot][4]);
    if (v.x < -1) { atomicExch(&status[kStDetail], 0x5C4ED); atomicExch(&status[kStTimeout], 1); *abort_flag = 1; return ti; }
    ti.tile = v.x; ti.expert = v.y; ti.m_block = v.z; ti.n_block = v.w; ti.count = w.x; ti.poff = w.y;
    return ti;
  }
  template <bool kPair>
  __device__ __forceinline__ void done(Bars* b, bool signal) {
    if (signal) {
      if (kPair) mbar_arrive_cluster(mapa(smem_u32(&b->sched_empty[slot]), 0));
      else mbar_arrive(smem_u32(&b->sched_empty[slot]));
    }
    if (++slot == kRing) { slot = 0; phase ^= 1u; }
  }
};

// kAcc (0: overwrite the accumulator, 1: add to it) is an immediate, so the issuing thread spends no instruction on it
template <int kAcc>
__device__ __forceinline__ void tc_mma_f8_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n}"
               ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "n"(kAcc) : "memory");
}
template <int kAcc>
__device__ __forceinline__ void tc_mma_f8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n}"
               ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "n"(kAcc) : "memory");
}
// the four K=32 MMAs of one 128-deep K block (a descriptor advances by 32 bytes = 2 units per MMA)
template <bool kPair>
__device__ __forceinline__ void issue_k_block(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc) {
  if (kPair) {
    tc_mma_f8_pair<0>(d_tmem, adesc, bdesc, idesc);
    tc_mma_f8_pair<1>(d_tmem, adesc + 2, bdesc + 2, idesc);
    tc_mma_f8_pair<1>(d_tmem, adesc + 4, bdesc + 4, idesc);
    tc_mma_f8_pair<1>(d_tmem, adesc + 6, bdesc + 6, idesc);
  } else {
    tc_mma_f8<0>(d_tmem, adesc, bdesc, idesc);
    tc_mma_f8<1>(d_tmem, adesc + 2, bdesc + 2, idesc);
    tc_mma_f8<1>(d_tmem, adesc + 4, bdesc + 4, idesc);
    tc_mma_f8<1>(d_tmem, adesc + 6, bdesc + 6, idesc);
  }
}
// kind::f8f6f4: fp32 accumulate, e4m3 x e4m3 (format code 0), both operands K-major
__host__ __device__ constexpr uint32_t make_idesc_e4m3(int m, int n) {
  return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void setmaxnreg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 232;" ::: "memory"); }
__device__ __forceinline__ void setmaxnreg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 40;" ::: "memory"); }

// packed pairs of fp32: one instruction does two independent round-to-nearest multiply-adds
__device__ __forceinline__ unsigned long long pack_f32x2(uint32_t lo, uint32_t hi) {
  unsigned long long r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi)); return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void fma_f32x2(unsigned long long& acc, unsigned long long v, unsigned long long s) {
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(v), "l"(s));
}

// two e4m3 codes (round-to-nearest-even, saturating to +-448) from two floats: lo in bits 0-7
__device__ __forceinline__ uint32_t cvt_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm volatile("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}

// A warp holds 64 bytes of output per lane (lane = row).  Written to global memory by the threads, every store
// instruction would touch 32 rows with 16 bytes each and the tile's 64 KiB would queue in the load/store unit while
// the MMAs wait for these warps.  Instead the warp lays its 32 x 64 bytes out in 2 KiB of shared memory (16-byte
// chunk index XOR row bits: the TMA engine's 64-byte swizzle, which also keeps the writes free of bank conflicts)
// and one lane hands the box to the TMA engine, which writes it out on its own.  The box covers all 32 rows: the
// caller skips warps whose rows lie wholly beyond the expert's count (they may belong to the next expert); rows
// between the count and the end of the expert's 128-row block are padding and receive the zeros computed for them.
__device__ __forceinline__ void stage_rows_64B(uint8_t* stage, int lane, const uint4 (&ch)[4]) {
#pragma unroll
  for (int q = 0; q < 4; ++q)
    *reinterpret_cast<uint4*>(stage + lane * 64 + ((q ^ ((lane >> 1) & 3)) << 4)) = ch[q];
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the writes, as the TMA engine must see them
  __syncwarp();
}
__device__ __forceinline__ void tma_store_box(const CUtensorMap* map, const uint8_t* stage, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(stage)) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// the staging buffer may be overwritten again (the engine has read it)
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// every store of this thread has reached global memory
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

template <bool kSwiglu, bool kPair>
__global__ void __launch_bounds__(kThreads, 1)
grouped_gemm_fp8_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                             const __grid_constant__ CUtensorMap tm_out /*codes (GEMM1) or bf16 (GEMM2), as boxes*/,
                             int num_kb, int n_blocks_n, int n_group, int n_experts, int n_out_cols,
                             const float* __restrict__ a_scales /*[rows, num_kb]*/,
                             const float* __restrict__ b_scales /*[E, N/128, num_kb]*/,
                             float* __restrict__ out_scales /*GEMM1: [rows, out cols/128]*/,
                             const int32_t* __restrict__ tile_prefix, const int32_t* __restrict__ counts,
                             const int32_t* __restrict__ padded_offsets, int32_t* __restrict__ tile_counter,
                             int32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  pdl_enter();
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  constexpr int kStages = Geo<kPair>::kStages, B_STAGE = Geo<kPair>::B_STAGE;
  constexpr int kRowsPerTile = kPair ? 2 * BM : BM;
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + kStages * A_STAGE;
  Bars* bars = reinterpret_cast<Bars*>(smem + kStages * (A_STAGE + B_STAGE));
  int32_t* pair_prefix = reinterpret_cast<int32_t*>(smem + kStages * (A_STAGE + B_STAGE) + kBarBytes);
  float* s_amax = reinterpret_cast<float*>(pair_prefix + kMaxExperts + 4);           // [tile parity][half][128]
  // [promotion warp][kStoreStage], on a 512-byte boundary: the swizzle pattern is a function of the address bits
  uint8_t* s_store = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(s_amax + 2 * 2 * BM) + 511) & ~(uintptr_t)511);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = kPair ? cluster_ctarank() : 0u;
  const bool is_peer = rank != 0;
  volatile int* abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&bars->full[s]), 1); mbar_init(smem_u32(&bars->done[s]), 1); }
    for (int s = 0; s < 2; ++s) mbar_init(smem_u32(&bars->part_empty[s]), Geo<kPair>::kPartArrivals);
    for (int s = 0; s < kRing; ++s) {
      mbar_init(smem_u32(&bars->sched_full[s]), 1); mbar_init(smem_u32(&bars->sched_empty[s]), Geo<kPair>::kRingReaders);
      bars->sched_tile[s][0] = kTilePoison;
    }
    for (int s = 0; s < 4; ++s) mbar_init(smem_u32(&bars->amax_bar[s]), 2);
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x == 32) {
    int run = 0;
    for (int e = 0; e < n_experts; ++e) {          // tiles per expert: pairs of 128-row blocks, or single blocks
      pair_prefix[e] = run;
      const int mt = tile_prefix[e + 1] - tile_prefix[e];
      run += kPair ? (mt + 1) >> 1 : mt;
    }
    pair_prefix[n_experts] = run;
  }
  __syncthreads();
  if (warp == 1) {
    if (kPair) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                   ::"r"(smem_u32(&bars->tmem_base)), "r"(kTmemCols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                   ::"r"(smem_u32(&bars->tmem_base)), "r"(kTmemCols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (kPair) cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  const int total_tiles = pair_prefix[n_experts] * n_blocks_n;

  if (warp < kPromoWarp0) {
    setmaxnreg_dec();
    if (warp == 0 && lane == 0) {
      // ---------------------------------------------------------------- TMA producer (both CTAs)
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      Ring rd;
      for (; ok;) {
        const TileInfo tc = rd.next(bars, is_peer, abort_flag, status);
        rd.template done<kPair>(bars, true);
        if (tc.tile < 0) break;
        const int row0 = tc.poff + tc.m_block * kRowsPerTile + (int)rank * BM;
        const int n0 = tc.n_block * BN + (int)rank * (BN / 2);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(smem_u32(&bars->done[stage]), phase ^ 1u, abort_flag, status)) { ok = false; break; }
          if (kPair) {
            const uint32_t full = mapa(smem_u32(&bars->full[stage]), 0);
            if (rank == 0) mbar_expect_tx(smem_u32(&bars->full[stage]), 2 * (A_STAGE + B_STAGE));
            tma_load_2d_pair(smem_u32(smem_a + stage * A_STAGE), &tm_a, kb * BKB, row0, full);
            tma_load_3d_pair(smem_u32(smem_b + stage * B_STAGE), &tm_b, kb * BKB, n0, tc.expert, full);
          } else {
            const uint32_t full = smem_u32(&bars->full[stage]);
            mbar_expect_tx(full, A_STAGE + B_STAGE);
            tma_load_2d(smem_u32(smem_a + stage * A_STAGE), &tm_a, kb * BKB, row0, full);
            tma_load_3d(smem_u32(smem_b + stage * B_STAGE), &tm_b, kb * BKB, n0, tc.expert, full);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    } else if ((warp == 1 || warp == 3) && lane == 0 && !is_peer) {
      // ---------------------------------------------------------------- MMA issuers (leader CTA)
      // warp 1 owns scratch buffer 0 and the even K blocks (counted across tiles), warp 3 buffer 1 and the odd ones
      constexpr uint32_t idesc = make_idesc_e4m3(kRowsPerTile, BN);
      const int mine = warp == 1 ? 0 : 1;
      const uint32_t d_tmem = tmem_base + (uint32_t)(mine * BN);
      // This thread's K blocks sit two apart, across tile borders: `skip` is 1 when the next tile starts with the
      // other thread's block.  kStages is even, so the stage index keeps this thread's parity.
      int stage = mine; uint32_t phase = 0;
      uint32_t pb_phase = 0;
      int skip = mine;
      bool ok = true;
      Ring rd;
      for (; ok;) {
        const TileInfo tc = rd.next(bars, false, abort_flag, status);
        rd.template done<kPair>(bars, true);
        if (tc.tile < 0) break;
        int kb = skip;
        for (; kb < num_kb; kb += 2) {
          const uint64_t adesc = make_smem_desc(smem_u32(smem_a + stage * A_STAGE));
          const uint64_t bdesc = make_smem_desc(smem_u32(smem_b + stage * B_STAGE));
          // both tests are in flight together; the operands have normally landed long before the buffer is free
          const bool have_ops = mbar_try_wait(smem_u32(&bars->full[stage]), phase);
          const bool have_buf = mbar_try_wait(smem_u32(&bars->part_empty[mine]), pb_phase ^ 1u);
          if (!have_ops && !mbar_wait(smem_u32(&bars->full[stage]), phase, abort_flag, status)) { ok = false; break; }
          if (!have_buf && !mbar_wait(smem_u32(&bars->part_empty[mine]), pb_phase ^ 1u, abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          issue_k_block<kPair>(d_tmem, adesc, bdesc, idesc);
          if (kPair) tc_commit_pair_both(smem_u32(&bars->done[stage]), 3);
          else tc_commit(smem_u32(&bars->done[stage]));
          pb_phase ^= 1u;
          stage += 2;
          if (stage >= kStages) { stage -= kStages; phase ^= 1u; }
        }
        skip = kb - num_kb;                              // 0 or 1
      }
    } else if (warp == 2 && lane == 0 && !is_peer) {
      // ---------------------------------------------------------------- tile scheduler (leader CTA)
      int slot = 0; uint32_t phase = 0;
      for (;;) {
        if (!mbar_wait(smem_u32(&bars->sched_empty[slot]), phase ^ 1u, abort_flag, status)) break;
        int t = atomicAdd(tile_counter, 1);
        if (t >= total_tiles) t = -1;
        int f[6] = {t, 0, 0, 0, 0, 0};
        TileCoord tc;
        if (t >= 0 && decode_tile(pair_prefix, n_experts, n_blocks_n, n_group, t, &tc)) {
          f[1] = tc.expert; f[2] = tc.m_block; f[3] = tc.n_block;
          f[4] = counts[tc.expert]; f[5] = padded_offsets[tc.expert];
        } else {
          f[0] = t = -1;
        }
#pragma unroll
        for (int i = 5; i >= 0; --i) {                   // the tile id, which readers test for poison, goes last
          bars->sched_tile[slot][i] = f[i];
          if (kPair) st_shared_cluster_u32(mapa(smem_u32(&bars->sched_tile[slot][i]), 1), (uint32_t)f[i]);
        }
        mbar_arrive(smem_u32(&bars->sched_full[slot]));
        if (kPair) mbar_arrive_release_cluster(mapa(smem_u32(&bars->sched_full[slot]), 1));
        if (t < 0) break;
        if (++slot == kRing) { slot = 0; phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------ promotion + epilogue warps
    setmaxnreg_inc();
    const int pw = warp - kPromoWarp0;                 // 0..7
    const int lane_grp = warp & 3;                     // tensor-memory lanes 32*lane_grp..+31
    const int half = pw >> 2;                          // which 2x64 columns of the tile
    uint8_t* my_store = s_store + pw * kStoreStage;
    // column groups: swiglu tile = [128 gate | 128 up] -> this thread owns gate cols 64*half..+63 and the
    // matching up cols; plain tile -> cols 128*half..+127 (two groups of 64 under one weight-scale block)
    const int col0 = kSwiglu ? 64 * half : 128 * half;
    const int col1 = kSwiglu ? 128 + 64 * half : 128 * half + 64;
    int stage = 0; uint32_t phase = 0;                 // K blocks are consumed in order; buffer = stage parity
    const uint32_t t_lane = tmem_base + ((uint32_t)(lane_grp * 32) << 16);
    // where the "buffer read out" arrivals go: the leader CTA's barriers
    const uint32_t part_empty0 = kPair ? mapa(smem_u32(&bars->part_empty[0]), 0) : smem_u32(&bars->part_empty[0]);
    const uint32_t part_empty1 = kPair ? mapa(smem_u32(&bars->part_empty[1]), 0) : smem_u32(&bars->part_empty[1]);
    uint32_t tile_parity = 0;
    Ring rd;
    unsigned long long acc2[64];                       // 128 fp32 accumulators as packed pairs
    for (;;) {
      const TileInfo tc = rd.next(bars, is_peer, abort_flag, status);
      __syncwarp();
      rd.template done<kPair>(bars, lane == 0);
      if (tc.tile < 0) break;
      const int r_warp = tc.m_block * kRowsPerTile + (int)rank * BM + lane_grp * 32;   // first row of this warp in the group
      const int r_in_group = r_warp + lane;
      const bool row_ok = r_in_group < tc.count;
      const size_t grow = (size_t)(tc.poff + r_in_group);
      const float* sa_row = a_scales + grow * num_kb;
      const int nb0 = 2 * tc.n_block + (kSwiglu ? 0 : half), nb1 = kSwiglu ? nb0 + 1 : nb0;
      const float* sw0_p = b_scales + ((size_t)tc.expert * (2 * n_blocks_n) + nb0) * num_kb;
      const float* sw1_p = b_scales + ((size_t)tc.expert * (2 * n_blocks_n) + nb1) * num_kb;
#pragma unroll
      for (int i = 0; i < 64; ++i) acc2[i] = 0ull;
      bool ok = true;
      // Promotion of one K block.  How long a scratch buffer stays with these warps is on the critical loop
      // MMA -> promotion -> MMA, so nothing but the reads themselves sits between "the block's MMAs have completed"
      // and "buffer handed back": this thread's 128 values are read in two 64-column loads, and only the first
      // half's multiply-adds (which free the staging registers for the second load) run in between.
#define CEP_FMA_HALF(BASE, S)                                                                       \
  {                                                                                                  \
    const unsigned long long s2_ = pack_f32x2(__float_as_uint(S), __float_as_uint(S));              \
    _Pragma("unroll") for (int i = 0; i < 32; ++i)                                                  \
        fma_f32x2(acc2[(BASE) + i], pack_f32x2(v[2 * i], v[2 * i + 1]), s2_);                      \
  }
      uint32_t v[64];
      // the scales of K block kb+1 are fetched while block kb is promoted: their L2 latency would otherwise sit
      // in front of every block's first multiply-add
      float sa_n = row_ok ? __ldg(sa_row) : 0.f, sw0_n = __ldg(sw0_p), sw1_n = __ldg(sw1_p);
      bool ready = false;                                // outcome of the early test of this K block's barrier
      for (int kb = 0; kb < num_kb; ++kb) {
        if (!__all_sync(0xffffffffu, ready)) {
          const bool got = mbar_wait(smem_u32(&bars->done[stage]), phase, abort_flag, status);
          if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
        }
        tc_fence_after();
        const int pb = stage & 1;
        const uint32_t t_addr = t_lane + (uint32_t)(pb * BN);
        tc_ld64(t_addr + (uint32_t)col0, v);
        const float s0 = sa_n * sw0_n, s1 = sa_n * sw1_n;
        const bool more = kb + 1 < num_kb;
        if (more) {
          sa_n = row_ok ? __ldg(sa_row + kb + 1) : 0.f;
          sw0_n = __ldg(sw0_p + kb + 1);
          sw1_n = __ldg(sw1_p + kb + 1);
        }
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
        tc_wait_ld();
        CEP_FMA_HALF(0, s0);
        tc_ld64(t_addr + (uint32_t)col1, v);
        tc_wait_ld();
        // every column of this scratch buffer is in registers: give it back
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (kPair) mbar_arrive_cluster(pb ? part_empty1 : part_empty0);
          else mbar_arrive(pb ? part_empty1 : part_empty0);
        }
        // the next K block's barrier is tested now: the test's latency hides behind the second half's arithmetic
        ready = more ? mbar_try_wait(smem_u32(&bars->done[stage]), phase) : false;
        CEP_FMA_HALF(32, s1);
      }
#undef CEP_FMA_HALF
      if (!ok) break;
      // ---------------------------------------------------------------- epilogue from registers
      float acc[128];
#pragma unroll
      for (int i = 0; i < 64; ++i) unpack_f32x2(acc2[i], acc[2 * i], acc[2 * i + 1]);
      if (kSwiglu) {
        // acc[0..63] = gate cols, acc[64..127] = up cols -> 64 activations of this row
        float amax = 0.f;
#pragma unroll
        for (int i = 0; i < 64; ++i) {
          acc[i] = silu_mul(acc[i], acc[64 + i]);
          amax = fmaxf(amax, fabsf(acc[i]));
        }
        // the row's other 64 columns belong to the partner warp of this lane group: exchange the amax
        // through shared memory (double-buffered by tile parity) and a two-arrival barrier, bounded wait
        const int r_tile = lane_grp * 32 + lane;
        float* mine = s_amax + (tile_parity * 2 + half) * BM + r_tile;
        const float* theirs = s_amax + (tile_parity * 2 + (half ^ 1)) * BM + r_tile;
        *mine = amax;
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->amax_bar[lane_grp]));
        const bool got_amax = mbar_wait(smem_u32(&bars->amax_bar[lane_grp]), tile_parity, abort_flag, status);
        if (!__all_sync(0xffffffffu, got_amax)) break;
        amax = fmaxf(amax, *theirs);
        tile_parity ^= 1u;
        const float scale = amax == 0.f ? 1.f : __fdiv_rn(amax, 448.f);
        const float inv = __fdiv_rn(1.f, scale);         // one division per row; the 64 quotients become products
        // 64 codes per row: through the warp's staging buffer, so that a store instruction covers 64 contiguous
        // bytes of 8 rows instead of 16 bytes of 32 rows
        uint4 ch[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t w[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int i = q * 16 + j * 4;
            const uint32_t lo = cvt_e4m3x2(acc[i] * inv, acc[i + 1] * inv);
            const uint32_t hi = cvt_e4m3x2(acc[i + 2] * inv, acc[i + 3] * inv);
            w[j] = lo | (hi << 16);
          }
          ch[q] = make_uint4(w[0], w[1], w[2], w[3]);
        }
        if (lane == 0) tma_store_wait_read();            // the previous tile's box has left the staging buffer
        __syncwarp();
        if (r_warp < tc.count) {
          stage_rows_64B(my_store, lane, ch);
          if (lane == 0) tma_store_box(&tm_out, my_store, tc.n_block * 128 + 64 * half, tc.poff + r_warp);
        }
        if (half == 0 && row_ok) out_scales[grow * (n_out_cols / 128) + tc.n_block] = scale;
      } else {
        // 128 bf16 per row, 32 columns (64 bytes) per pass through the staging buffer
#pragma unroll
        for (int pass = 0; pass < 4; ++pass) {
          uint4 ch[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int i = 32 * pass + 8 * q;
            ch[q].x = pack_bf16(acc[i + 0], acc[i + 1]);
            ch[q].y = pack_bf16(acc[i + 2], acc[i + 3]);
            ch[q].z = pack_bf16(acc[i + 4], acc[i + 5]);
            ch[q].w = pack_bf16(acc[i + 6], acc[i + 7]);
          }
          if (lane == 0) tma_store_wait_read();          // the previous box has left the staging buffer
          __syncwarp();
          if (r_warp < tc.count) {
            stage_rows_64B(my_store, lane, ch);
            if (lane == 0) tma_store_box(&tm_out, my_store, tc.n_block * BN + 128 * half + 32 * pass, tc.poff + r_warp);
          }
        }
      }
    }
    if (lane == 0) tma_store_wait_all();                 // this warp's boxes have reached global memory
  }
  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (kPair) cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    if (kPair) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------- weight-scale prepack
// s13p[e][2*ib + (0 gate | 1 up)][kb] <- s_gate/s_up[e][kb][ib];   s2p[e][hb][kb] <- s_down[e][kb][hb]
__global__ void pack_scales_kernel(const float* __restrict__ s_gate, const float* __restrict__ s_up,
                                   const float* __restrict__ s_down, float* __restrict__ s13p, float* __restrict__ s2p,
                                   int E, int HB, int IB) {
  const size_t n13 = (size_t)E * 2 * IB * HB, n2 = (size_t)E * HB * IB;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n13 + n2; i += (size_t)gridDim.x * blockDim.x) {
    if (i < n13) {
      const int kb = (int)(i % HB); const size_t r = i / HB; const int nb = (int)(r % (2 * IB)); const int e = (int)(r / (2 * IB));
      const float* src = (nb & 1) ? s_up : s_gate;
      s13p[i] = src[((size_t)e * HB + kb) * IB + (nb >> 1)];
    } else {
      const size_t j = i - n13;
      const int kb = (int)(j % IB); const size_t r = j / IB; const int hb = (int)(r % HB); const int e = (int)(r / HB);
      s2p[j] = s_down[((size_t)e * IB + kb) * HB + hb];
    }
  }
}

// cudaFuncSetAttribute and the occupancy answer hold per device: one slot per device ordinal
constexpr int kMaxDevices = 64;
int g_clusters[kMaxDevices];                           // co-resident CTA pairs + 1 (0: not set up yet)
bool g_single_ready[kMaxDevices];

template <bool kPair>
cudaError_t set_smem_attr() {
  cudaError_t e = cudaFuncSetAttribute(grouped_gemm_fp8_kernel<true, kPair>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       Geo<kPair>::kSmemBytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(grouped_gemm_fp8_kernel<false, kPair>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Geo<kPair>::kSmemBytes);
}

cudaError_t setup_pair(int dev, int n_sms) {
  if (g_clusters[dev] > 0) return cudaSuccess;
  cudaError_t e = set_smem_attr<true>();
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3(n_sms & ~1, 1, 1); cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = Geo<true>::kSmemBytes; cfg.attrs = attr; cfg.numAttrs = 1;
  int n = 0;
  e = cudaOccupancyMaxActiveClusters(&n, grouped_gemm_fp8_kernel<true, true>, &cfg);
  if (e != cudaSuccess) return e;
  g_clusters[dev] = n + 1;
  return cudaSuccess;
}

}  // namespace

int gemm_fp8_box_rows(int pair) { return pair ? BN / 2 : BN; }

cudaError_t launch_pack_scales(const cep_config& cfg, const float* s_gate, const float* s_up, const float* s_down,
                               float* s13p, float* s2p, cudaStream_t s, int64_t* launches) {
  pack_scales_kernel<<<256, 256, 0, s>>>(s_gate, s_up, s_down, s13p, s2p, cfg.n_experts_local, cfg.hidden / kQuantBlock,
                                         cfg.inter / kQuantBlock);
  *launches += 1;
  return cudaGetLastError();
}

template <bool kSwiglu, bool kPair>
static cudaError_t launch_one(cudaLaunchConfig_t* cfg, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& o, int num_kb, int n_blocks_n,
                              int n_group, int n_experts, int n_out_cols, const float* a_scales,
                              const float* b_scales, float* out_scales, const LayoutPtrs& lp, int32_t* counter) {
  return cudaLaunchKernelEx(cfg, grouped_gemm_fp8_kernel<kSwiglu, kPair>, a, b, o, num_kb, n_blocks_n, n_group, n_experts,
                            n_out_cols, a_scales, b_scales, kSwiglu ? out_scales : (float*)nullptr,
                            (const int32_t*)lp.tile_prefix, (const int32_t*)lp.counts, (const int32_t*)lp.padded_offsets,
                            counter, lp.status);
}

// pair != 0: CTA pairs on 256x256 tiles, max_tiles counts pair tiles; pair == 0: one CTA per 128x256 tile,
// max_tiles counts single tiles.  The weight operand map must have a box of gemm_fp8_box_rows(pair) rows.
cudaError_t launch_gemm_fp8(const GemmProblem& p, int pair, const GemmTensorMap& tm_a, const GemmTensorMap& tm_b,
                            const GemmTensorMap& tm_out, const float* a_scales, const float* b_scales, void* out, float* out_scales,
                            const LayoutPtrs& lp, int max_tiles, int n_sms, cudaStream_t s, int64_t* launches) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  int ctas;
  if (pair) {
    e = setup_pair(dev, n_sms);
    if (e != cudaSuccess) return e;
    const int clusters = g_clusters[dev] - 1;
    if (clusters < 1) return cudaErrorNotSupported;
    ctas = 2 * (max_tiles < clusters ? max_tiles : clusters);
  } else {
    if (!g_single_ready[dev]) {
      e = set_smem_attr<false>();
      if (e != cudaSuccess) return e;
      g_single_ready[dev] = true;
    }
    ctas = max_tiles < n_sms ? max_tiles : n_sms;
  }
  if (ctas < 1) return cudaSuccess;
  const int n_blocks_n = (p.N + BN - 1) / BN;
  const int n_out_cols = p.swiglu ? p.N / 2 : p.N;
  const int num_kb = p.K / BKB;
  const int n_group = n_group_for(n_blocks_n, BN, p.K, 1);
  int32_t* counter = lp.sched + (p.swiglu ? 0 : 1);
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = pair ? 2 : 1; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = dim3(ctas, 1, 1); cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = pair ? Geo<true>::kSmemBytes : Geo<false>::kSmemBytes;
  cfg.stream = s; cfg.attrs = attr; cfg.numAttrs = 2;
  const CUtensorMap& a = reinterpret_cast<const CUtensorMap&>(tm_a);
  const CUtensorMap& b = reinterpret_cast<const CUtensorMap&>(tm_b);
  const CUtensorMap& o = reinterpret_cast<const CUtensorMap&>(tm_out);
#define CEP_FP8_LAUNCH(SW, PR) launch_one<SW, PR>(&cfg, a, b, o, num_kb, n_blocks_n, n_group, p.n_experts, n_out_cols, \
                                                  a_scales, b_scales, out_scales, lp, counter)
  (void)out;                                             // the output tensor is reached through tm_out
  if (p.swiglu) e = pair ? CEP_FP8_LAUNCH(true, true) : CEP_FP8_LAUNCH(true, false);
  else e = pair ? CEP_FP8_LAUNCH(false, true) : CEP_FP8_LAUNCH(false, false);
#undef CEP_FP8_LAUNCH
  *launches += 1;
  return e;
}

}  // namespace cep
