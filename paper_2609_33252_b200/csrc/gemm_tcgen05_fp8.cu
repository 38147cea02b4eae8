// Grouped expert GEMM for block-scaled e4m3 operands (fp32 scales per 1x128 activation block and per
// 128x128 weight block), CTA pairs on 256x256 tiles:
//
//   D[m, n] = sum over 128-deep K blocks kb of  sa[m, kb] * sw[kb, n/128] * ( A_codes[m, kb] . B_codes[n, kb] )
//
// The scales are plain fp32, so they cannot ride on the tensor core's own (power-of-two, 1x32) block
// scaling.  Each K block is therefore multiplied on its own into a scratch accumulator in tensor memory
// (tcgen05.mma kind::f8f6f4, fp32 accumulate, two scratch buffers in flight), and eight "promotion"
// warps pull every partial product out of tensor memory and add it, scaled, into fp32 accumulators
// they hold in registers (128 per thread).  The same warps then run the epilogue:
//   GEMM1: SiLU(gate)*up, per-row amax over the tile's 128 columns, scale = amax/448, e4m3 codes
//          (round-to-nearest-even, saturating) + the scale: the "activation and quantization" step
//          between the two expert GEMMs (Appendix "Grouped FFN invocations")
//   GEMM2: bf16
// Roles (384 threads): warp 0 TMA producer, warp 1 MMA issuer (leader CTA), warp 2 tile scheduler
// (leader CTA), warps 4-11 promotion + epilogue.  Tiles come from a global counter, as in the bf16
// kernel.  All waits are bounded.
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
template <bool kPair> struct Geo {
  static constexpr int kStages = kPair ? 6 : 4;
  static constexpr int B_STAGE = (kPair ? BN / 2 : BN) * BKB;
  static constexpr int kRingReaders = kPair ? 19 : 10;    // producer, MMA, 8 promotion warps (+ peer: producer, 8)
  static constexpr int kPartArrivals = kPair ? 16 : 8;
  static constexpr int kSmemBytes = kStages * (A_STAGE + B_STAGE) + 256 + (1024 + 1) * 4 + 2 * 2 * BM * 4 + 1024;
};
constexpr int kMaxStages = 6;
constexpr int kThreads = 384;
constexpr int kPromoWarp0 = 4, kPromoWarps = 8;
constexpr int kTmemCols = 512;
constexpr int kMaxExperts = 1024;
constexpr int kRing = 4;
constexpr int kTilePoison = -2;

struct __align__(8) Bars {
  uint64_t full[kMaxStages], empty[kMaxStages];
  uint64_t part_full[2], part_empty[2];               // scratch accumulators in tensor memory
  uint64_t sched_full[kRing], sched_empty[kRing];
  uint64_t amax_bar[4];                               // per lane group: the two warps sharing its rows
  int32_t sched_tile[kRing];
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(Bars) <= 256, "barrier block");

struct Ring {
  int slot = 0; uint32_t phase = 0;
  __device__ __forceinline__ int next(Bars* b, bool is_peer, volatile int* abort_flag, int32_t* status) {
    const uint32_t bar = smem_u32(&b->sched_full[slot]);
    const bool ok = is_peer ? mbar_wait_acq_cluster(bar, phase, abort_flag, status) : mbar_wait(bar, phase, abort_flag, status);
    if (!ok) return -1;
    const int t = b->sched_tile[slot];
    if (t < -1) { atomicExch(&status[kStDetail], 0x5C4ED); atomicExch(&status[kStTimeout], 1); *abort_flag = 1; return -1; }
    return t;
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

__device__ __forceinline__ void tc_mma_f8_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n}"
               ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_mma_f8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n}"
               ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
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

template <bool kSwiglu, bool kPair>
__global__ void __launch_bounds__(kThreads, 1)
grouped_gemm_fp8_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                             int num_kb, int n_blocks_n, int n_group, int n_experts, int n_out_cols, int out_ld,
                             const float* __restrict__ a_scales /*[rows, num_kb]*/,
                             const float* __restrict__ b_scales /*[E, N/128, num_kb]*/,
                             uint8_t* __restrict__ out_codes, float* __restrict__ out_scales /*[rows, out cols/128]*/,
                             __nv_bfloat16* __restrict__ out_bf16,
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
  int32_t* pair_prefix = reinterpret_cast<int32_t*>(smem + kStages * (A_STAGE + B_STAGE) + 256);
  float* s_amax = reinterpret_cast<float*>(pair_prefix + kMaxExperts + 1);           // [tile parity][half][128]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = kPair ? cluster_ctarank() : 0u;
  const bool is_peer = rank != 0;
  volatile int* abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&bars->full[s]), 1); mbar_init(smem_u32(&bars->empty[s]), 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&bars->part_full[s]), 1); mbar_init(smem_u32(&bars->part_empty[s]), Geo<kPair>::kPartArrivals); }
    for (int s = 0; s < kRing; ++s) {
      mbar_init(smem_u32(&bars->sched_full[s]), 1); mbar_init(smem_u32(&bars->sched_empty[s]), Geo<kPair>::kRingReaders);
      bars->sched_tile[s] = kTilePoison;
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
        const int tile = rd.next(bars, is_peer, abort_flag, status);
        rd.template done<kPair>(bars, true);
        if (tile < 0) break;
        TileCoord tc;
        if (!decode_tile(pair_prefix, n_experts, n_blocks_n, n_group, tile, &tc)) break;
        const int row0 = padded_offsets[tc.expert] + tc.m_block * kRowsPerTile + (int)rank * BM;
        const int n0 = tc.n_block * BN + (int)rank * (BN / 2);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag, status)) { ok = false; break; }
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
    } else if (warp == 1 && lane == 0 && !is_peer) {
      // ---------------------------------------------------------------- MMA issuer (leader CTA)
      constexpr uint32_t idesc = make_idesc_e4m3(kRowsPerTile, BN);
      int stage = 0; uint32_t phase = 0;
      int pb = 0; uint32_t pb_phase = 0;
      bool ok = true;
      Ring rd;
      for (; ok;) {
        const int tile = rd.next(bars, false, abort_flag, status);
        rd.template done<kPair>(bars, true);
        if (tile < 0) break;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(smem_u32(&bars->part_empty[pb]), pb_phase ^ 1u, abort_flag, status)) { ok = false; break; }
          if (!mbar_wait(smem_u32(&bars->full[stage]), phase, abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(pb * BN);
          const uint64_t adesc = make_smem_desc(smem_u32(smem_a + stage * A_STAGE));
          const uint64_t bdesc = make_smem_desc(smem_u32(smem_b + stage * B_STAGE));
#pragma unroll
          for (int k4 = 0; k4 < BKB / 32; ++k4) {        // 32 e4m3 elements of K per MMA
            if (kPair) tc_mma_f8_pair(d_tmem, adesc + (uint64_t)(k4 * 2), bdesc + (uint64_t)(k4 * 2), idesc, k4 != 0 ? 1u : 0u);
            else tc_mma_f8(d_tmem, adesc + (uint64_t)(k4 * 2), bdesc + (uint64_t)(k4 * 2), idesc, k4 != 0 ? 1u : 0u);
          }
          if (kPair) {
            tc_commit_pair_both(smem_u32(&bars->empty[stage]), 3);
            tc_commit_pair_both(smem_u32(&bars->part_full[pb]), 3);
          } else {
            tc_commit(smem_u32(&bars->empty[stage]));
            tc_commit(smem_u32(&bars->part_full[pb]));
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
          if (++pb == 2) { pb = 0; pb_phase ^= 1u; }
        }
      }
    } else if (warp == 2 && lane == 0 && !is_peer) {
      // ---------------------------------------------------------------- tile scheduler (leader CTA)
      int slot = 0; uint32_t phase = 0;
      for (;;) {
        if (!mbar_wait(smem_u32(&bars->sched_empty[slot]), phase ^ 1u, abort_flag, status)) break;
        int t = atomicAdd(tile_counter, 1);
        if (t >= total_tiles) t = -1;
        bars->sched_tile[slot] = t;
        if (kPair) st_shared_cluster_u32(mapa(smem_u32(&bars->sched_tile[slot]), 1), (uint32_t)t);
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
    // column groups: swiglu tile = [128 gate | 128 up] -> this thread owns gate cols 64*half..+63 and the
    // matching up cols; plain tile -> cols 128*half..+127 (two groups of 64 under one weight-scale block)
    const int col0 = kSwiglu ? 64 * half : 128 * half;
    const int col1 = kSwiglu ? 128 + 64 * half : 128 * half + 64;
    int pb = 0; uint32_t pb_phase = 0;
    uint32_t tile_parity = 0;
    Ring rd;
    unsigned long long acc2[64];                       // 128 fp32 accumulators as packed pairs
    for (;;) {
      const int tile = rd.next(bars, is_peer, abort_flag, status);
      __syncwarp();
      rd.template done<kPair>(bars, lane == 0);
      if (tile < 0) break;
      TileCoord tc;
      if (!decode_tile(pair_prefix, n_experts, n_blocks_n, n_group, tile, &tc)) break;
      const int r_in_group = tc.m_block * kRowsPerTile + (int)rank * BM + lane_grp * 32 + lane;
      const bool row_ok = r_in_group < counts[tc.expert];
      const size_t grow = (size_t)(padded_offsets[tc.expert] + r_in_group);
      const float* sa_row = a_scales + grow * num_kb;
      const int nb0 = 2 * tc.n_block + (kSwiglu ? 0 : half), nb1 = kSwiglu ? nb0 + 1 : nb0;
      const float* sw0_p = b_scales + ((size_t)tc.expert * (2 * n_blocks_n) + nb0) * num_kb;
      const float* sw1_p = b_scales + ((size_t)tc.expert * (2 * n_blocks_n) + nb1) * num_kb;
#pragma unroll
      for (int i = 0; i < 64; ++i) acc2[i] = 0ull;
      bool ok = true;
      // Software-pipelined promotion: the partial tile is read in four 32-column chunks per K block; the
      // load of chunk i+1 is in flight while chunk i is multiplied and added, across K-block borders, and
      // the scratch buffer is handed back to the MMA warp as soon as its last chunk has been read.
#define CEP_FMA_CHUNK(V, BASE, S)                                                                   \
  {                                                                                                  \
    const unsigned long long s2_ = pack_f32x2(__float_as_uint(S), __float_as_uint(S));              \
    _Pragma("unroll") for (int i = 0; i < 16; ++i)                                                  \
        fma_f32x2(acc2[(BASE) + i], pack_f32x2((V)[2 * i], (V)[2 * i + 1]), s2_);                  \
  }
      uint32_t va[32], vb[32];
      {
        const bool got = mbar_wait(smem_u32(&bars->part_full[pb]), pb_phase, abort_flag, status);
        if (!__all_sync(0xffffffffu, got)) break;
        tc_fence_after();
        tc_ld32(tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(pb * BN + col0), va);
        tc_wait_ld();
      }
      // the scales of K block kb+1 are fetched while block kb is promoted: their L2 latency would otherwise sit
      // in front of every block's first multiply-add
      float sa_n = row_ok ? __ldg(sa_row) : 0.f, sw0_n = __ldg(sw0_p), sw1_n = __ldg(sw1_p);
      for (int kb = 0; kb < num_kb; ++kb) {
        const float s0 = sa_n * sw0_n, s1 = sa_n * sw1_n;
        if (kb + 1 < num_kb) {
          sa_n = row_ok ? __ldg(sa_row + kb + 1) : 0.f;
          sw0_n = __ldg(sw0_p + kb + 1);
          sw1_n = __ldg(sw1_p + kb + 1);
        }
        const uint32_t t_addr = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(pb * BN);
        tc_ld32(t_addr + (uint32_t)(col0 + 32), vb);
        CEP_FMA_CHUNK(va, 0, s0);
        tc_wait_ld();
        tc_ld32(t_addr + (uint32_t)col1, va);
        CEP_FMA_CHUNK(vb, 16, s0);
        tc_wait_ld();
        tc_ld32(t_addr + (uint32_t)(col1 + 32), vb);
        CEP_FMA_CHUNK(va, 32, s1);
        tc_wait_ld();
        // every column of this scratch buffer is in registers: give it back
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (kPair) mbar_arrive_cluster(mapa(smem_u32(&bars->part_empty[pb]), 0));
          else mbar_arrive(smem_u32(&bars->part_empty[pb]));
        }
        if (++pb == 2) { pb = 0; pb_phase ^= 1u; }
        if (kb + 1 < num_kb) {
          const bool got = mbar_wait(smem_u32(&bars->part_full[pb]), pb_phase, abort_flag, status);
          if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
          tc_fence_after();
          tc_ld32(tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(pb * BN + col0), va);
          CEP_FMA_CHUNK(vb, 48, s1);
          tc_wait_ld();
        } else {
          CEP_FMA_CHUNK(vb, 48, s1);
        }
      }
#undef CEP_FMA_CHUNK
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
        if (row_ok) {
          uint4* dst = reinterpret_cast<uint4*>(out_codes + grow * out_ld + tc.n_block * 128 + 64 * half);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int i = q * 16 + j * 4;
              const uint32_t lo = cvt_e4m3x2(__fdiv_rn(acc[i], scale), __fdiv_rn(acc[i + 1], scale));
              const uint32_t hi = cvt_e4m3x2(__fdiv_rn(acc[i + 2], scale), __fdiv_rn(acc[i + 3], scale));
              w[j] = lo | (hi << 16);
            }
            dst[q] = make_uint4(w[0], w[1], w[2], w[3]);
          }
          if (half == 0) out_scales[grow * (n_out_cols / 128) + tc.n_block] = scale;
        }
      } else {
        if (row_ok) {
          const int c_out = tc.n_block * BN + 128 * half;
          if (c_out < n_out_cols) {
            uint4* dst = reinterpret_cast<uint4*>(out_bf16 + grow * out_ld + c_out);
#pragma unroll
            for (int q = 0; q < 16; ++q) {
              uint4 v;
              v.x = pack_bf16(acc[8 * q + 0], acc[8 * q + 1]);
              v.y = pack_bf16(acc[8 * q + 2], acc[8 * q + 3]);
              v.z = pack_bf16(acc[8 * q + 4], acc[8 * q + 5]);
              v.w = pack_bf16(acc[8 * q + 6], acc[8 * q + 7]);
              dst[q] = v;
            }
          }
        }
      }
    }
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

int g_clusters = -1;
bool g_single_ready = false;

template <bool kPair>
cudaError_t set_smem_attr() {
  cudaError_t e = cudaFuncSetAttribute(grouped_gemm_fp8_kernel<true, kPair>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       Geo<kPair>::kSmemBytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(grouped_gemm_fp8_kernel<false, kPair>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Geo<kPair>::kSmemBytes);
}

cudaError_t setup_pair(int n_sms) {
  if (g_clusters >= 0) return cudaSuccess;
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
  g_clusters = n;
  return cudaSuccess;
}

}  // namespace

cudaError_t launch_pack_scales(const cep_config& cfg, const float* s_gate, const float* s_up, const float* s_down,
                               float* s13p, float* s2p, cudaStream_t s, int64_t* launches) {
  pack_scales_kernel<<<256, 256, 0, s>>>(s_gate, s_up, s_down, s13p, s2p, cfg.n_experts_local, cfg.hidden / kQuantBlock,
                                         cfg.inter / kQuantBlock);
  *launches += 1;
  return cudaGetLastError();
}

template <bool kSwiglu, bool kPair>
static cudaError_t launch_one(cudaLaunchConfig_t* cfg, const CUtensorMap& a, const CUtensorMap& b, int num_kb, int n_blocks_n,
                              int n_group, int n_experts, int n_out_cols, int out_ld, const float* a_scales,
                              const float* b_scales, void* out, float* out_scales, const LayoutPtrs& lp, int32_t* counter) {
  return cudaLaunchKernelEx(cfg, grouped_gemm_fp8_kernel<kSwiglu, kPair>, a, b, num_kb, n_blocks_n, n_group, n_experts,
                            n_out_cols, out_ld, a_scales, b_scales, kSwiglu ? (uint8_t*)out : (uint8_t*)nullptr,
                            kSwiglu ? out_scales : (float*)nullptr, kSwiglu ? (__nv_bfloat16*)nullptr : (__nv_bfloat16*)out,
                            (const int32_t*)lp.tile_prefix, (const int32_t*)lp.counts, (const int32_t*)lp.padded_offsets,
                            counter, lp.status);
}

// pair != 0: CTA pairs on 256x256 tiles (the weight operand map must have a 128-row box, max_tiles counts pair
// tiles); pair == 0: one CTA per 128x256 tile (256-row box, max_tiles counts single tiles).
cudaError_t launch_gemm_fp8(const GemmProblem& p, int pair, const GemmTensorMap& tm_a, const GemmTensorMap& tm_b,
                            const float* a_scales, const float* b_scales, void* out, float* out_scales,
                            const LayoutPtrs& lp, int max_tiles, int n_sms, cudaStream_t s, int64_t* launches) {
  cudaError_t e;
  int ctas;
  if (pair) {
    e = setup_pair(n_sms);
    if (e != cudaSuccess) return e;
    if (g_clusters < 1) return cudaErrorNotSupported;
    ctas = 2 * (max_tiles < g_clusters ? max_tiles : g_clusters);
  } else {
    if (!g_single_ready) {
      e = set_smem_attr<false>();
      if (e != cudaSuccess) return e;
      g_single_ready = true;
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
#define CEP_FP8_LAUNCH(SW, PR) launch_one<SW, PR>(&cfg, a, b, num_kb, n_blocks_n, n_group, p.n_experts, n_out_cols, p.out_ld, \
                                                  a_scales, b_scales, out, out_scales, lp, counter)
  if (p.swiglu) e = pair ? CEP_FP8_LAUNCH(true, true) : CEP_FP8_LAUNCH(true, false);
  else e = pair ? CEP_FP8_LAUNCH(false, true) : CEP_FP8_LAUNCH(false, false);
#undef CEP_FP8_LAUNCH
  *launches += 1;
  return e;
}

}  // namespace cep
