// Grouped expert GEMM for microscaling operands: e4m3 activations x e2m1 (MXFP4) weights, one ue8m0
// (power-of-two) scale per 32 elements of K on both sides, fp32 accumulate.  CTA pairs on 256x256 tiles.
//
//   D[m, n] = sum over 32-deep K blocks kb of  2^(sa[m,kb]-127) * 2^(sb[n,kb]-127) * ( A_codes[m,kb] . B_codes[n,kb] )
//
// The scaling is done by the tensor core itself (tcgen05.mma kind::mxf8f6f4.block_scale): the scale bytes of a
// stage are copied from shared memory into tensor memory (tcgen05.cp 32x128b.warpx4) right before the stage's
// four K=32 MMAs, so the whole K loop accumulates into one 256-column fp32 accumulator in tensor memory.  The
// weights stay packed (two codes per byte) in HBM; the TMA load expands every 16 codes into a 16-byte slot of
// shared memory (tensor-map type 16U4_ALIGN16B), which is the operand form the f8f6f4 kinds read.
//
// Tensor memory (512 columns): accumulator 0..255 (one stage: the epilogue warps pull a finished tile into
// registers, 128 values per thread, and hand the columns back before they do any arithmetic), scale factors
// from column 256 (a ring of 4 slots: 4 columns for this CTA's 128 rows, 8 for the tile's 256 weight rows).
//
// Epilogues:
//   GEMM1  SiLU(gate)*up, then the "activation and quantization" step between the two expert GEMMs
//          (Appendix "Grouped FFN invocations"): per row and 32 columns, scale = smallest power of two with
//          amax <= 448*scale, e4m3 codes round-to-nearest-even; codes row-major, scale bytes in atom order
//   GEMM2  bf16
// Roles (384 threads): warp 0 TMA producer (both CTAs), warp 1 MMA issuer (leader CTA), warp 2 tile scheduler
// (leader CTA), warps 4-11 epilogue.  Tiles come from a global counter.  All waits are bounded.
//
// Where the time goes (device-timer trace and profiler counters on the 7168x2048 shapes): a K=128 slab costs
// about 470 cycles of MMA, 115 cycles for its three scale copies (they run in the same in-order pipe as the MMAs;
// issuing them a slab ahead or leaving them out confirms it: 2640 TFLOP/s without copies, the same as an unscaled
// kind::f8f6f4 loop), and the rest is the issue thread's barrier round trip per group of slabs.  The tile-end
// bubble is small: the finished accumulator is in registers 160 cycles after the epilogue warps see it.
#include <cuda.h>
#include <cuda_bf16.h>

#include "cep_common.h"
#include "gemm_tcgen05.h"
#include "tcgen05_ptx.cuh"

namespace cep {
namespace {

using namespace ptx;

constexpr int BM = 128, BN = 256, BKE = 128;           // BKE elements of K per stage = 4 scale blocks
constexpr int A_STAGE = BM * BKE;                      // e4m3: 16 KiB
constexpr int B_STAGE = (BN / 2) * BKE;                // this CTA's half of the weight tile, 16 codes per 16-byte slot
constexpr int B_TX = (BN / 2) * BKE / 2;               // bytes the TMA engine counts for it (packed codes)
constexpr int SFA_STAGE = kSfAtomBytes;                // 128 rows x 4 scale blocks
constexpr int SFB_STAGE = 2 * kSfAtomBytes;            // 256 weight rows x 4 scale blocks
constexpr int kStages = 6;                             // K=128 slabs of operands in shared memory
// Slabs are handed between producer and MMA warp several at a time: one barrier round trip (wait, fence, commit) per
// eight or twelve MMAs instead of four.  Measured on the 7168x2048 expert shapes: two at a time GEMM1 2260 -> 2390
// TFLOP/s, GEMM2 2206 -> 2280; three at a time helps the K=7168 GEMM1 a little more (2420-2490) but leaves the
// K=2048 GEMM2 only two rounds deep (2100-2150).
// The group size is a template parameter: 3 for long K loops (at least kLongK slabs), 2 otherwise.
constexpr int kMaxRounds = 3;
constexpr int kLongK = 24;
constexpr int kThreads = 384;
constexpr int kEpiWarp0 = 4, kEpiWarps = 8;
constexpr int kTmemCols = 512;
constexpr int kSfCol0 = 256, kSfSlots = 4, kSfSlotCols = 16;   // per slot: SFA at +0 (4 columns), SFB at +4 (8 columns)
constexpr int kMaxExperts = 1024;
constexpr int kRing = 4;
constexpr int kTilePoison = -2;
constexpr int kRingReaders = 19;                       // producer, MMA, 8 epilogue warps (+ peer: producer, 8)
constexpr int kSmemBytes = kStages * (A_STAGE + B_STAGE + SFA_STAGE + SFB_STAGE) + 256 + (kMaxExperts + 1) * 4 + 1024;
constexpr uint32_t kStageTx = 2u * (A_STAGE + B_TX + SFA_STAGE + SFB_STAGE);   // both CTAs' bytes, counted at the leader

struct __align__(8) Bars {
  uint64_t full[kMaxRounds], empty[kMaxRounds];
  uint64_t acc_full, acc_empty;
  uint64_t sched_full[kRing], sched_empty[kRing];
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
  __device__ __forceinline__ void done(Bars* b, bool signal) {
    if (signal) mbar_arrive_cluster(mapa(smem_u32(&b->sched_empty[slot]), 0));
    if (++slot == kRing) { slot = 0; phase ^= 1u; }
  }
};

// kind::mxf8f6f4.block_scale: A e4m3 (format 0), B e2m1 (format 5), both K-major, ue8m0 scales (bit 23);
// the byte of each 32-bit scale word that an MMA uses (its K block within the stage) goes in bits 4-5 (B) and
// 29-30 (A)
__host__ __device__ constexpr uint32_t make_idesc_mx(int m, int n, int sf_id) {
  return ((uint32_t)sf_id << 4) | (0u << 7) | (5u << 10) | ((uint32_t)(n >> 3) << 17) | (1u << 23) |
         ((uint32_t)(m >> 4) << 24) | ((uint32_t)sf_id << 29);
}
__device__ __forceinline__ void tc_mma_mx_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %6, 0;\n"
               " tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%4], [%5], p;\n}"
               ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate) : "memory");
}
// Shared-memory descriptor of one scale atom: 32 rows of 16 bytes, no swizzle, 8-row groups 128 bytes apart.
__device__ __forceinline__ uint64_t make_sf_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(128 >> 4) << 32;                   // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                            // descriptor version (sm_100)
  return d;
}
// 32 rows x 128 bits of shared memory into 4 tensor-memory columns, repeated in all four 32-lane groups, in
// both CTAs of the pair (each from its own shared memory)
__device__ __forceinline__ void tc_cp_sf_pair(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void setmaxnreg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 232;" ::: "memory"); }
__device__ __forceinline__ void setmaxnreg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 40;" ::: "memory"); }

__device__ __forceinline__ uint32_t cvt_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm volatile("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
// ue8m0 code of the smallest power of two s with amax <= 448*s (448 = 1.75 * 2^8): biased exponent of amax
// minus 8, one more when its fraction exceeds 0.75; 127 for an all-zero block; clamped to 0..254.
__device__ __forceinline__ uint32_t mx_scale_code_e4m3(float amax) {
  const uint32_t u = __float_as_uint(amax);
  int code = (int)(u >> 23) - 8 + ((u & 0x7FFFFFu) > 0x600000u ? 1 : 0);
  code = code < 0 ? 0 : (code > 254 ? 254 : code);
  return amax == 0.f ? 127u : (uint32_t)code;
}
// 2^(127-code): the factor that brings a block onto the e4m3 grid
__device__ __forceinline__ float mx_inv_scale(uint32_t code) {
  return code <= 253u ? __uint_as_float((254u - code) << 23) : __uint_as_float(0x00400000u);
}

template <bool kSwiglu, int kGroup>
__global__ void __launch_bounds__(kThreads, 1)
grouped_gemm_mx_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                       const __grid_constant__ CUtensorMap tm_sfa, const __grid_constant__ CUtensorMap tm_sfb,
                       int num_kb /*K/128*/, int n_blocks_n, int n_group, int n_experts, int n_out_cols, int out_ld,
                       uint8_t* __restrict__ out_codes, uint8_t* __restrict__ out_sf /*atom order, out_ld/128 atoms per row block*/,
                       __nv_bfloat16* __restrict__ out_bf16,
                       const int32_t* __restrict__ tile_prefix, const int32_t* __restrict__ counts,
                       const int32_t* __restrict__ padded_offsets, int32_t* __restrict__ tile_counter,
                       int32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  pdl_enter();
  constexpr int kRounds = kStages / kGroup;
  static_assert(kStages % kGroup == 0 && kRounds <= kMaxRounds, "slabs per round");
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem_a + kStages * A_STAGE;
  uint8_t* smem_sfa = smem_b + kStages * B_STAGE;
  uint8_t* smem_sfb = smem_sfa + kStages * SFA_STAGE;
  Bars* bars = reinterpret_cast<Bars*>(smem_sfb + kStages * SFB_STAGE);
  int32_t* pair_prefix = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(bars) + 256);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool is_peer = rank != 0;
  volatile int* abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kRounds; ++s) { mbar_init(smem_u32(&bars->full[s]), 1); mbar_init(smem_u32(&bars->empty[s]), 1); }
    mbar_init(smem_u32(&bars->acc_full), 1);
    mbar_init(smem_u32(&bars->acc_empty), 2 * kEpiWarps);
    for (int s = 0; s < kRing; ++s) {
      mbar_init(smem_u32(&bars->sched_full[s]), 1); mbar_init(smem_u32(&bars->sched_empty[s]), kRingReaders);
      bars->sched_tile[s] = kTilePoison;
    }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x == 32) {
    int run = 0;
    for (int e = 0; e < n_experts; ++e) {          // pair tiles (two 128-row blocks) per expert
      pair_prefix[e] = run;
      run += (tile_prefix[e + 1] - tile_prefix[e] + 1) >> 1;
    }
    pair_prefix[n_experts] = run;
  }
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&bars->tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  const int total_tiles = pair_prefix[n_experts] * n_blocks_n;

  if (warp < kEpiWarp0) {
    setmaxnreg_dec();
    if (warp == 0 && lane == 0) {
      // ---------------------------------------------------------------- TMA producer (both CTAs)
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      Ring rd;
      for (; ok;) {
        const int tile = rd.next(bars, is_peer, abort_flag, status);
        rd.done(bars, true);
        if (tile < 0) break;
        TileCoord tc;
        if (!decode_tile(pair_prefix, n_experts, n_blocks_n, n_group, tile, &tc)) break;
        const int row0 = padded_offsets[tc.expert] + tc.m_block * (2 * BM) + (int)rank * BM;
        const int n0 = tc.n_block * BN + (int)rank * (BN / 2);
        const int sfa_atom0 = (row0 >> 7) * num_kb;                                   // atoms are [row block][k128]
        const int sfb_atom0 = (tc.expert * n_blocks_n + tc.n_block) * num_kb;         // [expert][n block of 256][k128]
        for (int kb0 = 0; kb0 < num_kb; kb0 += kGroup) {        // `stage` counts rounds of kGroup slabs here
          const int n_sub = num_kb - kb0 < kGroup ? num_kb - kb0 : kGroup;
          if (!mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag, status)) { ok = false; break; }
          const uint32_t full = mapa(smem_u32(&bars->full[stage]), 0);
          if (rank == 0) mbar_expect_tx(smem_u32(&bars->full[stage]), (uint32_t)n_sub * kStageTx);
          for (int sub = 0; sub < n_sub; ++sub) {
            const int slab = stage * kGroup + sub, kb = kb0 + sub;
            tma_load_2d_pair(smem_u32(smem_a + slab * A_STAGE), &tm_a, kb * BKE, row0, full);
            tma_load_3d_pair(smem_u32(smem_b + slab * B_STAGE), &tm_b, kb * BKE, n0, tc.expert, full);
            tma_load_2d_pair(smem_u32(smem_sfa + slab * SFA_STAGE), &tm_sfa, 0, sfa_atom0 + kb, full);
            tma_load_2d_pair(smem_u32(smem_sfb + slab * SFB_STAGE), &tm_sfb, 0, sfb_atom0 + kb, full);
          }
          if (++stage == kRounds) { stage = 0; phase ^= 1u; }
        }
      }
    } else if (warp == 1 && lane == 0 && !is_peer) {
      // ---------------------------------------------------------------- MMA issuer (leader CTA)
      int stage = 0; uint32_t phase = 0;
      uint32_t acc_phase = 0;
      int sf_slot = 0;
      bool ok = true;
      Ring rd;
      for (; ok;) {
        const int tile = rd.next(bars, false, abort_flag, status);
        rd.done(bars, true);
        if (tile < 0) break;
        if (!mbar_wait(smem_u32(&bars->acc_empty), acc_phase ^ 1u, abort_flag, status)) break;
        tc_fence_after();
        for (int kb0 = 0; kb0 < num_kb; kb0 += kGroup) {
          const int n_sub = num_kb - kb0 < kGroup ? num_kb - kb0 : kGroup;
          if (!mbar_wait(smem_u32(&bars->full[stage]), phase, abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          for (int sub = 0; sub < n_sub; ++sub) {
            const int slab = stage * kGroup + sub;
            const uint32_t sfa_t = tmem_base + (uint32_t)(kSfCol0 + sf_slot * kSfSlotCols);
            const uint32_t sfb_t = sfa_t + 4u;
            tc_cp_sf_pair(sfa_t, make_sf_desc(smem_u32(smem_sfa + slab * SFA_STAGE)));
            tc_cp_sf_pair(sfb_t, make_sf_desc(smem_u32(smem_sfb + slab * SFB_STAGE)));
            tc_cp_sf_pair(sfb_t + 4u, make_sf_desc(smem_u32(smem_sfb + slab * SFB_STAGE + kSfAtomBytes)));
            const uint64_t adesc = make_smem_desc(smem_u32(smem_a + slab * A_STAGE));
            const uint64_t bdesc = make_smem_desc(smem_u32(smem_b + slab * B_STAGE));
#pragma unroll
            for (int k4 = 0; k4 < BKE / 32; ++k4)        // 32 elements of K per MMA = one scale block
              tc_mma_mx_pair(tmem_base, adesc + (uint64_t)(k4 * 2), bdesc + (uint64_t)(k4 * 2), make_idesc_mx(2 * BM, BN, k4),
                             sfa_t, sfb_t, (kb0 | sub | k4) != 0 ? 1u : 0u);
            if (++sf_slot == kSfSlots) sf_slot = 0;
          }
          tc_commit_pair_both(smem_u32(&bars->empty[stage]), 3);
          if (++stage == kRounds) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit_pair_both(smem_u32(&bars->acc_full), 3);
        acc_phase ^= 1u;
      }
    } else if (warp == 2 && lane == 0 && !is_peer) {
      // ---------------------------------------------------------------- tile scheduler (leader CTA)
      int slot = 0; uint32_t phase = 0;
      for (;;) {
        if (!mbar_wait(smem_u32(&bars->sched_empty[slot]), phase ^ 1u, abort_flag, status)) break;
        int t = atomicAdd(tile_counter, 1);
        if (t >= total_tiles) t = -1;
        bars->sched_tile[slot] = t;
        st_shared_cluster_u32(mapa(smem_u32(&bars->sched_tile[slot]), 1), (uint32_t)t);
        mbar_arrive(smem_u32(&bars->sched_full[slot]));
        mbar_arrive_release_cluster(mapa(smem_u32(&bars->sched_full[slot]), 1));
        if (t < 0) break;
        if (++slot == kRing) { slot = 0; phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    setmaxnreg_inc();
    const int lane_grp = warp & 3;                     // tensor-memory lanes 32*lane_grp..+31
    const int half = (warp - kEpiWarp0) >> 2;
    // swiglu tile = [128 gate | 128 up]: this thread owns gate columns 64*half..+63 and the matching up columns;
    // plain tile: columns 128*half..+127
    const int col0 = kSwiglu ? 64 * half : 128 * half;
    const int col1 = kSwiglu ? 128 + 64 * half : 128 * half + 64;
    uint32_t acc_phase = 0;
    Ring rd;
    for (;;) {
      const int tile = rd.next(bars, is_peer, abort_flag, status);
      __syncwarp();
      rd.done(bars, lane == 0);
      if (tile < 0) break;
      TileCoord tc;
      if (!decode_tile(pair_prefix, n_experts, n_blocks_n, n_group, tile, &tc)) break;
      const int r_tile = lane_grp * 32 + lane;
      const int r_in_group = tc.m_block * (2 * BM) + (int)rank * BM + r_tile;
      const bool row_ok = r_in_group < counts[tc.expert];
      const size_t grow = (size_t)(padded_offsets[tc.expert] + r_in_group);
      // the lanes may leave the polling loop in different iterations; the tensor-memory loads are warp-collective
      const bool got = mbar_wait(smem_u32(&bars->acc_full), acc_phase, abort_flag, status);
      if (!__all_sync(0xffffffffu, got)) break;
      acc_phase ^= 1u;
      tc_fence_after();
      uint32_t v0[32], v1[32], v2[32], v3[32];
      const uint32_t t_addr = tmem_base + ((uint32_t)(lane_grp * 32) << 16);
      tc_ld32(t_addr + (uint32_t)col0, v0);
      tc_ld32(t_addr + (uint32_t)(col0 + 32), v1);
      tc_ld32(t_addr + (uint32_t)col1, v2);
      tc_ld32(t_addr + (uint32_t)(col1 + 32), v3);
      tc_wait_ld();
      // the tile is in registers: hand the accumulator columns back to the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa(smem_u32(&bars->acc_empty), 0));
      if (kSwiglu) {
        // v0,v1 = gate columns, v2,v3 = up columns -> 64 activations of this row = two scale blocks of 32
        uint32_t codes[16];
        uint32_t sf2 = 0;
#pragma unroll
        for (int b = 0; b < 2; ++b) {
          float a[32];
          float amax = 0.f;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            a[i] = silu_mul(__uint_as_float(b ? v1[i] : v0[i]), __uint_as_float(b ? v3[i] : v2[i]));
            amax = fmaxf(amax, fabsf(a[i]));
          }
          const uint32_t code = mx_scale_code_e4m3(amax);
          const float inv = mx_inv_scale(code);
          sf2 |= code << (8 * b);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint32_t lo = cvt_e4m3x2(a[4 * j] * inv, a[4 * j + 1] * inv);
            const uint32_t hi = cvt_e4m3x2(a[4 * j + 2] * inv, a[4 * j + 3] * inv);
            codes[8 * b + j] = lo | (hi << 16);
          }
        }
        if (row_ok) {
          uint4* dst = reinterpret_cast<uint4*>(out_codes + grow * out_ld + tc.n_block * 128 + 64 * half);
#pragma unroll
          for (int q = 0; q < 4; ++q) dst[q] = make_uint4(codes[4 * q], codes[4 * q + 1], codes[4 * q + 2], codes[4 * q + 3]);
          // the tile's 128 output columns are one atom column (4 scale blocks) of the next GEMM's A operand
          uint8_t* sf = out_sf + sf_atom_offset((long long)grow, 4 * tc.n_block + 2 * half, out_ld >> 7);
          *reinterpret_cast<uint16_t*>(sf) = (uint16_t)sf2;
        }
      } else {
        if (row_ok) {
          const int c_out = tc.n_block * BN + 128 * half;
          if (c_out < n_out_cols) {
            uint4* dst = reinterpret_cast<uint4*>(out_bf16 + grow * out_ld + c_out);
#define CEP_STORE32(V, Q0)                                                                               \
  _Pragma("unroll") for (int q = 0; q < 4; ++q) {                                                        \
    uint4 o;                                                                                             \
    o.x = pack_bf16(__uint_as_float((V)[8 * q + 0]), __uint_as_float((V)[8 * q + 1]));                   \
    o.y = pack_bf16(__uint_as_float((V)[8 * q + 2]), __uint_as_float((V)[8 * q + 3]));                   \
    o.z = pack_bf16(__uint_as_float((V)[8 * q + 4]), __uint_as_float((V)[8 * q + 5]));                   \
    o.w = pack_bf16(__uint_as_float((V)[8 * q + 6]), __uint_as_float((V)[8 * q + 7]));                   \
    dst[(Q0) + q] = o;                                                                                   \
  }
            CEP_STORE32(v0, 0)
            CEP_STORE32(v1, 4)
            CEP_STORE32(v2, 8)
            CEP_STORE32(v3, 12)
#undef CEP_STORE32
          }
        }
      }
    }
  }
  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------- weight prepack (one-off)
// Codes: src [E, R, C] one e2m1 code per byte (R = input dimension) -> dst [E, n_dst, R/2], two codes per byte
// (the element with the even K index in the low four bits), row n = packed_col(c, mode) as in the bf16 prepack:
// mode 0: n = c; mode 1 (gate): n = (c/128)*256 + c%128; mode 2 (up): that + 128.
__host__ __device__ inline int packed_col(int c, int mode) {
  if (mode == 0) return c;
  return (c >> 7) * 256 + (c & 127) + (mode == 2 ? 128 : 0);
}

__global__ void __launch_bounds__(256)
pack_codes_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, int R, int C, int n_dst, int mode) {
  __shared__ uint8_t tile[64][33];
  const int e = blockIdx.z;
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 64;
  const uint8_t* s = src + (size_t)e * R * C;
  uint8_t* d = dst + (size_t)e * n_dst * (R / 2);
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;          // 32 x 8
  for (int i = ty; i < 64; i += 8) {
    const int r = r0 + i, c = c0 + tx;
    tile[i][tx] = (r < R && c < C) ? s[(size_t)r * C + c] : (uint8_t)0;
  }
  __syncthreads();
  for (int i = ty; i < 32; i += 8) {
    const int c = c0 + i, rb = (r0 >> 1) + tx;                       // output byte rb holds rows 2rb, 2rb+1
    if (c < C && 2 * rb + 1 < R)
      d[(size_t)packed_col(c, mode) * (R / 2) + rb] = (uint8_t)((tile[2 * tx][i] & 15) | ((tile[2 * tx + 1][i] & 15) << 4));
  }
}

// Scales: src [E, R/32, C] ue8m0 -> atoms [E][n_dst/256][R/128][2][512]: weight row n of a 256-row block sits in
// atom (n%256)/128 at byte (n%32)*16 + ((n%128)/32)*4 + (K block % 4)
__global__ void pack_weight_sf_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, int E, int R, int C,
                                      int n_dst, int mode) {
  const int RB = R / kMxBlock;
  const size_t total = (size_t)E * RB * C;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int c = (int)(i % C); const size_t t = i / C; const int kb = (int)(t % RB); const int e = (int)(t / RB);
    const int n = packed_col(c, mode);
    const size_t atom2 = ((size_t)e * (n_dst / 256) + (n >> 8)) * (R / 128) + (kb >> 2);
    const int nl = n & 255;
    dst[atom2 * (2 * kSfAtomBytes) + (nl >> 7) * kSfAtomBytes + (nl & 31) * 16 + ((nl >> 5) & 3) * 4 + (kb & 3)] = src[i];
  }
}

// cudaFuncSetAttribute and the occupancy answer hold per device: one slot per device ordinal
constexpr int kMaxDevices = 64;
int g_clusters[kMaxDevices];                           // co-resident CTA pairs + 1 (0: not set up yet)

cudaError_t setup(int dev, int n_sms) {
  if (g_clusters[dev] > 0) return cudaSuccess;
  cudaError_t e = cudaSuccess;
#define CEP_MX_ATTR(SW, G) if (e == cudaSuccess) e = cudaFuncSetAttribute(grouped_gemm_mx_kernel<SW, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  CEP_MX_ATTR(true, 2) CEP_MX_ATTR(true, 3) CEP_MX_ATTR(false, 2) CEP_MX_ATTR(false, 3)
#undef CEP_MX_ATTR
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3(n_sms & ~1, 1, 1); cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes; cfg.attrs = attr; cfg.numAttrs = 1;
  int n = 0;
  e = cudaOccupancyMaxActiveClusters(&n, grouped_gemm_mx_kernel<true, 2>, &cfg);
  if (e != cudaSuccess) return e;
  g_clusters[dev] = n + 1;
  return cudaSuccess;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

}  // namespace

// Packed e2m1 weights [n_batch, rows, K/2 bytes]: tiles of 128 codes of K x box_rows rows; the load expands
// every 16 codes (8 bytes) into a 16-byte slot of shared memory, 128-byte swizzle.
int make_mx_weight_map(GemmTensorMap* out, const void* base, int K, long long rows, int n_batch, int box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return -1;
  CUtensorMap* m = reinterpret_cast<CUtensorMap*>(out);
  cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, (cuuint64_t)n_batch};
  cuuint64_t strides[2] = {(cuuint64_t)K / 2, (cuuint64_t)K / 2 * (cuuint64_t)rows};
  cuuint32_t box[3] = {128, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B, 3, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -2;
}

// Scale atoms as a 2-D tensor of 32-bit words: one row per load (atom_bytes = 512 or 1024), no swizzle.
int make_mx_sf_map(GemmTensorMap* out, const void* base, long long n_loads, int atom_bytes) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return -1;
  CUtensorMap* m = reinterpret_cast<CUtensorMap*>(out);
  cuuint64_t dims[2] = {(cuuint64_t)(atom_bytes / 4), (cuuint64_t)n_loads};
  cuuint64_t strides[1] = {(cuuint64_t)atom_bytes};
  cuuint32_t box[2] = {(cuuint32_t)(atom_bytes / 4), 1};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_INT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -2;
}

cudaError_t launch_prepack_mx(const cep_config& cfg, const void* w_gate, const void* w_up, const void* w_down,
                              const void* s_gate, const void* s_up, const void* s_down, void* w13p, void* w2p,
                              void* sf13p, void* sf2p, cudaStream_t s, int64_t* launches) {
  const int H = cfg.hidden, I = cfg.inter, E = cfg.n_experts_local;
  dim3 g1((I + 31) / 32, (H + 63) / 64, E), g2((H + 31) / 32, (I + 63) / 64, E);
  pack_codes_kernel<<<g1, 256, 0, s>>>((const uint8_t*)w_gate, (uint8_t*)w13p, H, I, 2 * I, 1);
  pack_codes_kernel<<<g1, 256, 0, s>>>((const uint8_t*)w_up, (uint8_t*)w13p, H, I, 2 * I, 2);
  pack_codes_kernel<<<g2, 256, 0, s>>>((const uint8_t*)w_down, (uint8_t*)w2p, I, H, H, 0);
  pack_weight_sf_kernel<<<512, 256, 0, s>>>((const uint8_t*)s_gate, (uint8_t*)sf13p, E, H, I, 2 * I, 1);
  pack_weight_sf_kernel<<<512, 256, 0, s>>>((const uint8_t*)s_up, (uint8_t*)sf13p, E, H, I, 2 * I, 2);
  pack_weight_sf_kernel<<<512, 256, 0, s>>>((const uint8_t*)s_down, (uint8_t*)sf2p, E, I, H, H, 0);
  *launches += 6;
  return cudaGetLastError();
}

cudaError_t launch_gemm_mx(const GemmProblem& p, const GemmTensorMap& tm_a, const GemmTensorMap& tm_b,
                           const GemmTensorMap& tm_sfa, const GemmTensorMap& tm_sfb, void* out, void* out_sf,
                           const LayoutPtrs& lp, int max_pair_tiles, int n_sms, cudaStream_t s, int64_t* launches) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  e = setup(dev, n_sms);
  if (e != cudaSuccess) return e;
  const int resident = g_clusters[dev] - 1;
  if (resident < 1) return cudaErrorNotSupported;
  const int ctas = 2 * (max_pair_tiles < resident ? max_pair_tiles : resident);
  if (ctas < 2) return cudaSuccess;
  const int n_blocks_n = p.N / BN;
  const int n_out_cols = p.swiglu ? p.N / 2 : p.N;
  const int num_kb = p.K / BKE;
  // packed codes: half a byte per element
  const int n_group = n_group_for(n_blocks_n, BN, p.K / 2, 1);
  int32_t* counter = lp.sched + (p.swiglu ? 0 : 1);
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = dim3(ctas, 1, 1); cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes; cfg.stream = s; cfg.attrs = attr; cfg.numAttrs = 2;
  const CUtensorMap& a = reinterpret_cast<const CUtensorMap&>(tm_a);
  const CUtensorMap& b = reinterpret_cast<const CUtensorMap&>(tm_b);
  const CUtensorMap& sa = reinterpret_cast<const CUtensorMap&>(tm_sfa);
  const CUtensorMap& sb = reinterpret_cast<const CUtensorMap&>(tm_sfb);
#define CEP_MX_LAUNCH(SW, G)                                                                                           \
  cudaLaunchKernelEx(&cfg, grouped_gemm_mx_kernel<SW, G>, a, b, sa, sb, num_kb, n_blocks_n, n_group, p.n_experts,          \
                     n_out_cols, p.out_ld, SW ? (uint8_t*)out : (uint8_t*)nullptr, SW ? (uint8_t*)out_sf : (uint8_t*)nullptr, \
                     SW ? (__nv_bfloat16*)nullptr : (__nv_bfloat16*)out, (const int32_t*)lp.tile_prefix,                   \
                     (const int32_t*)lp.counts, (const int32_t*)lp.padded_offsets, counter, lp.status)
  const bool long_k = num_kb >= kLongK;
  if (p.swiglu) e = long_k ? CEP_MX_LAUNCH(true, 3) : CEP_MX_LAUNCH(true, 2);
  else e = long_k ? CEP_MX_LAUNCH(false, 3) : CEP_MX_LAUNCH(false, 2);
#undef CEP_MX_LAUNCH
  *launches += 1;
  return e;
}

}  // namespace cep
