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
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s

struct __align__(8) Barriers {
  uint64_t full[kStages], empty[kStages], acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};
constexpr int kSmemBytes = kStages * (A_STAGE + B_STAGE) + 1024 /*alignment slack*/ + 256;
static_assert(sizeof(Barriers) <= 256, "barrier block");

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long globaltimer() {
  unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the wait was abandoned (this or another role timed out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer();
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 1023u) == 0u) {
      if (*abort_flag) return false;
      if (globaltimer() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(&status[kStTimeout], 1);
        return false;
      }
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
               ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes,
// 8-row groups 1024 bytes apart (stride byte offset), descriptor version 1.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);          // start address, 16-byte units
  d |= (uint64_t)1 << 16;                            // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset
  d |= (uint64_t)1 << 46;                            // descriptor version (sm_100)
  d |= (uint64_t)2 << 61;                            // 128-byte swizzle
  return d;
}
// Instruction descriptor for kind::f16: fp32 accumulate, bf16 x bf16, both K-major, M=128, N=256.
__host__ __device__ constexpr uint32_t make_idesc_bf16() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ float silu_mul(float g, float u) { return (g / (1.f + __expf(-g))) * u; }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// ------------------------------------------------------------------ the kernel
template <bool kSwiglu>
__global__ void __launch_bounds__(kThreads, 1)
grouped_gemm_bf16_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                         int num_kb /*K*2/128*/, int n_blocks_n, int n_experts, int n_out_cols, int out_ld,
                         __nv_bfloat16* __restrict__ out, const int32_t* __restrict__ tile_prefix,
                         const int32_t* __restrict__ counts, const int32_t* __restrict__ padded_offsets,
                         int32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
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
        if (!decode_tile(tile_prefix, n_experts, n_blocks_n, tile, &tc)) break;
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
      constexpr uint32_t idesc = make_idesc_bf16();
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
      if (!decode_tile(tile_prefix, n_experts, n_blocks_n, tile, &tc)) break;
      if (!mbar_wait(smem_u32(&bars->acc_full[acc]), acc_phase, abort_flag, status)) break;
      tc_fence_after();
      const int r_in_group = tc.m_block * BM + lane_grp * 32 + lane;
      const bool row_ok = r_in_group < counts[tc.expert];
      const size_t grow = (size_t)(padded_offsets[tc.expert] + r_in_group);
      const uint32_t t_addr = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(acc * BN);
      if (kSwiglu) {
        __nv_bfloat16* orow = out + grow * out_ld + tc.n_block * (BN / 2);
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t g[32], u[32];
          tc_ld32(t_addr + c * 32, g);
          tc_ld32(t_addr + 128 + c * 32, u);
          tc_wait_ld();
          if (row_ok && tc.n_block * (BN / 2) + c * 32 < n_out_cols) {
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
        __nv_bfloat16* orow = out + grow * out_ld + tc.n_block * BN;
#pragma unroll 1
        for (int c = 0; c < 8; ++c) {
          uint32_t d[32];
          tc_ld32(t_addr + c * 32, d);
          tc_wait_ld();
          if (row_ok && tc.n_block * BN + c * 32 < n_out_cols) {
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

}  // namespace

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

int gemm_tile_rows() { return BM; }
int gemm_tile_cols() { return BN; }

cudaError_t launch_gemm_tcgen05(const GemmProblem& p, const GemmTensorMap& tm_a, const GemmTensorMap& tm_b,
                                void* out, const LayoutPtrs& lp, int max_tiles, int n_sms, cudaStream_t s,
                                int64_t* launches) {
  if (p.is_fp8) return cudaErrorNotSupported;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(grouped_gemm_bf16_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(grouped_gemm_bf16_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int n_blocks_n = (p.N + BN - 1) / BN;
  const int n_out_cols = p.swiglu ? p.N / 2 : p.N;
  int grid = max_tiles < n_sms ? max_tiles : n_sms;
  if (grid < 1) return cudaSuccess;
  const int num_kb = p.K * 2 / BKB;
  const CUtensorMap& a = reinterpret_cast<const CUtensorMap&>(tm_a);
  const CUtensorMap& b = reinterpret_cast<const CUtensorMap&>(tm_b);
  if (p.swiglu)
    grouped_gemm_bf16_kernel<true><<<grid, kThreads, kSmemBytes, s>>>(a, b, num_kb, n_blocks_n, p.n_experts, n_out_cols,
        p.out_ld, (__nv_bfloat16*)out, lp.tile_prefix, lp.counts, lp.padded_offsets, lp.status);
  else
    grouped_gemm_bf16_kernel<false><<<grid, kThreads, kSmemBytes, s>>>(a, b, num_kb, n_blocks_n, p.n_experts, n_out_cols,
        p.out_ld, (__nv_bfloat16*)out, lp.tile_prefix, lp.counts, lp.padded_offsets, lp.status);
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace cep
