// Host interface of the tensor-core grouped GEMM (gemm_tcgen05.cu).
#pragma once
#include "cep_common.h"

namespace cep {

// Opaque 128-byte TMA descriptor (layout of the driver's CUtensorMap).
struct alignas(64) GemmTensorMap { unsigned long long opaque[16]; };

// Describes a K-major operand `rows x K` (n_batch == 0) or `n_batch x rows x K` (n_batch > 0)
// for 128-byte-of-K x box_rows tiles with 128-byte swizzle.  Returns 0, -1 when the driver
// entry point is unavailable, -2 when the driver rejects the description.
int make_operand_map(GemmTensorMap* out, const void* base, int elt_bytes, int K, long long rows, int n_batch,
                     int box_rows);
// One CTA that waits limit_ns on a barrier nobody signals, then records the timeout in status (test hook).
cudaError_t launch_wait_probe(unsigned long long limit_ns, int32_t* status, cudaStream_t s, int64_t* launches);
int gemm_tile_rows();
int gemm_tile_cols();

cudaError_t launch_gemm_tcgen05(const GemmProblem& p, const GemmTensorMap& tm_a, const GemmTensorMap& tm_b,
                                void* out, const LayoutPtrs& lp, int max_tiles, int n_sms, cudaStream_t s,
                                int64_t* launches);

// CTA-pair variant (256-row x 256-column tiles, tcgen05 cta_group::2).  box_rows of its weight operand
// map is gemm_tile_cols()/2.  max_pair_tiles bounds the number of pair tiles (for the grid size).
// src_row != NULL (GEMM1 only): tm_a describes the caller's token tensor with one-row boxes
// (make_operand_map with box_rows = 1) and physical row r of the operand is that tensor's row src_row[r].
cudaError_t launch_gemm_tcgen05_pair(const GemmProblem& p, const GemmTensorMap& tm_a, const GemmTensorMap& tm_b,
                                     void* out, const LayoutPtrs& lp, const int32_t* src_row, int max_pair_tiles,
                                     int n_sms, cudaStream_t s, int64_t* launches);

// Block-scaled e4m3 variant.  a_scales [rows, K/128], b_scales [E, N/128, K/128] fp32.  With p.swiglu the output is
// e4m3 codes [rows, N/2] plus out_scales [rows, N/256]; otherwise bf16 [rows, N].  pair != 0: CTA pairs on 256x256
// tiles; pair == 0: one CTA per 128x256 tile.  The weight map's box has gemm_fp8_box_rows(pair) rows (the weight
// rows one CTA loads per stage).
int gemm_fp8_box_rows(int pair);
// Output of the block-scaled kernels as the TMA engine stores it: a rows x cols tensor of elt_bytes elements
// written in boxes of 32 rows x 64 bytes (64-byte swizzle in shared memory).
int make_store_map(GemmTensorMap* out, void* base, int elt_bytes, int cols, long long rows);
cudaError_t launch_gemm_fp8(const GemmProblem& p, int pair, const GemmTensorMap& tm_a, const GemmTensorMap& tm_b,
                            const GemmTensorMap& tm_out, const float* a_scales, const float* b_scales, void* out, float* out_scales,
                            const LayoutPtrs& lp, int max_tiles, int n_sms, cudaStream_t s, int64_t* launches);
// s13p[e][2*ib + (0 gate | 1 up)][kb] and s2p[e][hb][kb] from the caller's [E, in/128, out/128] scale tensors
cudaError_t launch_pack_scales(const cep_config& cfg, const float* s_gate, const float* s_up, const float* s_down,
                               float* s13p, float* s2p, cudaStream_t s, int64_t* launches);

// Microscaling variant (e4m3 activations x packed e2m1 weights, ue8m0 scales per 32 elements of K, scaled by the
// tensor core).  CTA pairs on 256x256 tiles.  Scale factors of both operands are read through 2-D maps over
// their 512-byte atoms (see kSfAtomBytes); with p.swiglu the output is e4m3 codes [rows, N/2] plus their scale
// atoms out_sf, otherwise bf16 [rows, N].
int make_mx_weight_map(GemmTensorMap* out, const void* base, int K, long long rows, int n_batch, int box_rows);
int make_mx_sf_map(GemmTensorMap* out, const void* base, long long n_loads, int atom_bytes);
cudaError_t launch_gemm_mx(const GemmProblem& p, const GemmTensorMap& tm_a, const GemmTensorMap& tm_b,
                           const GemmTensorMap& tm_sfa, const GemmTensorMap& tm_sfb, void* out, void* out_sf,
                           const LayoutPtrs& lp, int max_pair_tiles, int n_sms, cudaStream_t s, int64_t* launches);
// codes [E,in,out] (one e2m1 code per byte) -> K-major packed nibbles; scales [E,in/32,out] -> scale atoms
cudaError_t launch_prepack_mx(const cep_config& cfg, const void* w_gate, const void* w_up, const void* w_down,
                              const void* s_gate, const void* s_up, const void* s_down, void* w13p, void* w2p,
                              void* sf13p, void* sf2p, cudaStream_t s, int64_t* launches);

}  // namespace cep
