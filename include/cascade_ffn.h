/*
 * cascade_ffn.h -- C ABI of the streamFFN routed-expert path for one B200 (sm_100a).
 *
 * The library runs the expert side of a prefill MoE layer the way the paper's
 * streamFFN does (Section 3.2 "Asynchronous EP and streaming FFN"; Appendix
 * "Runtime Implementation Details"): routed tokens arrive in per-replica chunks at
 * different times; ready chunks accumulate until a launch threshold theta is reached
 * (or everything has arrived: the final flush bypasses theta); every launch is one
 * *grouped FFN invocation* on its own CUDA stream and scratch slot:
 *
 *   layout transform  histogram -> exclusive scan -> stable scatter into expert-major,
 *                     tile-aligned groups, with an inverse map (Appendix "Grouped FFN
 *                     invocations")
 *   expert GEMM 1     [gate | up] projections, SiLU(gate)*up fused in the epilogue
 *   expert GEMM 2     down projection
 *   combine           every routed contribution weighted by its routing coefficient
 *                     exactly once, accumulated per token, written in token order
 *                     (Appendix "Output return and combine")
 *
 * Conventions
 *   - Every function returns 0 (CEP_OK) or a negative cep_status.  Nothing throws,
 *     aborts or traps.  cep_last_error() gives a human-readable reason.
 *   - Pointers marked [device] are CUDA device pointers, [host] are host pointers.
 *   - The CALLER owns every device buffer (workspace, packed weights, chunk inputs,
 *     output).  The library allocates no device memory; it owns only the host-side
 *     plan object and the CUDA streams/events it creates.
 *   - Chunk input buffers and the output buffer must stay valid and unmodified from
 *     ffn_submit_chunk() until the stream passed to combine() has completed: buffers
 *     remain live until their dependent computations have finished (Appendix "Output
 *     return and combine").
 *   - ffn_submit_chunk / ffn_flush / combine only enqueue work; none blocks the host
 *     on the device.
 *   - A plan is not thread-safe; use one plan per host thread or serialise calls.
 *   - Expert ids are *global*; ids 0..n_experts_local-1 live on this rank, larger ids
 *     belong to other ranks and their pairs are skipped.
 */
#ifndef CASCADE_FFN_H_
#define CASCADE_FFN_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define CEP_API __attribute__((visibility("default")))
#else
#define CEP_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cep_plan cep_plan;

typedef enum {
  CEP_OK = 0,
  CEP_ERR_ARG = -1,            /* null pointer, non-positive size, unsupported shape            */
  CEP_ERR_STATE = -2,          /* call out of order: submit before begin / after flush, double
                                  submit of a chunk id, begin while a layer is open             */
  CEP_ERR_WORKSPACE = -3,      /* workspace or packed-weight buffer too small or misaligned     */
  CEP_ERR_CAPACITY = -4,       /* more tokens or chunks than the plan was made for              */
  CEP_ERR_INCOMPLETE = -5,     /* flush/combine with fewer chunks than ffn_begin announced;
                                  the work already submitted still runs                          */
  CEP_ERR_BAD_ROUTING = -6,    /* device found an expert id outside [0, n_experts_global), or (plans
                                  made with debug_checks) a token naming one expert twice        */
  CEP_ERR_DEVICE_TIMEOUT = -7, /* a bounded wait inside a kernel expired; kernel exited cleanly */
  CEP_ERR_CUDA = -8,           /* a CUDA runtime/driver call failed                             */
  CEP_ERR_UNSUPPORTED = -9     /* valid request this build does not implement                   */
} cep_status;

typedef enum {
  CEP_BF16 = 0,                /* bf16 activations and weights, fp32 accumulate, bf16 output    */
  CEP_FP8_E4M3_BLOCK128 = 1,   /* e4m3 codes; fp32 scales per 1x128 activation block and per
                                  128x128 weight block; bf16 output                              */
  CEP_MXFP4_E4M3 = 2           /* microscaling: MXFP4 expert weights ("Evaluation Settings"), e2m1 codes with
                                  one ue8m0 scale (2^(s-127)) per 32 elements of the input
                                  dimension; e4m3 activations with one ue8m0 scale per 1x32 block
                                  along the hidden dimension; the intermediate is re-quantised the
                                  same way (scale = the smallest power of two that brings the
                                  block's largest magnitude to <= 448, round to nearest even);
                                  fp32 accumulate; bf16 output                                   */
} cep_dtype;

/* Execution modes of the ablation study ("Deep Dive"). */
typedef enum {
  CEP_MODE_SYNC = 0,           /* one invocation once all chunks have arrived                   */
  CEP_MODE_ASYNC = 1,          /* one invocation per chunk as it arrives                        */
  CEP_MODE_STREAMFFN = 2       /* accumulate to threshold_pairs, multi-stream, final flush      */
} cep_mode;

typedef enum {
  CEP_GEMM_TCGEN05 = 0,        /* tcgen05/TMEM tiles fed by TMA, CTA pairs on 256x256 tiles
                                  (the product path)                                            */
  CEP_GEMM_SIMT = 1,           /* slow CUDA-core kernel, kept for fault isolation in tests      */
  CEP_GEMM_TCGEN05_1CTA = 2    /* tcgen05 with one CTA per 128x256 tile (comparison variant)    */
} cep_gemm_impl;

#define CEP_MAX_CHUNKS_PER_INVOCATION 32   /* a batch is launched early when it holds this many */
#define CEP_ROW_ALIGN 128                  /* expert groups start on multiples of the GEMM tile */

typedef struct {
  int32_t hidden;              /* H; multiple of 128 (fp8, mxfp4: multiple of 256)              */
  int32_t inter;               /* I; multiple of 128                                            */
  int32_t n_experts_global;    /* E_g                                                           */
  int32_t n_experts_local;     /* E <= E_g, at most 1024                                        */
  int32_t top_k;               /* k, at most 32                                                 */
  int32_t max_tokens;          /* upper bound on tokens per layer call                          */
  int32_t max_chunks;          /* upper bound on chunks per layer call                          */
  int32_t dtype;               /* cep_dtype                                                     */
  int32_t mode;                /* cep_mode                                                      */
  int32_t n_streams;           /* S >= 1 compute streams / scratch slots (round-robin)          */
  int64_t threshold_pairs;     /* theta: ready local (token, expert) pairs per invocation       */
  int32_t gemm_impl;           /* cep_gemm_impl                                                 */
  int32_t debug_checks;        /* nonzero: every region of the workspace is followed by a 1 KiB gap
                                  filled with a byte pattern at moe_plan (cep_debug_check_guards
                                  verifies them), and the histogram kernel also checks that the
                                  top_k ids of a token are distinct (CEP_ERR_BAD_ROUTING).  The
                                  other in-kernel checks (expert ids in range, rows inside the
                                  scratch slot, tile-ring values) are always on and record in the
                                  status word instead of trapping                               */
  int32_t profile_kernels;     /* nonzero: record CUDA events between the kernels of every
                                  invocation so ffn_query can report per-kernel device times    */
  int32_t defer_while_busy;    /* CEP_MODE_STREAMFFN only.  0: a batch is launched the moment it reaches
                                  theta (the launch rule as Section 3.2 states it).  Nonzero: when theta
                                  is reached while the previous invocation of this layer call is still
                                  running on the GPU, the launch is put off and chunks keep accumulating:
                                  queued work gains nothing from being split, and fewer, larger batches
                                  keep the expert GEMMs efficient.  The batch goes out at the first later
                                  ffn_submit_chunk that finds that invocation finished, when it holds
                                  4*theta pairs or CEP_MAX_CHUNKS_PER_INVOCATION chunks, or at the flush.
                                  Batching then depends on GPU timing (results do not)             */
  int32_t gather_a;            /* bf16 with CEP_GEMM_TCGEN05 only (CEP_ERR_UNSUPPORTED otherwise).  Nonzero:
                                  the layout transform (Appendix "Grouped FFN invocations") computes the
                                  indices but moves no rows; the gate/up GEMM fetches each operand row
                                  from the caller's tokens through a TMA row gather.  All chunks of a
                                  layer call must then be row slices of ONE dense [n_tokens_total, H]
                                  tensor (chunk pointer = tensor + token_offset rows; CEP_ERR_UNSUPPORTED
                                  from ffn_submit_chunk otherwise), and that tensor must stay unchanged
                                  until the layer call's combine work has run.  Results are bit-identical
                                  to gather_a = 0; the workspace is smaller by the permuted copy      */
} cep_config;

/* Per-invocation record for tracing (ffn_query). */
typedef struct {
  int32_t n_chunks;            /* chunks in the batch                                           */
  int32_t first_chunk_pos;     /* submission position of its first chunk                        */
  int32_t stream_index;        /* compute stream / scratch slot used                            */
  int32_t n_tokens;            /* tokens in the batch                                           */
  int64_t pairs_bound;         /* host-side count of ready pairs that triggered the launch      */
  float elapsed_ms;            /* device time first kernel -> last kernel; < 0 if not finished  */
  float layout_ms;             /* histogram + scan + rank + scatter   (profile_kernels only,    */
  float gemm1_ms;              /* gate/up GEMM with fused SiLU*up      else < 0)                 */
  float gemm2_ms;              /* down GEMM                                                     */
  float combine_ms;            /* weighted combine + unpermute                                  */
  float index_ms;              /* histogram + scan + rank (the integer part of layout_ms)       */
  float scatter_ms;            /* row scatter (the payload part of layout_ms)                   */
} cep_invocation_info;

/* Bytes of device workspace a plan with this configuration needs.  [host] out. */
CEP_API int moe_plan_workspace_bytes(const cep_config* cfg, size_t* bytes);

/* Bytes of the packed (K-major, gate/up interleaved) copy of the expert weights. */
CEP_API int moe_packed_weight_bytes(const cep_config* cfg, size_t* bytes);

/*
 * moe_plan: create a plan ("routing" = the shapes and the streamFFN policy of one MoE
 * layer).  `workspace` [device], 256-byte aligned, at least moe_plan_workspace_bytes();
 * it is carved into S scratch slots (each invocation has its own scratch, Appendix
 * "Grouped FFN invocations") and stays owned by the caller.  Creates S non-blocking
 * streams and the events.  Must be called with the target device current.
 * If the environment variable CEP_NVTX is set to anything but "" or "0" when the plan is made,
 * the plan names its streams ("cep slot i") and wraps every layer call (ffn_begin .. combine) and
 * every FFN invocation's enqueue in NVTX ranges, for timeline tools (the paper reads its attention
 * and dispatch timings from such timelines, Appendix "Long-Tail Statistics of DEP Prefill"); without
 * a tool attached the annotations do nothing.
 */
CEP_API int moe_plan(const cep_config* cfg, void* workspace, size_t workspace_bytes, cep_plan** out);

/*
 * One-off weight prepack, off the hot path.  Inputs [device]:
 *   w_gate, w_up  [E, H, I]   w_down [E, I, H]     (bf16, or e4m3 codes, or for mxfp4 one
 *                                                   e2m1 code per byte in its low four bits)
 *   s_gate, s_up  [E, H/128, I/128]  s_down [E, I/128, H/128]   fp32, for fp8
 *   s_gate, s_up  [E, H/32, I]       s_down [E, I/32, H]        uint8 ue8m0, for mxfp4
 *                 (32 consecutive elements of the input dimension share a scale); NULL for bf16
 * `packed` [device], 256-byte aligned, moe_packed_weight_bytes() long, must outlive the
 * plan's use of it.  The transposes are enqueued on `stream` (cudaStream_t); later
 * layer calls are ordered after them.
 */
CEP_API int moe_load_weights(cep_plan* plan, const void* w_gate, const void* w_up, const void* w_down,
                     const void* s_gate, const void* s_up, const void* s_down,
                     void* packed, size_t packed_bytes, void* stream);

/*
 * Open a layer call.  `out` [device] bf16 [n_tokens_total, H] in token order, 16-byte aligned
 * (CEP_ERR_ARG otherwise); every row is written by combine work (rows of tokens with no local
 * expert become exact zeros).  n_chunks_expected chunks will be submitted, together covering the
 * n_tokens_total tokens exactly once: a chunk that would bring the submitted tokens above
 * n_tokens_total is refused with CEP_ERR_CAPACITY, and a flush or combine with all chunks in but
 * fewer tokens than announced reports CEP_ERR_INCOMPLETE.
 */
CEP_API int ffn_begin(cep_plan* plan, void* out, int32_t n_tokens_total, int32_t n_chunks_expected);

/*
 * Optional, between ffn_begin and the first ffn_submit_chunk: `addend` [device] bf16 [n_tokens_total, H] in
 * token order is added to every output row (fp32, before the single rounding).  This is the shared expert's
 * output, which the layer sums with the routed result (Appendix "Output return and combine").
 * The rows of a chunk's tokens must be complete on that chunk's stream when the chunk is submitted.  NULL
 * (the default after ffn_begin) adds nothing.
 */
CEP_API int ffn_set_addend(cep_plan* plan, const void* addend);

/*
 * Router step that precedes the path (benchmark definition; the paper does not describe its router):
 * softmax over all experts, keep the top_k most probable, renormalise over those.  Needs no plan.
 *   logits        [device] fp32 [n_tokens, n_experts_global], n_experts_global <= 1024
 *   topk_ids      [device] out int32 [n_tokens, top_k]  slots in descending probability, ties to the lower id
 *   topk_weights  [device] out fp32 [n_tokens, top_k]   softmax over the selected logits (sums to 1)
 * Enqueued on `stream`.
 */
CEP_API int moe_route(const float* logits, int32_t n_tokens, int32_t n_experts_global, int32_t top_k,
                      int32_t* topk_ids, float* topk_weights, void* stream);

/*
 * A replica's routed tokens have arrived (Section 3.2: per-replica completion signal).
 *   chunk_id       0..n_chunks_expected-1, each exactly once, any order
 *   token_offset   first token (row of `out`) this chunk covers
 *   tokens         [device] bf16 [n,H]  |  e4m3 [n,H]
 *   token_scales   [device] fp32 [n,H/128] for fp8; uint8 ue8m0 [n,H/32] for mxfp4 (4-byte aligned); else NULL
 *   topk_ids       [device] int32 [n,k] global expert ids, distinct per token
 *   topk_weights   [device] fp32 [n,k]
 *   n_local_pairs  number of (token,slot) pairs with id < n_experts_local, as known from
 *                  dispatch metadata; -1 => use the bound n*k.  Only the launch decision
 *                  uses it, never an index.
 *   stream         cudaStream_t on which the chunk's data becomes ready; the library
 *                  records an event there and its compute streams wait on it.
 * Returns immediately.  May launch an invocation (see cep_mode).
 */
CEP_API int ffn_submit_chunk(cep_plan* plan, int32_t chunk_id, int32_t token_offset, int32_t n_tokens,
                     const void* tokens, const void* token_scales, const int32_t* topk_ids,
                     const float* topk_weights, int64_t n_local_pairs, void* stream);

/* All tokens have arrived: launch whatever is pending regardless of theta
 * (Section 3.2 "Launch threshold", last sentence). */
CEP_API int ffn_flush(cep_plan* plan);

/*
 * Layer boundary (Appendix "Output return and combine": the common layer boundary is
 * retained).  Makes `stream` wait for every invocation of this layer call, then
 * enqueues the read-back of the device status word.  `out` is complete once `stream`
 * has completed.  Implies ffn_flush.  Closes the layer call.
 */
CEP_API int combine(cep_plan* plan, void* stream);

/* Device-side status of the last closed layer call.  Valid after the stream given to
 * combine() has completed (the caller synchronises); before that returns CEP_ERR_STATE.
 * CEP_OK, CEP_ERR_BAD_ROUTING, CEP_ERR_DEVICE_TIMEOUT, or CEP_ERR_CAPACITY (a row index left
 * the scratch slot: more local pairs than the plan was made for; the access was skipped). */
CEP_API int ffn_status(cep_plan* plan);

/*
 * Asynchronous output return (Appendix "Output return and combine": outputs are returned asynchronously,
 * readiness is tracked separately from the layer boundary).  Makes `stream` wait until invocation `inv` of the
 * current layer call has written the output rows of its chunks (ffn_query tells which chunks it holds), so a
 * caller can start consuming or copying those rows before the other invocations finish.  Does not block the host.
 */
CEP_API int ffn_wait_invocation(cep_plan* plan, int32_t inv, void* stream);

/* Number of invocations launched in the current / last layer call. */
CEP_API int ffn_num_invocations(const cep_plan* plan);

/* Trace record of invocation `inv` [host out]. elapsed_ms needs the invocation finished. */
CEP_API int ffn_query(cep_plan* plan, int32_t inv, cep_invocation_info* info);

/*
 * The same record for an earlier layer call: calls_back = 0 is the current (or last) call, 1 the one before,
 * up to 7 for plans made with profile_kernels (other plans keep only the current call: CEP_ERR_ARG).  Lets a
 * harness run several layer calls back to back without a host synchronisation in between and read every call's
 * per-kernel device times afterwards.  pairs_bound and the chunk fields are those of that call.
 */
CEP_API int ffn_query_call(cep_plan* plan, int32_t calls_back, int32_t inv, cep_invocation_info* info);

/*
 * Copy the layout transform's integers of invocation `inv` to [host] arrays (any may be
 * NULL): counts[E], offsets[E+1], padded_offsets[E+1], row_of_pair[n_tokens*k] (physical,
 * tile-aligned row of each pair in batch pair order, -1 if not local), pair_of_row[
 * padded_offsets[E]] (inverse, -1 on padding rows).  Synchronises the invocation's stream.
 * Only meaningful until the invocation's scratch slot is reused (S invocations later).
 */
CEP_API int ffn_debug_export(cep_plan* plan, int32_t inv, int32_t* counts, int32_t* offsets,
                     int32_t* padded_offsets, int32_t* row_of_pair, int32_t* pair_of_row);

/*
 * Use only the first `n` (1..n_streams) compute streams / scratch slots for the following layer calls
 * (round-robin over n instead of n_streams).  Between layer calls only.  A plan starts with all of them.
 */
CEP_API int ffn_set_active_streams(cep_plan* plan, int32_t n);

/* One point of the FFN-throughput profile (the quantity plotted against expert-token count in Section 3.2,
 * "Launch threshold"): every local expert gets the same number of rows. */
typedef struct {
  int32_t rows_per_expert;
  int32_t n_tokens;            /* tokens of the synthetic batch                                   */
  int64_t expert_tokens;       /* N: local (token, expert) pairs of the batch                     */
  float ffn_ms;                /* F(N): median device time of the two expert GEMMs                */
  float layer_ms;              /* median device time of the whole invocation                      */
  float tflops;                /* 6*H*I*N / F(N)                                                  */
  float eta;                   /* tflops / peak of the profile: F(N) = N / (eta(N) * P_peak)      */
} cep_profile_point;

typedef struct {
  float rho;                   /* throughput target given                                         */
  float peak_tflops;           /* best point of the profile (P_peak)                              */
  int64_t theta_pairs;         /* smallest profiled N with eta(N) >= rho                          */
  int32_t theta_rows_per_expert;
  int32_t best_streams;        /* fewest active streams within 2 % of the fastest probe; 0 if not probed */
  int32_t probe_invocations;   /* invocations of theta_pairs each in the stream probe             */
  float stream_ms[16];         /* median completion time of the probe with s+1 active streams; < 0: not run */
} cep_calibration;

/*
 * Launch-threshold calibration (Section 3.2: theta is the smallest profiled expert-token count whose FFN throughput
 * reaches the fraction rho of the best profiled one; Section 3.3, Eq. 2 models FFN latency from the same profile).  Runs the plan's OWN
 * kernels, with the weights it holds, on synthetic routing that gives every local expert rows_per_expert[i] rows
 * (ascending), `reps` timed layer calls per point after two warm-ups, and then probes how many compute streams a
 * chain of theta-sized invocations wants.  Blocks the host until done; not part of the hot path.  Needs a plan
 * made with profile_kernels != 0, loaded weights, no open layer call.  Caller-provided [device] scratch, for
 * T_max = max(rows_per_expert) * n_experts_local / min(top_k, n_experts_local) tokens (T_max <= max_tokens):
 *   tokens        [T_max, H] in the plan's activation format, any finite values (they are only timed)
 *   token_scales  as for ffn_submit_chunk, or NULL for bf16
 *   ids, weights  [T_max, top_k] int32 / fp32, overwritten with the synthetic routing
 *   out           [T_max, H] bf16, overwritten
 * [host] out: points[n_points], *result.  The plan's mode, threshold and active streams are restored on return.
 */
CEP_API int cep_calibrate(cep_plan* plan, float rho, const int32_t* rows_per_expert, int32_t n_points, int32_t reps,
                          const void* tokens, const void* token_scales, int32_t* ids, float* weights, void* out,
                          cep_profile_point* points, cep_calibration* result);

/*
 * The same calibration on the CALLER'S routing: the profile is taken on growing prefixes of one real batch
 * (the first n_tokens[i] tokens of tokens / ids / weights, ascending, each run as one synchronous invocation),
 * so theta reflects the expert skew the layer actually sees: with a skewed router the unpopular experts of a
 * batch get far fewer rows than the mean, and an invocation reaches a given throughput only at a larger
 * expert-token count than uniform routing suggests.  points[i].expert_tokens is the number of local
 * (token, expert) pairs in that prefix, rows_per_expert their mean per local expert.  No stream probe
 * (best_streams = 0).  Same requirements as cep_calibrate; ids and weights are read, not written.
 */
CEP_API int cep_calibrate_routed(cep_plan* plan, float rho, const int32_t* n_tokens, int32_t n_points, int32_t reps,
                                 const void* tokens, const void* token_scales, const int32_t* ids, const float* weights,
                                 void* out, cep_profile_point* points, cep_calibration* result);

/* Total kernel launches this plan has issued (layout, GEMM, combine, prepack). */
CEP_API int64_t cep_kernel_launches(const cep_plan* plan);

/* Destroys streams, events and the host object.  Synchronises the plan's streams. */
CEP_API int moe_plan_destroy(cep_plan* plan);

/* Static or plan-owned string describing the last error on this plan (or the last
 * plan-less error when plan is NULL). */
CEP_API const char* cep_last_error(const cep_plan* plan);

/*
 * layout_indices_noalloc: the integer half of the layout transform (per-expert counts, offsets,
 * tile-aligned offsets, the stable row of every pair and the inverse map) for callers that cannot
 * hand the library any scratch memory.  The paper has no counterpart: it exists for users who run
 * inside a process whose memory pool already owns the device (an extra cudaMalloc would fail or eat
 * into the KV cache) or who may not allocate on a latency-critical path.  It needs no plan and no
 * workspace and calls no allocator: its scratch is a fixed array inside the library, about 1 MiB
 * that every GPU loading the library holds until exit.
 *   topk_ids        [device] int32 [n_tokens, top_k] global ids (one contiguous batch)
 *   counts          [device] out int32 [E]
 *   offsets         [device] out int32 [E+1]
 *   padded_offsets  [device] out int32 [E+1]   group starts rounded up to CEP_ROW_ALIGN
 *   row_of_pair     [device] out int32 [n_tokens*top_k]  tile-aligned row of each pair, -1 if not local
 *   pair_of_row     [device] out int32 [pair_of_row_capacity]; entries of real rows are written,
 *                   padding rows are left untouched; capacity >= padded_offsets[E]
 *   status          [device] out int32 [2] or NULL: [0] != 0 an id was outside [0, n_experts_global),
 *                   [1] != 0 a row did not fit pair_of_row_capacity
 * Limits: n_experts_local <= 1024 and ceil(n_tokens*top_k / 2048) * n_experts_local <= 262144;
 * larger requests return CEP_ERR_CAPACITY.  The work is enqueued on `stream`; outputs are ready when
 * it completes.  The first call on each device looks up the array's device address: a blocking
 * runtime query that also loads the library's device code onto that GPU if nothing has yet, so make
 * that first call once at start-up, before any stream capture and off any latency-critical path.
 * All calls share the one array,
 * which keeps the previous call's contents (the part that must start at zero is cleared by every
 * call): calls whose GPU work may overlap must be ordered by the caller or they race.
 */
CEP_API int layout_indices_noalloc(const int32_t* topk_ids, int32_t n_tokens, int32_t top_k,
                                   int32_t n_experts_local, int32_t n_experts_global, int32_t* counts,
                                   int32_t* offsets, int32_t* padded_offsets, int32_t* row_of_pair,
                                   int32_t* pair_of_row, int32_t pair_of_row_capacity, int32_t* status,
                                   void* stream);

/*
 * Host-only helpers exported for CPU tests of the index arithmetic the kernels use.
 * cep_debug_decode_tile: maps a linear tile index to (expert, m_block, n_block) given the
 * per-expert m-tile prefix [E+1], the number of n blocks and the n blocks per L2-resident chunk;
 * returns 0 or CEP_ERR_ARG.
 * cep_debug_schedule: replays the host scheduler on a list of per-chunk pair counts and
 * writes, per chunk position, the invocation it lands in; returns the invocation count.
 */
CEP_API int cep_debug_decode_tile(const int32_t* tile_prefix, int32_t n_experts, int32_t n_blocks_n,
                          int32_t n_group, int32_t tile, int32_t* expert, int32_t* m_block,
                          int32_t* n_block);
/*
 * Test hook for failure detection (no counterpart in the paper).  Every wait inside the kernels is
 * bounded; this launches, on `stream`, one thread block that waits with the same routine on a barrier
 * nothing signals.  After limit_ms (1..1000) the wait gives up, the device status word records it and the
 * kernel exits normally.  Call between ffn_begin and combine and pass the same stream to combine:
 * ffn_status() then returns CEP_ERR_DEVICE_TIMEOUT, and the next layer call starts clean.
 */
CEP_API int cep_debug_wait_timeout(cep_plan* plan, int32_t limit_ms, void* stream);
/*
 * Out-of-bounds tripwire for plans made with debug_checks (no counterpart in the paper): synchronises
 * the plan's streams and compares every guard gap of the workspace with the pattern written at moe_plan.
 * n_damaged [host out] = number of gaps that changed; 0 means no kernel wrote past the end of a region.
 */
CEP_API int cep_debug_check_guards(cep_plan* plan, int32_t* n_damaged);
CEP_API int cep_debug_schedule(const int64_t* pairs, int32_t n_chunks, int32_t mode, int64_t theta,
                       int32_t* invocation_of_chunk);

#ifdef __cplusplus
}
#endif
#endif /* CASCADE_FFN_H_ */
