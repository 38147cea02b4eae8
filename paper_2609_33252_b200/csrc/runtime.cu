// Host runtime of the streamFFN library: plan object, workspace carving, the streamFFN
// accumulator (threshold batching, final flush, round-robin streams; Section 3.2) and the
// C ABI declared in include/cascade_ffn.h.  Host code only enqueues; it never waits for
// the device except in ffn_debug_export / ffn_query / moe_plan_destroy.
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <algorithm>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>
#include <nvtx3/nvToolsExtCudaRt.h>

#include "cep_common.h"
#include "gemm_tcgen05.h"

using namespace cep;

namespace {

thread_local char g_error[256] = "";          // last error of a call that had no plan to record it in
constexpr int kGuardByte = 0xA5;
constexpr size_t kStatusBlockBytes = 256;        // one status block (kStWords int32) per layer-call parity
constexpr int kTraceCalls = 8;                   // profile_kernels: layer calls whose per-kernel events are kept

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Slot {
  LayoutPtrs lp;
  uint8_t* xp; void* xp_scales;
  uint8_t* act; void* act_scales;
  uint8_t* y;
  GemmTensorMap tm_a1, tm_a2;
  GemmTensorMap tm_o1, tm_o2;                   // fp8: the intermediate and the down-projection output as store targets
  GemmTensorMap tm_sfa1, tm_sfa2;               // microscaling: scale atoms of the two activation operands
};

struct Invocation {
  int first_pos, n_chunks, slot, n_tokens;
  int64_t pairs_bound;
  cudaEvent_t start, done;
  cudaEvent_t mark[4];          // after layout, after GEMM1, after GEMM2, after the index kernels (profile_kernels)
  bool profiled;
};

struct PendingChunk {
  ChunkDesc d;
  int64_t pairs;
  int chunk_id;
};

// The launch rule, shared by the live path and cep_debug_schedule.
bool should_launch(int mode, int64_t pending_pairs, int pending_chunks, int64_t theta) {
  if (pending_chunks <= 0) return false;
  if (pending_chunks >= kMaxChunksPerInv) return true;
  if (mode == CEP_MODE_ASYNC) return true;
  if (mode == CEP_MODE_STREAMFFN) return pending_pairs >= theta;
  return false;                                   // CEP_MODE_SYNC: only at flush
}

struct Layout {                                   // byte offsets inside the workspace
  size_t status;
  size_t slot0, slot_bytes;
  size_t counts, offsets, padded, tile_prefix, sched, block_base, row_of_pair, pair_of_row, src_row, xp, xp_scales,
      act, act_scales, y;                         // offsets inside a slot
  size_t total;
  int cap_rows, n_seg_max;
  size_t guard;                                   // bytes of poisoned gap after every region (debug_checks)
  std::vector<size_t> guard_offsets;              // offsets inside a slot of those gaps
};

int validate(const cep_config* c, const char** why) {
  *why = nullptr;
  if (!c) { *why = "config is NULL"; return CEP_ERR_ARG; }
  if (c->dtype != CEP_BF16 && c->dtype != CEP_FP8_E4M3_BLOCK128 && c->dtype != CEP_MXFP4_E4M3) {
    *why = "unknown dtype"; return CEP_ERR_ARG; }
  if (c->hidden <= 0 || c->inter <= 0 || c->hidden % 128 || c->inter % 128) {
    *why = "hidden and inter must be positive multiples of 128"; return CEP_ERR_ARG; }
  if (c->n_experts_local <= 0 || c->n_experts_local > 1024 || c->n_experts_global < c->n_experts_local) {
    *why = "need 0 < n_experts_local <= min(1024, n_experts_global)"; return CEP_ERR_ARG; }
  if (c->top_k <= 0 || c->top_k > 32 || c->top_k > c->n_experts_global) { *why = "need 0 < top_k <= 32"; return CEP_ERR_ARG; }
  if (c->max_tokens <= 0 || c->max_chunks <= 0) { *why = "max_tokens and max_chunks must be positive"; return CEP_ERR_ARG; }
  if ((long long)c->max_tokens * c->top_k > (1ll << 30)) { *why = "max_tokens*top_k exceeds 2^30"; return CEP_ERR_ARG; }
  if (c->mode < CEP_MODE_SYNC || c->mode > CEP_MODE_STREAMFFN) { *why = "unknown mode"; return CEP_ERR_ARG; }
  if (c->n_streams < 1 || c->n_streams > 16) { *why = "n_streams must be in 1..16"; return CEP_ERR_ARG; }
  if (c->threshold_pairs < 0) { *why = "threshold_pairs must be >= 0"; return CEP_ERR_ARG; }
  if (c->gemm_impl < CEP_GEMM_TCGEN05 || c->gemm_impl > CEP_GEMM_TCGEN05_1CTA) { *why = "unknown gemm_impl"; return CEP_ERR_ARG; }
  if (c->gather_a && (c->dtype != CEP_BF16 || c->gemm_impl != CEP_GEMM_TCGEN05)) {
    *why = "gather_a is built for bf16 on the CTA-pair tensor-core kernel only"; return CEP_ERR_UNSUPPORTED; }
  return CEP_OK;
}

Layout make_layout(const cep_config& c) {
  Layout L{};
  const bool fp8 = dtype_is_bytes(c.dtype);       // one-byte codes + 4 bytes of scales per 128 elements
  const size_t elt = fp8 ? 1 : 2;
  const long long max_pairs = (long long)c.max_tokens * c.top_k;
  const long long pad_groups = c.n_experts_local < max_pairs ? c.n_experts_local : max_pairs;
  L.cap_rows = (int)align_up((size_t)(max_pairs + (kRowAlign - 1) * pad_groups), kRowAlign);
  L.n_seg_max = (int)((max_pairs + kSegPairs - 1) / kSegPairs);
  if (L.n_seg_max < 1) L.n_seg_max = 1;
  const size_t E = c.n_experts_local, A = 256;
  L.guard = c.debug_checks ? 1024 : 0;
  size_t o = 0;
  // every region ends on an A boundary; with debug_checks a poisoned gap follows it
  auto region = [&](size_t& field, size_t bytes, size_t align) {
    o = align_up(o, align);
    field = o;
    o = align_up(o + bytes, A);
    if (L.guard) { L.guard_offsets.push_back(o); o += L.guard; }
  };
  region(L.counts, E * 4, A);
  region(L.offsets, (E + 1) * 4, A);
  region(L.padded, (E + 1) * 4, A);
  region(L.tile_prefix, (E + 1) * 4, A);
  region(L.sched, 2 * 4, A);
  region(L.block_base, (size_t)L.n_seg_max * E * 4, A);
  region(L.row_of_pair, (size_t)max_pairs * 4, A);
  region(L.pair_of_row, (size_t)L.cap_rows * 4, A);
  // gather_a plans keep no permuted copy of the tokens: GEMM1 reads them where the caller put them
  region(L.src_row, c.gather_a ? (size_t)L.cap_rows * 4 : 0, A);
  region(L.xp, c.gather_a ? 0 : (size_t)L.cap_rows * c.hidden * elt, 1024);
  region(L.xp_scales, fp8 ? (size_t)L.cap_rows * (c.hidden / kQuantBlock) * 4 : 0, A);
  region(L.act, (size_t)L.cap_rows * c.inter * elt, 1024);
  region(L.act_scales, fp8 ? (size_t)L.cap_rows * (c.inter / kQuantBlock) * 4 : 0, A);
  region(L.y, (size_t)L.cap_rows * c.hidden * 2, 1024);
  o = align_up(o, 1024);
  L.slot_bytes = o;
  L.status = 0;
  L.slot0 = 1024;
  L.total = L.slot0 + L.slot_bytes * c.n_streams;
  return L;
}

struct PackedLayout { size_t w13, w2, s13, s2, total; };
PackedLayout make_packed_layout(const cep_config& c) {
  PackedLayout P{};
  const bool fp8 = c.dtype == CEP_FP8_E4M3_BLOCK128, mx = c.dtype == CEP_MXFP4_E4M3;
  const size_t elt = fp8 ? 1 : 2, E = c.n_experts_local, H = c.hidden, I = c.inter;
  size_t o = 0;
  // microscaling: two e2m1 codes per byte, one scale byte per 32 elements
  P.w13 = o; o = align_up(o + (mx ? E * 2 * I * H / 2 : E * 2 * I * H * elt), 1024);
  P.w2 = o; o = align_up(o + (mx ? E * H * I / 2 : E * H * I * elt), 1024);
  P.s13 = o; o = align_up(o + (mx ? E * 2 * I * H / kMxBlock : fp8 ? E * (2 * I / kQuantBlock) * (H / kQuantBlock) * 4 : 0), 1024);
  P.s2 = o; o = align_up(o + (mx ? E * H * I / kMxBlock : fp8 ? E * (H / kQuantBlock) * (I / kQuantBlock) * 4 : 0), 1024);
  P.total = o;
  return P;
}

}  // namespace

struct cep_plan {
  cep_config cfg;
  Layout L;
  uint8_t* ws;
  int n_sms;
  int active_streams;                           // round-robin over the first this-many streams / slots
  std::vector<cudaStream_t> streams;
  std::vector<Slot> slots;
  std::vector<cudaEvent_t> ready_evt;           // per chunk position
  std::vector<Invocation> inv;                  // the current (or last) layer call
  // Event pools: one set per possible invocation of a layer call.  With profile_kernels there are kTraceCalls
  // sets, used in turn, and `past` keeps the records of the calls before the current one, so per-kernel device
  // times of several back-to-back layer calls can be read after they have all run (ffn_query_call).
  std::vector<cudaEvent_t> inv_start, inv_done;
  std::vector<cudaEvent_t> inv_mark;            // 4 per possible invocation (profile_kernels)
  std::vector<Invocation> past[kTraceCalls];
  int trace_sets;                               // 1, or kTraceCalls with profile_kernels
  long long call_index;                         // layer calls opened so far
  // Two status blocks, used by alternate layer calls: a call clears its block without waiting for the previous
  // call's read-back (a small device-to-host copy that can sit behind the caller's own output copies in the copy
  // engine's queue), only for the read-back of the call before that.
  cudaEvent_t begin_evt, readback_evt[2], weights_evt;
  int status_idx;                               // block of the current / last layer call
  bool readback_pending[2];
  bool have_weights, layer_open, flushed, ever_closed;
  uint8_t* w13p; uint8_t* w2p;
  void* s13p; void* s2p;                        // fp8, mxfp4: packed weight scales
  GemmTensorMap tm_b1, tm_b2;
  GemmTensorMap tm_sfb1, tm_sfb2;               // mxfp4: scale atoms of the two weight operands
  // gather_a: the layer call's token tensor [n_tokens_total, H] as GEMM1's activation operand (one-row boxes);
  // its base is fixed by the first chunk of the call, every later chunk must be a row slice of the same tensor
  GemmTensorMap tm_src;
  const uint8_t* src_base;
  // current layer call
  void* out; const void* addend; int n_tokens_total, n_chunks_expected, n_submitted, tokens_submitted;
  std::vector<char> chunk_seen;
  std::vector<PendingChunk> pending;
  int64_t pending_pairs;
  int32_t* host_status;                         // pinned, two blocks of kStWords
  int64_t launches;
  bool nvtx;                                    // CEP_NVTX=1 when the plan was made: ranges for timeline tools
  nvtxRangeId_t call_range;
  char err[256];
};

namespace {

int fail(cep_plan* p, int code, const char* fmt, ...) {
  char* dst = p ? p->err : g_error;
  va_list ap; va_start(ap, fmt); vsnprintf(dst, 256, fmt, ap); va_end(ap);
  return code;
}
#define CUDA_TRY(p, call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) \
  return fail((p), CEP_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_)); } while (0)

// A named range on the calling thread for as long as the object lives (only with CEP_NVTX=1).
struct HostRange {
  bool on;
  HostRange(const cep_plan* p, const char* fmt, long long a, long long b, long long c) : on(p->nvtx) {
    if (!on) return;
    char name[96];
    snprintf(name, sizeof name, fmt, a, b, c);
    nvtxRangePushA(name);
  }
  ~HostRange() { if (on) nvtxRangePop(); }
};

int launch_invocation(cep_plan* p) {
  if (p->pending.empty()) return CEP_OK;
  const cep_config& c = p->cfg;
  const int idx = (int)p->inv.size();
  HostRange range(p, "cep invocation %lld: %lld chunks, %lld expert tokens", idx, (long long)p->pending.size(),
                  (long long)p->pending_pairs);
  if (idx >= c.max_chunks) return fail(p, CEP_ERR_CAPACITY, "more invocations than max_chunks");
  const int ev = (int)(p->call_index % p->trace_sets) * c.max_chunks + idx;      // this call's set of events
  const int slot_i = idx % p->active_streams;
  Slot& sl = p->slots[slot_i];
  cudaStream_t st = p->streams[slot_i];
  BatchDesc batch{};
  int tok = 0;
  const int first_pos = p->n_submitted - (int)p->pending.size();
  for (size_t i = 0; i < p->pending.size(); ++i) {
    batch.chunk[i] = p->pending[i].d;
    batch.chunk[i].token_base = tok;
    tok += p->pending[i].d.n_tokens;
  }
  batch.n_chunks = (int)p->pending.size();
  batch.n_tokens = tok;
  // nothing is launched for a batch the scratch slot was not carved for
  if (tok > c.max_tokens || ((long long)tok * c.top_k + kSegPairs - 1) / kSegPairs > p->L.n_seg_max)
    return fail(p, CEP_ERR_CAPACITY, "a batch of %d tokens exceeds the plan's max_tokens = %d", tok, c.max_tokens);
  CUDA_TRY(p, cudaStreamWaitEvent(st, p->begin_evt, 0));
  CUDA_TRY(p, cudaStreamWaitEvent(st, p->weights_evt, 0));
  for (size_t i = 0; i < p->pending.size(); ++i) CUDA_TRY(p, cudaStreamWaitEvent(st, p->ready_evt[first_pos + (int)i], 0));
  Invocation iv{first_pos, batch.n_chunks, slot_i, tok, p->pending_pairs, p->inv_start[ev], p->inv_done[ev],
                {nullptr, nullptr, nullptr, nullptr}, false};
  const bool prof = c.profile_kernels != 0 && tok > 0;
  if (prof) { for (int m = 0; m < 4; ++m) iv.mark[m] = p->inv_mark[4 * ev + m]; iv.profiled = true; }
  CUDA_TRY(p, cudaEventRecord(iv.start, st));
  if (tok > 0) {
    const long long n_pairs = (long long)tok * c.top_k;
    const int n_seg = (int)((n_pairs + kSegPairs - 1) / kSegPairs);
    CUDA_TRY(p, launch_layout(batch, c, sl.lp, sl.xp, sl.xp_scales, p->L.cap_rows, n_seg, st, prof ? iv.mark[3] : nullptr,
                              &p->launches));
    if (prof) CUDA_TRY(p, cudaEventRecord(iv.mark[0], st));
    const bool fp8 = c.dtype == CEP_FP8_E4M3_BLOCK128, mx = c.dtype == CEP_MXFP4_E4M3;
    const long long groups = c.n_experts_local < n_pairs ? c.n_experts_local : n_pairs;
    const long long m_tiles_bound = (n_pairs + (kRowAlign - 1) * groups + kRowAlign - 1) / kRowAlign;
    GemmProblem g1{c.hidden, 2 * c.inter, c.n_experts_local, 1, c.inter, p->L.cap_rows, fp8 || mx};
    GemmProblem g2{c.inter, c.hidden, c.n_experts_local, 0, c.hidden, p->L.cap_rows, fp8 || mx};
    if (c.gemm_impl == CEP_GEMM_SIMT) {
      CUDA_TRY(p, launch_gemm_simt(g1, sl.xp, p->w13p, sl.act, sl.lp, st, &p->launches));
      if (prof) CUDA_TRY(p, cudaEventRecord(iv.mark[1], st));
      CUDA_TRY(p, launch_gemm_simt(g2, sl.act, p->w2p, sl.y, sl.lp, st, &p->launches));
    } else if (mx) {
      const int bn = gemm_tile_cols();
      const long long pair_bound = (m_tiles_bound + groups + 1) / 2;
      const long long t1 = pair_bound * (g1.N / bn), t2 = pair_bound * (g2.N / bn);
      CUDA_TRY(p, launch_gemm_mx(g1, sl.tm_a1, p->tm_b1, sl.tm_sfa1, p->tm_sfb1, sl.act, sl.act_scales, sl.lp,
                                 (int)(t1 > (1 << 30) ? (1 << 30) : t1), p->n_sms, st, &p->launches));
      if (prof) CUDA_TRY(p, cudaEventRecord(iv.mark[1], st));
      CUDA_TRY(p, launch_gemm_mx(g2, sl.tm_a2, p->tm_b2, sl.tm_sfa2, p->tm_sfb2, sl.y, nullptr, sl.lp,
                                 (int)(t2 > (1 << 30) ? (1 << 30) : t2), p->n_sms, st, &p->launches));
    } else if (fp8) {
      const int pair = c.gemm_impl == CEP_GEMM_TCGEN05 ? 1 : 0;
      const int bn = gemm_tile_cols();
      const long long m_bound = pair ? (m_tiles_bound + groups + 1) / 2 : m_tiles_bound;
      const long long t1 = m_bound * ((g1.N + bn - 1) / bn), t2 = m_bound * ((g2.N + bn - 1) / bn);
      CUDA_TRY(p, launch_gemm_fp8(g1, pair, sl.tm_a1, p->tm_b1, sl.tm_o1, (const float*)sl.xp_scales, (const float*)p->s13p, sl.act,
                                  (float*)sl.act_scales, sl.lp,
                                  (int)(t1 > (1 << 30) ? (1 << 30) : t1), p->n_sms, st, &p->launches));
      if (prof) CUDA_TRY(p, cudaEventRecord(iv.mark[1], st));
      CUDA_TRY(p, launch_gemm_fp8(g2, pair, sl.tm_a2, p->tm_b2, sl.tm_o2, (const float*)sl.act_scales, (const float*)p->s2p, sl.y, nullptr, sl.lp,
                                  (int)(t2 > (1 << 30) ? (1 << 30) : t2), p->n_sms, st, &p->launches));
    } else if (c.gemm_impl == CEP_GEMM_TCGEN05) {
      const int bn = gemm_tile_cols();
      const long long pair_bound = (m_tiles_bound + groups + 1) / 2;
      const long long t1 = pair_bound * ((g1.N + bn - 1) / bn), t2 = pair_bound * ((g2.N + bn - 1) / bn);
      CUDA_TRY(p, launch_gemm_tcgen05_pair(g1, c.gather_a ? p->tm_src : sl.tm_a1, p->tm_b1, sl.act, sl.lp,
                                           c.gather_a ? sl.lp.src_row : nullptr, (int)(t1 > (1 << 30) ? (1 << 30) : t1),
                                           p->n_sms, st, &p->launches));
      if (prof) CUDA_TRY(p, cudaEventRecord(iv.mark[1], st));
      CUDA_TRY(p, launch_gemm_tcgen05_pair(g2, sl.tm_a2, p->tm_b2, sl.y, sl.lp, nullptr, (int)(t2 > (1 << 30) ? (1 << 30) : t2),
                                           p->n_sms, st, &p->launches));
    } else {
      const int bn = gemm_tile_cols();
      const long long t1 = m_tiles_bound * ((g1.N + bn - 1) / bn), t2 = m_tiles_bound * ((g2.N + bn - 1) / bn);
      CUDA_TRY(p, launch_gemm_tcgen05(g1, sl.tm_a1, p->tm_b1, sl.act, sl.lp, (int)(t1 > (1 << 30) ? (1 << 30) : t1),
                                      p->n_sms, st, &p->launches));
      if (prof) CUDA_TRY(p, cudaEventRecord(iv.mark[1], st));
      CUDA_TRY(p, launch_gemm_tcgen05(g2, sl.tm_a2, p->tm_b2, sl.y, sl.lp, (int)(t2 > (1 << 30) ? (1 << 30) : t2),
                                      p->n_sms, st, &p->launches));
    }
    if (prof) CUDA_TRY(p, cudaEventRecord(iv.mark[2], st));
    CUDA_TRY(p, launch_combine(batch, c, sl.lp, sl.y, p->addend, p->out, st, &p->launches));
  }
  CUDA_TRY(p, cudaEventRecord(iv.done, st));
  p->inv.push_back(iv);
  p->pending.clear();
  p->pending_pairs = 0;
  return CEP_OK;
}

}  // namespace

extern "C" {

const char* cep_last_error(const cep_plan* plan) { return plan ? plan->err : g_error; }

int moe_plan_workspace_bytes(const cep_config* cfg, size_t* bytes) {
  const char* why;
  int rc = validate(cfg, &why);
  if (rc) return fail(nullptr, rc, "%s", why);
  if (!bytes) return fail(nullptr, CEP_ERR_ARG, "bytes is NULL");
  *bytes = make_layout(*cfg).total;
  return CEP_OK;
}

int moe_packed_weight_bytes(const cep_config* cfg, size_t* bytes) {
  const char* why;
  int rc = validate(cfg, &why);
  if (rc) return fail(nullptr, rc, "%s", why);
  if (!bytes) return fail(nullptr, CEP_ERR_ARG, "bytes is NULL");
  *bytes = make_packed_layout(*cfg).total;
  return CEP_OK;
}

int moe_plan(const cep_config* cfg, void* workspace, size_t workspace_bytes, cep_plan** out) {
  const char* why;
  int rc = validate(cfg, &why);
  if (rc) return fail(nullptr, rc, "%s", why);
  if (!out) return fail(nullptr, CEP_ERR_ARG, "out is NULL");
  *out = nullptr;
  if (!workspace) return fail(nullptr, CEP_ERR_ARG, "workspace is NULL");
  if (cfg->dtype == CEP_FP8_E4M3_BLOCK128) {
    if (cfg->gemm_impl == CEP_GEMM_SIMT)
      return fail(nullptr, CEP_ERR_UNSUPPORTED, "block-scaled fp8 runs on the tensor-core kernels only");
    if (cfg->hidden % 256) return fail(nullptr, CEP_ERR_ARG, "fp8 needs hidden to be a multiple of 256");
  }
  if (cfg->dtype == CEP_MXFP4_E4M3) {
    if (cfg->gemm_impl != CEP_GEMM_TCGEN05)
      return fail(nullptr, CEP_ERR_UNSUPPORTED, "microscaling operands run on the CTA-pair tensor-core kernel only");
    if (cfg->hidden % 256) return fail(nullptr, CEP_ERR_ARG, "mxfp4 needs hidden to be a multiple of 256");
  }
  Layout L = make_layout(*cfg);
  if (workspace_bytes < L.total) return fail(nullptr, CEP_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, L.total);
  if (reinterpret_cast<uintptr_t>(workspace) % 256) return fail(nullptr, CEP_ERR_WORKSPACE, "workspace must be 256-byte aligned");
  cep_plan* p = new (std::nothrow) cep_plan();
  if (!p) return fail(nullptr, CEP_ERR_ARG, "out of host memory");
  p->cfg = *cfg; p->L = L; p->ws = static_cast<uint8_t*>(workspace);
  p->err[0] = 0; p->launches = 0; p->active_streams = cfg->n_streams;
  p->have_weights = p->layer_open = p->flushed = p->ever_closed = false;
  p->readback_pending[0] = p->readback_pending[1] = false; p->status_idx = 0;
  p->trace_sets = cfg->profile_kernels ? kTraceCalls : 1; p->call_index = -1;
  p->host_status = nullptr; p->begin_evt = p->readback_evt[0] = p->readback_evt[1] = p->weights_evt = nullptr;
  p->out = nullptr; p->addend = nullptr; p->pending_pairs = 0; p->n_submitted = 0;
  const char* nvtx_env = getenv("CEP_NVTX");
  p->nvtx = nvtx_env && nvtx_env[0] && nvtx_env[0] != '0'; p->call_range = 0;
  int dev = 0;
#define PLAN_TRY(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { \
    fail(nullptr, CEP_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_)); moe_plan_destroy(p); return CEP_ERR_CUDA; } } while (0)
  PLAN_TRY(cudaGetDevice(&dev));
  PLAN_TRY(cudaDeviceGetAttribute(&p->n_sms, cudaDevAttrMultiProcessorCount, dev));
  PLAN_TRY(cudaHostAlloc(reinterpret_cast<void**>(&p->host_status), 2 * kStWords * sizeof(int32_t), cudaHostAllocDefault));
  memset(p->host_status, 0, 2 * kStWords * sizeof(int32_t));
  PLAN_TRY(cudaEventCreateWithFlags(&p->begin_evt, cudaEventDisableTiming));
  PLAN_TRY(cudaEventCreateWithFlags(&p->readback_evt[0], cudaEventDisableTiming));
  PLAN_TRY(cudaEventCreateWithFlags(&p->readback_evt[1], cudaEventDisableTiming));
  PLAN_TRY(cudaEventCreateWithFlags(&p->weights_evt, cudaEventDisableTiming));
  for (int s = 0; s < cfg->n_streams; ++s) {
    cudaStream_t st;
    PLAN_TRY(cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking));
    p->streams.push_back(st);
    if (p->nvtx) { char name[32]; snprintf(name, sizeof name, "cep slot %d", s); nvtxNameCudaStreamA(st, name); }
  }
  for (int i = 0; i < cfg->max_chunks; ++i) {
    cudaEvent_t e;
    PLAN_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming)); p->ready_evt.push_back(e);
  }
  for (int i = 0; i < cfg->max_chunks * p->trace_sets; ++i) {
    cudaEvent_t e;
    PLAN_TRY(cudaEventCreate(&e)); p->inv_start.push_back(e);
    PLAN_TRY(cudaEventCreate(&e)); p->inv_done.push_back(e);
    if (cfg->profile_kernels)
      for (int m = 0; m < 4; ++m) { PLAN_TRY(cudaEventCreate(&e)); p->inv_mark.push_back(e); }
  }
  const bool mx = cfg->dtype == CEP_MXFP4_E4M3;
  const int elt = dtype_is_bytes(cfg->dtype) ? 1 : 2;
  for (int s = 0; s < cfg->n_streams; ++s) {
    uint8_t* b = p->ws + L.slot0 + L.slot_bytes * s;
    Slot sl{};
    sl.lp.counts = reinterpret_cast<int32_t*>(b + L.counts);
    sl.lp.offsets = reinterpret_cast<int32_t*>(b + L.offsets);
    sl.lp.padded_offsets = reinterpret_cast<int32_t*>(b + L.padded);
    sl.lp.tile_prefix = reinterpret_cast<int32_t*>(b + L.tile_prefix);
    sl.lp.block_base = reinterpret_cast<int32_t*>(b + L.block_base);
    sl.lp.row_of_pair = reinterpret_cast<int32_t*>(b + L.row_of_pair);
    sl.lp.pair_of_row = reinterpret_cast<int32_t*>(b + L.pair_of_row);
    sl.lp.src_row = cfg->gather_a ? reinterpret_cast<int32_t*>(b + L.src_row) : nullptr;
    sl.lp.status = reinterpret_cast<int32_t*>(p->ws + L.status);
    sl.lp.sched = reinterpret_cast<int32_t*>(b + L.sched);
    sl.xp = b + L.xp; sl.xp_scales = b + L.xp_scales;
    sl.act = b + L.act; sl.act_scales = b + L.act_scales;
    sl.y = b + L.y;
    if (cfg->gemm_impl != CEP_GEMM_SIMT) {
      int r1 = cfg->gather_a ? 0 : make_operand_map(&sl.tm_a1, sl.xp, elt, cfg->hidden, L.cap_rows, 0, gemm_tile_rows());
      int r2 = make_operand_map(&sl.tm_a2, sl.act, elt, cfg->inter, L.cap_rows, 0, gemm_tile_rows());
      if (cfg->dtype == CEP_FP8_E4M3_BLOCK128 && !r1 && !r2) {
        r1 = make_store_map(&sl.tm_o1, sl.act, 1, cfg->inter, L.cap_rows);
        r2 = make_store_map(&sl.tm_o2, sl.y, 2, cfg->hidden, L.cap_rows);
      }
      if (mx && !r1 && !r2) {
        r1 = make_mx_sf_map(&sl.tm_sfa1, sl.xp_scales, (long long)(L.cap_rows / kRowAlign) * (cfg->hidden / 128), kSfAtomBytes);
        r2 = make_mx_sf_map(&sl.tm_sfa2, sl.act_scales, (long long)(L.cap_rows / kRowAlign) * (cfg->inter / 128), kSfAtomBytes);
      }
      if (r1 || r2) {
        fail(nullptr, CEP_ERR_CUDA, "cuTensorMapEncodeTiled for the activation operands failed (%d, %d)", r1, r2);
        moe_plan_destroy(p);
        return CEP_ERR_CUDA;
      }
    }
    p->slots.push_back(sl);
  }
  if (L.guard) PLAN_TRY(cudaMemsetAsync(p->ws, kGuardByte, L.total, p->streams[0]));   // gaps keep this pattern
  // status word starts clean
  PLAN_TRY(cudaMemsetAsync(p->ws + L.status, 0, 2 * kStatusBlockBytes, p->streams[0]));
  PLAN_TRY(cudaEventRecord(p->begin_evt, p->streams[0]));
  PLAN_TRY(cudaEventRecord(p->weights_evt, p->streams[0]));
#undef PLAN_TRY
  *out = p;
  return CEP_OK;
}

int moe_load_weights(cep_plan* p, const void* w_gate, const void* w_up, const void* w_down, const void* s_gate,
                     const void* s_up, const void* s_down, void* packed, size_t packed_bytes, void* stream) {
  if (!p) return fail(nullptr, CEP_ERR_ARG, "plan is NULL");
  if (!w_gate || !w_up || !w_down || !packed) return fail(p, CEP_ERR_ARG, "a weight pointer is NULL");
  if (p->layer_open) return fail(p, CEP_ERR_STATE, "weights cannot change while a layer call is open");
  const cep_config& c = p->cfg;
  const bool fp8 = c.dtype == CEP_FP8_E4M3_BLOCK128, mx = c.dtype == CEP_MXFP4_E4M3;
  if ((fp8 || mx) && (!s_gate || !s_up || !s_down)) return fail(p, CEP_ERR_ARG, "quantised weights need their scale tensors");
  PackedLayout P = make_packed_layout(c);
  if (packed_bytes < P.total) return fail(p, CEP_ERR_WORKSPACE, "packed buffer has %zu bytes, %zu needed", packed_bytes, P.total);
  if (reinterpret_cast<uintptr_t>(packed) % 256) return fail(p, CEP_ERR_WORKSPACE, "packed buffer must be 256-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  p->w13p = static_cast<uint8_t*>(packed) + P.w13;
  p->w2p = static_cast<uint8_t*>(packed) + P.w2;
  p->s13p = static_cast<uint8_t*>(packed) + P.s13;
  p->s2p = static_cast<uint8_t*>(packed) + P.s2;
  if (mx) {
    CUDA_TRY(p, launch_prepack_mx(c, w_gate, w_up, w_down, s_gate, s_up, s_down, p->w13p, p->w2p, p->s13p, p->s2p, st,
                                  &p->launches));
    CUDA_TRY(p, cudaEventRecord(p->weights_evt, st));
    const int box = gemm_tile_cols() / 2, E = c.n_experts_local;
    int r1 = make_mx_weight_map(&p->tm_b1, p->w13p, c.hidden, 2 * c.inter, E, box);
    int r2 = make_mx_weight_map(&p->tm_b2, p->w2p, c.inter, c.hidden, E, box);
    int r3 = make_mx_sf_map(&p->tm_sfb1, p->s13p, (long long)E * (2 * c.inter / 256) * (c.hidden / 128), 2 * kSfAtomBytes);
    int r4 = make_mx_sf_map(&p->tm_sfb2, p->s2p, (long long)E * (c.hidden / 256) * (c.inter / 128), 2 * kSfAtomBytes);
    if (r1 || r2 || r3 || r4)
      return fail(p, CEP_ERR_CUDA, "cuTensorMapEncodeTiled for the weight operands failed (%d, %d, %d, %d)", r1, r2, r3, r4);
    p->have_weights = true;
    return CEP_OK;
  }
  CUDA_TRY(p, launch_prepack(c, w_gate, w_up, w_down, p->w13p, p->w2p, st, &p->launches));
  if (fp8) CUDA_TRY(p, launch_pack_scales(c, (const float*)s_gate, (const float*)s_up, (const float*)s_down, (float*)p->s13p,
                                          (float*)p->s2p, st, &p->launches));
  CUDA_TRY(p, cudaEventRecord(p->weights_evt, st));
  if (c.gemm_impl != CEP_GEMM_SIMT) {
    const int elt = fp8 ? 1 : 2;
    // the CTA-pair kernel loads half a weight tile per CTA
    const int box = fp8 ? gemm_fp8_box_rows(c.gemm_impl == CEP_GEMM_TCGEN05)
                        : c.gemm_impl == CEP_GEMM_TCGEN05 ? gemm_tile_cols() / 2 : gemm_tile_cols();
    int r1 = make_operand_map(&p->tm_b1, p->w13p, elt, c.hidden, 2 * c.inter, c.n_experts_local, box);
    int r2 = make_operand_map(&p->tm_b2, p->w2p, elt, c.inter, c.hidden, c.n_experts_local, box);
    if (r1 || r2) return fail(p, CEP_ERR_CUDA, "cuTensorMapEncodeTiled for the weight operands failed (%d, %d)", r1, r2);
  }
  p->have_weights = true;
  return CEP_OK;
}

int ffn_begin(cep_plan* p, void* out, int32_t n_tokens_total, int32_t n_chunks_expected) {
  if (!p) return fail(nullptr, CEP_ERR_ARG, "plan is NULL");
  if (p->layer_open) return fail(p, CEP_ERR_STATE, "ffn_begin while a layer call is open (call combine first)");
  if (!p->have_weights) return fail(p, CEP_ERR_STATE, "ffn_begin before moe_load_weights");
  if (!out || n_tokens_total < 0 || n_chunks_expected < 0) return fail(p, CEP_ERR_ARG, "bad ffn_begin arguments");
  if (reinterpret_cast<uintptr_t>(out) % 16) return fail(p, CEP_ERR_ARG, "out must be 16-byte aligned");
  if (n_tokens_total > p->cfg.max_tokens) return fail(p, CEP_ERR_CAPACITY, "%d tokens, plan made for %d", n_tokens_total, p->cfg.max_tokens);
  if (n_chunks_expected > p->cfg.max_chunks) return fail(p, CEP_ERR_CAPACITY, "%d chunks, plan made for %d", n_chunks_expected, p->cfg.max_chunks);
  cudaStream_t s0 = p->streams[0];
  // the previous layer's status read-back must finish before the status word is cleared
  p->status_idx ^= 1;
  const int sb = p->status_idx;
  // the read-back of the call that last used this status block must finish before the block is cleared
  if (p->readback_pending[sb]) CUDA_TRY(p, cudaStreamWaitEvent(s0, p->readback_evt[sb], 0));
  int32_t* status_dev = reinterpret_cast<int32_t*>(p->ws + p->L.status + (size_t)sb * kStatusBlockBytes);
  for (Slot& sl : p->slots) sl.lp.status = status_dev;
  CUDA_TRY(p, cudaMemsetAsync(status_dev, 0, kStWords * sizeof(int32_t), s0));
  CUDA_TRY(p, cudaEventRecord(p->begin_evt, s0));
  p->out = out; p->addend = nullptr; p->n_tokens_total = n_tokens_total; p->n_chunks_expected = n_chunks_expected;
  p->n_submitted = 0; p->tokens_submitted = 0; p->src_base = nullptr;
  p->chunk_seen.assign(n_chunks_expected, 0);
  if (p->call_index >= 0) p->past[p->call_index % kTraceCalls] = p->inv;    // the call that just ended
  p->call_index += 1;
  p->pending.clear(); p->pending_pairs = 0; p->inv.clear();
  p->layer_open = true; p->flushed = false;
  if (p->nvtx) {
    char name[64];
    snprintf(name, sizeof name, "cep layer call %lld: %d tokens", p->call_index, n_tokens_total);
    p->call_range = nvtxRangeStartA(name);
  }
  return CEP_OK;
}

int ffn_submit_chunk(cep_plan* p, int32_t chunk_id, int32_t token_offset, int32_t n_tokens, const void* tokens,
                     const void* token_scales, const int32_t* topk_ids, const float* topk_weights,
                     int64_t n_local_pairs, void* stream) {
  if (!p) return fail(nullptr, CEP_ERR_ARG, "plan is NULL");
  if (!p->layer_open) return fail(p, CEP_ERR_STATE, "ffn_submit_chunk before ffn_begin");
  if (p->flushed) return fail(p, CEP_ERR_STATE, "ffn_submit_chunk after ffn_flush");
  if (chunk_id < 0 || chunk_id >= p->n_chunks_expected) return fail(p, CEP_ERR_ARG, "chunk_id %d outside 0..%d", chunk_id, p->n_chunks_expected - 1);
  if (p->chunk_seen[chunk_id]) return fail(p, CEP_ERR_STATE, "chunk %d submitted twice", chunk_id);
  if (n_tokens < 0 || token_offset < 0) return fail(p, CEP_ERR_ARG, "negative n_tokens or token_offset");
  if ((long long)token_offset + n_tokens > p->n_tokens_total) return fail(p, CEP_ERR_CAPACITY, "chunk %d covers tokens beyond n_tokens_total", chunk_id);
  // chunks cover the layer call's tokens exactly once: together they can never hold more than n_tokens_total
  // (which also keeps every batch within max_tokens, the size the scratch slots were carved for)
  if ((long long)p->tokens_submitted + n_tokens > p->n_tokens_total)
    return fail(p, CEP_ERR_CAPACITY, "chunk %d brings the submitted tokens to %lld, the layer call has %d", chunk_id,
                (long long)p->tokens_submitted + n_tokens, p->n_tokens_total);
  if (n_tokens > 0 && (!tokens || !topk_ids || !topk_weights)) return fail(p, CEP_ERR_ARG, "a chunk pointer is NULL");
  if (reinterpret_cast<uintptr_t>(tokens) % 16) return fail(p, CEP_ERR_ARG, "chunk tokens must be 16-byte aligned");
  const bool fp8 = dtype_is_bytes(p->cfg.dtype);
  if (fp8 && n_tokens > 0 && !token_scales) return fail(p, CEP_ERR_ARG, "quantised chunk without token_scales");
  if (fp8 && reinterpret_cast<uintptr_t>(token_scales) % 4) return fail(p, CEP_ERR_ARG, "token_scales must be 4-byte aligned");
  if (p->cfg.gather_a && n_tokens > 0) {
    // the chunk must be rows token_offset.. of one tensor that holds the whole layer call
    const uint8_t* base = static_cast<const uint8_t*>(tokens) - (size_t)token_offset * p->cfg.hidden * 2;
    if (!p->src_base) {
      if (make_operand_map(&p->tm_src, base, 2, p->cfg.hidden, p->n_tokens_total, 0, 1))
        return fail(p, CEP_ERR_CUDA, "cuTensorMapEncodeTiled for the token tensor failed");
      p->src_base = base;
    } else if (base != p->src_base) {
      return fail(p, CEP_ERR_UNSUPPORTED, "gather_a: chunk %d is not a row slice of the layer call's token tensor", chunk_id);
    }
  }
  const int64_t bound = (int64_t)n_tokens * p->cfg.top_k;
  if (n_local_pairs > bound) return fail(p, CEP_ERR_ARG, "n_local_pairs exceeds n_tokens*top_k");
  const int64_t pairs = n_local_pairs < 0 ? bound : n_local_pairs;
  CUDA_TRY(p, cudaEventRecord(p->ready_evt[p->n_submitted], static_cast<cudaStream_t>(stream)));
  PendingChunk pc{};
  pc.d.tokens = tokens; pc.d.scales = token_scales; pc.d.ids = topk_ids; pc.d.weights = topk_weights;
  pc.d.n_tokens = n_tokens; pc.d.token_offset = token_offset;
  pc.pairs = pairs; pc.chunk_id = chunk_id;
  p->pending.push_back(pc);
  p->pending_pairs += pairs;
  p->chunk_seen[chunk_id] = 1;
  p->n_submitted += 1;
  p->tokens_submitted += n_tokens;
  if (should_launch(p->cfg.mode, p->pending_pairs, (int)p->pending.size(), p->cfg.threshold_pairs)) {
    // Work that would only queue behind a running invocation is not split off: see cep_config::defer_while_busy.
    if (p->cfg.defer_while_busy && p->cfg.mode == CEP_MODE_STREAMFFN && !p->inv.empty() &&
        (int)p->pending.size() < kMaxChunksPerInv && p->pending_pairs < 4 * p->cfg.threshold_pairs) {
      const cudaError_t q = cudaEventQuery(p->inv.back().done);
      if (q == cudaErrorNotReady) { (void)cudaGetLastError(); return CEP_OK; }
      if (q != cudaSuccess) return fail(p, CEP_ERR_CUDA, "cudaEventQuery failed: %s", cudaGetErrorString(q));
    }
    return launch_invocation(p);
  }
  return CEP_OK;
}

int ffn_set_addend(cep_plan* p, const void* addend) {
  if (!p) return fail(nullptr, CEP_ERR_ARG, "plan is NULL");
  if (!p->layer_open) return fail(p, CEP_ERR_STATE, "ffn_set_addend before ffn_begin");
  if (p->n_submitted > 0) return fail(p, CEP_ERR_STATE, "ffn_set_addend after the first chunk was submitted");
  if (addend && reinterpret_cast<uintptr_t>(addend) % 16) return fail(p, CEP_ERR_ARG, "addend must be 16-byte aligned");
  p->addend = addend;
  return CEP_OK;
}

int moe_route(const float* logits, int32_t n_tokens, int32_t n_experts_global, int32_t top_k, int32_t* topk_ids,
              float* topk_weights, void* stream) {
  if (!logits || !topk_ids || !topk_weights) return fail(nullptr, CEP_ERR_ARG, "a router pointer is NULL");
  if (n_tokens < 0 || n_experts_global <= 0 || n_experts_global > 1024 || top_k <= 0 || top_k > 32 || top_k > n_experts_global)
    return fail(nullptr, CEP_ERR_ARG, "router needs 0 < top_k <= min(32, n_experts_global) and n_experts_global <= 1024");
  cudaError_t e = launch_route(logits, n_tokens, n_experts_global, top_k, topk_ids, topk_weights, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fail(nullptr, CEP_ERR_CUDA, "router launch failed: %s", cudaGetErrorString(e));
  return CEP_OK;
}

int ffn_flush(cep_plan* p) {
  if (!p) return fail(nullptr, CEP_ERR_ARG, "plan is NULL");
  if (!p->layer_open) return fail(p, CEP_ERR_STATE, "ffn_flush before ffn_begin");
  p->flushed = true;
  int rc = launch_invocation(p);
  if (rc) return rc;
  if (p->n_submitted < p->n_chunks_expected)
    return fail(p, CEP_ERR_INCOMPLETE, "flush after %d of %d chunks", p->n_submitted, p->n_chunks_expected);
  if (p->tokens_submitted < p->n_tokens_total)
    return fail(p, CEP_ERR_INCOMPLETE, "the chunks cover %d of the layer call's %d tokens", p->tokens_submitted, p->n_tokens_total);
  return CEP_OK;
}

int combine(cep_plan* p, void* stream) {
  if (!p) return fail(nullptr, CEP_ERR_ARG, "plan is NULL");
  if (!p->layer_open) return fail(p, CEP_ERR_STATE, "combine before ffn_begin");
  int rc = CEP_OK;
  if (!p->flushed) { rc = ffn_flush(p); if (rc && rc != CEP_ERR_INCOMPLETE) return rc; }
  else if (p->n_submitted < p->n_chunks_expected)
    rc = fail(p, CEP_ERR_INCOMPLETE, "combine after %d of %d chunks", p->n_submitted, p->n_chunks_expected);
  else if (p->tokens_submitted < p->n_tokens_total)
    rc = fail(p, CEP_ERR_INCOMPLETE, "the chunks cover %d of the layer call's %d tokens", p->tokens_submitted, p->n_tokens_total);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CUDA_TRY(p, cudaStreamWaitEvent(st, p->begin_evt, 0));
  for (const Invocation& iv : p->inv) CUDA_TRY(p, cudaStreamWaitEvent(st, iv.done, 0));
  const int sb = p->status_idx;
  CUDA_TRY(p, cudaMemcpyAsync(p->host_status + sb * kStWords, p->ws + p->L.status + (size_t)sb * kStatusBlockBytes,
                              kStWords * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  CUDA_TRY(p, cudaEventRecord(p->readback_evt[sb], st));
  p->readback_pending[sb] = true; p->ever_closed = true;
  p->layer_open = false;
  if (p->nvtx) nvtxRangeEnd(p->call_range);
  return rc;
}

int ffn_status(cep_plan* p) {
  if (!p) return fail(nullptr, CEP_ERR_ARG, "plan is NULL");
  if (!p->ever_closed || p->layer_open) return fail(p, CEP_ERR_STATE, "no closed layer call to report on");
  const int32_t* hs = p->host_status + p->status_idx * kStWords;
  cudaError_t q = cudaEventQuery(p->readback_evt[p->status_idx]);
  if (q == cudaErrorNotReady) return fail(p, CEP_ERR_STATE, "the stream given to combine has not completed yet");
  if (q != cudaSuccess) return fail(p, CEP_ERR_CUDA, "cudaEventQuery failed: %s", cudaGetErrorString(q));
  if (hs[kStTimeout]) return fail(p, CEP_ERR_DEVICE_TIMEOUT, "a bounded wait inside a kernel expired");
  if (hs[kStBoundsViolation]) return fail(p, CEP_ERR_CAPACITY, "a row index left the scratch slot (more local pairs than planned)");
  if (hs[kStBadRouting] & 1) return fail(p, CEP_ERR_BAD_ROUTING, "an expert id was outside [0, n_experts_global)");
  if (hs[kStBadRouting] & 2) return fail(p, CEP_ERR_BAD_ROUTING, "a token names the same expert in two of its slots");
  return CEP_OK;
}

int ffn_wait_invocation(cep_plan* p, int32_t inv, void* stream) {
  if (!p) return fail(nullptr, CEP_ERR_ARG, "plan is NULL");
  if (inv < 0 || inv >= (int)p->inv.size()) return fail(p, CEP_ERR_ARG, "invocation %d does not exist", inv);
  CUDA_TRY(p, cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), p->inv[inv].done, 0));
  return CEP_OK;
}

int ffn_num_invocations(const cep_plan* p) { return p ? (int)p->inv.size() : CEP_ERR_ARG; }

static void fill_info(const Invocation& iv, cep_invocation_info* info) {
  info->n_chunks = iv.n_chunks; info->first_chunk_pos = iv.first_pos; info->stream_index = iv.slot;
  info->n_tokens = iv.n_tokens; info->pairs_bound = iv.pairs_bound; info->elapsed_ms = -1.f;
  info->layout_ms = info->gemm1_ms = info->gemm2_ms = info->combine_ms = info->index_ms = info->scatter_ms = -1.f;
  if (cudaEventQuery(iv.done) == cudaSuccess) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, iv.start, iv.done) == cudaSuccess) info->elapsed_ms = ms;
    if (iv.profiled) {
      if (cudaEventElapsedTime(&ms, iv.start, iv.mark[0]) == cudaSuccess) info->layout_ms = ms;
      if (cudaEventElapsedTime(&ms, iv.start, iv.mark[3]) == cudaSuccess) info->index_ms = ms;
      if (cudaEventElapsedTime(&ms, iv.mark[3], iv.mark[0]) == cudaSuccess) info->scatter_ms = ms;
      if (cudaEventElapsedTime(&ms, iv.mark[0], iv.mark[1]) == cudaSuccess) info->gemm1_ms = ms;
      if (cudaEventElapsedTime(&ms, iv.mark[1], iv.mark[2]) == cudaSuccess) info->gemm2_ms = ms;
      if (cudaEventElapsedTime(&ms, iv.mark[2], iv.done) == cudaSuccess) info->combine_ms = ms;
    }
  }
}

int ffn_query(cep_plan* p, int32_t inv, cep_invocation_info* info) {
  if (!p || !info) return fail(p, CEP_ERR_ARG, "NULL argument");
  if (inv < 0 || inv >= (int)p->inv.size()) return fail(p, CEP_ERR_ARG, "invocation %d does not exist", inv);
  fill_info(p->inv[inv], info);
  return CEP_OK;
}

int ffn_query_call(cep_plan* p, int32_t calls_back, int32_t inv, cep_invocation_info* info) {
  if (!p || !info) return fail(p, CEP_ERR_ARG, "NULL argument");
  if (calls_back == 0) return ffn_query(p, inv, info);
  if (calls_back < 0 || calls_back >= p->trace_sets || calls_back > p->call_index)
    return fail(p, CEP_ERR_ARG, "the records of %d layer calls ago are not kept", calls_back);
  const std::vector<Invocation>& v = p->past[(p->call_index - calls_back) % kTraceCalls];
  if (inv < 0 || inv >= (int)v.size()) return fail(p, CEP_ERR_ARG, "invocation %d does not exist in that layer call", inv);
  fill_info(v[inv], info);
  return CEP_OK;
}

int ffn_debug_export(cep_plan* p, int32_t inv, int32_t* counts, int32_t* offsets, int32_t* padded_offsets,
                     int32_t* row_of_pair, int32_t* pair_of_row) {
  if (!p) return fail(nullptr, CEP_ERR_ARG, "plan is NULL");
  if (inv < 0 || inv >= (int)p->inv.size()) return fail(p, CEP_ERR_ARG, "invocation %d does not exist", inv);
  const Invocation& iv = p->inv[inv];
  if ((int)p->inv.size() - inv > p->active_streams) return fail(p, CEP_ERR_STATE, "scratch slot of invocation %d was reused", inv);
  CUDA_TRY(p, cudaEventSynchronize(iv.done));
  const Slot& sl = p->slots[iv.slot];
  const int E = p->cfg.n_experts_local;
  std::vector<int32_t> po(E + 1, 0);
  if (iv.n_tokens > 0) CUDA_TRY(p, cudaMemcpy(po.data(), sl.lp.padded_offsets, (E + 1) * 4, cudaMemcpyDeviceToHost));
  if (iv.n_tokens == 0) {
    if (counts) memset(counts, 0, E * 4);
    if (offsets) memset(offsets, 0, (E + 1) * 4);
    if (padded_offsets) memset(padded_offsets, 0, (E + 1) * 4);
    return CEP_OK;
  }
  if (counts) CUDA_TRY(p, cudaMemcpy(counts, sl.lp.counts, E * 4, cudaMemcpyDeviceToHost));
  if (offsets) CUDA_TRY(p, cudaMemcpy(offsets, sl.lp.offsets, (E + 1) * 4, cudaMemcpyDeviceToHost));
  if (padded_offsets) memcpy(padded_offsets, po.data(), (E + 1) * 4);
  if (row_of_pair) CUDA_TRY(p, cudaMemcpy(row_of_pair, sl.lp.row_of_pair, (size_t)iv.n_tokens * p->cfg.top_k * 4, cudaMemcpyDeviceToHost));
  if (pair_of_row && po[E] > 0) CUDA_TRY(p, cudaMemcpy(pair_of_row, sl.lp.pair_of_row, (size_t)po[E] * 4, cudaMemcpyDeviceToHost));
  return CEP_OK;
}

int ffn_set_active_streams(cep_plan* p, int32_t n) {
  if (!p) return fail(nullptr, CEP_ERR_ARG, "plan is NULL");
  if (p->layer_open) return fail(p, CEP_ERR_STATE, "the number of active streams cannot change while a layer call is open");
  if (n < 1 || n > p->cfg.n_streams) return fail(p, CEP_ERR_ARG, "active streams must be in 1..%d", p->cfg.n_streams);
  p->active_streams = n;
  return CEP_OK;
}

static float median_of(std::vector<float>& v) {
  std::sort(v.begin(), v.end());
  const size_t n = v.size();
  return n == 0 ? -1.f : (n & 1) ? v[n / 2] : 0.5f * (v[n / 2 - 1] + v[n / 2]);
}

int cep_calibrate(cep_plan* p, float rho, const int32_t* rows_per_expert, int32_t n_points, int32_t reps,
                  const void* tokens, const void* token_scales, int32_t* ids, float* weights, void* out,
                  cep_profile_point* points, cep_calibration* res) {
  if (!p) return fail(nullptr, CEP_ERR_ARG, "plan is NULL");
  if (!rows_per_expert || !tokens || !ids || !weights || !out || !points || !res) return fail(p, CEP_ERR_ARG, "a calibration pointer is NULL");
  if (!(rho > 0.f && rho <= 1.f) || n_points < 1 || reps < 1 || reps > 100) return fail(p, CEP_ERR_ARG, "need 0 < rho <= 1, n_points >= 1, 1 <= reps <= 100");
  if (p->layer_open) return fail(p, CEP_ERR_STATE, "cep_calibrate while a layer call is open");
  if (!p->have_weights) return fail(p, CEP_ERR_STATE, "cep_calibrate before moe_load_weights");
  if (!p->cfg.profile_kernels) return fail(p, CEP_ERR_STATE, "cep_calibrate needs a plan made with profile_kernels != 0");
  const cep_config saved = p->cfg;
  const int saved_active = p->active_streams;
  const int E = saved.n_experts_local, k = saved.top_k, k_loc = k < E ? k : E;
  for (int i = 0; i < n_points; ++i) {
    if (rows_per_expert[i] < 1 || (i > 0 && rows_per_expert[i] <= rows_per_expert[i - 1]))
      return fail(p, CEP_ERR_ARG, "rows_per_expert must be positive and ascending");
  }
  auto tokens_for = [&](long long rows) { long long t = rows * E / k_loc; return t < 1 ? 1ll : t; };
  const long long T_max = tokens_for(rows_per_expert[n_points - 1]);
  if (T_max > saved.max_tokens) return fail(p, CEP_ERR_CAPACITY, "largest point needs %lld tokens, plan made for %d", T_max, saved.max_tokens);
  cudaStream_t s0 = p->streams[0];
  cudaEvent_t ea = nullptr, eb = nullptr;
  int rc = CEP_OK;
  const size_t act_row = (size_t)saved.hidden * (dtype_is_bytes(saved.dtype) ? 1 : 2);
  const size_t scale_row = saved.dtype == CEP_BF16 ? 0 : (size_t)saved.hidden / kQuantBlock * 4;   // bytes of scales per token
  auto restore = [&]() {
    p->cfg.mode = saved.mode; p->cfg.threshold_pairs = saved.threshold_pairs; p->active_streams = saved_active;
    if (p->layer_open) { p->pending.clear(); p->pending_pairs = 0; p->layer_open = false; }   // a probe call that failed half-way
    if (ea) cudaEventDestroy(ea);
    if (eb) cudaEventDestroy(eb);
  };
#define CAL_TRY(call) do { rc = (call); if (rc != CEP_OK) { restore(); return rc; } } while (0)
#define CAL_CUDA(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { restore(); \
    return fail(p, CEP_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_)); } } while (0)
  CAL_CUDA(launch_uniform_routing(ids, weights, (int)T_max, k, k_loc, E, s0));
  CAL_CUDA(cudaEventCreate(&ea));
  CAL_CUDA(cudaEventCreate(&eb));
  // ---- the profile: one synchronous invocation per point
  p->cfg.mode = CEP_MODE_SYNC;
  float peak = 0.f;
  for (int i = 0; i < n_points; ++i) {
    const int T = (int)tokens_for(rows_per_expert[i]);
    std::vector<float> ffn, layer;
    for (int r = 0; r < reps + 2; ++r) {
      CAL_TRY(ffn_begin(p, out, T, 1));
      CAL_TRY(ffn_submit_chunk(p, 0, 0, T, tokens, token_scales, ids, weights, (int64_t)T * k_loc, s0));
      CAL_TRY(combine(p, s0));
      CAL_CUDA(cudaStreamSynchronize(s0));
      CAL_TRY(ffn_status(p));
      cep_invocation_info info;
      CAL_TRY(ffn_query(p, 0, &info));
      if (r >= 2) { ffn.push_back(info.gemm1_ms + info.gemm2_ms); layer.push_back(info.elapsed_ms); }
    }
    cep_profile_point& pt = points[i];
    pt.rows_per_expert = rows_per_expert[i]; pt.n_tokens = T; pt.expert_tokens = (int64_t)T * k_loc;
    pt.ffn_ms = median_of(ffn); pt.layer_ms = median_of(layer);
    pt.tflops = pt.ffn_ms > 0.f ? (float)(6.0 * saved.hidden * saved.inter * (double)pt.expert_tokens / (pt.ffn_ms * 1e-3) / 1e12) : 0.f;
    pt.eta = 0.f;
    if (pt.tflops > peak) peak = pt.tflops;
  }
  res->rho = rho; res->peak_tflops = peak; res->theta_pairs = points[n_points - 1].expert_tokens;
  res->theta_rows_per_expert = points[n_points - 1].rows_per_expert;
  for (int i = 0; i < n_points; ++i) points[i].eta = peak > 0.f ? points[i].tflops / peak : 0.f;
  for (int i = 0; i < n_points; ++i)
    if (points[i].eta >= rho) { res->theta_pairs = points[i].expert_tokens; res->theta_rows_per_expert = points[i].rows_per_expert; break; }
  // ---- stream probe: a chain of theta-sized invocations, all chunks present, 1..S active streams
  for (int s = 0; s < 16; ++s) res->stream_ms[s] = -1.f;
  res->best_streams = 0; res->probe_invocations = 0;
  const int T_theta = (int)tokens_for(res->theta_rows_per_expert);
  int n_inv = (int)(T_max / T_theta);
  if (n_inv > 8) n_inv = 8;
  if (n_inv > saved.max_chunks) n_inv = saved.max_chunks;
  if (n_inv >= 2 && saved.n_streams > 1) {
    res->probe_invocations = n_inv;
    p->cfg.mode = CEP_MODE_STREAMFFN;
    p->cfg.threshold_pairs = (int64_t)T_theta * k_loc;
    float best = -1.f;
    for (int s = 1; s <= saved.n_streams; ++s) {
      p->active_streams = s;
      std::vector<float> ms;
      for (int r = 0; r < reps + 2; ++r) {
        CAL_CUDA(cudaEventRecord(ea, s0));
        CAL_TRY(ffn_begin(p, out, n_inv * T_theta, n_inv));
        for (int c = 0; c < n_inv; ++c) {
          const uint8_t* tk = static_cast<const uint8_t*>(tokens) + (size_t)c * T_theta * act_row;
          const uint8_t* sc = token_scales ? static_cast<const uint8_t*>(token_scales) + (size_t)c * T_theta * scale_row : nullptr;
          CAL_TRY(ffn_submit_chunk(p, c, c * T_theta, T_theta, tk, sc, ids + (size_t)c * T_theta * k,
                                   weights + (size_t)c * T_theta * k, (int64_t)T_theta * k_loc, s0));
        }
        CAL_TRY(combine(p, s0));
        CAL_CUDA(cudaEventRecord(eb, s0));
        CAL_CUDA(cudaStreamSynchronize(s0));
        CAL_TRY(ffn_status(p));
        float t = 0.f;
        CAL_CUDA(cudaEventElapsedTime(&t, ea, eb));
        if (r >= 2) ms.push_back(t);
      }
      res->stream_ms[s - 1] = median_of(ms);
      if (best < 0.f || res->stream_ms[s - 1] < best) best = res->stream_ms[s - 1];
    }
    for (int s = 1; s <= saved.n_streams; ++s)
      if (res->stream_ms[s - 1] <= 1.02f * best) { res->best_streams = s; break; }
  }
#undef CAL_TRY
#undef CAL_CUDA
  restore();
  return CEP_OK;
}

int cep_calibrate_routed(cep_plan* p, float rho, const int32_t* n_tokens, int32_t n_points, int32_t reps,
                         const void* tokens, const void* token_scales, const int32_t* ids, const float* weights,
                         void* out, cep_profile_point* points, cep_calibration* res) {
  if (!p) return fail(nullptr, CEP_ERR_ARG, "plan is NULL");
  if (!n_tokens || !tokens || !ids || !weights || !out || !points || !res) return fail(p, CEP_ERR_ARG, "a calibration pointer is NULL");
  if (!(rho > 0.f && rho <= 1.f) || n_points < 1 || reps < 1 || reps > 100) return fail(p, CEP_ERR_ARG, "need 0 < rho <= 1, n_points >= 1, 1 <= reps <= 100");
  if (p->layer_open) return fail(p, CEP_ERR_STATE, "cep_calibrate_routed while a layer call is open");
  if (!p->have_weights) return fail(p, CEP_ERR_STATE, "cep_calibrate_routed before moe_load_weights");
  if (!p->cfg.profile_kernels) return fail(p, CEP_ERR_STATE, "cep_calibrate_routed needs a plan made with profile_kernels != 0");
  for (int i = 0; i < n_points; ++i)
    if (n_tokens[i] < 1 || (i > 0 && n_tokens[i] <= n_tokens[i - 1]) || n_tokens[i] > p->cfg.max_tokens)
      return fail(p, CEP_ERR_ARG, "n_tokens must be positive, ascending and at most max_tokens");
  const int saved_mode = p->cfg.mode;
  const int E = p->cfg.n_experts_local;
  cudaStream_t s0 = p->streams[0];
  p->cfg.mode = CEP_MODE_SYNC;
  int rc = CEP_OK;
  float peak = 0.f;
  for (int i = 0; i < n_points && rc == CEP_OK; ++i) {
    const int T = n_tokens[i];
    std::vector<float> ffn, layer;
    int32_t n_local = 0;
    for (int r = 0; r < reps + 2 && rc == CEP_OK; ++r) {
      rc = ffn_begin(p, out, T, 1);
      if (rc == CEP_OK) rc = ffn_submit_chunk(p, 0, 0, T, tokens, token_scales, ids, weights, -1, s0);
      if (rc == CEP_OK) rc = combine(p, s0);
      if (rc == CEP_OK && cudaStreamSynchronize(s0) != cudaSuccess) rc = fail(p, CEP_ERR_CUDA, "cudaStreamSynchronize failed");
      if (rc == CEP_OK) rc = ffn_status(p);
      cep_invocation_info info;
      if (rc == CEP_OK) rc = ffn_query(p, 0, &info);
      if (rc == CEP_OK && r >= 2) { ffn.push_back(info.gemm1_ms + info.gemm2_ms); layer.push_back(info.elapsed_ms); }
    }
    // the expert tokens of this prefix of the batch: the last entry of the offsets the layout transform just made
    if (rc == CEP_OK && cudaMemcpy(&n_local, p->slots[p->inv[0].slot].lp.offsets + E, sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess)
      rc = fail(p, CEP_ERR_CUDA, "cudaMemcpy of the pair count failed");
    if (rc != CEP_OK) break;
    cep_profile_point& pt = points[i];
    pt.n_tokens = T; pt.expert_tokens = n_local; pt.rows_per_expert = n_local / E;
    pt.ffn_ms = median_of(ffn); pt.layer_ms = median_of(layer);
    pt.tflops = pt.ffn_ms > 0.f ? (float)(6.0 * p->cfg.hidden * p->cfg.inter * (double)n_local / (pt.ffn_ms * 1e-3) / 1e12) : 0.f;
    pt.eta = 0.f;
    if (pt.tflops > peak) peak = pt.tflops;
  }
  p->cfg.mode = saved_mode;
  if (rc != CEP_OK) {
    if (p->layer_open) { p->pending.clear(); p->pending_pairs = 0; p->layer_open = false; }
    return rc;
  }
  res->rho = rho; res->peak_tflops = peak;
  res->theta_pairs = points[n_points - 1].expert_tokens; res->theta_rows_per_expert = points[n_points - 1].rows_per_expert;
  for (int i = 0; i < n_points; ++i) points[i].eta = peak > 0.f ? points[i].tflops / peak : 0.f;
  for (int i = 0; i < n_points; ++i)
    if (points[i].eta >= rho) { res->theta_pairs = points[i].expert_tokens; res->theta_rows_per_expert = points[i].rows_per_expert; break; }
  for (int s = 0; s < 16; ++s) res->stream_ms[s] = -1.f;
  res->best_streams = 0; res->probe_invocations = 0;
  return CEP_OK;
}

int64_t cep_kernel_launches(const cep_plan* p) { return p ? p->launches : 0; }

int moe_plan_destroy(cep_plan* p) {
  if (!p) return CEP_OK;
  for (cudaStream_t s : p->streams) cudaStreamSynchronize(s);
  for (cudaEvent_t e : p->ready_evt) cudaEventDestroy(e);
  for (cudaEvent_t e : p->inv_start) cudaEventDestroy(e);
  for (cudaEvent_t e : p->inv_done) cudaEventDestroy(e);
  for (cudaEvent_t e : p->inv_mark) cudaEventDestroy(e);
  if (p->begin_evt) cudaEventDestroy(p->begin_evt);
  for (int i = 0; i < 2; ++i)
    if (p->readback_evt[i]) { cudaEventSynchronize(p->readback_evt[i]); cudaEventDestroy(p->readback_evt[i]); }
  if (p->weights_evt) cudaEventDestroy(p->weights_evt);
  for (cudaStream_t s : p->streams) cudaStreamDestroy(s);
  if (p->host_status) cudaFreeHost(p->host_status);
  delete p;
  return CEP_OK;
}

int cep_debug_wait_timeout(cep_plan* p, int32_t limit_ms, void* stream) {
  if (!p) return fail(nullptr, CEP_ERR_ARG, "plan is NULL");
  if (!p->layer_open) return fail(p, CEP_ERR_STATE, "cep_debug_wait_timeout needs an open layer call");
  if (limit_ms < 1 || limit_ms > 1000) return fail(p, CEP_ERR_ARG, "limit_ms must be in 1..1000");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CUDA_TRY(p, cudaStreamWaitEvent(st, p->begin_evt, 0));          // after this call's status reset
  CUDA_TRY(p, launch_wait_probe((unsigned long long)limit_ms * 1000000ull,
                                reinterpret_cast<int32_t*>(p->ws + p->L.status + (size_t)p->status_idx * kStatusBlockBytes), st,
                                &p->launches));
  return CEP_OK;
}

int cep_debug_check_guards(cep_plan* p, int32_t* n_damaged) {
  if (!p || !n_damaged) return fail(p, CEP_ERR_ARG, "NULL argument");
  *n_damaged = 0;
  if (!p->L.guard) return fail(p, CEP_ERR_STATE, "the plan was made without debug_checks: it has no guard gaps");
  for (cudaStream_t s : p->streams) CUDA_TRY(p, cudaStreamSynchronize(s));
  std::vector<uint8_t> host(p->L.guard);
  for (int s = 0; s < p->cfg.n_streams; ++s)
    for (size_t off : p->L.guard_offsets) {
      CUDA_TRY(p, cudaMemcpy(host.data(), p->ws + p->L.slot0 + p->L.slot_bytes * s + off, p->L.guard, cudaMemcpyDeviceToHost));
      for (uint8_t b : host)
        if (b != kGuardByte) { *n_damaged += 1; break; }
    }
  return CEP_OK;
}

int cep_debug_decode_tile(const int32_t* tile_prefix, int32_t n_experts, int32_t n_blocks_n, int32_t n_group,
                          int32_t tile, int32_t* expert, int32_t* m_block, int32_t* n_block) {
  if (!tile_prefix || n_experts <= 0 || !expert || !m_block || !n_block) return CEP_ERR_ARG;
  TileCoord tc;
  if (!decode_tile(tile_prefix, n_experts, n_blocks_n, n_group, tile, &tc)) return CEP_ERR_ARG;
  *expert = tc.expert; *m_block = tc.m_block; *n_block = tc.n_block;
  return CEP_OK;
}

int cep_debug_schedule(const int64_t* pairs, int32_t n_chunks, int32_t mode, int64_t theta,
                       int32_t* invocation_of_chunk) {
  if (n_chunks < 0 || (n_chunks > 0 && (!pairs || !invocation_of_chunk))) return CEP_ERR_ARG;
  int inv = 0, pending = 0;
  int64_t acc = 0;
  for (int c = 0; c < n_chunks; ++c) {
    invocation_of_chunk[c] = inv;
    ++pending; acc += pairs[c];
    if (should_launch(mode, acc, pending, theta)) { ++inv; pending = 0; acc = 0; }
  }
  if (pending) ++inv;                             // final flush
  return inv;
}

}  // extern "C"
