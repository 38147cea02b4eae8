"""ctypes binding of include/cascade_ffn.h: same names, argument marshalling only.

Every step of the path runs inside the library's CUDA kernels.  torch is used for
device memory and streams.  If the library cannot be loaded the import of a symbol
raises: there is no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libcascade_ffn.so")

CEP_BF16, CEP_FP8_E4M3_BLOCK128, CEP_MXFP4_E4M3 = 0, 1, 2
DTYPE_OF = {"bf16": CEP_BF16, "fp8": CEP_FP8_E4M3_BLOCK128, "mxfp4": CEP_MXFP4_E4M3}   # workload dtype names
CEP_MODE_SYNC, CEP_MODE_ASYNC, CEP_MODE_STREAMFFN = 0, 1, 2
CEP_GEMM_TCGEN05, CEP_GEMM_SIMT, CEP_GEMM_TCGEN05_1CTA = 0, 1, 2
STATUS_NAMES = {0: "CEP_OK", -1: "CEP_ERR_ARG", -2: "CEP_ERR_STATE", -3: "CEP_ERR_WORKSPACE",
                -4: "CEP_ERR_CAPACITY", -5: "CEP_ERR_INCOMPLETE", -6: "CEP_ERR_BAD_ROUTING",
                -7: "CEP_ERR_DEVICE_TIMEOUT", -8: "CEP_ERR_CUDA", -9: "CEP_ERR_UNSUPPORTED"}

EXPORTS = ["moe_plan_workspace_bytes", "moe_packed_weight_bytes", "moe_plan", "moe_load_weights",
           "ffn_begin", "ffn_submit_chunk", "ffn_flush", "combine", "ffn_status", "ffn_num_invocations",
           "ffn_query", "ffn_debug_export", "cep_kernel_launches", "moe_plan_destroy", "cep_last_error",
           "cep_debug_decode_tile", "cep_debug_schedule", "layout_indices_noalloc", "cep_debug_wait_timeout", "ffn_set_addend", "moe_route", "cep_debug_check_guards", "ffn_wait_invocation",
           "ffn_set_active_streams", "cep_calibrate", "ffn_query_call", "cep_calibrate_routed"]


class CepConfig(ctypes.Structure):
    _fields_ = [("hidden", ctypes.c_int32), ("inter", ctypes.c_int32),
                ("n_experts_global", ctypes.c_int32), ("n_experts_local", ctypes.c_int32),
                ("top_k", ctypes.c_int32), ("max_tokens", ctypes.c_int32), ("max_chunks", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("mode", ctypes.c_int32), ("n_streams", ctypes.c_int32),
                ("threshold_pairs", ctypes.c_int64), ("gemm_impl", ctypes.c_int32),
                ("debug_checks", ctypes.c_int32), ("profile_kernels", ctypes.c_int32),
                ("defer_while_busy", ctypes.c_int32), ("gather_a", ctypes.c_int32)]


class InvocationInfo(ctypes.Structure):
    _fields_ = [("n_chunks", ctypes.c_int32), ("first_chunk_pos", ctypes.c_int32),
                ("stream_index", ctypes.c_int32), ("n_tokens", ctypes.c_int32),
                ("pairs_bound", ctypes.c_int64), ("elapsed_ms", ctypes.c_float),
                ("layout_ms", ctypes.c_float), ("gemm1_ms", ctypes.c_float), ("gemm2_ms", ctypes.c_float),
                ("combine_ms", ctypes.c_float), ("index_ms", ctypes.c_float), ("scatter_ms", ctypes.c_float)]


class ProfilePoint(ctypes.Structure):
    _fields_ = [("rows_per_expert", ctypes.c_int32), ("n_tokens", ctypes.c_int32), ("expert_tokens", ctypes.c_int64),
                ("ffn_ms", ctypes.c_float), ("layer_ms", ctypes.c_float), ("tflops", ctypes.c_float),
                ("eta", ctypes.c_float)]


class Calibration(ctypes.Structure):
    _fields_ = [("rho", ctypes.c_float), ("peak_tflops", ctypes.c_float), ("theta_pairs", ctypes.c_int64),
                ("theta_rows_per_expert", ctypes.c_int32), ("best_streams", ctypes.c_int32),
                ("probe_invocations", ctypes.c_int32), ("stream_ms", ctypes.c_float * 16)]


class CepError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__("%s: %s" % (STATUS_NAMES.get(code, str(code)), msg))
        self.code = code


_lib = None


def load_library(build_if_missing: bool = True):
    """dlopen the C-ABI library (building it with nvcc first if it is absent or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing:
        from .build import build
        try:
            build()
        except Exception:
            if not os.path.exists(LIB_PATH):
                raise
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libcascade_ffn.so is missing: build it with `python -m paper_2609_33252_b200.build`")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    cfgp = ctypes.POINTER(CepConfig)
    sig = {
        "moe_plan_workspace_bytes": (ctypes.c_int, [cfgp, ctypes.POINTER(sz)]),
        "moe_packed_weight_bytes": (ctypes.c_int, [cfgp, ctypes.POINTER(sz)]),
        "moe_plan": (ctypes.c_int, [cfgp, vp, sz, ctypes.POINTER(vp)]),
        "moe_load_weights": (ctypes.c_int, [vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]),
        "ffn_begin": (ctypes.c_int, [vp, vp, i32, i32]),
        "ffn_submit_chunk": (ctypes.c_int, [vp, i32, i32, i32, vp, vp, vp, vp, i64, vp]),
        "ffn_flush": (ctypes.c_int, [vp]),
        "combine": (ctypes.c_int, [vp, vp]),
        "ffn_status": (ctypes.c_int, [vp]),
        "ffn_num_invocations": (ctypes.c_int, [vp]),
        "ffn_wait_invocation": (ctypes.c_int, [vp, i32, vp]),
        "ffn_query": (ctypes.c_int, [vp, i32, ctypes.POINTER(InvocationInfo)]),
        "ffn_query_call": (ctypes.c_int, [vp, i32, i32, ctypes.POINTER(InvocationInfo)]),
        "ffn_debug_export": (ctypes.c_int, [vp, i32, vp, vp, vp, vp, vp]),
        "cep_kernel_launches": (i64, [vp]),
        "moe_plan_destroy": (ctypes.c_int, [vp]),
        "cep_last_error": (ctypes.c_char_p, [vp]),
        "cep_debug_decode_tile": (ctypes.c_int, [vp, i32, i32, i32, i32] + [ctypes.POINTER(i32)] * 3),
        "cep_debug_schedule": (ctypes.c_int, [vp, i32, i32, i64, vp]),
        "cep_debug_wait_timeout": (ctypes.c_int, [vp, i32, vp]),
        "ffn_set_addend": (ctypes.c_int, [vp, vp]),
        "cep_debug_check_guards": (ctypes.c_int, [vp, ctypes.POINTER(i32)]),
        "moe_route": (ctypes.c_int, [vp, i32, i32, i32, vp, vp, vp]),
        "ffn_set_active_streams": (ctypes.c_int, [vp, i32]),
        "cep_calibrate": (ctypes.c_int, [vp, ctypes.c_float, vp, i32, i32, vp, vp, vp, vp, vp,
                                         ctypes.POINTER(ProfilePoint), ctypes.POINTER(Calibration)]),
        "cep_calibrate_routed": (ctypes.c_int, [vp, ctypes.c_float, vp, i32, i32, vp, vp, vp, vp, vp,
                                                ctypes.POINTER(ProfilePoint), ctypes.POINTER(Calibration)]),
        "layout_indices_noalloc": (ctypes.c_int, [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, i32, vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(L, name)
        fn.restype, fn.argtypes = res, args
    _lib = L
    return L


def lib():
    return load_library()


def _check(rc: int, plan=None, allow: Sequence[int] = ()):
    if rc != 0 and rc not in allow:
        msg = lib().cep_last_error(plan)
        raise CepError(rc, msg.decode() if msg else "")
    return rc


def _dptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream_handle(stream) -> int:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


# ---------------------------------------------------------------- same-named wrappers
def moe_plan_workspace_bytes(cfg: CepConfig) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().moe_plan_workspace_bytes(ctypes.byref(cfg), ctypes.byref(n)))
    return n.value


def moe_packed_weight_bytes(cfg: CepConfig) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().moe_packed_weight_bytes(ctypes.byref(cfg), ctypes.byref(n)))
    return n.value


def moe_plan(cfg: CepConfig, workspace) -> int:
    """workspace: torch uint8 CUDA tensor.  Returns the plan handle."""
    h = ctypes.c_void_p()
    _check(lib().moe_plan(ctypes.byref(cfg), workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                          ctypes.byref(h)))
    return h.value


def moe_load_weights(plan, w_gate, w_up, w_down, s_gate, s_up, s_down, packed, stream=None):
    _check(lib().moe_load_weights(plan, _dptr(w_gate), _dptr(w_up), _dptr(w_down), _dptr(s_gate), _dptr(s_up),
                                  _dptr(s_down), packed.data_ptr(), packed.numel() * packed.element_size(),
                                  _stream_handle(stream)), plan)


def ffn_begin(plan, out, n_tokens_total: int, n_chunks_expected: int):
    _check(lib().ffn_begin(plan, out.data_ptr(), n_tokens_total, n_chunks_expected), plan)


def ffn_set_addend(plan, addend):
    _check(lib().ffn_set_addend(plan, _dptr(addend)), plan)


def moe_route(logits, top_k: int, topk_ids, topk_weights, stream=None):
    n_tokens, n_experts_global = logits.shape
    _check(lib().moe_route(logits.data_ptr(), n_tokens, n_experts_global, top_k, topk_ids.data_ptr(),
                           topk_weights.data_ptr(), _stream_handle(stream)))


def ffn_submit_chunk(plan, chunk_id: int, token_offset: int, n_tokens: int, tokens, token_scales, topk_ids,
                     topk_weights, n_local_pairs: int = -1, stream=None):
    _check(lib().ffn_submit_chunk(plan, chunk_id, token_offset, n_tokens, _dptr(tokens), _dptr(token_scales),
                                  _dptr(topk_ids), _dptr(topk_weights), n_local_pairs, _stream_handle(stream)),
           plan)


def ffn_flush(plan, allow_incomplete: bool = False) -> int:
    return _check(lib().ffn_flush(plan), plan, allow=(-5,) if allow_incomplete else ())


def combine(plan, stream=None, allow_incomplete: bool = False) -> int:
    return _check(lib().combine(plan, _stream_handle(stream)), plan, allow=(-5,) if allow_incomplete else ())


def ffn_status(plan) -> int:
    return lib().ffn_status(plan)


def ffn_wait_invocation(plan, inv: int, stream=None):
    _check(lib().ffn_wait_invocation(plan, inv, _stream_handle(stream)), plan)


def ffn_num_invocations(plan) -> int:
    return lib().ffn_num_invocations(plan)


def ffn_query(plan, inv: int) -> InvocationInfo:
    info = InvocationInfo()
    _check(lib().ffn_query(plan, inv, ctypes.byref(info)), plan)
    return info


def ffn_query_call(plan, calls_back: int, inv: int) -> InvocationInfo:
    info = InvocationInfo()
    _check(lib().ffn_query_call(plan, calls_back, inv, ctypes.byref(info)), plan)
    return info


def ffn_debug_export(plan, inv: int, n_experts_local: int, n_pairs: int):
    """Returns dict of numpy int32 arrays: counts, offsets, padded_offsets, row_of_pair, pair_of_row."""
    import numpy as np
    E = n_experts_local
    counts = np.zeros(E, np.int32)
    offsets = np.zeros(E + 1, np.int32)
    padded = np.zeros(E + 1, np.int32)
    rop = np.full(max(n_pairs, 1), -1, np.int32)
    p = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    _check(lib().ffn_debug_export(plan, inv, p(counts), p(offsets), p(padded), p(rop), None), plan)
    por = np.full(max(int(padded[E]), 1), -1, np.int32)
    _check(lib().ffn_debug_export(plan, inv, None, None, None, None, p(por)), plan)
    return dict(counts=counts, offsets=offsets, padded_offsets=padded, row_of_pair=rop[:n_pairs],
                pair_of_row=por[:int(padded[E])])


def ffn_set_active_streams(plan, n: int):
    _check(lib().ffn_set_active_streams(plan, n), plan)


def cep_calibrate(plan, rho: float, rows_per_expert: Sequence[int], reps: int, tokens, token_scales, ids, weights, out):
    """Returns (list of profile-point dicts, calibration dict); the tensors are device scratch (see the header)."""
    n = len(rows_per_expert)
    rows = (ctypes.c_int32 * n)(*[int(r) for r in rows_per_expert])
    pts = (ProfilePoint * n)()
    cal = Calibration()
    _check(lib().cep_calibrate(plan, float(rho), ctypes.cast(rows, ctypes.c_void_p), n, reps, _dptr(tokens),
                               _dptr(token_scales), _dptr(ids), _dptr(weights), _dptr(out), pts, ctypes.byref(cal)), plan)
    points = [{f: getattr(p, f) for f, _ in ProfilePoint._fields_} for p in pts]
    result = {f: getattr(cal, f) for f, _ in Calibration._fields_ if f != "stream_ms"}
    result["stream_ms"] = [v for v in cal.stream_ms if v >= 0]
    return points, result


def cep_calibrate_routed(plan, rho: float, n_tokens: Sequence[int], reps: int, tokens, token_scales, ids, weights, out):
    """Calibration on the caller's routing: profile on growing prefixes of one real batch (see the header)."""
    n = len(n_tokens)
    nt = (ctypes.c_int32 * n)(*[int(v) for v in n_tokens])
    pts = (ProfilePoint * n)()
    cal = Calibration()
    _check(lib().cep_calibrate_routed(plan, float(rho), ctypes.cast(nt, ctypes.c_void_p), n, reps, _dptr(tokens),
                                      _dptr(token_scales), _dptr(ids), _dptr(weights), _dptr(out), pts, ctypes.byref(cal)), plan)
    points = [{f: getattr(p, f) for f, _ in ProfilePoint._fields_} for p in pts]
    result = {f: getattr(cal, f) for f, _ in Calibration._fields_ if f != "stream_ms"}
    return points, result


def cep_kernel_launches(plan) -> int:
    return lib().cep_kernel_launches(plan)


def moe_plan_destroy(plan):
    _check(lib().moe_plan_destroy(plan))


def cep_last_error(plan=None) -> str:
    m = lib().cep_last_error(plan)
    return m.decode() if m else ""


def cep_debug_check_guards(plan) -> int:
    """Number of damaged guard gaps of a plan made with debug_checks (0 = no overrun)."""
    n = ctypes.c_int32(-1)
    _check(lib().cep_debug_check_guards(plan, ctypes.byref(n)), plan)
    return n.value


def cep_debug_wait_timeout(plan, limit_ms: int, stream=None):
    _check(lib().cep_debug_wait_timeout(plan, limit_ms, _stream_handle(stream)), plan)


def cep_debug_decode_tile(tile_prefix, n_blocks_n: int, tile: int, n_group: int = 0):
    import numpy as np
    tp = np.ascontiguousarray(tile_prefix, dtype=np.int32)
    e, m, n = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    rc = lib().cep_debug_decode_tile(tp.ctypes.data_as(ctypes.c_void_p), tp.shape[0] - 1, n_blocks_n,
                                     n_group if n_group > 0 else n_blocks_n, tile,
                                     ctypes.byref(e), ctypes.byref(m), ctypes.byref(n))
    return None if rc else (e.value, m.value, n.value)


def cep_debug_schedule(pairs: Sequence[int], mode: int, theta: int) -> List[int]:
    import numpy as np
    pr = np.ascontiguousarray(pairs, dtype=np.int64)
    out = np.zeros(max(len(pr), 1), np.int32)
    n = lib().cep_debug_schedule(pr.ctypes.data_as(ctypes.c_void_p), len(pr), mode, theta,
                                 out.ctypes.data_as(ctypes.c_void_p))
    if n < 0:
        raise CepError(n, "cep_debug_schedule")
    return out[:len(pr)].tolist()


def layout_indices_noalloc(topk_ids, n_experts_local: int, n_experts_global: int, counts, offsets,
                           padded_offsets, row_of_pair, pair_of_row, status=None, stream=None) -> int:
    """Index half of the layout transform with no workspace (all arguments are CUDA tensors the
    caller allocated beforehand).  Returns the library's status code instead of raising, so a caller
    can test the size limit."""
    n_tokens, top_k = topk_ids.shape
    return lib().layout_indices_noalloc(topk_ids.data_ptr(), n_tokens, top_k, n_experts_local, n_experts_global,
                                        counts.data_ptr(), offsets.data_ptr(), padded_offsets.data_ptr(),
                                        row_of_pair.data_ptr(), pair_of_row.data_ptr(), pair_of_row.numel(),
                                        _dptr(status), _stream_handle(stream))


# ---------------------------------------------------------------- convenience owner of the buffers
class MoELayer:
    """Owns the torch-allocated workspace and packed weights of one plan.

    Plumbing only: allocation and pointer passing.  ``run`` submits the chunks of one
    layer call in the given order on the given streams and joins on ``stream``.
    """

    def __init__(self, hidden, inter, n_experts_global, n_experts_local, top_k, max_tokens, max_chunks,
                 dtype=CEP_BF16, mode=CEP_MODE_STREAMFFN, n_streams=2, threshold_pairs=0,
                 gemm_impl=CEP_GEMM_TCGEN05, debug_checks=0, profile_kernels=0, defer_while_busy=0, gather_a=0,
                 device="cuda"):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("the streamFFN library needs a CUDA device; there is no CPU path")
        self.cfg = CepConfig(hidden, inter, n_experts_global, n_experts_local, top_k, max_tokens, max_chunks,
                             dtype, mode, n_streams, threshold_pairs, gemm_impl, debug_checks, profile_kernels,
                             defer_while_busy, gather_a)
        self.device = torch.device(device)
        self.workspace = torch.empty(moe_plan_workspace_bytes(self.cfg), dtype=torch.uint8, device=self.device)
        self.packed = torch.empty(moe_packed_weight_bytes(self.cfg), dtype=torch.uint8, device=self.device)
        self.plan = moe_plan(self.cfg, self.workspace)

    def load_weights(self, w_gate, w_up, w_down, s_gate=None, s_up=None, s_down=None, stream=None):
        moe_load_weights(self.plan, w_gate, w_up, w_down, s_gate, s_up, s_down, self.packed, stream)

    def run(self, out, chunks, order=None, streams=None, stream=None, n_local_pairs=None, addend=None):
        """chunks: list of (token_offset, x, x_scale, ids, w).  Returns the number of invocations."""
        n_tok = sum(c[1].shape[0] for c in chunks)
        ffn_begin(self.plan, out, n_tok, len(chunks))
        if addend is not None:
            ffn_set_addend(self.plan, addend)
        order = list(range(len(chunks))) if order is None else order
        for c in order:
            off, x, xs, ids, w = chunks[c]
            ffn_submit_chunk(self.plan, c, off, x.shape[0], x, xs, ids, w,
                             -1 if n_local_pairs is None else n_local_pairs[c],
                             None if streams is None else streams[c])
        ffn_flush(self.plan)
        combine(self.plan, stream)
        return ffn_num_invocations(self.plan)

    def close(self):
        if getattr(self, "plan", None):
            moe_plan_destroy(self.plan)
            self.plan = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
