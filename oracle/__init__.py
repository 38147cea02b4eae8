"""CPU oracle for the streamFFN routed-expert path -- TEST INFRASTRUCTURE, not product.

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It shares no code with the CUDA path and never calls it.

Contents (each function cites the passage of the paper it restates):

* ``route``            softmax -> top-k -> renormalise (benchmark definition; the paper
                       does not describe the router)
* ``permute``          per-invocation layout transform: counts, offsets, tile-aligned
                       offsets, stable expert-major row of every (token, slot) pair and
                       the inverse map (Appendix "Grouped FFN invocations")
* ``schedule``         streamFFN launch decisions: threshold batching, final flush, the
                       Sync / Async / Async+streamFFN modes, round-robin streams
                       (Section 3.2 "Launch threshold", "Multi-stream execution";
                       "Deep Dive", ablation study: the three modes)
* ``moe_forward``      the fp64 layer result (C, ``oracle_moe.c``)
* codecs               bf16 / e4m3 / e2m1 / ue8m0 decode and encode, the microscaling block
                       scale rule (C)

Parity pins live in ``tests/test_oracle_*.py``; nothing here is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "liboracle_moe.so")
_SRC = os.path.join(_HERE, "oracle_moe.c")

F64, BF16, FP8, MXFP4 = 0, 1, 2, 3
MIRROR_FP8_ACT, MIRROR_MXFP8_ACT = 1, 4


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc -O2 -fopenmp) next to its source."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.oracle_bf16_to_f64.restype = ctypes.c_double
        L.oracle_bf16_to_f64.argtypes = [ctypes.c_uint16]
        L.oracle_e4m3_to_f64.restype = ctypes.c_double
        L.oracle_e4m3_to_f64.argtypes = [ctypes.c_uint8]
        L.oracle_f64_to_e4m3.restype = ctypes.c_uint8
        L.oracle_f64_to_e4m3.argtypes = [ctypes.c_double]
        L.oracle_f64_to_bf16.restype = ctypes.c_uint16
        L.oracle_f64_to_bf16.argtypes = [ctypes.c_double]
        L.oracle_e2m1_to_f64.restype = ctypes.c_double
        L.oracle_e2m1_to_f64.argtypes = [ctypes.c_uint8]
        L.oracle_f64_to_e2m1.restype = ctypes.c_uint8
        L.oracle_f64_to_e2m1.argtypes = [ctypes.c_double]
        L.oracle_ue8m0_to_f64.restype = ctypes.c_double
        L.oracle_ue8m0_to_f64.argtypes = [ctypes.c_uint8]
        L.oracle_mx_scale_code.restype = ctypes.c_uint8
        L.oracle_mx_scale_code.argtypes = [ctypes.c_float, ctypes.c_int, ctypes.c_double]
        L.oracle_silu.restype = ctypes.c_double
        L.oracle_silu.argtypes = [ctypes.c_double]
        L.oracle_num_threads.restype = ctypes.c_int
        L.oracle_moe_forward.restype = ctypes.c_int
        L.oracle_moe_forward.argtypes = [ctypes.c_int] + [ctypes.c_int64] * 5 + \
            [ctypes.c_void_p] * 10 + [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int,
                                      ctypes.c_void_p, ctypes.c_int]
        _lib = L
    return _lib


# --------------------------------------------------------------------------- codecs
def bf16_to_f64(bits: int) -> float:
    return lib().oracle_bf16_to_f64(int(bits))


def e4m3_to_f64(code: int) -> float:
    return lib().oracle_e4m3_to_f64(int(code))


def f64_to_e4m3(x: float) -> int:
    return lib().oracle_f64_to_e4m3(float(x))


def f64_to_bf16(x: float) -> int:
    return lib().oracle_f64_to_bf16(float(x))


def e2m1_to_f64(code: int) -> float:
    return lib().oracle_e2m1_to_f64(int(code))


def f64_to_e2m1(x: float) -> int:
    return lib().oracle_f64_to_e2m1(float(x))


def ue8m0_to_f64(code: int) -> float:
    return lib().oracle_ue8m0_to_f64(int(code))


def mx_scale_code(amax: float, elem: str) -> int:
    """ue8m0 code of a 32-element block whose largest magnitude is ``amax`` (binary32)."""
    emax, top = {"e4m3": (8, 0.75), "e2m1": (2, 0.5)}[elem]
    return lib().oracle_mx_scale_code(float(np.float32(amax)), emax, top)


def silu(x: float) -> float:
    return lib().oracle_silu(float(x))


# --------------------------------------------------------------------------- routing
def route(logits: np.ndarray, k: int) -> Tuple[np.ndarray, np.ndarray]:
    """Softmax over all experts, keep the k most probable, renormalise over those k.

    Ties go to the lower expert id; slots are in descending probability.  Computed in
    fp64 and stored as int32 ids and fp32 weights.  Renormalisation is over the global
    top-k, before any expert is dropped for living on another rank.
    """
    T, E = logits.shape
    ids = np.zeros((T, k), dtype=np.int32)
    w = np.zeros((T, k), dtype=np.float32)
    for t in range(T):
        l = logits[t].astype(np.float64)
        p = np.exp(l - l.max())
        p = p / p.sum()
        taken: List[int] = []
        for _ in range(k):
            best = -1
            for e in range(E):
                if e in taken:
                    continue
                if best < 0 or p[e] > p[best]:      # strict: lower id wins ties
                    best = e
            taken.append(best)
        psel = np.array([p[e] for e in taken])
        ids[t] = taken
        w[t] = (psel / psel.sum()).astype(np.float32)
    return ids, w


# --------------------------------------------------------------------------- permutation
def permute(ids_batch: np.ndarray, E_local: int, align: int = 128):
    """Layout transform of one grouped invocation.

    ``ids_batch`` is int32 [n_tokens_in_batch, k] with the batch's chunks concatenated
    in batch order, so pair p = t*k + j enumerates (chunk, token, slot) lexicographically.

    Returns dict with
      counts[E]            pairs routed to local expert e
      offsets[E+1]         exclusive scan of counts
      padded_offsets[E+1]  exclusive scan of counts rounded up to ``align`` (tile-aligned
                           group starts)
      row_of_pair[P_all]   compact row offsets[e]+rank, -1 for pairs of non-local experts
      prow_of_pair[P_all]  physical row padded_offsets[e]+rank, -1 likewise
      pair_of_row[P]       inverse of row_of_pair
      pair_of_prow[M_pad]  inverse of prow_of_pair, -1 on padding rows
    rank = number of earlier pairs (pair order) with the same expert: a stable counting
    sort.  The paper aligns each group to the GEMM tile and keeps an inverse map but does
    not fix the order inside a group; stable order is the reading taken.
    """
    flat = np.asarray(ids_batch, dtype=np.int64).reshape(-1)
    E = int(E_local)
    counts = np.zeros(E, dtype=np.int32)
    for e in flat:
        if 0 <= e < E:
            counts[e] += 1
    offsets = np.zeros(E + 1, dtype=np.int32)
    padded = np.zeros(E + 1, dtype=np.int32)
    for e in range(E):
        offsets[e + 1] = offsets[e] + counts[e]
        padded[e + 1] = padded[e] + ((int(counts[e]) + align - 1) // align) * align
    seen = np.zeros(E, dtype=np.int64)
    row_of_pair = np.full(flat.shape[0], -1, dtype=np.int32)
    prow_of_pair = np.full(flat.shape[0], -1, dtype=np.int32)
    pair_of_row = np.full(int(offsets[E]), -1, dtype=np.int32)
    pair_of_prow = np.full(int(padded[E]), -1, dtype=np.int32)
    for p, e in enumerate(flat):
        if 0 <= e < E:
            r = int(seen[e])
            seen[e] += 1
            row_of_pair[p] = offsets[e] + r
            prow_of_pair[p] = padded[e] + r
            pair_of_row[offsets[e] + r] = p
            pair_of_prow[padded[e] + r] = p
    return dict(counts=counts, offsets=offsets, padded_offsets=padded,
                row_of_pair=row_of_pair, prow_of_pair=prow_of_pair,
                pair_of_row=pair_of_row, pair_of_prow=pair_of_prow)


# --------------------------------------------------------------------------- scheduler
MODE_SYNC, MODE_ASYNC, MODE_STREAMFFN = 0, 1, 2


def schedule(pairs_in_submission_order: Sequence[int], mode: int, theta: int, n_streams: int,
             max_chunks_per_invocation: Optional[int] = None):
    """streamFFN launch decisions for one layer call.

    Chunks become ready in submission order, each bringing ``pairs`` ready expert
    tokens.  Ready work accumulates; an invocation is launched as soon as the
    accumulated count reaches theta (Async+streamFFN), at every chunk (Async), or only
    once everything has arrived (Sync).  After the last chunk the threshold is bypassed
    and the remainder runs.  Invocation i uses stream / scratch slot i mod S.

    Returns a list of (chunk positions in the batch, stream) per invocation.
    """
    inv: List[Tuple[List[int], int]] = []
    pending: List[int] = []
    n = 0

    def launch():
        nonlocal pending, n
        inv.append((pending, len(inv) % max(1, n_streams)))
        pending, n = [], 0

    for pos, pairs in enumerate(pairs_in_submission_order):
        pending.append(pos)
        n += int(pairs)
        if mode == MODE_ASYNC or (mode == MODE_STREAMFFN and n >= theta):
            launch()
        elif max_chunks_per_invocation and len(pending) >= max_chunks_per_invocation:
            launch()
    if pending:
        launch()                       # final flush bypasses the threshold
    return inv


# --------------------------------------------------------------------------- the layer
def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def moe_forward(dtype: int, X, Xs, ids, w, Wg, Wgs, Wu, Wus, Wd, Wds, E_local: int,
                sel: Optional[np.ndarray] = None, mirror: int = 0, nthreads: int = 0) -> np.ndarray:
    """fp64 result of the layer for tokens ``sel`` (all tokens when None).

    bf16 tensors are passed as uint16 bit patterns, fp8 tensors as uint8 codes plus fp32
    block scales, F64 tensors as float64.  MXFP4: X e4m3 codes with ue8m0 scales [T,H/32];
    weights one e2m1 code per byte with ue8m0 scales [E,in/32,out].
    Weight layouts: Wg,Wu [E,H,I]; Wd [E,I,H].
    """
    X = np.ascontiguousarray(X)
    T, H = X.shape
    E, H2, I = Wg.shape
    assert H2 == H and Wd.shape == (E, I, H) and Wu.shape == (E, H, I) and E == E_local
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    k = ids.shape[1]
    want = {F64: np.float64, BF16: np.uint16, FP8: np.uint8, MXFP4: np.uint8}[dtype]
    arrs = []
    for a in (X, Wg, Wu, Wd):
        assert a.dtype == want, (a.dtype, want)
        arrs.append(np.ascontiguousarray(a))
    X, Wg, Wu, Wd = arrs
    sdt = np.uint8 if dtype == MXFP4 else np.float32
    for s_ in (Xs, Wgs, Wus, Wds):
        assert s_ is None or s_.dtype == sdt, (s_.dtype, sdt)
    scal = [None if s is None else np.ascontiguousarray(s) for s in (Xs, Wgs, Wus, Wds)]
    if dtype in (FP8, MXFP4):
        assert all(s is not None for s in scal)
    if dtype == MXFP4:
        assert scal[0].shape == (T, H // 32) and scal[1].shape == (E, H // 32, I) and scal[3].shape == (E, I // 32, H)
    if sel is None:
        sel_arr, n_sel = None, T
    else:
        sel_arr = np.ascontiguousarray(sel, dtype=np.int64)
        n_sel = sel_arr.shape[0]
    out = np.empty((n_sel, H), dtype=np.float64)
    rc = lib().oracle_moe_forward(dtype, T, H, I, E, k, _ptr(X), _ptr(scal[0]), _ptr(ids), _ptr(w),
                                  _ptr(Wg), _ptr(scal[1]), _ptr(Wu), _ptr(scal[2]),
                                  _ptr(Wd), _ptr(scal[3]), _ptr(sel_arr), n_sel, mirror,
                                  _ptr(out), nthreads)
    if rc != 0:
        raise ValueError("oracle_moe_forward: bad expert id")
    return out


def num_threads() -> int:
    return lib().oracle_num_threads()


# ------------------------------------------------------------------- torch conveniences
def from_inputs(inp, sel=None, mirror=None, nthreads=0) -> np.ndarray:
    """Run ``moe_forward`` on a ``workloads.MoEInputs`` (tensors are copied to host)."""
    import torch
    fp8 = inp.cfg.dtype == "fp8"
    mx = inp.cfg.dtype == "mxfp4"

    def bits(t):
        t = t.detach().cpu().contiguous()
        return t.view(torch.uint8).numpy() if (fp8 or mx) else t.view(torch.int16).numpy().view(np.uint16)

    def f32(t):
        if t is None:
            return None
        t = t.detach().cpu().contiguous()
        return t.view(torch.uint8).numpy() if mx else t.float().numpy()

    if mirror is None:
        mirror = MIRROR_FP8_ACT if fp8 else (MIRROR_MXFP8_ACT if mx else 0)
    return moe_forward(FP8 if fp8 else (MXFP4 if mx else BF16), bits(inp.x), f32(inp.x_scale),
                       inp.topk_ids.cpu().numpy(), inp.topk_w.cpu().numpy(),
                       bits(inp.w_gate), f32(inp.s_gate), bits(inp.w_up), f32(inp.s_up),
                       bits(inp.w_down), f32(inp.s_down), inp.cfg.E_local, sel=sel,
                       mirror=mirror, nthreads=nthreads)
