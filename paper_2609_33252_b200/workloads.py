"""Seeded synthetic inputs for the streamFFN routed-expert path.

This module only *draws inputs*: random logits, activations and weights with the
shapes and distributions of the benchmark configurations, the router decision
that turns logits into (topk_ids, topk_weights), dtype casts (bf16, block-scaled
e4m3) and the chunk / arrival schedule.  It contains none of the arithmetic of the
path itself (no permutation, no expert FFN, no combine) and is the one module the
CUDA path's harnesses and the CPU oracle's tests both use.

Inputs stand in for the serving traces the paper evaluates on ("Evaluation Settings", workloads):
those traces are not available, so every tensor is synthetic and seeded.

Representation: all tensors are torch tensors on ``device``.  bf16 tensors are
``torch.bfloat16``; block-scaled fp8 tensors are a ``torch.float8_e4m3fn`` code
tensor plus an fp32 scale tensor (``value = code * scale``).  Microscaling ("mxfp4")
configurations: activations are ``torch.float8_e4m3fn`` codes with ``uint8`` ue8m0
scales per 1x32 block along the hidden dimension; weights are ``uint8`` tensors holding
one e2m1 code (low four bits) per element with ``uint8`` ue8m0 scales per 32 elements of
the input (contraction) dimension and per output column (``value = code * 2^(scale-127)``).
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence

import torch

SEED_BASE = 0xCA5CADE0
FP8_MAX = 448.0
BLOCK = 128


@dataclasses.dataclass(frozen=True)
class MoEConfig:
    """One benchmark configuration (shapes of the MoE layer and its chunking)."""
    name: str
    index: int                 # position in the benchmark's config list (seeds derive from it)
    T: int                     # tokens in the layer call
    H: int                     # hidden size
    I: int                     # expert intermediate size
    E_global: int              # routed experts in the whole layer
    E_local: int               # experts resident on this rank: ids 0..E_local-1
    k: int                     # experts per token
    chunks: Sequence[int]      # tokens per replica chunk, in chunk-id order
    dtype: str = "bf16"        # "bf16" | "fp8" | "mxfp4"
    zipf_s: float = 0.0        # 0 => N(0,1) logits; >0 => logits biased by -s*ln(rank)
    zipf_strided: bool = False  # popularity rank strided across ranks instead of literal
    arrival_sigma: float = 0.5  # lognormal(0, sigma) arrival offsets
    straggler_last: bool = False

    @property
    def n_chunks(self) -> int:
        return len(self.chunks)


def _equal_chunks(T: int, n: int) -> List[int]:
    base = T // n
    out = [base] * n
    out[-1] += T - base * n
    return out


CONFIGS = {
    "tiny": MoEConfig("tiny", 0, T=256, H=512, I=256, E_global=8, E_local=8, k=2,
                      chunks=(160, 96)),
    "mid": MoEConfig("mid", 1, T=4096, H=2048, I=768, E_global=64, E_local=64, k=6,
                     chunks=(1536, 1024, 1024, 512)),
    "ep_shard": MoEConfig("ep_shard", 2, T=16384, H=7168, I=2048, E_global=256, E_local=32, k=8,
                          chunks=tuple(_equal_chunks(16384, 8)), zipf_s=1.1),
    "ep_shard_strided": MoEConfig("ep_shard_strided", 2, T=16384, H=7168, I=2048, E_global=256,
                                  E_local=32, k=8, chunks=tuple(_equal_chunks(16384, 8)),
                                  zipf_s=1.1, zipf_strided=True),
    "straggler": MoEConfig("straggler", 3, T=16384, H=7168, I=2048, E_global=256, E_local=32, k=8,
                           chunks=(1404,) * 7 + (16384 - 7 * 1404,), zipf_s=1.1,
                           straggler_last=True),
    # reduced EP shard (same H, I, k and routing recipe; 8 of 64 experts, 2048 tokens): the case small
    # enough for multi-pass profiler captures while its weights (0.7 GB) still exceed the L2
    "ep_shard_small": MoEConfig("ep_shard_small", 2, T=2048, H=7168, I=2048, E_global=64, E_local=8, k=8,
                                chunks=tuple(_equal_chunks(2048, 8)), zipf_s=1.1),
    "fp8_shard_small": MoEConfig("fp8_shard_small", 4, T=2048, H=7168, I=3072, E_global=64, E_local=8, k=8,
                                 chunks=tuple(_equal_chunks(2048, 8)), dtype="fp8", zipf_s=1.1),
    "fp8_shard": MoEConfig("fp8_shard", 4, T=32768, H=7168, I=3072, E_global=512, E_local=64, k=8,
                           chunks=tuple(_equal_chunks(32768, 8)), dtype="fp8", zipf_s=1.1),
    # microscaling variant of the EP shard ("Evaluation Settings", models and environments: MXFP4 routed-expert weights): same shapes and routing
    "mxfp4_tiny": MoEConfig("mxfp4_tiny", 5, T=256, H=512, I=256, E_global=8, E_local=8, k=2,
                            chunks=(160, 96), dtype="mxfp4"),
    "mxfp4_shard_small": MoEConfig("mxfp4_shard_small", 5, T=2048, H=7168, I=2048, E_global=64, E_local=8, k=8,
                                   chunks=tuple(_equal_chunks(2048, 8)), dtype="mxfp4", zipf_s=1.1),
    "mxfp4_straggler": MoEConfig("mxfp4_straggler", 5, T=16384, H=7168, I=2048, E_global=256, E_local=32, k=8,
                                 chunks=(1404,) * 7 + (16384 - 7 * 1404,), dtype="mxfp4", zipf_s=1.1, straggler_last=True),
    "mxfp4_shard": MoEConfig("mxfp4_shard", 5, T=16384, H=7168, I=2048, E_global=256, E_local=32, k=8,
                             chunks=tuple(_equal_chunks(16384, 8)), dtype="mxfp4", zipf_s=1.1),
    # one EP rank's shard of the larger MXFP4 model of the paper's model table ("Evaluation Settings": 384 routed
    # experts per layer, 6 per token, expert intermediate size 3072); the hidden size is not in the paper: 7168 assumed
    "mxfp4_pro_shard": MoEConfig("mxfp4_pro_shard", 6, T=16384, H=7168, I=3072, E_global=384, E_local=48, k=6,
                                 chunks=tuple(_equal_chunks(16384, 8)), dtype="mxfp4", zipf_s=1.1),
}


def scaled(cfg: MoEConfig, **kw) -> MoEConfig:
    """A copy of ``cfg`` with some fields replaced (used for reduced test shapes)."""
    return dataclasses.replace(cfg, **kw)


@dataclasses.dataclass
class MoEInputs:
    cfg: MoEConfig
    x: torch.Tensor                 # [T,H] bf16 or e4m3 codes
    x_scale: Optional[torch.Tensor]  # fp8: [T,H/128] fp32
    topk_ids: torch.Tensor          # [T,k] int32 global expert ids, slot order = descending prob
    topk_w: torch.Tensor            # [T,k] fp32, renormalised over the k selected
    w_gate: torch.Tensor            # [E_local,H,I]
    w_up: torch.Tensor              # [E_local,H,I]
    w_down: torch.Tensor            # [E_local,I,H]
    s_gate: Optional[torch.Tensor]  # fp8: [E_local,H/128,I/128] fp32
    s_up: Optional[torch.Tensor]
    s_down: Optional[torch.Tensor]  # fp8: [E_local,I/128,H/128] fp32
    logits: Optional[torch.Tensor]  # [T,E_global] fp32 (kept for routing tests)
    chunk_offsets: List[int]        # first token of each chunk
    arrival: List[float]            # unitless arrival offset per chunk (scaled by the harness)

    def n_local_pairs(self) -> int:
        return int((self.topk_ids < self.cfg.E_local).sum().item())


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _randn_chunked(shape, std, gen, device, out_dtype, chunk_elems=1 << 27):
    """N(0, std) drawn in fp32 slabs along dim 0 and cast, to bound peak memory."""
    n0 = shape[0]
    rest = 1
    for s in shape[1:]:
        rest *= s
    out = torch.empty(shape, dtype=out_dtype, device=device)
    rows = max(1, chunk_elems // max(rest, 1))
    for r0 in range(0, n0, rows):
        r1 = min(n0, r0 + rows)
        blk = torch.randn((r1 - r0,) + tuple(shape[1:]), generator=gen, device=device,
                          dtype=torch.float32)
        if std != 1.0:
            blk.mul_(std)
        out[r0:r1].copy_(blk)
    return out


def make_logits(cfg: MoEConfig, device="cpu") -> torch.Tensor:
    """Router logits fp32 [T,E_global]: N(0,1), minus s*ln(popularity rank) when skewed."""
    g = _gen(SEED_BASE + 16 * cfg.index + 0, device)
    logits = torch.randn((cfg.T, cfg.E_global), generator=g, device=device, dtype=torch.float32)
    if cfg.zipf_s > 0.0:
        e = torch.arange(cfg.E_global, device=device, dtype=torch.float64)
        if cfg.zipf_strided:
            ranks_per = cfg.E_global // cfg.E_local
            rank = 1 + (e % cfg.E_local) * ranks_per + torch.floor(e / cfg.E_local)
        else:
            rank = e + 1
        logits = (logits.double() - cfg.zipf_s * torch.log(rank)[None, :]).float()
    return logits


def route(logits: torch.Tensor, k: int):
    """Router decision for the synthetic inputs: softmax, top-k, renormalise.

    Ties go to the lower expert id; slots are ordered by descending probability.
    Weights are the selected probabilities divided by their sum (computed in fp64,
    stored fp32).  This is input preparation, not part of the timed path.
    """
    l64 = logits.double()
    order = torch.sort(l64, dim=1, descending=True, stable=True).indices[:, :k]
    sel = torch.gather(l64, 1, order)
    p = torch.exp(sel - l64.max(dim=1, keepdim=True).values)
    w = p / p.sum(dim=1, keepdim=True)
    return order.to(torch.int32).contiguous(), w.to(torch.float32).contiguous()


def quantize_rows_1x128(x: torch.Tensor):
    """Block-scale an fp32 [R,C] matrix along C in 1x128 blocks to e4m3 codes + fp32 scales."""
    R, C = x.shape
    assert C % BLOCK == 0
    xb = x.float().view(R, C // BLOCK, BLOCK)
    amax = xb.abs().amax(dim=2)
    scale = (amax / FP8_MAX).float()
    scale = torch.where(amax == 0, torch.ones_like(scale), scale)
    q = (xb / scale[:, :, None]).clamp_(-FP8_MAX, FP8_MAX).to(torch.float8_e4m3fn)
    return q.view(R, C), scale.contiguous()


def quantize_blocks_128x128(w: torch.Tensor):
    """Block-scale an fp32 [E,R,C] tensor in 128x128 blocks over (R,C)."""
    E, R, C = w.shape
    assert R % BLOCK == 0 and C % BLOCK == 0
    wb = w.float().view(E, R // BLOCK, BLOCK, C // BLOCK, BLOCK)
    amax = wb.abs().amax(dim=(2, 4))
    scale = (amax / FP8_MAX).float()
    scale = torch.where(amax == 0, torch.ones_like(scale), scale)
    q = (wb / scale[:, :, None, :, None]).clamp_(-FP8_MAX, FP8_MAX).to(torch.float8_e4m3fn)
    return q.view(E, R, C), scale.contiguous()


MX_BLOCK = 32


def mx_scale_codes(amax: torch.Tensor, elem: str) -> torch.Tensor:
    """ue8m0 code of the smallest power of two s with amax <= elem_max * s (127 for amax == 0)."""
    emax, top = {"e4m3": (8, 0x600000), "e2m1": (2, 0x400000)}[elem]
    bits = amax.float().contiguous().view(torch.int32)
    code = ((bits >> 23) & 0xFF) - emax + ((bits & 0x7FFFFF) > top).to(torch.int32)
    code = code.clamp_(0, 254)
    return torch.where(amax == 0, torch.full_like(code, 127), code).to(torch.uint8)


def _to_e2m1(y: torch.Tensor) -> torch.Tensor:
    """Round-to-nearest-even of fp32 values with |y| <= 6 onto the e2m1 grid; uint8 codes."""
    a = y.abs()
    code = ((a > 0.25).to(torch.uint8) + (a >= 0.75).to(torch.uint8) + (a > 1.25).to(torch.uint8) +
            (a >= 1.75).to(torch.uint8) + (a > 2.5).to(torch.uint8) + (a >= 3.5).to(torch.uint8) +
            (a > 5.0).to(torch.uint8))
    return code | (torch.signbit(y).to(torch.uint8) << 3)


def quantize_mx(x: torch.Tensor, elem: str, dim: int):
    """Microscaling quantisation of an fp32 tensor in blocks of 32 along ``dim``.

    Returns (codes, scales): codes have the shape of x (``float8_e4m3fn`` for "e4m3", ``uint8``
    with the code in the low four bits for "e2m1"); scales are uint8 ue8m0 codes with ``dim``
    shrunk by 32.
    """
    x = x.float().movedim(dim, -1)
    shp = x.shape
    assert shp[-1] % MX_BLOCK == 0
    xb = x.reshape(shp[:-1] + (shp[-1] // MX_BLOCK, MX_BLOCK))
    sc = mx_scale_codes(xb.abs().amax(dim=-1), elem)
    y = xb * torch.exp2(127.0 - sc.float())[..., None]          # exact: a power of two
    if elem == "e4m3":
        q = y.clamp_(-FP8_MAX, FP8_MAX).to(torch.float8_e4m3fn)
    else:
        q = _to_e2m1(y)
    return q.reshape(shp).movedim(-1, dim).contiguous(), sc.movedim(-1, dim).contiguous()


def make_arrivals(cfg: MoEConfig) -> List[float]:
    """Unitless lognormal(0, sigma) arrival offsets, one per chunk (CPU generator)."""
    g = _gen(SEED_BASE + 16 * cfg.index + 5, "cpu")
    z = torch.randn(cfg.n_chunks, generator=g, dtype=torch.float64)
    a = torch.exp(cfg.arrival_sigma * z)
    a = a - a.min()
    if cfg.straggler_last:
        # the chunk holding the most tokens arrives last
        big = max(range(cfg.n_chunks), key=lambda c: cfg.chunks[c])
        a[big] = a.max() + 0.25
    return [float(v) for v in a]


def make_inputs(cfg: MoEConfig, device="cpu", keep_logits=True) -> MoEInputs:
    """Draw every tensor of one configuration.  Deterministic for (cfg, device type)."""
    assert sum(cfg.chunks) == cfg.T
    seed = SEED_BASE + 16 * cfg.index
    logits = make_logits(cfg, device)
    ids, w = route(logits, cfg.k)
    H, I, E = cfg.H, cfg.I, cfg.E_local
    fp8 = cfg.dtype == "fp8"
    sg = su = sd = xs = None
    if cfg.dtype == "mxfp4":
        x32 = torch.randn((cfg.T, H), generator=_gen(seed + 1, device), device=device)
        x, xs = quantize_mx(x32, "e4m3", 1)
        del x32

        def mxweights(shape, std, sd_):
            g = _gen(sd_, device)
            codes = torch.empty(shape, dtype=torch.uint8, device=device)
            scales = torch.empty((shape[0], shape[1] // MX_BLOCK, shape[2]), dtype=torch.uint8, device=device)
            for e in range(shape[0]):
                blk = torch.randn(tuple(shape[1:]), generator=g, device=device) * std
                codes[e], scales[e] = quantize_mx(blk, "e2m1", 0)
            return codes, scales
        wg, sg = mxweights((E, H, I), H ** -0.5, seed + 2)
        wu, su = mxweights((E, H, I), H ** -0.5, seed + 3)
        wd, sd = mxweights((E, I, H), I ** -0.5, seed + 4)
    elif not fp8:
        x = _randn_chunked((cfg.T, H), 1.0, _gen(seed + 1, device), device, torch.bfloat16)
        wg = _randn_chunked((E, H, I), H ** -0.5, _gen(seed + 2, device), device, torch.bfloat16)
        wu = _randn_chunked((E, H, I), H ** -0.5, _gen(seed + 3, device), device, torch.bfloat16)
        wd = _randn_chunked((E, I, H), I ** -0.5, _gen(seed + 4, device), device, torch.bfloat16)
    else:
        x32 = torch.randn((cfg.T, H), generator=_gen(seed + 1, device), device=device)
        x, xs = quantize_rows_1x128(x32)
        del x32

        def qweights(shape, std, sd_):
            g = _gen(sd_, device)
            codes = torch.empty(shape, dtype=torch.float8_e4m3fn, device=device)
            scales = torch.empty((shape[0], shape[1] // BLOCK, shape[2] // BLOCK),
                                 dtype=torch.float32, device=device)
            for e in range(shape[0]):
                blk = torch.randn((1,) + tuple(shape[1:]), generator=g, device=device) * std
                q, s = quantize_blocks_128x128(blk)
                codes[e] = q[0]
                scales[e] = s[0]
            return codes, scales
        wg, sg = qweights((E, H, I), H ** -0.5, seed + 2)
        wu, su = qweights((E, H, I), H ** -0.5, seed + 3)
        wd, sd = qweights((E, I, H), I ** -0.5, seed + 4)
    offs, acc = [], 0
    for c in cfg.chunks:
        offs.append(acc)
        acc += c
    return MoEInputs(cfg, x, xs, ids, w, wg, wu, wd, sg, su, sd,
                     logits if keep_logits else None, offs, make_arrivals(cfg))


def submission_order(arrival: Sequence[float]) -> List[int]:
    """Chunk ids ordered by arrival offset (ties by id)."""
    return sorted(range(len(arrival)), key=lambda c: (arrival[c], c))
