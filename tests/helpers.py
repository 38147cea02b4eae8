"""Shared helpers of the GPU parity tests (no arithmetic of the path lives here)."""
import numpy as np
import torch

import paper_2609_33252_b200 as cep
from paper_2609_33252_b200 import workloads as wl

REL_FRO_TOL = 5e-3          # relative Frobenius error against the fp64 oracle
ELEM_TOL = 2e-2             # |delta| <= ELEM_TOL * max(1, |ref|) per element


def chunks_of(inp):
    cfg = inp.cfg
    out = []
    for off, n in zip(inp.chunk_offsets, cfg.chunks):
        xs = None if inp.x_scale is None else inp.x_scale[off:off + n]
        out.append((off, inp.x[off:off + n], xs, inp.topk_ids[off:off + n], inp.topk_w[off:off + n]))
    return out


def make_layer(cfg, mode=cep.CEP_MODE_SYNC, theta=0, n_streams=2, gemm_impl=cep.CEP_GEMM_TCGEN05, max_chunks=None,
               debug_checks=0, gather_a=0):
    dt = cep.DTYPE_OF[cfg.dtype]
    return cep.MoELayer(cfg.H, cfg.I, cfg.E_global, cfg.E_local, cfg.k, cfg.T, max_chunks or max(cfg.n_chunks, 1),
                        dtype=dt, mode=mode, n_streams=n_streams, threshold_pairs=theta, gemm_impl=gemm_impl,
                        debug_checks=debug_checks, gather_a=gather_a)


def run_layer(inp, layer, order=None, local_pairs=False):
    cfg = inp.cfg
    out = torch.full((cfg.T, cfg.H), float("nan"), dtype=torch.bfloat16, device=inp.x.device)
    ch = chunks_of(inp)
    nlp = None
    if local_pairs:
        nlp = [int((c[3] < cfg.E_local).sum().item()) for c in ch]
    n_inv = layer.run(out, ch, order=order, n_local_pairs=nlp)
    torch.cuda.synchronize()
    st = cep.ffn_status(layer.plan)
    assert st == 0, cep.STATUS_NAMES.get(st, st)
    return out, n_inv


def to_device(inp, device="cuda"):
    import dataclasses
    kw = {}
    for f in dataclasses.fields(inp):
        v = getattr(inp, f.name)
        kw[f.name] = v.to(device) if isinstance(v, torch.Tensor) else v
    return type(inp)(**kw)


def check_close(got_bf16: torch.Tensor, ref: np.ndarray, what=""):
    got = got_bf16.detach().double().cpu().numpy()
    assert np.isfinite(got).all(), what + ": non-finite output"
    num = np.linalg.norm(got - ref)
    den = max(np.linalg.norm(ref), 1e-30)
    rel = num / den
    worst = np.max(np.abs(got - ref) / np.maximum(1.0, np.abs(ref)))
    assert rel <= REL_FRO_TOL, "%s: relative Frobenius error %.3e > %.1e" % (what, rel, REL_FRO_TOL)
    assert worst <= ELEM_TOL, "%s: worst element error %.3e > %.1e" % (what, worst, ELEM_TOL)
    return rel, worst


def batch_ids(inp, chunk_positions):
    """ids of a batch with its chunks concatenated in batch order (numpy int32 [n,k])."""
    cfg = inp.cfg
    parts = []
    for c in chunk_positions:
        off, n = inp.chunk_offsets[c], cfg.chunks[c]
        parts.append(inp.topk_ids[off:off + n].cpu().numpy())
    return np.concatenate(parts) if parts else np.zeros((0, cfg.k), np.int32)
