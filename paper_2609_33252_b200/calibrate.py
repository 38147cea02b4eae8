"""Launch-threshold calibration (Section 3.2 "Launch threshold"; Section 3.3, Eq. 2: FFN latency model).

The measurement itself lives in the library (``cep_calibrate``: uniform rows per expert, plus the stream
probe; ``cep_calibrate_routed``: growing prefixes of a real batch, so theta reflects the router's skew).  It
profiles the expert-FFN throughput of THIS library on THIS GPU as a function of the expert-token count of
one invocation, sets theta to the smallest profiled count that reaches a fraction rho of the observed peak,
and returns the normalised efficiency eta(N) = throughput(N) / peak, from which the paper's latency model
F(N) = N / (eta(N) * P_peak) follows.  The functions here only draw a configuration's inputs, allocate the
scratch tensors and forward the pointers.
"""
from __future__ import annotations

import json
import sys
from typing import Dict, Sequence

from . import binding as cep
from . import workloads as wl


def calibrate_in_library(cfg: wl.MoEConfig, rho: float = 0.90, rows: Sequence[int] = (64, 128, 256, 512, 1024, 2048),
                         reps: int = 5, n_streams: int = 4, device="cuda") -> Dict:
    """``cep_calibrate`` on a configuration's shapes: profile with uniform rows per expert, theta(rho) and the number
    of compute streams a chain of theta-sized invocations wants."""
    import torch
    inp = wl.make_inputs(wl.scaled(cfg, T=8, chunks=(8,)), device=device, keep_logits=False)   # weights only
    E, k, H, I = cfg.E_local, cfg.k, cfg.H, cfg.I
    k_loc = min(k, E)
    T_max = max(1, max(rows) * E // k_loc)
    layer = cep.MoELayer(H, I, cfg.E_global, E, k, T_max, 8, dtype=cep.DTYPE_OF[cfg.dtype], mode=cep.CEP_MODE_SYNC,
                         n_streams=n_streams, profile_kernels=1)
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)
    x32 = torch.randn((T_max, H), generator=torch.Generator(device=device).manual_seed(wl.SEED_BASE + 99), device=device)
    if cfg.dtype == "fp8":
        x, xs = wl.quantize_rows_1x128(x32)
    elif cfg.dtype == "mxfp4":
        x, xs = wl.quantize_mx(x32, "e4m3", 1)
    else:
        x, xs = x32.to(torch.bfloat16), None
    del x32
    ids = torch.empty((T_max, k), dtype=torch.int32, device=device)
    w = torch.empty((T_max, k), dtype=torch.float32, device=device)
    out = torch.empty((T_max, H), dtype=torch.bfloat16, device=device)
    points, result = cep.cep_calibrate(layer.plan, rho, list(rows), reps, x, xs, ids, w, out)
    layer.close()
    result.update({"config": cfg.name, "profile": points})
    return result


def calibrate_on_routing(cfg: wl.MoEConfig, rho: float = 0.90, fractions: Sequence[float] = (1 / 32, 1 / 16, 1 / 8, 1 / 4, 3 / 8, 1 / 2, 3 / 4, 1.0),
                         reps: int = 5, device="cuda") -> Dict:
    """``cep_calibrate_routed`` on a configuration's own (skewed) routing: the profile points are prefixes of the
    configuration's batch holding the given fractions of its tokens."""
    import torch
    inp = wl.make_inputs(cfg, device=device, keep_logits=False)
    layer = cep.MoELayer(cfg.H, cfg.I, cfg.E_global, cfg.E_local, cfg.k, cfg.T, 1, dtype=cep.DTYPE_OF[cfg.dtype],
                         mode=cep.CEP_MODE_SYNC, n_streams=1, profile_kernels=1)
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)
    out = torch.empty((cfg.T, cfg.H), dtype=torch.bfloat16, device=device)
    n_tokens = sorted({max(1, int(round(f * cfg.T))) for f in fractions})
    points, result = cep.cep_calibrate_routed(layer.plan, rho, n_tokens, reps, inp.x, inp.x_scale, inp.topk_ids, inp.topk_w, out)
    layer.close()
    result.update({"config": cfg.name, "profile": points})
    return result


if __name__ == "__main__":
    name = sys.argv[1] if len(sys.argv) > 1 else "ep_shard"
    if len(sys.argv) > 2 and sys.argv[2] == "routed":
        print(json.dumps(calibrate_on_routing(wl.CONFIGS[name])))
    else:
        print(json.dumps(calibrate_in_library(wl.CONFIGS[name])))
