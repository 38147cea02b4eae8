"""Launch-threshold calibration (Section 3.2 "Launch threshold"; Section 4.2 FFN latency model).

Profiles the expert-FFN throughput of THIS library on THIS GPU as a function of the expert-token
count of one invocation (uniform rows per expert, the shapes of a configuration), and sets theta to the
smallest profiled count that reaches a fraction rho of the observed peak.  Also returns the normalised
efficiency eta(N) = throughput(N) / peak, from which the paper's FFN latency model
F(N) = N / (eta(N) * P_peak) follows.  This is a measurement harness over the C ABI: every timed
kernel is the library's.
"""
from __future__ import annotations

import json
import statistics
import sys
from typing import Dict, List, Sequence

from . import binding as cep
from . import workloads as wl


def uniform_routing(rows_per_expert: int, E: int, k: int, device):
    """ids [T,k] giving every local expert exactly rows_per_expert rows (T = rows*E/k tokens)."""
    import torch
    T = max(1, rows_per_expert * E // k)
    t = torch.arange(T, device=device, dtype=torch.int64)[:, None]
    j = torch.arange(k, device=device, dtype=torch.int64)[None, :]
    ids = ((t * k + j) % E).to(torch.int32).contiguous()
    w = torch.full((T, k), 1.0 / k, dtype=torch.float32, device=device)
    return ids, w


def profile(cfg: wl.MoEConfig, rows: Sequence[int] = (16, 32, 64, 128, 256, 512, 1024, 2048, 4096),
            reps: int = 5, device="cuda") -> List[Dict]:
    import torch
    inp = wl.make_inputs(wl.scaled(cfg, T=8, chunks=(8,)), device=device, keep_logits=False)   # weights only
    E, k, H, I = cfg.E_local, min(cfg.k, cfg.E_local), cfg.H, cfg.I
    fp8 = cfg.dtype == "fp8"
    max_T = max(rows) * E // k
    layer = cep.MoELayer(H, I, E, E, k, max_T, 1, dtype=cep.DTYPE_OF[cfg.dtype],
                         mode=cep.CEP_MODE_SYNC, n_streams=1, profile_kernels=1)
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)
    g = torch.Generator(device=device).manual_seed(wl.SEED_BASE + 99)
    out_rows = []
    for m in rows:
        ids, w = uniform_routing(m, E, k, device)
        T = ids.shape[0]
        x32 = torch.randn((T, H), generator=g, device=device)
        if fp8:
            x, xs = wl.quantize_rows_1x128(x32)
        elif cfg.dtype == "mxfp4":
            x, xs = wl.quantize_mx(x32, "e4m3", 1)
        else:
            x, xs = x32.to(torch.bfloat16), None
        out = torch.empty((T, H), dtype=torch.bfloat16, device=device)
        g1, g2, tot = [], [], []
        for r in range(reps + 2):
            layer.run(out, [(0, x, xs, ids, w)])
            torch.cuda.synchronize()
            info = cep.ffn_query(layer.plan, 0)
            if r >= 2:
                g1.append(info.gemm1_ms); g2.append(info.gemm2_ms); tot.append(info.elapsed_ms)
        pairs = T * k
        ffn_ms = statistics.median(g1) + statistics.median(g2)
        out_rows.append({"rows_per_expert": m, "expert_tokens": pairs, "ffn_ms": ffn_ms,
                         "layer_ms": statistics.median(tot), "tflops": 6.0 * H * I * pairs / (ffn_ms * 1e-3) / 1e12})
    layer.close()
    return out_rows


def calibrate(cfg: wl.MoEConfig, rho: float = 0.90, **kw) -> Dict:
    """theta = smallest profiled expert-token count whose throughput is >= rho * observed peak."""
    prof = profile(cfg, **kw)
    peak = max(p["tflops"] for p in prof)
    for p in prof:
        p["eta"] = p["tflops"] / peak
    theta = next(p["expert_tokens"] for p in prof if p["eta"] >= rho)
    return {"config": cfg.name, "rho": rho, "peak_tflops": peak, "theta_pairs": theta,
            "theta_rows_per_expert": theta // cfg.E_local, "profile": prof}


def calibrate_in_library(cfg: wl.MoEConfig, rho: float = 0.90, rows: Sequence[int] = (64, 128, 256, 512, 1024, 2048),
                         reps: int = 5, n_streams: int = 4, device="cuda") -> Dict:
    """The same calibration done by the library itself (``cep_calibrate``): profile, theta(rho) and the number of
    compute streams a chain of theta-sized invocations wants.  This wrapper only allocates the scratch tensors."""
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


if __name__ == "__main__":
    name = sys.argv[1] if len(sys.argv) > 1 else "ep_shard"
    if len(sys.argv) > 2 and sys.argv[2] == "library":
        print(json.dumps(calibrate_in_library(wl.CONFIGS[name])))
    else:
        print(json.dumps(calibrate(wl.CONFIGS[name])))
