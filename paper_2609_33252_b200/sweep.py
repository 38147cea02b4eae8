"""Threshold sweep on the attention-imbalance configuration (8 replicas, one straggler holding 40 % of the
tokens and arriving last): completion latency of Async+streamFFN for each batch threshold, under both readings
of "tokens per expert batch" (theta in ready local pairs per invocation, and theta = E_local x that many rows
per expert), against one synchronous launch once everything has arrived (Section 5.4 modes; Section 3.2
threshold and multi-stream execution).  A measurement harness over the C ABI; prints one JSON object.
"""
from __future__ import annotations

import json
import statistics
import sys

from . import binding as cep
from . import workloads as wl
from .arrivals import run_with_arrivals


def sweep(name="straggler", taus=(0.0, 0.5), streams=(1, 2, 4), warm=3, reps=10, device="cuda"):
    import torch
    cfg = wl.CONFIGS[name]
    inp = wl.make_inputs(cfg, device=device, keep_logits=False)
    chunks = [(o, inp.x[o:o + n], None if inp.x_scale is None else inp.x_scale[o:o + n], inp.topk_ids[o:o + n],
               inp.topk_w[o:o + n]) for o, n in zip(inp.chunk_offsets, cfg.chunks)]
    pairs = [int((c[3] < cfg.E_local).sum().item()) for c in chunks]
    out = torch.empty(cfg.T, cfg.H, dtype=torch.bfloat16, device=device)
    rstreams = [torch.cuda.Stream() for _ in chunks]
    dt = cep.DTYPE_OF[cfg.dtype]

    def measure(mode, theta, S, arrival):
        L = cep.MoELayer(cfg.H, cfg.I, cfg.E_global, cfg.E_local, cfg.k, cfg.T, cfg.n_chunks, dtype=dt, mode=mode,
                         n_streams=S, threshold_pairs=theta)
        L.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)
        ts, ninv = [], 0
        for r in range(warm + reps):
            t, ninv = run_with_arrivals(L, out, chunks, arrival, pairs, rstreams)
            if r >= warm:
                ts.append(t)
        L.close()
        return {"median_ms": statistics.median(ts) * 1e3, "min_ms": min(ts) * 1e3, "invocations": ninv}

    t_sync = measure(cep.CEP_MODE_SYNC, 0, 1, [0.0] * cfg.n_chunks)["median_ms"] * 1e-3
    report = {"config": name, "chunk_tokens": list(cfg.chunks), "chunk_local_pairs": pairs, "t_sync_ms": t_sync * 1e3,
              "arrival_offsets_unitless": inp.arrival, "cases": []}
    thetas = [("pairs", t) for t in (256, 512, 1024, 2048)] + [("rows_per_expert", cfg.E_local * t) for t in (256, 512, 1024, 2048)]
    for tau in taus:
        arrival = [tau * t_sync * a for a in inp.arrival]
        case = {"tau": tau, "last_arrival_ms": max(arrival) * 1e3,
                "sync": measure(cep.CEP_MODE_SYNC, 0, 1, arrival),
                "async": measure(cep.CEP_MODE_ASYNC, 0, 1, arrival), "streamffn": []}
        for reading, theta in thetas:
            for S in streams:
                m = measure(cep.CEP_MODE_STREAMFFN, theta, S, arrival)
                m.update({"reading": reading, "theta_pairs": theta, "streams": S})
                case["streamffn"].append(m)
        report["cases"].append(case)
    return report


if __name__ == "__main__":
    print(json.dumps(sweep(sys.argv[1] if len(sys.argv) > 1 else "straggler")))
