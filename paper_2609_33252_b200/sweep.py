"""Threshold sweep on the attention-imbalance configuration (8 replicas, one straggler holding 40 % of the
tokens and arriving last): completion latency of Async+streamFFN for each batch threshold, under both readings
of "tokens per expert batch" (theta in ready local pairs per invocation, and theta = E_local x that many rows
per expert), against one synchronous launch once everything has arrived ("Deep Dive", ablation study: the modes; Section 3.2:
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

    def make(mode, theta, S, defer=0):
        L = cep.MoELayer(cfg.H, cfg.I, cfg.E_global, cfg.E_local, cfg.k, cfg.T, cfg.n_chunks, dtype=dt, mode=mode,
                         n_streams=S, threshold_pairs=theta, defer_while_busy=defer)
        L.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)
        return L

    sync_layer = make(cep.CEP_MODE_SYNC, 0, 1)

    def measure(L, arrival):
        """The cell and the synchronous launch take turns, so both see the same clock and power state."""
        ts, ts_sync, ninv = [], [], 0
        for r in range(warm + reps):
            t_s, _ = run_with_arrivals(sync_layer, out, chunks, arrival, pairs, rstreams)
            t, ninv = run_with_arrivals(L, out, chunks, arrival, pairs, rstreams)
            if r >= warm:
                ts.append(t); ts_sync.append(t_s)
        med, med_sync = statistics.median(ts) * 1e3, statistics.median(ts_sync) * 1e3
        return {"median_ms": med, "min_ms": min(ts) * 1e3, "invocations": ninv, "sync_alongside_ms": med_sync,
                "sync_over_cell": med_sync / med}

    zero = [0.0] * cfg.n_chunks
    t_sync = statistics.median([run_with_arrivals(sync_layer, out, chunks, zero, pairs, rstreams)[0] for _ in range(warm + reps)][warm:])
    report = {"config": name, "chunk_tokens": list(cfg.chunks), "chunk_local_pairs": pairs, "t_sync_ms": t_sync * 1e3,
              "arrival_offsets_unitless": inp.arrival, "cases": []}
    thetas = [("pairs", t) for t in (256, 512, 1024, 2048)] + [("rows_per_expert", cfg.E_local * t) for t in (256, 512, 1024, 2048)]
    for tau in taus:
        arrival = [tau * t_sync * a for a in inp.arrival]
        L = make(cep.CEP_MODE_ASYNC, 0, 1)
        case = {"tau": tau, "last_arrival_ms": max(arrival) * 1e3, "async": measure(L, arrival), "streamffn": []}
        L.close()
        for reading, theta in thetas:
            for S, defer in [(S_, 0) for S_ in streams] + [(2, 1)]:
                L = make(cep.CEP_MODE_STREAMFFN, theta, S, defer)
                m = measure(L, arrival)
                L.close()
                m.update({"reading": reading, "theta_pairs": theta, "streams": S, "defer_while_busy": defer})
                case["streamffn"].append(m)
        report["cases"].append(case)
    sync_layer.close()
    return report


if __name__ == "__main__":
    print(json.dumps(sweep(sys.argv[1] if len(sys.argv) > 1 else "straggler")))
