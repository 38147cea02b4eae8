#!/usr/bin/env python
"""Benchmark of the streamFFN routed-expert path on B200.

One "step" = one pass of the whole hot path (layout transform, both expert GEMMs with the
fused activation, weighted combine) over one batch of synthetic routed tokens, all chunks
present, through the C ABI.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config ep_shard|mid|...]
  python bench.py --impl reference ...     # times the CPU oracle on a bounded sample
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "MoE-layer prefill tokens/s (streamFFN routed-expert path: permute + grouped SwiGLU expert FFN + combine)"
UNIT = "tokens/s"
NOMINAL_BF16_TFLOPS = 2250.0
# measured DRAM traffic of GEMM1 per launch: one record per workload, each naming the profiler command, date,
# commit and the hash of the kernel source it was captured from
TRAFFIC_RECORD = os.path.join(ROOT, "profiles", "gemm1_dram_traffic.json")
KERNEL_SOURCE = {"bf16": "gemm_tcgen05.cu", "fp8": "gemm_tcgen05_fp8.cu", "mxfp4": "gemm_tcgen05_mx.cu"}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


class ClockSampler:
    """Samples SM clock, power and throttle reasons with nvidia-smi (a read-only query) while the timed region
    runs.  The GPU is addressed by its UUID (an index would ignore CUDA_VISIBLE_DEVICES); every sample carries
    the host time it was read at, and only samples taken between the region's two synchronisation points count."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.gpu_id, self.rows, self.proc = gpu_id, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.gpu_id, "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t_begin: float, t_end: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

        def fold(rows):
            sm, mx, reasons, power = [], [], set(), []
            for _, r in rows:
                try:
                    sm.append(float(r[0])); mx.append(float(r[1])); power.append(float(r[2]))
                except Exception:
                    continue
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            return sm, mx, reasons, power
        # a sample is printed a little after it was taken: allow one sampling period of slack at the front
        inside = [x for x in self.rows if t_begin + 0.02 <= x[0] <= t_end + 0.01]
        sm, mx, reasons, power = fold(inside)
        all_sm, all_mx, all_reasons, _ = fold(self.rows)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_mhz_min": min(sm) if sm else None,
                "sm_max_mhz": max(all_mx) if all_mx else None,
                "power_w_max": max(power) if power else None, "power_w_median": statistics.median(power) if power else None,
                "samples": len(sm), "samples_outside_region": len(all_sm) - len(sm),
                "reasons": sorted(reasons), "reasons_outside_region": sorted(all_reasons - reasons)}


def gpu_identifier(local_rank: int) -> str:
    import torch
    try:
        u = str(torch.cuda.get_device_properties(local_rank).uuid)
        return u if u.startswith("GPU-") else "GPU-" + u
    except Exception:
        return str(local_rank)


def sha256_of(path: str) -> str:
    import hashlib
    with open(path, "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()


def recorded_traffic(cfg, gather_a=0):
    """GEMM1's measured DRAM bytes per launch for this workload, if a capture of the CURRENT kernel source is on
    record; (None, reason) otherwise."""
    try:
        with open(TRAFFIC_RECORD) as f:
            rec = json.load(f)
    except Exception:
        return None, "no traffic record"
    ent = rec.get(cfg.name + ("+gather_a" if gather_a else ""))
    if ent is None:
        return None, "no capture of this workload on record"
    src = KERNEL_SOURCE[cfg.dtype]
    now = sha256_of(os.path.join(ROOT, "paper_2609_33252_b200", "csrc", src))
    if ent.get("source_sha256", {}).get(src) != now:
        return None, "%s changed since the capture of %s (commit %s)" % (src, ent.get("date"), ent.get("commit"))
    return float(ent["dram_bytes_read"]) + float(ent["dram_bytes_write"]), \
        "ncu capture of %s, commit %s%s" % (ent.get("date"), ent.get("commit"),
                                           (", " + ent["note"]) if ent.get("note") else "")


def workload_numbers(cfg, n_pairs):
    """Algorithmic work of one step: 6*H*I FLOP per kept (token, expert) pair; bytes per kernel as the method
    itself must move them (each row read/written once, each touched expert's weights read once)."""
    H, I, T, E = cfg.H, cfg.I, cfg.T, cfg.E_local
    s = 2 if cfg.dtype == "bf16" else 1 + 4.0 / 128      # bytes per element (fp8: code + its share of a 1x128 scale;
    #                                                      mxfp4 activations: e4m3 code + 1/32 of a scale byte: the same)
    sw = 0.5 + 1.0 / 32 if cfg.dtype == "mxfp4" else s   # bytes per weight element (mxfp4: a nibble + 1/32 scale byte)
    return {
        "pairs": n_pairs,
        "flops": 6.0 * H * I * n_pairs,
        "gemm1_flops": 4.0 * H * I * n_pairs,
        "gemm2_flops": 2.0 * H * I * n_pairs,
        "layout_bytes": (T + n_pairs) * H * s + T * cfg.k * 4.0,
        "combine_bytes": (n_pairs + T) * H * 2.0 + n_pairs * 4.0,
        "gemm1_bytes": n_pairs * H * s + 2.0 * H * I * sw * E + n_pairs * I * s,
        "gemm2_bytes": n_pairs * I * s + 1.0 * H * I * sw * E + n_pairs * H * 2,
    }


def max_over_ranks(value: float, dist, device) -> float:
    """Every rank contributes its own time; the job's time is the slowest rank's."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def host_copy(inp):
    """The same inputs with every tensor on the host (for the CPU oracle)."""
    import dataclasses
    import torch
    kw = {}
    for f in dataclasses.fields(inp):
        v = getattr(inp, f.name)
        kw[f.name] = v.cpu() if isinstance(v, torch.Tensor) else v
    return type(inp)(**kw)


def run_reference(args):
    """The CPU oracle, as it stands, on a bounded sample of the same workload."""
    import numpy as np
    import oracle
    from paper_2609_33252_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import torch
    cfg = wl.CONFIGS[args.config]
    n_sample = args.oracle_tokens
    inp = wl.make_inputs(cfg, device="cuda" if torch.cuda.is_available() else "cpu", keep_logits=False)
    inp = host_copy(inp)
    cores = oracle.num_threads()
    sel = np.linspace(0, cfg.T - 1, n_sample).astype(np.int64)
    times = []
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        oracle.from_inputs(inp, sel=sel)
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt)
    dt = sum(times) / len(times)
    val = n_sample / dt
    sample = "%d evenly spaced tokens of the %s workload, all their local routed pairs, fp64" % (n_sample, cfg.name)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "T": cfg.T, "H": cfg.H, "I": cfg.I, "E_local": cfg.E_local,
                       "E_global": cfg.E_global, "top_k": cfg.k, "sample_tokens": n_sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def stream_section(cep, wl, cfg, inp, out, chunks, ch_pairs, t_sync_s, args):
    """Completion latency of Sync / Async / Async+streamFFN when the chunks arrive at seeded offsets
    (lognormal, scaled to tau x the one-shot time), the matched-work retention at tau = 0, and the gate
    "chunked asynchronous execution is no slower than one synchronous launch over the same tokens"."""
    import torch
    from paper_2609_33252_b200.arrivals import run_with_arrivals
    theta = args.theta if args.theta >= 0 else cfg.E_local * 1024
    rstreams = [torch.cuda.Stream() for _ in chunks]
    # streamffn: the launch rule as the paper states it; streamffn_defer: a batch that has reached theta while the
    # GPU is still busy with the previous invocation keeps accumulating (cep_config::defer_while_busy)
    modes = [("sync", cep.CEP_MODE_SYNC, 0, 1, 0), ("async", cep.CEP_MODE_ASYNC, 0, 1, 0),
             ("streamffn", cep.CEP_MODE_STREAMFFN, theta, args.streams, 0),
             ("streamffn_defer", cep.CEP_MODE_STREAMFFN, theta, args.streams, 1)]
    layers = {}
    for name, mode, th, S, defer in modes:
        L = cep.MoELayer(cfg.H, cfg.I, cfg.E_global, cfg.E_local, cfg.k, cfg.T, cfg.n_chunks, mode=mode,
                         dtype=cep.DTYPE_OF[cfg.dtype],
                         n_streams=S, threshold_pairs=th, gemm_impl=args.gemm_impl, defer_while_busy=defer)
        L.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)
        layers[name] = L
    torch.cuda.synchronize()
    base = inp.arrival
    report = {"theta_pairs": theta, "streams": args.streams, "t_sync_ms": t_sync_s * 1e3,
              "arrival_offsets_unitless": base, "cases": []}
    for tau in (0.0, 0.25, 0.5, 1.0):
        arr = [tau * t_sync_s * a for a in base]
        case = {"tau": tau, "last_arrival_ms": max(arr) * 1e3}
        # the modes take turns inside every repetition, so that all of them see the same clock and power state
        ts = {name: [] for name, _, _, _, _ in modes}
        ninv = {}
        for rep in range(13):                      # 3 warm-up + 10 timed
            for name, _, _, _, _ in modes:
                dt, ninv[name] = run_with_arrivals(layers[name], out, chunks, arr, ch_pairs, rstreams)
                if rep >= 3:
                    ts[name].append(dt)
        for name, _, _, _, _ in modes:
            case[name] = {"completion_ms": statistics.median(ts[name]) * 1e3, "min_ms": min(ts[name]) * 1e3,
                          "invocations": ninv[name]}
        report["cases"].append(case)
    c0 = report["cases"][0]
    report["matched_work_retention"] = {m: c0["sync"]["completion_ms"] / c0[m]["completion_ms"]
                                        for m in ("async", "streamffn", "streamffn_defer")}
    staggered = report["cases"][1:]
    report["gate"] = {
        "statement": "completion latency of chunked asynchronous execution <= one synchronous launch over the same "
                     "tokens, for every staggered arrival pattern (tau > 0); at tau = 0 (everything present at once) "
                     "the synchronous launch is the best possible schedule and the retention is reported instead",
        "tolerance": "1 % (run-to-run spread of the medians)",
        "streamffn_no_slower_than_sync": {str(c["tau"]): bool(c["streamffn"]["completion_ms"] <= 1.01 * c["sync"]["completion_ms"])
                                          for c in staggered},
        "streamffn_defer_no_slower_than_sync": {str(c["tau"]): bool(c["streamffn_defer"]["completion_ms"] <= 1.01 * c["sync"]["completion_ms"])
                                                for c in staggered},
        "retention_at_tau0": {"streamffn": report["matched_work_retention"]["streamffn"],
                              "streamffn_defer": report["matched_work_retention"]["streamffn_defer"],
                              "paper_other_system_and_hardware": 0.973}}
    for L in layers.values():
        L.close()
    return report


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="ep_shard")
    ap.add_argument("--streams", type=int, default=2)
    ap.add_argument("--oracle-tokens", type=int, default=48)
    ap.add_argument("--gemm-impl", type=int, default=0, help="0: CTA-pair tcgen05 (product), 2: one-CTA tcgen05")
    ap.add_argument("--gather-a", type=int, default=0, choices=[0, 1],
                    help="bf16 only: no permuted copy, GEMM1 gathers its rows from the token tensor (cep_config::gather_a); "
                         "applies to the device-resident timing, the end-to-end and arrival sections keep the default")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-stream", action="store_true", help="skip the arrival-offset (streamFFN) section")
    ap.add_argument("--theta", type=int, default=-1, help="streamFFN threshold in local pairs (default: E_local*1024)")
    ap.add_argument("--profile-in-region", type=int, default=-1,
                    help="1: the timed plan itself records events between its kernels, so the per-kernel times come from "
                         "the timed steps; 0: a second plan is profiled after the timed region; default: 1 for workloads "
                         "of at least 2 TFLOP per step (the events cost a few microseconds of launch overlap per step)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3 if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        if args.steps > 3:
            args.steps = 3
        args.warmup = min(args.warmup, 1)
        return run_reference(args)

    import numpy as np
    import torch
    import paper_2609_33252_b200 as cep
    from paper_2609_33252_b200 import workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist = dist_
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    cfg = wl.CONFIGS[args.config]
    peaks = load_peaks()
    inp = wl.make_inputs(cfg, device="cuda", keep_logits=False)
    n_pairs = inp.n_local_pairs()
    work = workload_numbers(cfg, n_pairs)
    ch_pairs = [int((inp.topk_ids[o:o + n] < cfg.E_local).sum().item()) for o, n in zip(inp.chunk_offsets, cfg.chunks)]

    dt = cep.DTYPE_OF[cfg.dtype]
    in_region = args.profile_in_region == 1 or (args.profile_in_region < 0 and work["flops"] >= 2e12)
    layer = cep.MoELayer(cfg.H, cfg.I, cfg.E_global, cfg.E_local, cfg.k, cfg.T, cfg.n_chunks, dtype=dt,
                         mode=cep.CEP_MODE_SYNC, n_streams=args.streams, gemm_impl=args.gemm_impl,
                         profile_kernels=1 if in_region else 0, gather_a=args.gather_a)
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)
    prof_layer = None
    if not in_region:
        # small workloads: a second plan records events between the kernels, run right after the timed region
        prof_layer = cep.MoELayer(cfg.H, cfg.I, cfg.E_global, cfg.E_local, cfg.k, cfg.T, cfg.n_chunks, dtype=dt,
                                  mode=cep.CEP_MODE_SYNC, n_streams=1, profile_kernels=1, gemm_impl=args.gemm_impl,
                                  gather_a=args.gather_a)
        prof_layer.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)
    torch.cuda.synchronize()
    out = torch.empty(cfg.T, cfg.H, dtype=torch.bfloat16, device="cuda")
    chunks = [(o, inp.x[o:o + n], None if inp.x_scale is None else inp.x_scale[o:o + n], inp.topk_ids[o:o + n],
               inp.topk_w[o:o + n]) for o, n in zip(inp.chunk_offsets, cfg.chunks)]

    def step():
        layer.run(out, chunks, n_local_pairs=ch_pairs)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    assert cep.ffn_status(layer.plan) == 0, cep.cep_last_error(layer.plan)

    names = ("layout_ms", "gemm1_ms", "gemm2_ms", "combine_ms", "index_ms", "scatter_ms", "elapsed_ms")
    kern = {k_: [] for k_ in names}
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    bad_reasons = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}
    gpu_id = gpu_identifier(local_rank)
    for attempt in range(2):            # a run that saw a thermal or hardware slowdown is taken once more
        sampler = ClockSampler(gpu_id)
        if rank == 0:
            sampler.start()
            time.sleep(0.1)
        launches0 = cep.cep_kernel_launches(layer.plan)
        barrier()
        t_begin = time.time()
        step_ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
        ev0.record()
        for i in range(args.steps):
            step()
            step_ev[i].record()                    # the join stream: complete when this step's output is
        ev1.record()
        barrier()
        t_end = time.time()
        total_ms = ev0.elapsed_time(ev1)
        step_ms = [(ev0 if i == 0 else step_ev[i - 1]).elapsed_time(step_ev[i]) for i in range(args.steps)]
        launches = cep.cep_kernel_launches(layer.plan) - launches0
        timed_clocks = sampler.stop(t_begin, t_end) if rank == 0 else None
        redo = 1 if (rank == 0 and timed_clocks and bad_reasons & set(timed_clocks.get("reasons", []))) else 0
        if dist is not None:
            flag = torch.tensor([redo], device="cuda")
            dist.broadcast(flag, 0)
            redo = int(flag.item())
        if not redo:
            break
    assert cep.ffn_status(layer.plan) == 0, cep.cep_last_error(layer.plan)
    if in_region:
        # the plan keeps the events of its last layer calls: per-kernel device times of the last timed steps themselves
        kernel_source = "events recorded between the kernels of the last %d timed steps" % min(args.steps, 8)
        for back in range(min(args.steps, 8)):
            for i in range(cep.ffn_num_invocations(layer.plan)):
                info = cep.ffn_query_call(layer.plan, back, i)
                for k_ in kern:
                    kern[k_].append(getattr(info, k_))
    else:
        kernel_source = "a second, event-instrumented plan run back to back right after the timed region (the timed " \
                        "plan records no events: they would cost this short step its launch overlap)"
        for rep in range(3):
            for _ in range(max(args.steps // 3, 1)):
                prof_layer.run(out, chunks, n_local_pairs=ch_pairs)
            torch.cuda.synchronize()
            for i in range(cep.ffn_num_invocations(prof_layer.plan)):
                info = cep.ffn_query(prof_layer.plan, i)
                for k_ in kern:
                    kern[k_].append(getattr(info, k_))
    clocks = timed_clocks
    if clocks is not None:
        clocks["remeasured"] = attempt == 1
    ms = max_over_ranks(total_ms / args.steps, dist, "cuda")
    value = world * cfg.T / (ms * 1e-3)

    # ---- end to end: pinned host buffers -> device -> path -> host, every step
    e2e = None
    if not args.no_e2e:
        hx = inp.x.cpu().pin_memory(); hid = inp.topk_ids.cpu().pin_memory(); hw = inp.topk_w.cpu().pin_memory()
        hxs = None if inp.x_scale is None else inp.x_scale.cpu().pin_memory()
        # two sets of device input / output buffers and host output buffers: layer call i+1 may copy its inputs in
        # while call i still computes and copies out (consecutive micro-batches of a serving loop)
        sets = []
        for _ in range(2):
            sets.append({"dx": torch.empty_like(inp.x), "did": torch.empty_like(inp.topk_ids), "dw": torch.empty_like(inp.topk_w),
                         "dxs": None if inp.x_scale is None else torch.empty_like(inp.x_scale),
                         "out": torch.empty_like(out), "hout": torch.empty(cfg.T, cfg.H, dtype=torch.bfloat16).pin_memory(),
                         "in_free": torch.cuda.Event(), "out_free": torch.cuda.Event()})
        rstreams = [torch.cuda.Stream() for _ in chunks]
        main = torch.cuda.current_stream()
        for b_ in sets:
            b_["in_free"].record(main)
            b_["out_free"].record(main)

        # chunks are consumed as they land (Async+streamFFN, theta = two chunks' worth of pairs) and every
        # invocation's output rows are copied back as soon as that invocation has written them
        e2e_theta = max(1, 2 * (sum(ch_pairs) // max(len(ch_pairs), 1)))
        e2e_layer = cep.MoELayer(cfg.H, cfg.I, cfg.E_global, cfg.E_local, cfg.k, cfg.T, cfg.n_chunks, dtype=dt,
                                 mode=cep.CEP_MODE_STREAMFFN, n_streams=args.streams, threshold_pairs=e2e_theta,
                                 gemm_impl=args.gemm_impl)
        e2e_layer.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)
        # with two calls in flight the copies of neighbouring calls hide behind the compute anyway, so one synchronous
        # invocation per call (the most efficient GEMM shapes) is also tried
        sync_layer = cep.MoELayer(cfg.H, cfg.I, cfg.E_global, cfg.E_local, cfg.k, cfg.T, cfg.n_chunks, dtype=dt,
                                  mode=cep.CEP_MODE_SYNC, n_streams=2, gemm_impl=args.gemm_impl)
        sync_layer.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)
        d2h = torch.cuda.Stream()
        free_s = torch.cuda.Stream()

        def e2e_step(i, overlap, e2e_layer=e2e_layer):
            b_ = sets[i % 2 if overlap else 0]
            dx, did, dw, dxs, dout, hout = b_["dx"], b_["did"], b_["dw"], b_["dxs"], b_["out"], b_["hout"]
            cep.ffn_begin(e2e_layer.plan, dout, cfg.T, len(chunks))
            seen = 0
            for c, (o, n) in enumerate(zip(inp.chunk_offsets, cfg.chunks)):
                st = rstreams[c]
                if overlap:
                    st.wait_event(b_["in_free"])        # the call that last used these input buffers has consumed them
                else:
                    st.wait_stream(main)                # one layer call at a time
                with torch.cuda.stream(st):
                    dx[o:o + n].copy_(hx[o:o + n], non_blocking=True)
                    did[o:o + n].copy_(hid[o:o + n], non_blocking=True)
                    dw[o:o + n].copy_(hw[o:o + n], non_blocking=True)
                    if dxs is not None:
                        dxs[o:o + n].copy_(hxs[o:o + n], non_blocking=True)
                if overlap:
                    st.wait_event(b_["out_free"])       # ... and its output rows have left the output buffer
                cep.ffn_submit_chunk(e2e_layer.plan, c, o, n, dx[o:o + n], None if dxs is None else dxs[o:o + n],
                                     did[o:o + n], dw[o:o + n], ch_pairs[c], st)
                if c == len(chunks) - 1:
                    cep.ffn_flush(e2e_layer.plan)
                # copy back the rows of every invocation launched so far (chunks are submitted in id order)
                while seen < cep.ffn_num_invocations(e2e_layer.plan):
                    info = cep.ffn_query(e2e_layer.plan, seen)
                    cep.ffn_wait_invocation(e2e_layer.plan, seen, d2h)
                    lo = inp.chunk_offsets[info.first_chunk_pos]
                    last = info.first_chunk_pos + info.n_chunks - 1
                    hi = inp.chunk_offsets[last] + cfg.chunks[last]
                    with torch.cuda.stream(d2h):
                        hout[lo:hi].copy_(dout[lo:hi], non_blocking=True)
                    seen += 1
            for j in range(cep.ffn_num_invocations(e2e_layer.plan)):
                cep.ffn_wait_invocation(e2e_layer.plan, j, free_s)
            b_["in_free"].record(free_s)                # every invocation of this call has finished reading its inputs
            cep.combine(e2e_layer.plan, main)
            main.wait_stream(d2h)
            b_["out_free"].record(main)

        def e2e_run(overlap, layer_):
            for i in range(4):
                e2e_step(i, overlap, layer_)
            barrier()
            ev0.record()
            for i in range(args.steps):
                e2e_step(i, overlap, layer_)
            ev1.record()
            barrier()
            return max_over_ranks(ev0.elapsed_time(ev1) / args.steps, dist, "cuda")

        serial_ms = e2e_run(False, e2e_layer)
        stream_ms = e2e_run(True, e2e_layer)
        sync_ms = e2e_run(True, sync_layer)
        assert torch.equal(sets[0]["hout"].view(torch.int16), sets[1]["hout"].view(torch.int16))   # both buffer sets hold the result
        e2e_ms = min(stream_ms, sync_ms)
        sync_layer.close()
        h2d = hx.numel() * hx.element_size() + hid.numel() * 4 + hw.numel() * 4 + \
            (0 if hxs is None else hxs.numel() * hxs.element_size())
        e2e_layer.close()
        e2e = {"value": world * cfg.T / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
               "mode": "two layer calls in flight (double-buffered inputs and outputs), output rows copied back per "
                       "invocation; " + ("one synchronous invocation per call" if sync_ms <= stream_ms else
                                         "Async+streamFFN, theta=%d pairs" % e2e_theta),
               "ms_per_step_two_calls_streamffn": stream_ms, "ms_per_step_two_calls_sync": sync_ms,
               "ms_per_step_one_call_at_a_time_streamffn": serial_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": sets[0]["hout"].numel() * 2}

    # ---- chunked asynchronous execution under seeded arrival offsets (rank 0 only, outside the timed step)
    stream_report = None
    if rank == 0 and not args.no_stream and cfg.n_chunks > 1:
        stream_report = stream_section(cep, wl, cfg, inp, out, chunks, ch_pairs, ms * 1e-3, args)

    if prof_layer is not None:
        prof_layer.close()
    if rank != 0:
        layer.close()
        if dist is not None:
            dist.barrier()                      # rank 0 is still measuring its rank-0-only legs
            dist.destroy_process_group()
        return 0

    med = {k_: (statistics.median(v) if v else None) for k_, v in kern.items()}
    g1_ms, g2_ms = med["gemm1_ms"], med["gemm2_ms"]
    ffn_tflops = work["flops"] / ((g1_ms + g2_ms) * 1e-3) / 1e12
    g1_tflops = work["gemm1_flops"] / (g1_ms * 1e-3) / 1e12
    g2_tflops = work["gemm2_flops"] / (g2_ms * 1e-3) / 1e12
    # Which measured peak the fraction is taken of: the burst figure for a short region at full clocks, the
    # sustained one once the steps ran under the power cap (cap reported by a sample INSIDE the region, its median
    # clock well below the maximum, or more than a second of back-to-back steps).  The power controller needs on
    # the order of 100 ms of load before it pulls the clocks down.  All three fractions are printed side by side.
    sm, smx = (clocks or {}).get("sm_mhz"), (clocks or {}).get("sm_max_mhz")
    capped = "sw_power_cap" in ((clocks or {}).get("reasons") or [])
    sustained = total_ms > 100.0 and (capped or total_ms > 1000.0 or bool(sm and smx and sm < 0.9 * smx))
    mult = 2.0 if cfg.dtype in ("fp8", "mxfp4") else 1.0   # no measured fp8 peak: measured bf16 peak x the nominal fp8:bf16
    #                                                        ratio; the mxf8f6f4 MMA kind (e4m3 x e2m1) runs at the fp8 rate
    burst_tf, sust_tf, nominal_tf = mult * peaks["bf16_tflops"], mult * peaks["bf16_tflops_sustained"], mult * NOMINAL_BF16_TFLOPS
    peak_tf = sust_tf if sustained else burst_tf
    traffic, traffic_note = recorded_traffic(cfg, args.gather_a)
    kernel_sum = sum(med[k_] for k_ in ("layout_ms", "gemm1_ms", "gemm2_ms", "combine_ms"))
    roofline = {"bound": "tensor", "kernel": "grouped GEMM1 (gate/up + SiLU*up%s), CTA-pair tcgen05" %
                          (" + e4m3 re-quantisation" if cfg.dtype != "bf16" else ""),
                "achieved": g1_tflops, "peak": peak_tf, "unit": "TFLOP/s", "frac": g1_tflops / peak_tf,
                "peak_kind": ("sustained" if sustained else "burst") + " bf16 cuBLAS" +
                             (" x2 (nominal fp8:bf16 ratio)" if cfg.dtype != "bf16" else "") + ", of " + peaks["source"],
                "frac_of_burst": g1_tflops / burst_tf, "frac_of_sustained": g1_tflops / sust_tf,
                "frac_of_nominal": g1_tflops / nominal_tf, "nominal_tflops": nominal_tf,
                "duration_ms": g1_ms, "share_of_step": g1_ms / ms, "traffic": traffic, "traffic_source": traffic_note,
                "algorithmic_bytes": work["gemm1_bytes"]}
    n_last = min(args.steps, 8)
    last_ms = statistics.median(step_ms[-n_last:])          # the steps the per-kernel times were read from
    timing = {"timed_region_ms": total_ms, "kernel_times_from": kernel_source,
              "kernel_sum_ms": kernel_sum, "invocation_elapsed_ms": med["elapsed_ms"],
              "ms_per_step_first": step_ms[0], "ms_per_step_median": statistics.median(step_ms),
              "ms_per_step_median_of_last_%d" % n_last: last_ms,
              "kernel_sum_within_those_steps": bool(kernel_sum <= last_ms * 1.005) if in_region else None,
              "note": "the first steps of a region run at burst clocks, the later ones under the power cap: ms_per_step "
                      "is the mean over all timed steps, the per-kernel times are medians over the last ones",
              "sm_mhz_median_in_region": sm, "ms_per_step_x_sm_mhz": (ms * sm) if sm else None}
    kernels = {
        "layout": {"ms": med["layout_ms"], "GB/s": work["layout_bytes"] / (med["layout_ms"] * 1e-3) / 1e9,
                   "frac_of_hbm": work["layout_bytes"] / (med["layout_ms"] * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "index (hist+scan+rank)": {"ms": med["index_ms"]},
        "scatter_rows": {"ms": med["scatter_ms"], "GB/s": work["layout_bytes"] / (med["scatter_ms"] * 1e-3) / 1e9,
                         "frac_of_hbm": work["layout_bytes"] / (med["scatter_ms"] * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "gemm1": {"ms": g1_ms, "TFLOP/s": g1_tflops},
        "gemm2": {"ms": g2_ms, "TFLOP/s": g2_tflops, "frac": g2_tflops / peak_tf},
        "combine": {"ms": med["combine_ms"], "GB/s": work["combine_bytes"] / (med["combine_ms"] * 1e-3) / 1e9,
                    "frac_of_hbm": work["combine_bytes"] / (med["combine_ms"] * 1e-3) / 1e9 / peaks["hbm_gbs"]},
    }
    if args.gather_a:           # index kernels only: no rows move, a bandwidth figure would mean nothing
        kernels["layout"] = {"ms": med["layout_ms"], "note": "indices only (gather_a)"}
        kernels["scatter_rows"] = {"ms": med["scatter_ms"], "note": "padding marks only (gather_a)"}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": {"bf16": "bf16", "fp8": "fp8_e4m3", "mxfp4": "e4m3 x e2m1 (ue8m0 1x32 scales)"}[cfg.dtype], "data": "synthetic",
            "config": {"workload": cfg.name, "T": cfg.T, "H": cfg.H, "I": cfg.I, "E_local": cfg.E_local,
                       "E_global": cfg.E_global, "top_k": cfg.k, "local_pairs": n_pairs, "chunks": list(cfg.chunks),
                       "mode": "sync (one invocation, all chunks present)", "parallelism": "replicas only",
                       "gather_a": args.gather_a,
                       "l2": "inputs larger than L2 (weights %.2f GB re-read every step)" %
                             (3.0 * cfg.H * cfg.I * {"bf16": 2, "fp8": 1, "mxfp4": 0.5}[cfg.dtype] * cfg.E_local / 1e9)},
            "ffn_tflops": {"value": ffn_tflops, "frac_of_nominal": ffn_tflops / nominal_tf, "nominal_tflops": nominal_tf,
                           "frac_of_measured": ffn_tflops / peak_tf, "flops_per_step": work["flops"]},
            "roofline": roofline, "timing": timing, "kernels": kernels, "clocks": clocks, "e2e": e2e, "streamffn": stream_report,
            "gpu_launches": int(launches)}
    if not args.no_cpu_baseline:
        import oracle
        n_s = args.oracle_tokens
        hin = host_copy(inp)
        sel = np.linspace(0, cfg.T - 1, n_s).astype(np.int64)
        t0 = time.perf_counter()
        ref = oracle.from_inputs(hin, sel=sel)
        dt = time.perf_counter() - t0
        got = out[torch.as_tensor(sel, device="cuda")].double().cpu().numpy()
        rel = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30))
        line["cpu_baseline"] = {"value": n_s / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                                "sample": "%d evenly spaced tokens of the %s workload, all their local routed "
                                          "pairs, fp64, %.1f s" % (n_s, cfg.name, dt),
                                "rel_fro_error_of_gpu_on_sample": rel}
    print(json.dumps(line), flush=True)
    layer.close()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
