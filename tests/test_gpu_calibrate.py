"""Launch-threshold calibration done by the library (Section 3.2 "Launch threshold"): profile, theta(rho), stream
probe; and the switch that limits the round-robin to the first n compute streams."""
import numpy as np
import pytest
import torch

import paper_2609_33252_b200 as cep
from paper_2609_33252_b200 import calibrate, workloads as wl

from helpers import make_layer, run_layer, to_device

pytestmark = pytest.mark.gpu

CFG = wl.MoEConfig("cal", 1, T=2048, H=1024, I=512, E_global=16, E_local=8, k=4, chunks=(2048,))


@pytest.mark.parametrize("dtype", ["bf16", "fp8", "mxfp4"])
def test_library_calibration_profile_and_threshold(dtype):
    cfg = wl.scaled(CFG, dtype=dtype)
    rows = (16, 64, 256, 1024)
    res = calibrate.calibrate_in_library(cfg, rho=0.9, rows=rows, reps=3, n_streams=3)
    prof = res["profile"]
    assert [p["rows_per_expert"] for p in prof] == list(rows)
    assert [p["expert_tokens"] for p in prof] == [r * cfg.E_local for r in rows]
    assert all(p["ffn_ms"] > 0 and p["layer_ms"] >= p["ffn_ms"] for p in prof)
    assert max(p["eta"] for p in prof) == pytest.approx(1.0)
    assert prof[-1]["tflops"] > 4 * prof[0]["tflops"]            # throughput rises steeply with rows per expert
    # theta is the smallest profiled count that reaches rho of the peak
    reach = [p for p in prof if p["eta"] >= 0.9]
    assert res["theta_pairs"] == reach[0]["expert_tokens"] and res["theta_rows_per_expert"] == reach[0]["rows_per_expert"]
    for p in prof:                                               # F(N) = N / (eta(N) * P_peak)
        f_model = 6.0 * cfg.H * cfg.I * p["expert_tokens"] / (p["eta"] * res["peak_tflops"] * 1e12) * 1e3
        assert f_model == pytest.approx(p["ffn_ms"], rel=1e-3)
    if res["probe_invocations"] >= 2:
        assert 1 <= res["best_streams"] <= 3 and len(res["stream_ms"]) == 3
        assert res["stream_ms"][res["best_streams"] - 1] <= 1.02 * min(res["stream_ms"]) + 1e-6


def test_calibration_restores_the_plan_and_rejects_bad_calls():
    cfg = CFG
    inp = to_device(wl.make_inputs(cfg))
    layer = cep.MoELayer(cfg.H, cfg.I, cfg.E_global, cfg.E_local, cfg.k, cfg.T, 4, mode=cep.CEP_MODE_ASYNC, n_streams=2,
                         profile_kernels=1)
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down)
    before, n_before = run_layer(inp, layer)
    ids = torch.empty((cfg.T, cfg.k), dtype=torch.int32, device="cuda")
    w = torch.empty((cfg.T, cfg.k), dtype=torch.float32, device="cuda")
    out = torch.empty((cfg.T, cfg.H), dtype=torch.bfloat16, device="cuda")
    cep.cep_calibrate(layer.plan, 0.9, [32, 128, 512], 2, inp.x, None, ids, w, out)
    after, n_after = run_layer(inp, layer)                        # same mode, same result as before the calibration
    assert n_after == n_before and torch.equal(before.view(torch.int16), after.view(torch.int16))
    with pytest.raises(cep.CepError):
        cep.cep_calibrate(layer.plan, 0.9, [128, 64], 2, inp.x, None, ids, w, out)        # not ascending
    with pytest.raises(cep.CepError):
        cep.cep_calibrate(layer.plan, 0.9, [1 << 20], 2, inp.x, None, ids, w, out)        # beyond max_tokens
    with pytest.raises(cep.CepError):
        cep.cep_calibrate(layer.plan, 1.5, [64], 2, inp.x, None, ids, w, out)
    layer.close()
    plain = make_layer(cfg)                                       # no profile_kernels: refused
    plain.load_weights(inp.w_gate, inp.w_up, inp.w_down)
    with pytest.raises(cep.CepError):
        cep.cep_calibrate(plain.plan, 0.9, [64], 2, inp.x, None, ids, w, out)
    plain.close()


def test_active_streams_changes_the_slots_not_the_result():
    cfg = wl.scaled(CFG, chunks=(512, 512, 512, 512))
    inp = to_device(wl.make_inputs(cfg))
    layer = make_layer(cfg, mode=cep.CEP_MODE_ASYNC, n_streams=3)
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down)
    ref, n = run_layer(inp, layer)
    assert n == 4 and [cep.ffn_query(layer.plan, i).stream_index for i in range(4)] == [0, 1, 2, 0]
    cep.ffn_set_active_streams(layer.plan, 1)
    one, _ = run_layer(inp, layer)
    assert [cep.ffn_query(layer.plan, i).stream_index for i in range(4)] == [0, 0, 0, 0]
    cep.ffn_set_active_streams(layer.plan, 2)
    two, _ = run_layer(inp, layer)
    assert [cep.ffn_query(layer.plan, i).stream_index for i in range(4)] == [0, 1, 0, 1]
    assert torch.equal(ref.view(torch.int16), one.view(torch.int16)) and torch.equal(ref.view(torch.int16), two.view(torch.int16))
    for bad in (0, 4):
        with pytest.raises(cep.CepError):
            cep.ffn_set_active_streams(layer.plan, bad)
    layer.close()


def test_calibration_on_the_callers_routing_counts_the_real_expert_tokens():
    # growing prefixes of one skewed batch: expert_tokens are the local pairs of each prefix, theta the first
    # profiled count that reaches rho of the best throughput seen on THIS routing
    cfg = wl.scaled(CFG, zipf_s=1.1)
    res = calibrate.calibrate_on_routing(cfg, rho=0.9, fractions=(1 / 16, 1 / 4, 1.0), reps=3)
    host_ids = wl.make_inputs(cfg, device="cuda", keep_logits=False).topk_ids.cpu().numpy()
    prof = res["profile"]
    assert [p["n_tokens"] for p in prof] == [128, 512, 2048]
    for p in prof:
        assert p["expert_tokens"] == int((host_ids[:p["n_tokens"]] < cfg.E_local).sum())
        assert p["ffn_ms"] > 0 and 0 < p["eta"] <= 1.0 + 1e-6
    reach = [p for p in prof if p["eta"] >= 0.9]
    assert res["theta_pairs"] == reach[0]["expert_tokens"] and res["best_streams"] == 0


def test_per_kernel_times_of_earlier_layer_calls_are_kept():
    cfg = wl.scaled(CFG, chunks=(1024, 1024))
    inp = to_device(wl.make_inputs(cfg))
    layer = cep.MoELayer(cfg.H, cfg.I, cfg.E_global, cfg.E_local, cfg.k, cfg.T, 2, mode=cep.CEP_MODE_ASYNC, n_streams=2,
                         profile_kernels=1)
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down)
    out = torch.empty((cfg.T, cfg.H), dtype=torch.bfloat16, device="cuda")
    from helpers import chunks_of
    for _ in range(5):                                            # back to back, no host synchronisation in between
        layer.run(out, chunks_of(inp))
    torch.cuda.synchronize()
    for back in range(5):
        for i in range(2):
            q = cep.ffn_query_call(layer.plan, back, i)
            assert q.n_tokens == 1024 and q.first_chunk_pos == i
            assert q.elapsed_ms > 0 and q.gemm1_ms > 0 and q.gemm2_ms > 0 and q.combine_ms > 0
            assert q.layout_ms + q.gemm1_ms + q.gemm2_ms + q.combine_ms == pytest.approx(q.elapsed_ms, rel=1e-3, abs=1e-3)
    with pytest.raises(cep.CepError):
        cep.ffn_query_call(layer.plan, 5, 0)                      # only five calls were made
    with pytest.raises(cep.CepError):
        cep.ffn_query_call(layer.plan, 8, 0)                      # never kept
    layer.close()
    plain = make_layer(cfg)                                       # plans without profile_kernels keep the current call only
    plain.load_weights(inp.w_gate, inp.w_up, inp.w_down)
    run_layer(inp, plain); run_layer(inp, plain)
    with pytest.raises(cep.CepError):
        cep.ffn_query_call(plain.plan, 1, 0)
    plain.close()


def test_deferring_launches_while_the_gpu_is_busy_changes_batching_not_results():
    cfg = wl.scaled(CFG, chunks=(256,) * 8)
    inp = to_device(wl.make_inputs(cfg))
    pairs = int((inp.topk_ids[:256] < cfg.E_local).sum().item())
    outs, n_inv = [], []
    for defer in (0, 1):
        layer = cep.MoELayer(cfg.H, cfg.I, cfg.E_global, cfg.E_local, cfg.k, cfg.T, 8, mode=cep.CEP_MODE_STREAMFFN, n_streams=2,
                             threshold_pairs=pairs, defer_while_busy=defer)
        layer.load_weights(inp.w_gate, inp.w_up, inp.w_down)
        o, n = run_layer(inp, layer, local_pairs=True)
        outs.append(o); n_inv.append(n)
        layer.close()
    assert 1 <= n_inv[1] <= n_inv[0]                              # never more invocations than the plain threshold rule
    assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16))


def test_timeline_ranges_are_host_annotations_only(monkeypatch):
    """CEP_NVTX=1 names the plan's streams and wraps layer calls and invocations in ranges for timeline tools; with no
    tool attached the calls are no-ops and the output is bit-identical."""
    cfg = wl.scaled(CFG, chunks=(256,) * 8)
    inp = to_device(wl.make_inputs(cfg))
    outs = []
    for flag in ("0", "1"):
        monkeypatch.setenv("CEP_NVTX", flag)
        layer = cep.MoELayer(cfg.H, cfg.I, cfg.E_global, cfg.E_local, cfg.k, cfg.T, 8, mode=cep.CEP_MODE_ASYNC, n_streams=2)
        layer.load_weights(inp.w_gate, inp.w_up, inp.w_down)
        o, n = run_layer(inp, layer)
        assert n == 8
        outs.append(o)
        layer.close()
    assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16))
