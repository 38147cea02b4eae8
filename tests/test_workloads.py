"""The seeded input generator: shapes, determinism, and the fp8 block quantiser's pins."""
import numpy as np
import torch

from paper_2609_33252_b200 import workloads as wl


def test_configs_are_consistent():
    for cfg in wl.CONFIGS.values():
        assert sum(cfg.chunks) == cfg.T
        assert cfg.E_local <= cfg.E_global and cfg.k <= cfg.E_global
    s = wl.CONFIGS["straggler"]
    assert max(s.chunks) == s.chunks[-1] and abs(s.chunks[-1] / s.T - 0.4) < 1e-3


def test_tiny_inputs_deterministic_and_shaped():
    a = wl.make_inputs(wl.CONFIGS["tiny"])
    b = wl.make_inputs(wl.CONFIGS["tiny"])
    assert a.x.dtype == torch.bfloat16 and a.x.shape == (256, 512)
    assert a.w_gate.shape == (8, 512, 256) and a.w_down.shape == (8, 256, 512)
    assert torch.equal(a.x.view(torch.int16), b.x.view(torch.int16))
    assert torch.equal(a.topk_ids, b.topk_ids) and torch.equal(a.topk_w, b.topk_w)
    assert a.topk_ids.dtype == torch.int32 and a.topk_w.dtype == torch.float32
    assert a.n_local_pairs() == 256 * 2
    assert abs(a.w_gate.float().std().item() - 512 ** -0.5) < 2e-3      # std = fan_in^-1/2
    assert abs(a.w_down.float().std().item() - 256 ** -0.5) < 2e-3
    # ids distinct per token
    s, _ = torch.sort(a.topk_ids, dim=1)
    assert (s[:, 1:] != s[:, :-1]).all()


def test_zipf_routing_favours_low_ids_and_shard_keeps_a_subset():
    cfg = wl.scaled(wl.CONFIGS["ep_shard"], T=512, H=128, I=128, chunks=(512,))
    inp = wl.make_inputs(cfg)
    local = (inp.topk_ids < cfg.E_local).float().mean().item()
    assert 0.8 < local <= 1.0                  # the literal Zipf reading makes shard 0 the hot shard
    cfgs = wl.scaled(cfg, zipf_strided=True)
    inps = wl.make_inputs(cfgs)
    local_s = (inps.topk_ids < cfg.E_local).float().mean().item()
    assert local_s < 0.5


def test_fp8_block_quantiser_pins():
    g = torch.Generator().manual_seed(0)
    x = torch.randn(16, 256, generator=g)
    x[3, :128] = 0
    q, s = wl.quantize_rows_1x128(x)
    assert q.dtype == torch.float8_e4m3fn and s.shape == (16, 2)
    assert s[3, 0] == 1.0 and (q[3, :128].float() == 0).all()           # all-zero block -> scale 1
    codes = q.float().view(16, 2, 128)
    amax_pos = x.view(16, 2, 128).abs().argmax(dim=2)
    top = torch.gather(codes.abs(), 2, amax_pos[:, :, None])[:, :, 0]
    assert (top[s != 1.0] == 448).all()                                  # block max maps to 448
    deq = codes * s[:, :, None]
    err = (deq - x.view(16, 2, 128)).abs()
    assert (err <= 2 ** -4 * x.view(16, 2, 128).abs() + 2 ** -10 * s[:, :, None]).all()
    w = torch.randn(2, 256, 128, generator=g)
    qw, sw = wl.quantize_blocks_128x128(w)
    assert sw.shape == (2, 2, 1)
    assert torch.allclose(sw[:, :, 0], w.view(2, 2, 128, 128).abs().amax(dim=(2, 3)) / 448)


def test_arrivals_and_submission_order():
    cfg = wl.CONFIGS["straggler"]
    a = wl.make_arrivals(cfg)
    assert len(a) == 8 and min(a) == 0.0
    assert wl.submission_order(a)[-1] == 7                               # the straggler arrives last
    assert a == wl.make_arrivals(cfg)
