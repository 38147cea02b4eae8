"""Pins for the oracle's codecs and silu: closed forms and exhaustive tables."""
import math

import numpy as np
import pytest
import torch

import oracle


def test_bf16_decode_exhaustive_closed_form():
    # every finite bf16 code equals (-1)^s 2^(e-127) (1+m/128), subnormals m/128 * 2^-126
    for bits in range(0, 65536, 1):
        s, e, m = bits >> 15, (bits >> 7) & 0xFF, bits & 0x7F
        if e == 255:
            continue
        v = (m / 128.0) * 2.0 ** -126 if e == 0 else (1 + m / 128.0) * 2.0 ** (e - 127)
        v = -v if s else v
        got = oracle.bf16_to_f64(bits)
        assert got == v, bits


def test_bf16_decode_matches_torch_cast():
    bits = torch.arange(0, 65536, dtype=torch.int32).to(torch.int16)
    ref = bits.view(torch.bfloat16).double().numpy()
    for b in range(0, 65536, 7):
        r = ref[b]
        g = oracle.bf16_to_f64(b)
        assert (math.isnan(r) and math.isnan(g)) or r == g


def test_e4m3_decode_exhaustive_closed_form_and_torch():
    ref = torch.arange(256, dtype=torch.int32).to(torch.uint8).view(torch.float8_e4m3fn).double().numpy()
    for c in range(256):
        s, e, m = c >> 7, (c >> 3) & 15, c & 7
        got = oracle.e4m3_to_f64(c)
        if e == 15 and m == 7:
            assert math.isnan(got) and math.isnan(ref[c])
            continue
        v = (m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7)
        v = -v if s else v
        assert got == v == ref[c]
    assert oracle.e4m3_to_f64(0x7E) == 448.0


def test_e4m3_encode_roundtrip_ties_and_saturation():
    for c in range(256):
        if (c & 0x7F) == 0x7F:
            continue
        v = oracle.e4m3_to_f64(c)
        assert oracle.f64_to_e4m3(v) == c or v == 0.0
    # round-to-nearest-even ties: 1.0625 is halfway 1.0/1.125 -> 1.0 ; 1.1875 -> 1.25
    assert oracle.e4m3_to_f64(oracle.f64_to_e4m3(1.0625)) == 1.0
    assert oracle.e4m3_to_f64(oracle.f64_to_e4m3(1.1875)) == 1.25
    assert oracle.e4m3_to_f64(oracle.f64_to_e4m3(500.0)) == 448.0
    assert oracle.e4m3_to_f64(oracle.f64_to_e4m3(-1e9)) == -448.0
    assert oracle.e4m3_to_f64(oracle.f64_to_e4m3(464.0)) == 448.0
    # subnormal grid: spacing 2^-9; tie 1.5*2^-9 -> 2*2^-9 (even), 0.5*2^-9 -> 0
    assert oracle.e4m3_to_f64(oracle.f64_to_e4m3(1.5 * 2 ** -9)) == 2 * 2 ** -9
    assert oracle.e4m3_to_f64(oracle.f64_to_e4m3(0.5 * 2 ** -9)) == 0.0


def test_e4m3_encode_matches_torch_cast_on_random_values():
    g = torch.Generator().manual_seed(3)
    x = (torch.randn(4000, generator=g, dtype=torch.float64) * 60).clamp(-448, 448)
    x = torch.cat([x, torch.randn(2000, generator=g, dtype=torch.float64) * 0.02])
    # torch casts double -> float -> e4m3; keep inputs exactly representable in fp32 to avoid double rounding
    x = x.float().double()
    ref = x.float().to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    for i, v in enumerate(x.numpy()):
        assert oracle.f64_to_e4m3(float(v)) == int(ref[i]), v


def test_e4m3_encode_error_bound():
    # relative error of RNE to a 3-bit mantissa is at most 2^-4 in the normal range
    g = np.random.default_rng(0)
    for v in g.uniform(2 ** -6, 448, size=2000):
        q = oracle.e4m3_to_f64(oracle.f64_to_e4m3(v))
        assert abs(q - v) <= 2 ** -4 * v


def test_bf16_encode_rne():
    assert oracle.bf16_to_f64(oracle.f64_to_bf16(1.00390625)) == 1.0      # tie -> even
    assert oracle.bf16_to_f64(oracle.f64_to_bf16(1.01171875)) == 1.015625  # tie -> even (up)
    g = torch.Generator().manual_seed(5)
    x = torch.randn(3000, generator=g)
    ref = x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    for i, v in enumerate(x.numpy()):
        assert oracle.f64_to_bf16(float(v)) == int(ref[i])


def test_silu_closed_forms():
    assert oracle.silu(0.0) == 0.0
    for x in [0.1, 1.0, 2.5, 7.0, 30.0]:
        assert oracle.silu(x) - oracle.silu(-x) == pytest.approx(x, rel=1e-15)
        assert oracle.silu(x) == pytest.approx(x * (0.5 * (1 + math.tanh(x / 2))), rel=1e-14)
    assert oracle.silu(50.0) == pytest.approx(50.0, rel=1e-15)
    assert abs(oracle.silu(-50.0)) < 1e-19
    # value worked by hand: silu(1) = 1/(1+e^-1)
    assert oracle.silu(1.0) == pytest.approx(0.7310585786300049, rel=1e-15)
