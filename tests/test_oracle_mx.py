"""Pins for the oracle's microscaling pieces (e2m1 / ue8m0 codecs, the block-scale rule, MXFP4
tensors in the layer, the MXFP8 re-quantisation of the intermediate).

The pins are closed forms of the formats, library casts (torch's e8m0 and e4m3 dtypes), numpy
de-quantisation through a lookup table, and properties that fix the block-scale rule uniquely.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_33252_b200 import workloads as wl

E2M1_VALUES = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


def test_e2m1_table_is_the_closed_form():
    for c in range(16):
        s, e, m = c >> 3, (c >> 1) & 3, c & 1
        v = 0.5 * m if e == 0 else (1.0 + 0.5 * m) * 2.0 ** (e - 1)
        assert oracle.e2m1_to_f64(c) == (-v if s else v)
        assert abs(oracle.e2m1_to_f64(c)) == E2M1_VALUES[c & 7]
        assert oracle.e2m1_to_f64(c | 0xF0) == oracle.e2m1_to_f64(c)      # high nibble ignored by the layer
    assert np.signbit(oracle.e2m1_to_f64(8))


def test_e2m1_encoder_nearest_even_and_saturation():
    for c in range(16):
        assert oracle.f64_to_e2m1(oracle.e2m1_to_f64(c)) == c
    # midpoints go to the neighbour whose mantissa bit is 0
    for lo, hi, want in ((0.0, 0.5, 0.0), (0.5, 1.0, 1.0), (1.0, 1.5, 1.0), (1.5, 2.0, 2.0), (2.0, 3.0, 2.0),
                         (3.0, 4.0, 4.0), (4.0, 6.0, 4.0)):
        mid = (lo + hi) / 2
        assert oracle.e2m1_to_f64(oracle.f64_to_e2m1(mid)) == want
        assert oracle.e2m1_to_f64(oracle.f64_to_e2m1(-mid)) == -want
        assert oracle.e2m1_to_f64(oracle.f64_to_e2m1(np.nextafter(mid, 10.0))) == hi
        assert oracle.e2m1_to_f64(oracle.f64_to_e2m1(np.nextafter(mid, 0.0))) == lo
    assert oracle.f64_to_e2m1(6.0) == 7 and oracle.f64_to_e2m1(1e9) == 7 and oracle.f64_to_e2m1(-7.0) == 15
    # brute force: the decoded value is a nearest grid point for a dense sweep
    grid = np.array(E2M1_VALUES)
    for x in np.linspace(-6.5, 6.5, 2601):
        v = oracle.e2m1_to_f64(oracle.f64_to_e2m1(float(x)))
        assert abs(abs(x) - abs(v)) <= np.min(np.abs(grid - abs(x))) + 1e-15


def test_ue8m0_matches_library_dtype_and_closed_form():
    codes = torch.arange(0, 255, dtype=torch.uint8)
    lib_vals = codes.view(torch.float8_e8m0fnu).double().numpy()
    for c in range(255):
        assert oracle.ue8m0_to_f64(c) == np.ldexp(1.0, c - 127)
        if c > 0:                      # 2^-127 is a binary32 subnormal; the library cast may flush it
            assert oracle.ue8m0_to_f64(c) == lib_vals[c]
    assert np.isnan(oracle.ue8m0_to_f64(255))


@pytest.mark.parametrize("elem,elem_max", [("e4m3", 448.0), ("e2m1", 6.0)])
def test_block_scale_is_the_smallest_power_of_two_that_fits(elem, elem_max):
    r = np.random.default_rng(11)
    amaxes = list(np.exp(r.uniform(-30, 30, size=400)).astype(np.float32))
    for q in (-20, -1, 0, 1, 9):
        edge = np.float32(elem_max * 2.0 ** q)
        amaxes += [edge, np.nextafter(edge, np.float32(np.inf)), np.nextafter(edge, np.float32(0))]
    for a in amaxes:
        code = oracle.mx_scale_code(float(a), elem)
        s = 2.0 ** (code - 127)
        assert float(a) <= elem_max * s                   # fits: nothing saturates
        assert float(a) > elem_max * s / 2                # and no smaller power of two would
    assert oracle.mx_scale_code(0.0, elem) == 127
    assert oracle.mx_scale_code(float(np.float32(elem_max)), elem) == 127
    assert oracle.mx_scale_code(float(np.nextafter(np.float32(elem_max), np.float32(np.inf))), elem) == 128
    assert oracle.mx_scale_code(1e-45, elem) == 0          # clamped at the bottom of the range


def test_input_quantiser_agrees_with_the_oracle_codecs():
    g = torch.Generator().manual_seed(3)
    x = torch.randn((6, 96), generator=g) * torch.exp(2.0 * torch.randn((6, 1), generator=g))
    x[2, 32:64] = 0.0
    for elem in ("e4m3", "e2m1"):
        codes, scales = wl.quantize_mx(x, elem, 1)
        cb = codes.view(torch.uint8).numpy() if elem == "e4m3" else codes.numpy()
        for r in range(6):
            for b in range(3):
                blk = x[r, 32 * b:32 * b + 32].double().numpy()
                sc = oracle.mx_scale_code(float(np.abs(blk).max()), elem)
                assert int(scales[r, b]) == sc
                for i in range(32):
                    y = blk[i] / 2.0 ** (sc - 127)
                    want = oracle.f64_to_e4m3(y) if elem == "e4m3" else oracle.f64_to_e2m1(y)
                    got = int(cb[r, 32 * b + i])
                    if y == 0.0:
                        assert got & 0x7F == 0 if elem == "e4m3" else got & 7 == 0
                    else:
                        assert got == want, (elem, r, b, i, y, got, want)
    # blocks along another dimension: scales follow the blocked dimension
    w = torch.randn((64, 5), generator=g)
    c0, s0 = wl.quantize_mx(w, "e2m1", 0)
    c1, s1 = wl.quantize_mx(w.t().contiguous(), "e2m1", 1)
    assert s0.shape == (2, 5) and torch.equal(c0, c1.t()) and torch.equal(s0, s1.t())


def _dequant_np(codes, scales, table, block_axis):
    """numpy de-quantisation through a lookup table and ldexp (independent of the C decoders)."""
    vals = table[codes.astype(np.int64)]
    exp = np.repeat(scales.astype(np.int64) - 127, 32, axis=block_axis)
    return np.ldexp(vals, exp)


def _tables():
    e2m1 = np.array(E2M1_VALUES + [-v for v in E2M1_VALUES])
    e4m3 = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).double().numpy()   # library decode
    return e2m1, e4m3


def test_mxfp4_layer_equals_the_f64_layer_on_dequantised_tensors():
    inp = wl.make_inputs(wl.scaled(wl.CONFIGS["mxfp4_tiny"], T=12, chunks=(12,), H=64, I=96, E_global=4, E_local=3))
    e2m1, e4m3 = _tables()
    X = _dequant_np(inp.x.view(torch.uint8).numpy(), inp.x_scale.numpy(), e4m3, 1)
    Wg = _dequant_np(inp.w_gate.numpy(), inp.s_gate.numpy(), e2m1, 1)
    Wu = _dequant_np(inp.w_up.numpy(), inp.s_up.numpy(), e2m1, 1)
    Wd = _dequant_np(inp.w_down.numpy(), inp.s_down.numpy(), e2m1, 1)
    ids, w = inp.topk_ids.numpy(), inp.topk_w.numpy()
    ref = oracle.moe_forward(oracle.F64, X, None, ids, w, Wg, None, Wu, None, Wd, None, 3)
    got = oracle.from_inputs(inp, mirror=0)
    assert np.array_equal(got, ref)                        # same loop, exactly de-quantised operands
    assert np.abs(ref).max() > 0


def test_mxfp8_mirror_requantises_the_intermediate_per_row_and_32_block():
    # one expert, k=1, w=1, down projection = identity (1.0 is e2m1 code 2, scale 1): the layer's output IS the
    # re-quantised intermediate.  The expected values come from numpy amax + torch's e4m3 cast.
    T, H, I = 5, 64, 64
    g = torch.Generator().manual_seed(8)
    x, xs = wl.quantize_mx(torch.randn((T, H), generator=g) * 3.0, "e4m3", 1)
    wg, sg = wl.quantize_mx(torch.randn((H, I), generator=g) * 0.4, "e2m1", 0)
    wu, su = wl.quantize_mx(torch.randn((H, I), generator=g) * 0.4, "e2m1", 0)
    wd = (torch.eye(I, dtype=torch.uint8) * 2)[None]
    sd = torch.full((1, I // 32, H), 127, dtype=torch.uint8)
    ids = np.zeros((T, 1), np.int32)
    w = np.ones((T, 1), np.float32)
    args = (x.view(torch.uint8).numpy(), xs.numpy(), ids, w, wg[None].numpy(), sg[None].numpy(), wu[None].numpy(),
            su[None].numpy(), wd.numpy(), sd.numpy(), 1)
    a = oracle.moe_forward(oracle.MXFP4, *args, mirror=0)                     # = silu(g)*u, unrounded
    got = oracle.moe_forward(oracle.MXFP4, *args, mirror=oracle.MIRROR_MXFP8_ACT)
    want = np.empty_like(a)
    for t in range(T):
        for b in range(I // 32):
            blk = a[t, 32 * b:32 * b + 32]
            amax = float(np.float32(np.abs(blk).max()))
            q = int(np.ceil(np.log2(amax / 448.0)))                          # smallest power of two that fits
            y = torch.tensor(blk / 2.0 ** q, dtype=torch.float64).to(torch.float8_e4m3fn).double().numpy()
            want[t, 32 * b:32 * b + 32] = y * 2.0 ** q
    assert np.array_equal(got, want)
    rel = np.linalg.norm(got - a) / np.linalg.norm(a)
    assert 1e-3 < rel < 5e-2                                                  # e4m3 step, 3 mantissa bits
