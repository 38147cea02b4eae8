"""Microscaling path (MXFP4 expert weights, e4m3 activations, ue8m0 scales per 32 elements) against the fp64
oracle that mirrors the re-quantisation of the intermediate."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_33252_b200 as cep
from paper_2609_33252_b200 import workloads as wl

from helpers import check_close, make_layer, run_layer, to_device, batch_ids

pytestmark = pytest.mark.gpu

MX_MID = wl.MoEConfig("mx_mid", 5, T=640, H=1024, I=384, E_global=16, E_local=6, k=4, chunks=(200, 250, 190),
                      dtype="mxfp4", zipf_s=1.1)


def _layer_with_weights(inp, **kw):
    layer = make_layer(inp.cfg, **kw)
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)
    return layer


@pytest.mark.parametrize("cfg", [wl.CONFIGS["mxfp4_tiny"], MX_MID], ids=lambda c: c.name)
def test_mxfp4_layer_matches_the_oracle(cfg):
    inp = to_device(wl.make_inputs(cfg))
    layer = _layer_with_weights(inp)
    out, n_inv = run_layer(inp, layer)
    assert n_inv == 1
    ref = oracle.from_inputs(wl.make_inputs(cfg))            # mirror of the e4m3 re-quantisation is the default
    rel, worst = check_close(out, ref, cfg.name)
    # integers of the layout transform are the same as for every other dtype
    ids_np = batch_ids(inp, list(range(cfg.n_chunks)))
    exp = oracle.permute(ids_np, cfg.E_local, align=128)
    got = cep.ffn_debug_export(layer.plan, 0, cfg.E_local, ids_np.size)
    assert np.array_equal(got["counts"], exp["counts"]) and np.array_equal(got["row_of_pair"], exp["prow_of_pair"])
    assert np.array_equal(got["pair_of_row"], exp["pair_of_prow"])
    layer.close()


def test_mxfp4_chunked_streamffn_is_bitwise_the_one_shot_result():
    inp = to_device(wl.make_inputs(MX_MID))
    one = _layer_with_weights(inp)
    ref, _ = run_layer(inp, one)
    one.close()
    for mode, theta, order in ((cep.CEP_MODE_ASYNC, 0, [2, 0, 1]), (cep.CEP_MODE_STREAMFFN, 900, None)):
        layer = _layer_with_weights(inp, mode=mode, theta=theta, n_streams=2)
        out, n_inv = run_layer(inp, layer, order=order, local_pairs=True)
        assert n_inv >= 2
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16))
        layer.close()


def test_mxfp4_power_of_two_input_scaling_is_exact():
    # multiplying every activation scale by 2 (code + 1) doubles nothing but exponents on the way in; the
    # intermediate's scales move with it only through the non-linear SiLU, so compare against the oracle again
    cfg = wl.CONFIGS["mxfp4_tiny"]
    inp = wl.make_inputs(cfg)
    inp.x_scale = (inp.x_scale.to(torch.int16) + 1).to(torch.uint8)
    dev = to_device(inp)
    layer = _layer_with_weights(dev)
    out, _ = run_layer(dev, layer)
    check_close(out, oracle.from_inputs(inp), "scaled inputs")
    layer.close()


def test_mxfp4_rejects_unsupported_shapes_and_kernels():
    with pytest.raises(cep.CepError):
        cep.MoELayer(384, 256, 8, 8, 2, 64, 1, dtype=cep.CEP_MXFP4_E4M3)
    with pytest.raises(cep.CepError):
        cep.MoELayer(512, 256, 8, 8, 2, 64, 1, dtype=cep.CEP_MXFP4_E4M3, gemm_impl=cep.CEP_GEMM_TCGEN05_1CTA)
