"""The steps either side of the routed-expert path: the router kernel in front (softmax, top-k, renormalise;
ids bit-exact against the oracle's routing, ties to the lower id) and the shared expert's output added by the
combine (Appendix "Output return and combine": routed result and shared-expert output are summed)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_33252_b200 as cep
from paper_2609_33252_b200 import workloads as wl

from helpers import check_close, chunks_of, make_layer, to_device

pytestmark = pytest.mark.gpu


def gpu_route(logits, k):
    T = logits.shape[0]
    ids = torch.full((T, k), -1, dtype=torch.int32, device="cuda")
    w = torch.full((T, k), float("nan"), dtype=torch.float32, device="cuda")
    cep.moe_route(logits.cuda().contiguous(), k, ids, w)
    torch.cuda.synchronize()
    return ids.cpu(), w.cpu()


@pytest.mark.parametrize("name", ["mid", "ep_shard", "fp8_shard"])
def test_router_matches_oracle_routing(name):
    cfg = wl.CONFIGS[name]
    logits = wl.make_logits(wl.scaled(cfg, T=512, chunks=(512,)))
    logits[7, 3] = logits[7, 11] = logits[7].max() + 2.0          # an exact tie for the top slot
    logits[9, :] = 0.25                                            # every expert tied: ids 0..k-1 in order
    ids, w = gpu_route(logits, cfg.k)
    sel = np.concatenate([np.arange(0, 24), np.arange(500, 512)])
    oid, ow = oracle.route(logits.numpy()[sel], cfg.k)
    assert (ids.numpy()[sel] == oid).all()
    np.testing.assert_allclose(w.numpy()[sel], ow, rtol=5e-6)
    assert ids[7, 0] == 3 and ids[7, 1] == 11
    assert ids[9].tolist() == list(range(cfg.k))
    # every row against the generator's routing (library sort + fp64 softmax)
    gid, gw = wl.route(logits, cfg.k)
    assert torch.equal(ids, gid)
    assert torch.allclose(w, gw, rtol=5e-6, atol=0)
    assert torch.allclose(w.double().sum(1), torch.ones(512, dtype=torch.float64), atol=1e-6)
    assert (w[:, 1:] <= w[:, :-1]).all()


def test_router_feeds_the_layer_end_to_end():
    cfg = wl.CONFIGS["tiny"]
    host = wl.make_inputs(cfg)
    inp = to_device(host)
    ids = torch.empty_like(inp.topk_ids)
    w = torch.empty_like(inp.topk_w)
    cep.moe_route(inp.logits, cfg.k, ids, w)
    layer = make_layer(cfg, mode=cep.CEP_MODE_SYNC)
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down)
    out = torch.empty(cfg.T, cfg.H, dtype=torch.bfloat16, device="cuda")
    layer.run(out, [(0, inp.x, None, ids, w)])
    torch.cuda.synchronize()
    assert cep.ffn_status(layer.plan) == 0
    assert torch.equal(ids.cpu(), host.topk_ids)
    check_close(out, oracle.from_inputs(host), "router -> layer")
    layer.close()


def test_shared_expert_output_is_added_by_the_combine():
    cfg = wl.CONFIGS["tiny"]
    host = wl.make_inputs(cfg)
    inp = to_device(host)
    # the shared expert: a dense SwiGLU MLP over every token = one expert, k = 1, weight 1
    g = torch.Generator().manual_seed(77)
    sg = (torch.randn(1, cfg.H, cfg.I, generator=g) * cfg.H ** -0.5).to(torch.bfloat16)
    su = (torch.randn(1, cfg.H, cfg.I, generator=g) * cfg.H ** -0.5).to(torch.bfloat16)
    sd = (torch.randn(1, cfg.I, cfg.H, generator=g) * cfg.I ** -0.5).to(torch.bfloat16)
    ones_ids = torch.zeros(cfg.T, 1, dtype=torch.int32)
    ones_w = torch.ones(cfg.T, 1, dtype=torch.float32)
    bits = lambda t: t.view(torch.int16).numpy().view(np.uint16)
    ref_shared = oracle.moe_forward(oracle.BF16, bits(host.x), None, ones_ids.numpy(), ones_w.numpy(), bits(sg), None,
                                    bits(su), None, bits(sd), None, 1)
    ref = oracle.from_inputs(host) + ref_shared
    shared = cep.MoELayer(cfg.H, cfg.I, 1, 1, 1, cfg.T, 1, mode=cep.CEP_MODE_SYNC, n_streams=1)
    shared.load_weights(sg.cuda(), su.cuda(), sd.cuda())
    y_shared = torch.empty(cfg.T, cfg.H, dtype=torch.bfloat16, device="cuda")
    shared.run(y_shared, [(0, inp.x, None, ones_ids.cuda(), ones_w.cuda())])
    check_close(y_shared, ref_shared, "shared expert alone")
    layer = make_layer(cfg, mode=cep.CEP_MODE_ASYNC, n_streams=2)
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down)
    out = torch.empty(cfg.T, cfg.H, dtype=torch.bfloat16, device="cuda")
    n_inv = layer.run(out, chunks_of(inp), addend=y_shared)
    torch.cuda.synchronize()
    assert n_inv == 2 and cep.ffn_status(layer.plan) == 0
    check_close(out, ref, "routed + shared")
    # the addend is per layer call: the next call without it gives the routed result alone
    layer.run(out, chunks_of(inp))
    torch.cuda.synchronize()
    check_close(out, oracle.from_inputs(host), "routed only")
    with pytest.raises(cep.CepError) as e:
        cep.ffn_set_addend(layer.plan, y_shared)           # no layer call open
    assert e.value.code == -2
    shared.close(); layer.close()
