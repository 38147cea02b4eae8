"""GPU: many chunked layer calls in a row on the same plans, with shuffled arrival orders: overlapping invocations on
several streams, the tile rings and the scratch-slot reuse must give the synchronous result bit for bit every time
(Section 3.2: chunked asynchronous execution changes when work runs, not what it computes)."""
import random

import pytest
import torch

import paper_2609_33252_b200 as cep
from paper_2609_33252_b200 import workloads as wl

from helpers import make_layer, run_layer, to_device

pytestmark = pytest.mark.gpu

CALLS = 120


@pytest.mark.parametrize("name,gather", [("ep_shard_small", 0), ("ep_shard_small", 1), ("fp8_shard_small", 0),
                                         ("mxfp4_shard_small", 0), ("mid", 0)])
def test_repeated_chunked_calls_are_bitwise_stable(name, gather):
    cfg = wl.CONFIGS[name]
    if cfg.n_chunks < 4:
        cfg = wl.scaled(cfg, chunks=(cfg.T // 8,) * 8)
    inp = to_device(wl.make_inputs(cfg))
    weights = (inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)
    sync = make_layer(cfg, mode=cep.CEP_MODE_SYNC, gather_a=gather)
    sync.load_weights(*weights)
    base, _ = run_layer(inp, sync)
    sync.close()
    pairs = int((inp.topk_ids < cfg.E_local).sum().item())
    rng = random.Random(7)
    for mode, theta, streams in ((cep.CEP_MODE_ASYNC, 0, 2), (cep.CEP_MODE_STREAMFFN, max(1, pairs // 3), 2),
                                 (cep.CEP_MODE_STREAMFFN, max(1, pairs // 5), 3)):
        layer = make_layer(cfg, mode=mode, theta=theta, n_streams=streams, gather_a=gather)
        layer.load_weights(*weights)
        for call in range(CALLS):
            order = list(range(cfg.n_chunks))
            rng.shuffle(order)
            out, _ = run_layer(inp, layer, order=order, local_pairs=True)
            assert torch.equal(out.view(torch.int16), base.view(torch.int16)), (mode, theta, call, order)
        layer.close()
