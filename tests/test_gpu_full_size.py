"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (one synchronous
invocation, CTA-pair tensor-core GEMMs): layout integers in full, floats on a seeded sample of tokens the
oracle can compute one by one, plus properties that need no oracle (no NaN, exact-zero rows, chunked ==
one-shot bitwise)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_33252_b200 as cep
from paper_2609_33252_b200 import workloads as wl

from helpers import batch_ids, check_close, chunks_of, make_layer, run_layer

pytestmark = pytest.mark.gpu


def host_view(inp):
    import dataclasses
    kw = {}
    for f in dataclasses.fields(inp):
        v = getattr(inp, f.name)
        kw[f.name] = v.cpu() if isinstance(v, torch.Tensor) else v
    return type(inp)(**kw)


def sample_tokens(inp, n_random=40, seed=0):
    """Random tokens plus tokens routed to the largest, the smallest non-empty and a tile-boundary expert."""
    cfg = inp.cfg
    ids = inp.topk_ids.cpu().numpy()
    counts = np.bincount(ids[ids < cfg.E_local], minlength=cfg.E_local)
    picks = [int(np.argmax(counts)), int(np.argmin(np.where(counts > 0, counts, 1 << 30)))]
    rng = np.random.default_rng(seed)
    sel = list(rng.integers(0, cfg.T, n_random))
    for e in picks:
        toks = np.nonzero((ids == e).any(axis=1))[0]
        sel += [int(toks[0]), int(toks[-1]), int(toks[len(toks) // 2])]     # first / last / middle row of the group
    none_local = np.nonzero((ids >= cfg.E_local).all(axis=1))[0]
    sel += [int(t) for t in none_local[:2]]
    return np.unique(np.array(sel, dtype=np.int64))


@pytest.mark.parametrize("name", ["ep_shard", "ep_shard_strided", "mxfp4_shard", "fp8_shard", "mxfp4_pro_shard"])
def test_ep_shard_full_size(name):
    cfg = wl.CONFIGS[name]
    inp = wl.make_inputs(cfg, device="cuda", keep_logits=False)
    host = host_view(inp)
    layer = make_layer(cfg, mode=cep.CEP_MODE_SYNC, debug_checks=1)
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)
    out, n_inv = run_layer(inp, layer, local_pairs=True)
    assert n_inv == 1
    assert cep.cep_debug_check_guards(layer.plan) == 0
    # integers: every count, offset and row of all T*k pairs
    want = oracle.permute(batch_ids(host, list(range(cfg.n_chunks))), cfg.E_local, align=128)
    got = cep.ffn_debug_export(layer.plan, 0, cfg.E_local, cfg.T * cfg.k)
    for k_, w_ in (("counts", "counts"), ("offsets", "offsets"), ("padded_offsets", "padded_offsets"),
                   ("row_of_pair", "prow_of_pair"), ("pair_of_row", "pair_of_prow")):
        assert (got[k_] == want[w_]).all(), k_
    assert int(want["counts"].sum()) == host.n_local_pairs()
    # floats on the sample
    sel = sample_tokens(host)
    ref = oracle.from_inputs(host, sel=sel)
    check_close(out[torch.as_tensor(sel, device="cuda")], ref, name + " sample")
    # whole-tensor properties
    assert torch.isfinite(out.float()).all()
    none_local = (inp.topk_ids >= cfg.E_local).all(dim=1)
    assert (out[none_local].view(torch.int16) == 0).all()
    assert (out[~none_local].float().abs().sum(dim=1) > 0).all()
    # chunked asynchronous execution gives the same bits as the one synchronous launch
    stream = make_layer(cfg, mode=cep.CEP_MODE_STREAMFFN, theta=max(1, host.n_local_pairs() // 3), n_streams=2)
    stream.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)
    out2, n_inv2 = run_layer(inp, stream, order=wl.submission_order(host.arrival), local_pairs=True)
    assert n_inv2 > 1
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
    layer.close(); stream.close()
    if cfg.dtype == "bf16":
        # the plan without a permuted copy (GEMM1 gathers its rows from the token tensor): same bits, guards intact
        gathered = make_layer(cfg, mode=cep.CEP_MODE_STREAMFFN, theta=max(1, host.n_local_pairs() // 3), n_streams=2,
                              debug_checks=1, gather_a=1)
        gathered.load_weights(inp.w_gate, inp.w_up, inp.w_down)
        out3, n_inv3 = run_layer(inp, gathered, order=wl.submission_order(host.arrival), local_pairs=True)
        assert n_inv3 == n_inv2
        assert cep.cep_debug_check_guards(gathered.plan) == 0
        assert torch.equal(out.view(torch.int16), out3.view(torch.int16))
        gathered.close()


def test_straggler_config_threshold_sweep_is_bitwise_stable():
    cfg = wl.CONFIGS["straggler"]
    inp = wl.make_inputs(cfg, device="cuda", keep_logits=False)
    order = wl.submission_order(inp.arrival)
    assert order[-1] == cfg.n_chunks - 1                 # the 40 % straggler is submitted last
    base = None
    sweep = [(cep.CEP_MODE_STREAMFFN, 256), (cep.CEP_MODE_STREAMFFN, 2048), (cep.CEP_MODE_STREAMFFN, 32 * 512),
             (cep.CEP_MODE_STREAMFFN, 32 * 2048)]
    # repeated: overlapping invocations on two streams must give the same bits every time
    for mode, theta in [(cep.CEP_MODE_SYNC, 0)] + sweep * 6:
        layer = make_layer(cfg, mode=mode, theta=theta, n_streams=2)
        layer.load_weights(inp.w_gate, inp.w_up, inp.w_down)
        out, n_inv = run_layer(inp, layer, order=order, local_pairs=True)
        pairs = [int((inp.topk_ids[o:o + n] < cfg.E_local).sum().item()) for o, n in zip(inp.chunk_offsets, cfg.chunks)]
        assert n_inv == len(oracle.schedule([pairs[c] for c in order], mode, theta, 2))
        if base is None:
            base = out.clone()
            # these inputs are drawn with their own seeds: the synchronous result meets the oracle on a sample
            host = host_view(inp)
            sel = sample_tokens(host, n_random=12)
            check_close(base[torch.as_tensor(sel, device="cuda")], oracle.from_inputs(host, sel=sel), "straggler sample")
        else:
            assert torch.equal(base.view(torch.int16), out.view(torch.int16)), (mode, theta)
        layer.close()
