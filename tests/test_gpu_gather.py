"""GPU: plans made with gather_a (the gate/up GEMM gathers its rows from the caller's token tensor instead of
reading a permuted copy; layout transform of Appendix "Grouped FFN invocations") give the same bits as the default
plans, the same index arrays as the oracle, and refuse what they are not built for."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_33252_b200 as cep
from paper_2609_33252_b200 import workloads as wl

from helpers import batch_ids, check_close, chunks_of, make_layer, run_layer, to_device

pytestmark = pytest.mark.gpu

UNSUPPORTED = -9        # CEP_ERR_UNSUPPORTED


def load(layer, inp):
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)


def both(cfg, inp, order=None, **kw):
    outs, layers = [], []
    for g in (0, 1):
        layer = make_layer(cfg, gather_a=g, **kw)
        load(layer, inp)
        out, n_inv = run_layer(inp, layer, order=order)
        outs.append((out, n_inv)); layers.append(layer)
    return outs, layers


def test_tiny_two_chunks_out_of_order_bitwise_and_index_arrays():
    cfg = wl.CONFIGS["tiny"]
    host = wl.make_inputs(cfg)
    inp = to_device(host)
    (plain, gathered), layers = both(cfg, inp, order=[1, 0], mode=cep.CEP_MODE_ASYNC, n_streams=2)
    assert plain[1] == gathered[1] == 2
    assert torch.equal(plain[0].view(torch.int16), gathered[0].view(torch.int16))
    check_close(gathered[0], oracle.from_inputs(host), "tiny/gather")
    for inv, chunk in ((0, 1), (1, 0)):                     # padding entries of the inverse map are marked without the scatter
        ids = batch_ids(host, [chunk])
        want = oracle.permute(ids, cfg.E_local, align=128)
        got = cep.ffn_debug_export(layers[1].plan, inv, cfg.E_local, ids.size)
        assert (got["row_of_pair"] == want["prow_of_pair"]).all()
        assert (got["pair_of_row"] == want["pair_of_prow"]).all()
    for layer in layers:
        layer.close()


@pytest.mark.parametrize("mode,order", [(cep.CEP_MODE_SYNC, None), (cep.CEP_MODE_STREAMFFN, [3, 0, 2, 1, 5, 4, 7, 6])],
                         ids=["sync", "streamffn_shuffled"])
def test_several_tiles_ragged_groups_and_chunks_bitwise(mode, order):
    """8 experts with a few hundred to a few thousand rows each: several 256-row tiles per expert, ragged last
    blocks, odd block counts (a pair tile whose second half is all padding)."""
    cfg = wl.scaled(wl.CONFIGS["ep_shard_small"], chunks=(256,) * 8)
    host = wl.make_inputs(cfg)
    inp = to_device(host)
    theta = 3 * int((host.topk_ids[:256] < cfg.E_local).sum().item())
    (plain, gathered), layers = both(cfg, inp, order=order, mode=mode, theta=theta, n_streams=2)
    assert plain[1] == gathered[1]
    assert torch.equal(plain[0].view(torch.int16), gathered[0].view(torch.int16))
    counts = np.bincount(host.topk_ids.numpy()[host.topk_ids.numpy() < cfg.E_local], minlength=cfg.E_local)
    assert (counts % 128 != 0).any() and (counts > 256).any()
    # a second call on the same plans: the token tensor's descriptor is rebuilt per layer call
    again, _ = run_layer(inp, layers[1], order=order)
    assert torch.equal(plain[0].view(torch.int16), again.view(torch.int16))
    for layer in layers:
        layer.close()


def test_experts_without_tokens_and_single_row_groups():
    T, k, E = 384, 2, 8
    ids = np.full((T, k), 100, dtype=np.int32)              # not local
    ids[:, 0] = 100 + np.arange(T) % 20
    ids[:, 1] = 120 + np.arange(T) % 20
    ids[0, 0] = 3                                           # expert 3: one row
    ids[5:5 + 129, 1] = 6                                   # expert 6: 129 rows (one full block + 1)
    ids[200:328, 0] = 1                                     # expert 1: exactly 128 rows
    cfg = wl.MoEConfig("edge", 0, T=T, H=512, I=256, E_global=256, E_local=E, k=k, chunks=(128, 256))
    host = wl.make_inputs(cfg)
    host.topk_ids = torch.as_tensor(ids).contiguous()
    inp = to_device(host)
    (plain, gathered), layers = both(cfg, inp, order=[1, 0], mode=cep.CEP_MODE_SYNC)
    assert torch.equal(plain[0].view(torch.int16), gathered[0].view(torch.int16))
    check_close(gathered[0], oracle.from_inputs(host), "edge/gather")
    for layer in layers:
        layer.close()


def test_workspace_is_smaller_by_the_permuted_copy():
    c = wl.CONFIGS["ep_shard_small"]
    mk = lambda g: cep.CepConfig(c.H, c.I, c.E_global, c.E_local, c.k, c.T, 8, cep.CEP_BF16, cep.CEP_MODE_SYNC, 1, 0,
                                 cep.CEP_GEMM_TCGEN05, 0, 0, 0, g)
    plain, gathered = cep.moe_plan_workspace_bytes(mk(0)), cep.moe_plan_workspace_bytes(mk(1))
    cap_rows = c.T * c.k + 127 * c.E_local
    assert plain - gathered >= cap_rows * (c.H * 2 - 4) - 4096


def test_refusals():
    c = wl.CONFIGS["tiny"]
    for dtype, impl in ((cep.CEP_FP8_E4M3_BLOCK128, cep.CEP_GEMM_TCGEN05), (cep.CEP_BF16, cep.CEP_GEMM_TCGEN05_1CTA),
                        (cep.CEP_BF16, cep.CEP_GEMM_SIMT)):
        with pytest.raises(cep.CepError) as e:
            cep.MoELayer(c.H, c.I, c.E_global, c.E_local, c.k, c.T, 2, dtype=dtype, gemm_impl=impl, gather_a=1)
        assert e.value.code == UNSUPPORTED
    # chunks that are not row slices of one tensor
    host = wl.make_inputs(c)
    inp = to_device(host)
    layer = make_layer(c, gather_a=1)
    load(layer, inp)
    out = torch.empty(c.T, c.H, dtype=torch.bfloat16, device="cuda")
    (o0, x0, _, i0, w0), (o1, x1, _, i1, w1) = chunks_of(inp)
    elsewhere = x1.clone()
    cep.ffn_begin(layer.plan, out, c.T, 2)
    cep.ffn_submit_chunk(layer.plan, 0, o0, x0.shape[0], x0, None, i0, w0, -1, None)
    with pytest.raises(cep.CepError) as e:
        cep.ffn_submit_chunk(layer.plan, 1, o1, elsewhere.shape[0], elsewhere, None, i1, w1, -1, None)
    assert e.value.code == UNSUPPORTED
    cep.ffn_submit_chunk(layer.plan, 1, o1, x1.shape[0], x1, None, i1, w1, -1, None)     # the plan is still usable
    cep.ffn_flush(layer.plan); cep.combine(layer.plan, None)
    torch.cuda.synchronize()
    assert cep.ffn_status(layer.plan) == 0
    check_close(out, oracle.from_inputs(host), "tiny/gather after a refusal")
    layer.close()


def test_library_calibration_runs_on_a_gathering_plan():
    """The calibration's probe chunks are row slices of one caller buffer, so a gather_a plan profiles itself too."""
    cfg = wl.MoEConfig("cal", 1, T=2048, H=1024, I=512, E_global=16, E_local=8, k=4, chunks=(2048,))
    inp = to_device(wl.make_inputs(cfg))
    layer = cep.MoELayer(cfg.H, cfg.I, cfg.E_global, cfg.E_local, cfg.k, cfg.T, 4, mode=cep.CEP_MODE_ASYNC, n_streams=2,
                         profile_kernels=1, gather_a=1)
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down)
    ids = torch.empty((cfg.T, cfg.k), dtype=torch.int32, device="cuda")
    w = torch.empty((cfg.T, cfg.k), dtype=torch.float32, device="cuda")
    out = torch.empty((cfg.T, cfg.H), dtype=torch.bfloat16, device="cuda")
    points, res = cep.cep_calibrate(layer.plan, 0.9, [32, 128, 512], 2, inp.x, None, ids, w, out)
    assert [p["rows_per_expert"] for p in points] == [32, 128, 512]
    assert all(p["ffn_ms"] > 0 for p in points) and res["theta_pairs"] > 0
    got, _ = run_layer(inp, layer)
    check_close(got, oracle.from_inputs(wl.make_inputs(cfg)), "gather plan after its calibration")
    layer.close()
