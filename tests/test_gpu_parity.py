"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Integers bit-exact; floats within the stated tolerance of the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_33252_b200 as cep
from paper_2609_33252_b200 import workloads as wl

from helpers import (batch_ids, check_close, chunks_of, make_layer, run_layer, to_device)

pytestmark = pytest.mark.gpu

IMPLS = [cep.CEP_GEMM_SIMT, cep.CEP_GEMM_TCGEN05, cep.CEP_GEMM_TCGEN05_1CTA]


def load(layer, inp):
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down, inp.s_gate, inp.s_up, inp.s_down)


def assert_layout_matches(layer, inv, ids_np, E):
    want = oracle.permute(ids_np, E, align=128)
    got = cep.ffn_debug_export(layer.plan, inv, E, ids_np.size)
    assert (got["counts"] == want["counts"]).all()
    assert (got["offsets"] == want["offsets"]).all()
    assert (got["padded_offsets"] == want["padded_offsets"]).all()
    assert (got["row_of_pair"] == want["prow_of_pair"]).all()
    assert (got["pair_of_row"] == want["pair_of_prow"]).all()


# ------------------------------------------------------------------ config 0 (tiny), whole tensor
@pytest.mark.parametrize("impl", IMPLS, ids=["simt", "tcgen05", "tcgen05_1cta"])
def test_tiny_sync_matches_oracle(impl):
    cfg = wl.CONFIGS["tiny"]
    host = wl.make_inputs(cfg)
    ref = oracle.from_inputs(host)
    inp = to_device(host)
    layer = make_layer(cfg, mode=cep.CEP_MODE_SYNC, gemm_impl=impl)
    load(layer, inp)
    out, n_inv = run_layer(inp, layer)
    assert n_inv == 1
    assert_layout_matches(layer, 0, batch_ids(host, [0, 1]), cfg.E_local)
    check_close(out, ref, "tiny/sync")
    layer.close()


@pytest.mark.parametrize("impl", IMPLS, ids=["simt", "tcgen05", "tcgen05_1cta"])
def test_tiny_chunked_equals_one_shot_bitwise_and_layouts_per_invocation(impl):
    cfg = wl.CONFIGS["tiny"]
    host = wl.make_inputs(cfg)
    inp = to_device(host)
    sync = make_layer(cfg, mode=cep.CEP_MODE_SYNC, gemm_impl=impl)
    load(sync, inp)
    one, _ = run_layer(inp, sync)
    asy = make_layer(cfg, mode=cep.CEP_MODE_ASYNC, n_streams=2, gemm_impl=impl)
    load(asy, inp)
    two, n_inv = run_layer(inp, asy, order=[1, 0])          # chunk 1 arrives first
    assert n_inv == 2
    assert_layout_matches(asy, 0, batch_ids(host, [1]), cfg.E_local)
    assert_layout_matches(asy, 1, batch_ids(host, [0]), cfg.E_local)
    assert torch.equal(one.view(torch.int16), two.view(torch.int16))
    # a second layer call on the same plan gives the same bits (scratch reuse, status reset)
    again, _ = run_layer(inp, asy, order=[0, 1])
    assert torch.equal(one.view(torch.int16), again.view(torch.int16))
    sync.close(); asy.close()


# ------------------------------------------------------------------ edge cases of the layout transform
def edge_inputs(T, k, E_global, E_local, H, I, ids, seed=0, chunks=None):
    cfg = wl.MoEConfig("edge", 0, T=T, H=H, I=I, E_global=E_global, E_local=E_local, k=k,
                       chunks=tuple(chunks or (T,)))
    inp = wl.make_inputs(cfg)
    inp.topk_ids = torch.as_tensor(ids, dtype=torch.int32).contiguous()
    g = torch.Generator().manual_seed(seed)
    w = torch.rand(T, k, generator=g) + 0.1
    inp.topk_w = (w / w.sum(1, keepdim=True)).float().contiguous()
    return inp


def distinct_ids(T, k, E, seed):
    r = np.random.default_rng(seed)
    return np.stack([r.permutation(E)[:k] for _ in range(T)]).astype(np.int32)


EDGE_CASES = {
    "one_token": lambda: edge_inputs(1, 2, 8, 8, 256, 128, distinct_ids(1, 2, 8, 1)),
    "k1_all_to_one_expert": lambda: edge_inputs(300, 1, 4, 4, 256, 128, np.full((300, 1), 2, np.int32)),
    "count_127_128_129": lambda: edge_inputs(
        384, 1, 4, 4, 256, 128,
        np.concatenate([np.full(127, 0), np.full(128, 1), np.full(129, 3)]).astype(np.int32)[:, None]),
    "empty_experts_and_remote": lambda: edge_inputs(200, 3, 16, 5, 256, 128, distinct_ids(200, 3, 16, 3)),
    "nothing_local": lambda: edge_inputs(50, 2, 16, 4, 256, 128, 8 + distinct_ids(50, 2, 8, 4)),
    "ragged_three_chunks": lambda: edge_inputs(333, 4, 12, 12, 384, 256, distinct_ids(333, 4, 12, 5),
                                               chunks=(1, 300, 32)),
    "many_experts": lambda: edge_inputs(700, 8, 96, 96, 256, 128, distinct_ids(700, 8, 96, 6)),
}


@pytest.mark.parametrize("impl", IMPLS, ids=["simt", "tcgen05", "tcgen05_1cta"])
@pytest.mark.parametrize("case", sorted(EDGE_CASES))
def test_edge_cases(case, impl):
    host = EDGE_CASES[case]()
    cfg = host.cfg
    ref = oracle.from_inputs(host)
    inp = to_device(host)
    layer = make_layer(cfg, mode=cep.CEP_MODE_SYNC, gemm_impl=impl, debug_checks=1)
    load(layer, inp)
    out, n_inv = run_layer(inp, layer)
    assert n_inv == 1
    assert_layout_matches(layer, 0, batch_ids(host, list(range(cfg.n_chunks))), cfg.E_local)
    check_close(out, ref, case)
    assert cep.cep_debug_check_guards(layer.plan) == 0         # no kernel wrote past the end of a workspace region
    none_local = (host.topk_ids >= cfg.E_local).all(dim=1)
    if none_local.any():                                   # exact zeros, written not skipped
        assert (out.cpu()[none_local].view(torch.int16) == 0).all()
    layer.close()


def test_k1_weight1_identical_experts_is_dense_mlp_rowwise():
    # k=1, weight 1: the combine is a pure un-permutation, so every token's output must be the
    # dense SwiGLU MLP of that token, whatever expert (all hold the same weights) it went to.
    T, H, I, E = 260, 256, 128, 4
    host = edge_inputs(T, 1, E, E, H, I, np.random.default_rng(0).integers(0, E, (T, 1)).astype(np.int32))
    host.topk_w = torch.ones(T, 1)
    for t in (host.w_gate, host.w_up, host.w_down):
        t[1:] = t[0]
    x = host.x.double()
    g, u, d = host.w_gate[0].double(), host.w_up[0].double(), host.w_down[0].double()
    ref = ((torch.nn.functional.silu(x @ g) * (x @ u)) @ d).numpy()
    inp = to_device(host)
    layer = make_layer(host.cfg, mode=cep.CEP_MODE_SYNC)
    load(layer, inp)
    out, _ = run_layer(inp, layer)
    check_close(out, ref, "k1 dense")
    layer.close()


# ------------------------------------------------------------------ config 1 (mid): modes, streams, sampled floats
def test_mid_modes_agree_bitwise_and_match_oracle_on_a_sample():
    cfg = wl.CONFIGS["mid"]
    host = wl.make_inputs(cfg)
    inp = to_device(host)
    sel = np.unique(np.concatenate([np.arange(0, 8), np.arange(1530, 1542), np.arange(4088, 4096),
                                    np.random.default_rng(0).integers(0, cfg.T, 100)]))
    ref = oracle.from_inputs(host, sel=sel)
    sync = make_layer(cfg, mode=cep.CEP_MODE_SYNC)
    load(sync, inp)
    base, n = run_layer(inp, sync)
    assert n == 1
    assert_layout_matches(sync, 0, batch_ids(host, [0, 1, 2, 3]), cfg.E_local)
    check_close(base[torch.as_tensor(sel, device=base.device)], ref, "mid/sync sample")
    order = wl.submission_order(host.arrival)
    pairs = [c * cfg.k for c in cfg.chunks]
    for mode, theta, S in [(cep.CEP_MODE_ASYNC, 0, 1), (cep.CEP_MODE_STREAMFFN, 9000, 2),
                           (cep.CEP_MODE_STREAMFFN, 12288, 3)]:
        layer = make_layer(cfg, mode=mode, theta=theta, n_streams=S)
        load(layer, inp)
        out, n_inv = run_layer(inp, layer, order=order)
        want = oracle.schedule([pairs[c] for c in order], mode, theta, S)
        assert n_inv == len(want)
        for i, (pos, stream) in enumerate(want):
            info = cep.ffn_query(layer.plan, i)
            assert info.n_chunks == len(pos) and info.first_chunk_pos == pos[0] and info.stream_index == stream
            assert info.elapsed_ms >= 0
        for i in range(max(0, n_inv - S), n_inv):          # slots still holding their invocation
            assert_layout_matches(layer, i, batch_ids(host, [order[p] for p in want[i][0]]), cfg.E_local)
        assert torch.equal(out.view(torch.int16), base.view(torch.int16)), (mode, theta, S)
        layer.close()
    sync.close()


def test_simt_and_tensor_core_paths_agree_closely_on_mid():
    cfg = wl.scaled(wl.CONFIGS["mid"], T=1024, chunks=(1024,))
    inp = to_device(wl.make_inputs(cfg))
    outs = []
    for impl in IMPLS:
        layer = make_layer(cfg, gemm_impl=impl)
        load(layer, inp)
        outs.append(run_layer(inp, layer)[0].float())
        layer.close()
    rel = (outs[0] - outs[1]).norm() / outs[0].norm()
    assert rel < 3e-3            # both round the intermediate and the output to bf16 once
    # the two tensor-core variants accumulate every row in the same K order: identical bits
    assert torch.equal(outs[1], outs[2])


# ------------------------------------------------------------------ errors are reported, never faults
def test_error_paths():
    cfg = wl.CONFIGS["tiny"]
    host = wl.make_inputs(cfg)
    inp = to_device(host)
    layer = make_layer(cfg, mode=cep.CEP_MODE_SYNC)
    out = torch.zeros(cfg.T, cfg.H, dtype=torch.bfloat16, device="cuda")
    ch = chunks_of(inp)
    with pytest.raises(cep.CepError) as e:                 # no weights yet
        cep.ffn_begin(layer.plan, out, cfg.T, 2)
    assert e.value.code == -2
    load(layer, inp)
    with pytest.raises(cep.CepError) as e:                 # submit before begin
        cep.ffn_submit_chunk(layer.plan, 0, 0, 160, ch[0][1], None, ch[0][3], ch[0][4])
    assert e.value.code == -2
    with pytest.raises(cep.CepError) as e:
        cep.ffn_begin(layer.plan, out, cfg.T + 1, 2)
    assert e.value.code == -4
    cep.ffn_begin(layer.plan, out, cfg.T, 2)
    with pytest.raises(cep.CepError) as e:
        cep.ffn_begin(layer.plan, out, cfg.T, 2)
    assert e.value.code == -2
    with pytest.raises(cep.CepError) as e:
        cep.ffn_submit_chunk(layer.plan, 5, 0, 160, ch[0][1], None, ch[0][3], ch[0][4])
    assert e.value.code == -1
    cep.ffn_submit_chunk(layer.plan, 0, 0, 160, ch[0][1], None, ch[0][3], ch[0][4])
    with pytest.raises(cep.CepError) as e:                 # double submit
        cep.ffn_submit_chunk(layer.plan, 0, 0, 160, ch[0][1], None, ch[0][3], ch[0][4])
    assert e.value.code == -2
    assert cep.ffn_flush(layer.plan, allow_incomplete=True) == -5      # one chunk missing
    with pytest.raises(cep.CepError) as e:                 # submit after flush
        cep.ffn_submit_chunk(layer.plan, 1, 160, 96, ch[1][1], None, ch[1][3], ch[1][4])
    assert e.value.code == -2
    assert cep.combine(layer.plan, allow_incomplete=True) == -5
    torch.cuda.synchronize()
    assert cep.ffn_status(layer.plan) == 0
    ref = oracle.from_inputs(host, sel=np.arange(160))      # the submitted chunk still completed
    check_close(out[:160], ref, "incomplete layer")
    # an expert id outside [0, E_global) is flagged by the device, not dereferenced
    bad = inp.topk_ids.clone()
    bad[3, 1] = 99
    cep.ffn_begin(layer.plan, out, cfg.T, 1)
    cep.ffn_submit_chunk(layer.plan, 0, 0, cfg.T, inp.x, None, bad, inp.topk_w)
    cep.combine(layer.plan)
    torch.cuda.synchronize()
    assert cep.ffn_status(layer.plan) == -6
    # and the next layer call starts clean
    out2, _ = run_layer(inp, layer)
    check_close(out2, oracle.from_inputs(host), "after bad routing")
    layer.close()
    # workspace too small / misaligned
    c = layer.cfg
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(cep.CepError) as e:
        cep.moe_plan(c, ws)
    assert e.value.code == -3


def test_chunk_coverage_and_alignment_are_checked_on_the_host():
    # return codes only: nothing that could write out of bounds is ever launched
    cfg = wl.CONFIGS["tiny"]
    host = wl.make_inputs(cfg)
    inp = to_device(host)
    layer = make_layer(cfg, mode=cep.CEP_MODE_SYNC)
    load(layer, inp)
    out = torch.zeros(cfg.T + 8, cfg.H, dtype=torch.bfloat16, device="cuda")
    ch = chunks_of(inp)
    with pytest.raises(cep.CepError) as e:                 # output rows are stored 16 bytes at a time
        cep.ffn_begin(layer.plan, out.view(-1)[1:], cfg.T, 2)
    assert e.value.code == -1
    cep.ffn_begin(layer.plan, out, cfg.T, 2)
    cep.ffn_submit_chunk(layer.plan, 0, 0, 160, ch[0][1], None, ch[0][3], ch[0][4])
    with pytest.raises(cep.CepError) as e:                 # overlaps chunk 0: 160 + 156 tokens > 256
        cep.ffn_submit_chunk(layer.plan, 1, 100, 156, inp.x[100:256], None, inp.topk_ids[100:256], inp.topk_w[100:256])
    assert e.value.code == -4
    # a short last chunk leaves rows uncovered: reported, the submitted work still completes
    cep.ffn_submit_chunk(layer.plan, 1, 160, 90, inp.x[160:250], None, inp.topk_ids[160:250], inp.topk_w[160:250])
    assert cep.ffn_flush(layer.plan, allow_incomplete=True) == -5
    assert cep.combine(layer.plan, allow_incomplete=True) == -5
    torch.cuda.synchronize()
    assert cep.ffn_status(layer.plan) == 0
    check_close(out[:250], oracle.from_inputs(host, sel=np.arange(250)), "short coverage")
    layer.close()


def test_duplicate_expert_in_a_token_is_reported_by_debug_plans():
    cfg = wl.CONFIGS["tiny"]
    host = wl.make_inputs(cfg)
    inp = to_device(host)
    dup = inp.topk_ids.clone()
    dup[7, 1] = dup[7, 0]
    out = torch.zeros(cfg.T, cfg.H, dtype=torch.bfloat16, device="cuda")
    for debug, want in ((1, -6), (0, 0)):
        layer = make_layer(cfg, mode=cep.CEP_MODE_SYNC, debug_checks=debug)
        load(layer, inp)
        cep.ffn_begin(layer.plan, out, cfg.T, 1)
        cep.ffn_submit_chunk(layer.plan, 0, 0, cfg.T, inp.x, None, dup, inp.topk_w)
        cep.combine(layer.plan)
        torch.cuda.synchronize()
        assert cep.ffn_status(layer.plan) == want
        if debug:
            assert "same expert" in cep.cep_last_error(layer.plan)
            assert cep.cep_debug_check_guards(layer.plan) == 0
            out2, _ = run_layer(inp, layer)                  # clean ids: clean status, right answer
            check_close(out2, oracle.from_inputs(host), "after duplicate ids")
        layer.close()


def test_bounded_wait_expiry_is_reported_and_the_context_stays_usable():
    # failure detection without a fault: a wait that nothing satisfies runs out after its limit, the kernel
    # exits normally, the host reads CEP_ERR_DEVICE_TIMEOUT, and the next layer call is clean and correct
    import time
    cfg = wl.CONFIGS["tiny"]
    host = wl.make_inputs(cfg)
    inp = to_device(host)
    layer = make_layer(cfg, mode=cep.CEP_MODE_SYNC)
    load(layer, inp)
    out = torch.zeros(cfg.T, cfg.H, dtype=torch.bfloat16, device="cuda")
    cep.ffn_begin(layer.plan, out, cfg.T, 1)
    cep.ffn_submit_chunk(layer.plan, 0, 0, cfg.T, inp.x, None, inp.topk_ids, inp.topk_w)
    t0 = time.perf_counter()
    cep.cep_debug_wait_timeout(layer.plan, 200)
    cep.combine(layer.plan)
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    assert 0.15 < waited < 5.0
    assert cep.ffn_status(layer.plan) == -7
    assert "bounded wait" in cep.cep_last_error(layer.plan)
    check_close(out, oracle.from_inputs(host), "layer call that carried the probe")   # the real work still ran
    out2, _ = run_layer(inp, layer)                                                     # status was reset
    check_close(out2, oracle.from_inputs(host), "after a timeout")
    layer.close()


def test_kernel_launch_counter_counts_our_kernels():
    cfg = wl.CONFIGS["tiny"]
    inp = to_device(wl.make_inputs(cfg))
    layer = make_layer(cfg, mode=cep.CEP_MODE_ASYNC)
    load(layer, inp)
    before = cep.cep_kernel_launches(layer.plan)
    assert before == 3                                      # the three prepack transposes
    run_layer(inp, layer)
    assert cep.cep_kernel_launches(layer.plan) - before == 2 * 7   # 4 layout + 2 GEMM + 1 combine per invocation
    layer.close()


# ------------------------------------------------------------------ limits of the configuration space
def test_many_experts_and_wide_top_k():
    # the largest expert count the plan accepts, most experts empty; then the widest top-k
    T, H, I = 600, 256, 128
    for E_global, E_local, k in [(1024, 1024, 4), (64, 40, 32)]:
        host = edge_inputs(T, k, E_global, E_local, H, I, distinct_ids(T, k, E_global, 11), seed=3)
        ref = oracle.from_inputs(host)
        inp = to_device(host)
        layer = make_layer(host.cfg, mode=cep.CEP_MODE_SYNC)
        load(layer, inp)
        out, _ = run_layer(inp, layer)
        assert_layout_matches(layer, 0, batch_ids(host, [0]), E_local)
        check_close(out, ref, "E=%d k=%d" % (E_local, k))
        layer.close()


def test_more_chunks_than_one_invocation_holds_and_empty_chunks():
    # 40 chunks (some empty) under Sync: a batch is launched early when it holds 32 chunks
    sizes = [7] * 20 + [0, 0, 13] + [5] * 17
    T = sum(sizes)
    cfg = wl.MoEConfig("chunks40", 0, T=T, H=256, I=128, E_global=8, E_local=8, k=2, chunks=tuple(sizes))
    host = wl.make_inputs(cfg)
    ref = oracle.from_inputs(host)
    inp = to_device(host)
    layer = make_layer(cfg, mode=cep.CEP_MODE_SYNC, n_streams=2)
    load(layer, inp)
    out, n_inv = run_layer(inp, layer)
    assert n_inv == 2                                        # 32 chunks, then the remaining 8 at the flush
    assert cep.ffn_query(layer.plan, 0).n_chunks == 32 and cep.ffn_query(layer.plan, 1).n_chunks == 8
    assert_layout_matches(layer, 1, batch_ids(host, list(range(32, 40))), cfg.E_local)
    check_close(out, ref, "40 chunks")
    layer.close()


def test_guard_gaps_trip_when_something_writes_past_a_region():
    cfg = wl.CONFIGS["tiny"]
    inp = to_device(wl.make_inputs(cfg))
    layer = make_layer(cfg, mode=cep.CEP_MODE_SYNC, n_streams=1, debug_checks=1)
    load(layer, inp)
    run_layer(inp, layer)
    assert cep.cep_debug_check_guards(layer.plan) == 0
    # the last gap of the slot lies within its final 2 KiB: one of these two bytes is inside it
    ws = layer.workspace
    ws[ws.numel() - 1030] = 0
    ws[ws.numel() - 600] = 0
    assert cep.cep_debug_check_guards(layer.plan) >= 1
    layer.close()
    plain = make_layer(cfg, mode=cep.CEP_MODE_SYNC)
    with pytest.raises(cep.CepError) as e:                   # a plan without debug_checks has no gaps to check
        cep.cep_debug_check_guards(plain.plan)
    assert e.value.code == -2
    plain.close()


def test_outputs_can_be_consumed_per_invocation():
    # asynchronous output return: after waiting on one invocation only, the rows of its chunks are final
    cfg = wl.CONFIGS["mid"]
    host = wl.make_inputs(cfg)
    inp = to_device(host)
    sync = make_layer(cfg, mode=cep.CEP_MODE_SYNC)
    load(sync, inp)
    base, _ = run_layer(inp, sync)
    layer = make_layer(cfg, mode=cep.CEP_MODE_ASYNC, n_streams=2)
    load(layer, inp)
    out = torch.full((cfg.T, cfg.H), float("nan"), dtype=torch.bfloat16, device="cuda")
    ch = chunks_of(inp)
    cep.ffn_begin(layer.plan, out, cfg.T, len(ch))
    side = torch.cuda.Stream()
    copies = []
    for c, (off, x, xs, ids, w) in enumerate(ch):
        cep.ffn_submit_chunk(layer.plan, c, off, x.shape[0], x, xs, ids, w)
        info = cep.ffn_query(layer.plan, c)
        assert info.first_chunk_pos == c and info.n_chunks == 1
        cep.ffn_wait_invocation(layer.plan, c, side)
        with torch.cuda.stream(side):
            copies.append((off, x.shape[0], out[off:off + x.shape[0]].clone()))
    side.synchronize()                                      # only the side stream: the layer is still open
    for off, n, rows in copies:
        assert torch.equal(rows.view(torch.int16), base[off:off + n].view(torch.int16))
    with pytest.raises(cep.CepError) as e:
        cep.ffn_wait_invocation(layer.plan, 99, side)
    assert e.value.code == -1
    cep.combine(layer.plan)
    torch.cuda.synchronize()
    assert cep.ffn_status(layer.plan) == 0
    assert torch.equal(out.view(torch.int16), base.view(torch.int16))
    sync.close(); layer.close()
