"""The allocation-free index entry point against the regular path, through the C ABI.

Who needs it: code that runs where device memory is already spoken for (a plug-in inside a serving
process whose pool owns the GPU) or where allocating is not allowed at that moment.  Such a caller
passes only its own pre-made input and output buffers; the library's scratch is a fixed array inside
the library.  The test makes two calls in a row on different inputs (the array keeps the first call's
contents) and compares every integer with what the plan-based path exports for the same ids, and
with the CPU oracle's layout transform directly.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_33252_b200 as cep
from paper_2609_33252_b200 import workloads as wl

from helpers import make_layer, run_layer, to_device

pytestmark = pytest.mark.gpu


def reference_layout(inp):
    cfg = inp.cfg
    layer = make_layer(cfg, mode=cep.CEP_MODE_SYNC)
    layer.load_weights(inp.w_gate, inp.w_up, inp.w_down)
    run_layer(inp, layer)
    ref = cep.ffn_debug_export(layer.plan, 0, cfg.E_local, cfg.T * cfg.k)
    layer.close()
    return ref


def test_noalloc_layout_matches_plan_path_on_two_calls_in_a_row():
    cases = []
    mid = to_device(wl.make_inputs(wl.CONFIGS["mid"]))
    cases.append(mid)
    shard = wl.scaled(wl.CONFIGS["ep_shard"], T=3000, H=256, I=128, chunks=(3000,))
    cases.append(to_device(wl.make_inputs(shard)))            # remote experts: rows of -1, other E
    refs = [reference_layout(c) for c in cases]
    # the caller's buffers, made before the calls; the calls themselves allocate nothing
    bufs = []
    for c in cases:
        E, n_pairs = c.cfg.E_local, c.cfg.T * c.cfg.k
        i32 = dict(dtype=torch.int32, device="cuda")
        bufs.append(dict(counts=torch.full((E,), -7, **i32), offsets=torch.full((E + 1,), -7, **i32),
                         padded=torch.full((E + 1,), -7, **i32), rop=torch.full((n_pairs,), -7, **i32),
                         por=torch.full((n_pairs + 127 * E + 128,), -1, **i32), status=torch.full((2,), -7, **i32)))
    torch.cuda.synchronize()
    for c, b in zip(cases, bufs):                              # two calls back to back, same stream
        rc = cep.layout_indices_noalloc(c.topk_ids, c.cfg.E_local, c.cfg.E_global, b["counts"], b["offsets"],
                                        b["padded"], b["rop"], b["por"], b["status"])
        assert rc == 0
    torch.cuda.synchronize()
    for c, b, ref in zip(cases, bufs, refs):
        assert b["status"].tolist() == [0, 0]
        assert (b["counts"].cpu().numpy() == ref["counts"]).all()
        assert (b["offsets"].cpu().numpy() == ref["offsets"]).all()
        assert (b["padded"].cpu().numpy() == ref["padded_offsets"]).all()
        assert (b["rop"].cpu().numpy() == ref["row_of_pair"]).all()
        n_rows = int(ref["padded_offsets"][-1])
        assert (b["por"][:n_rows].cpu().numpy() == ref["pair_of_row"]).all()   # padding rows stay -1
        # and against the oracle itself, so this check does not lean on the plan path being right
        want = oracle.permute(c.topk_ids.cpu().numpy(), c.cfg.E_local, align=128)
        assert (b["counts"].cpu().numpy() == want["counts"]).all()
        assert (b["offsets"].cpu().numpy() == want["offsets"]).all()
        assert (b["padded"].cpu().numpy() == want["padded_offsets"]).all()
        assert (b["rop"].cpu().numpy() == want["prow_of_pair"]).all()
        assert (b["por"][:n_rows].cpu().numpy() == want["pair_of_prow"]).all()


def test_noalloc_reports_bad_ids_and_a_short_inverse_map_without_touching_memory_past_it():
    i32 = dict(dtype=torch.int32, device="cuda")
    E, E_g, k, T = 4, 6, 2, 300
    g = torch.Generator(device="cpu"); g.manual_seed(7)
    ids = torch.stack([torch.randperm(E_g, generator=g)[:k] for _ in range(T)]).to(torch.int32)
    want = oracle.permute(ids.numpy(), E, align=128)
    n_rows = int(want["padded_offsets"][-1])

    def call(ids_dev, por):
        b = dict(counts=torch.zeros(E, **i32), offsets=torch.zeros(E + 1, **i32), padded=torch.zeros(E + 1, **i32),
                 rop=torch.full((T * k,), -7, **i32), status=torch.full((2,), -7, **i32))
        assert cep.layout_indices_noalloc(ids_dev, E, E_g, b["counts"], b["offsets"], b["padded"], b["rop"], por,
                                          b["status"]) == 0
        torch.cuda.synchronize()
        return b
    # (1) an id equal to n_experts_global: flagged in status[0], counted nowhere
    bad = ids.clone(); bad[5, 1] = E_g
    b = call(bad.cuda(), torch.full((n_rows,), -1, **i32))
    assert b["status"].tolist() == [1, 0]
    # (2) an inverse map shorter than the rows needed: status[1], rows that do not fit get -1 and are not stored;
    #     the entries past the capacity handed in keep their sentinel
    cap = n_rows - 200
    assert cap > 0
    store = torch.full((n_rows + 64,), 12345, **i32)
    b = call(ids.cuda(), store[:cap])
    assert b["status"].tolist() == [0, 1]
    assert (store[cap:] == 12345).all()
    rop, prow = b["rop"].cpu().numpy(), want["prow_of_pair"]
    fits = (prow >= 0) & (prow < cap)
    assert (rop[fits] == prow[fits]).all() and (rop[~fits] == -1).all()
    got_por, want_por = store[:cap].cpu().numpy(), want["pair_of_prow"][:cap]
    real = want_por >= 0
    assert (got_por[real] == want_por[real]).all() and (got_por[~real] == 12345).all()   # padding rows are left untouched
    assert (b["counts"].cpu().numpy() == want["counts"]).all()


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch_and_bad_arguments():
    ids = torch.zeros((4, 2), dtype=torch.int32, device="cuda")
    o = torch.zeros(2048, dtype=torch.int32, device="cuda")
    big = torch.zeros((600000, 2), dtype=torch.int32, device="cuda")          # 586 segments * 1024 experts
    assert cep.layout_indices_noalloc(big, 1024, 1024, o, o, o, o, o) == -4
    assert cep.layout_indices_noalloc(ids, 2000, 2000, o, o, o, o, o) == -1
    assert cep.layout_indices_noalloc(ids, 8, 4, o, o, o, o, o) == -1
