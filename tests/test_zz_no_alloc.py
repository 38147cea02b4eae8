"""The allocation-free index entry point against the regular path, through the C ABI.

Who needs it: code that runs where device memory is already spoken for (a plug-in inside a serving
process whose pool owns the GPU) or where allocating is not allowed at that moment.  Such a caller
passes only its own pre-made input and output buffers; the library's scratch is a fixed array inside
the library.  The test makes two calls in a row on different inputs (the array keeps the first call's
contents) and compares every integer with what the plan-based path exports for the same ids.
"""
import pytest
import torch

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


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch_and_bad_arguments():
    ids = torch.zeros((4, 2), dtype=torch.int32, device="cuda")
    o = torch.zeros(2048, dtype=torch.int32, device="cuda")
    big = torch.zeros((600000, 2), dtype=torch.int32, device="cuda")          # 586 segments * 1024 experts
    assert cep.layout_indices_noalloc(big, 1024, 1024, o, o, o, o, o) == -4
    assert cep.layout_indices_noalloc(ids, 2000, 2000, o, o, o, o, o) == -1
    assert cep.layout_indices_noalloc(ids, 8, 4, o, o, o, o, o) == -1
