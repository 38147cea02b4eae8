"""CPU-only checks of the library's host side: exported symbols, index arithmetic, the
launch rule, argument validation.  No kernel is launched."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2609_33252_b200 as cep

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cascade_ffn.h")).read()
    return re.findall(r"CEP_API\s+[\w\s\*]+?\b(\w+)\s*\(", text)


def test_library_loads_and_exports_every_declared_symbol():
    L = cep.load_library()
    names = declared_functions()
    assert len(names) >= 17 and "moe_plan" in names and "ffn_submit_chunk" in names and "combine" in names
    for n in names:
        assert hasattr(L, n), n
    assert sorted(names) == sorted(cep.binding.EXPORTS)


@pytest.mark.parametrize("ng", [0, 1, 3, 8])
@pytest.mark.parametrize("mt,nb", [([3, 0, 17, 1, 0, 40], 4), ([1], 1), ([0, 0, 5], 16), ([33, 16, 15], 3)])
def test_tile_decode_covers_every_tile_exactly_once(mt, nb, ng):
    prefix = np.concatenate([[0], np.cumsum(mt)]).astype(np.int32)
    total = int(prefix[-1]) * nb
    seen = set()
    for t in range(total):
        e, m, n = cep.cep_debug_decode_tile(prefix, nb, t, ng)
        assert 0 <= m < mt[e] and 0 <= n < nb
        seen.add((e, m, n))
    assert len(seen) == total
    assert cep.cep_debug_decode_tile(prefix, nb, total) is None
    assert cep.cep_debug_decode_tile(prefix, nb, -1) is None
    # tiles of one expert are contiguous and experts appear in order
    last_e = -1
    for t in range(total):
        e = cep.cep_debug_decode_tile(prefix, nb, t, ng)[0]
        assert e >= last_e
        last_e = e


def test_tile_decode_order_keeps_an_experts_weight_panel_hot():
    # inside an expert the n block is the fast index: consecutive tiles sweep all n blocks of one m block
    prefix = np.array([0, 40, 43], np.int32)
    assert [cep.cep_debug_decode_tile(prefix, 4, t) for t in range(5)] == \
        [(0, 0, 0), (0, 0, 1), (0, 0, 2), (0, 0, 3), (0, 1, 0)]
    assert cep.cep_debug_decode_tile(prefix, 4, 159) == (0, 39, 3)
    assert cep.cep_debug_decode_tile(prefix, 4, 160) == (1, 0, 0)
    assert cep.cep_debug_decode_tile(prefix, 4, 171) == (1, 2, 3)
    # chunks of 3 n blocks: the chunk is swept over every m block before the next chunk starts
    p2 = np.array([0, 2], np.int32)
    assert [cep.cep_debug_decode_tile(p2, 4, t, 3) for t in range(8)] == \
        [(0, 0, 0), (0, 0, 1), (0, 0, 2), (0, 1, 0), (0, 1, 1), (0, 1, 2), (0, 0, 3), (0, 1, 3)]


@pytest.mark.parametrize("seed", range(6))
def test_launch_rule_matches_the_scheduler_oracle(seed):
    r = np.random.default_rng(seed)
    n = int(r.integers(1, 70))
    pairs = r.integers(0, 400, size=n).tolist()
    theta = int(r.integers(0, 1200))
    for mode in (cep.CEP_MODE_SYNC, cep.CEP_MODE_ASYNC, cep.CEP_MODE_STREAMFFN):
        got = cep.cep_debug_schedule(pairs, mode, theta)
        want = oracle.schedule(pairs, mode, theta, 2, max_chunks_per_invocation=32)
        inv_of = [None] * n
        for i, (chunks, _) in enumerate(want):
            for c in chunks:
                inv_of[c] = i
        assert got == inv_of


def test_config_validation_and_sizes():
    good = cep.CepConfig(512, 256, 8, 8, 2, 256, 2, 0, 0, 2, 0, 0, 0)
    n = cep.moe_plan_workspace_bytes(good)
    assert n > 0 and n % 256 == 0
    assert cep.moe_packed_weight_bytes(good) >= 8 * 3 * 512 * 256 * 2
    bad = [dict(hidden=500), dict(inter=100), dict(n_experts_local=9), dict(top_k=0), dict(top_k=33),
           dict(max_tokens=0), dict(mode=7), dict(n_streams=0), dict(threshold_pairs=-1), dict(dtype=5),
           dict(gemm_impl=4), dict(n_experts_local=2000, n_experts_global=4000)]
    for kw in bad:
        c = cep.CepConfig(512, 256, 8, 8, 2, 256, 2, 0, 0, 2, 0, 0, 0)
        for k_, v in kw.items():
            setattr(c, k_, v)
        with pytest.raises(cep.CepError) as ei:
            cep.moe_plan_workspace_bytes(c)
        assert ei.value.code == -1
    # workspace grows with the number of scratch slots
    more = cep.CepConfig(512, 256, 8, 8, 2, 256, 2, 0, 0, 4, 0, 0, 0)
    assert cep.moe_plan_workspace_bytes(more) > n


def test_null_plan_is_rejected_without_touching_a_device():
    L = cep.load_library()
    assert L.ffn_flush(None) == -1
    assert L.combine(None, None) == -1
    assert L.ffn_status(None) == -1
    assert L.moe_plan_destroy(None) == 0
    assert b"NULL" in L.cep_last_error(None)
    assert L.ffn_set_active_streams(None, 1) == -1
    assert L.cep_calibrate(None, 0.9, None, 0, 0, None, None, None, None, None, None, None) == -1


def test_microscaling_config_is_validated_on_the_host():
    ok = cep.CepConfig(512, 256, 8, 8, 2, 256, 2, cep.CEP_MXFP4_E4M3, 0, 2, 0, 0, 0)
    assert cep.moe_plan_workspace_bytes(ok) > 0
    bf16 = cep.CepConfig(512, 256, 8, 8, 2, 256, 2, cep.CEP_BF16, 0, 2, 0, 0, 0)
    # packed weights: a nibble + 1/32 scale byte per element against two bytes
    assert cep.moe_packed_weight_bytes(ok) < cep.moe_packed_weight_bytes(bf16) // 3
    with pytest.raises(cep.CepError):
        cep.moe_plan_workspace_bytes(cep.CepConfig(512, 256, 8, 8, 2, 256, 2, 3, 0, 2, 0, 0, 0))     # unknown dtype
