"""Host-only checks of the weight-fetching planner simulation: Algorithm 1 on hand cases, the admission rule,
the latency model, and the non-degradation property (sequential admissible updates never raise max_r T_r)."""
import math

import numpy as np
import pytest

from paper_2609_33252_b200 import oewf


def flat_F(tokens_per_s=1000.0):
    return oewf.FFNLatency([1, 10 ** 6], [tokens_per_s, tokens_per_s])


def test_ffn_latency_model():
    F = oewf.FFNLatency([100, 1000, 10000], [1e5, 8e5, 1e6])
    assert F(0) == 0.0
    assert F.eta(10000) == 1.0 and F.eta(50) == pytest.approx(0.1) and F.eta(10 ** 7) == 1.0
    assert F(10000) == pytest.approx(10000 / 1e6)
    assert F(100) == pytest.approx(100 / 1e5)
    mid = F.eta(math.sqrt(100 * 1000))                      # halfway in log N
    assert mid == pytest.approx((1e5 + 8e5) / 2 / 1e6)
    calib = {"profile": [{"expert_tokens": 512, "ffn_ms": 0.5}, {"expert_tokens": 32768, "ffn_ms": 2.0}]}
    G = oewf.FFNLatency.from_calibration(calib)
    assert G(32768) == pytest.approx(2.0e-3) and G(512) == pytest.approx(0.5e-3)


def test_remaining_attention_is_clamped():
    assert oewf.remaining_attention(5.0, 2.0) == 3.0
    assert oewf.remaining_attention(5.0, 7.0) == 0.0


def test_select_weights_hand_cases():
    donors = {1: 9.0, 2: 12.0, 3: 12.0}                     # tie between 2 and 3 -> lower rank
    tokens = {2: {10: 300, 11: 50, 12: 400, 13: 0}, 3: {20: 999}}
    size = {10: 100, 11: 100, 12: 200, 13: 100, 20: 100}
    p = oewf.select_weights(0, donors, tokens, size, budget=250)
    # densities: e10 3.0, e12 2.0, e11 0.5 ; e10 fits (150 left), e12 (200) does not -> stop, e11 never considered
    assert p.donor == 2 and p.experts == [10] and p.bytes_used == 100 and p.tokens == {10: 300}
    p = oewf.select_weights(0, donors, tokens, size, budget=400)
    assert p.experts == [10, 12, 11] and p.bytes_used == 400
    assert oewf.select_weights(0, donors, tokens, size, budget=50) is None        # nothing fits
    assert oewf.select_weights(0, {}, tokens, size, budget=400) is None           # no donor still in attention
    assert oewf.select_weights(0, {1: 5.0}, tokens, size, budget=400) is None     # no tokens on that donor


def test_admission_rule():
    F = flat_F(1000.0)                                       # F(N) = N / 1000
    # donor: A=2, D=0, N=4000 -> T_d = 6; helper finishes at 3
    ok, Td, Th = oewf.admit(2.0, 0.0, 4000, 3.0, 1000, s_h=1.0, F=F)
    assert ok and Td == pytest.approx(5.0) and Th == pytest.approx(3.0)           # fully hidden: alpha = 0
    ok, Td, Th = oewf.admit(2.0, 0.0, 4000, 3.0, 3000, s_h=3.0, F=F)
    assert ok and Td == pytest.approx(3.0) and Th == pytest.approx(6.0)           # serial: alpha = 1, max unchanged
    ok, _, Th = oewf.admit(2.0, 0.0, 4000, 3.0, 3500, s_h=3.0, F=F)
    assert not ok and Th == pytest.approx(6.5)                                    # helper would finish later than the donor did
    assert oewf.overlap_fraction(3.0, 1.0, 1.0) == 0.0 and oewf.overlap_fraction(3.0, 3.0, 2.0) == 1.0
    assert oewf.overlap_fraction(3.0, 2.5, 1.0) == pytest.approx(0.5)


@pytest.mark.parametrize("seed", range(20))
def test_sequential_admissible_updates_never_increase_the_layer_time(seed):
    r = np.random.default_rng(seed)
    n = int(r.integers(2, 9))
    counts = np.sort(r.uniform(100, 50000, 5))
    F = oewf.FFNLatency(counts, counts / np.sort(r.uniform(1e-4, 5e-3, 5)))       # sub-linear latency profile
    ranks = [oewf.Rank(A=float(r.uniform(0, 5e-3)) if r.random() < 0.6 else 0.0, D=float(r.uniform(0, 5e-4)),
                       N=float(r.integers(0, 60000))) for _ in range(n)]
    base = max(x.T(F) for x in ranks)
    total = sum(x.N for x in ranks)
    props = [(int(r.integers(n)), int(r.integers(n)), float(r.integers(0, 30000)), float(r.uniform(0, 5e-3)))
             for _ in range(30)]
    accepted, hist = oewf.apply_updates(ranks, props, F)
    assert all(b <= a + 1e-15 for a, b in zip(hist, hist[1:]))                    # max_r T_r is non-increasing
    assert hist[-1] <= base + 1e-15
    assert sum(x.N for x in ranks) + sum(a[2] for a in accepted) == pytest.approx(total)   # tokens are conserved
    assert all(x.N >= 0 for x in ranks)
