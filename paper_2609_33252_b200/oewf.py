"""Host-only simulation of opportunistic expert weight fetching (Section 3.3 "Opportunistic Expert Weight Fetching"; Algorithm 1; Eqs. 1-6; the
non-degradation proposition of the appendix).

Nothing here touches a GPU or moves weights: cross-GPU fetching is outside what this library runs.  The module
restates the planner's decisions so that they can be exercised with this library's own FFN latency profile
(``calibrate.calibrate_in_library`` / ``calibrate_on_routing`` give eta(N) and the observed peak) and synthetic attention / dispatch times:

* ``FFNLatency``            F(N) = N / (eta(N) * P_peak), F(0) = 0                       (Eq. 2)
* ``remaining_attention``   A_d = [f(I_d, P_d) - t_att]^+                                 (Eq. 1)
* ``donor_completion``      T_d(S) = A_d + D_d + F(N_d)                                   (Eq. 3)
* ``select_weights``        greedy donor and expert choice under a byte budget           (Algorithm 1, Eq. 4)
* ``admit``                 the cost-based reassignment test                             (Eqs. 5-6)
* ``apply_updates``         sequential admissible updates on a joint plan                (appendix proposition)
"""
from __future__ import annotations

import bisect
import dataclasses
import math
from typing import Dict, List, Optional, Sequence, Tuple


class FFNLatency:
    """F(N) from a throughput profile: points (expert_tokens, tokens_per_second).  eta(N) is the profile's
    throughput at N, interpolated linearly in log N between profiled counts and held flat outside them,
    divided by the observed peak."""

    def __init__(self, counts: Sequence[float], tokens_per_s: Sequence[float]):
        assert len(counts) == len(tokens_per_s) >= 1 and all(c > 0 for c in counts)
        order = sorted(range(len(counts)), key=lambda i: counts[i])
        self.n = [float(counts[i]) for i in order]
        self.tp = [float(tokens_per_s[i]) for i in order]
        self.peak = max(self.tp)

    @classmethod
    def from_calibration(cls, calib: Dict) -> "FFNLatency":
        prof = calib["profile"]
        return cls([p["expert_tokens"] for p in prof], [p["expert_tokens"] / (p["ffn_ms"] * 1e-3) for p in prof])

    def eta(self, n: float) -> float:
        if n <= self.n[0]:
            return self.tp[0] / self.peak
        if n >= self.n[-1]:
            return self.tp[-1] / self.peak
        i = bisect.bisect_right(self.n, n)
        x0, x1 = math.log(self.n[i - 1]), math.log(self.n[i])
        w = (math.log(n) - x0) / (x1 - x0)
        return ((1 - w) * self.tp[i - 1] + w * self.tp[i]) / self.peak

    def __call__(self, n: float) -> float:
        return 0.0 if n <= 0 else n / (self.eta(n) * self.peak)


def remaining_attention(predicted_total: float, elapsed: float) -> float:
    """Remaining attention-stage time of a donor, clamped at zero."""
    return max(0.0, predicted_total - elapsed)


def donor_completion(A_d: float, D_d: float, N_d: float, F) -> float:
    return A_d + D_d + F(N_d)


@dataclasses.dataclass
class FetchPlan:
    helper: int
    donor: int
    experts: List[int]
    tokens: Dict[int, int]          # expert -> tokens the helper dispatched to it on the donor
    bytes_used: int


def select_weights(helper: int, donors_T: Dict[int, float], tokens_h: Dict[int, Dict[int, int]],
                   bytes_per_expert: Dict[int, int], budget: int) -> Optional[FetchPlan]:
    """Algorithm 1.  donors_T: predicted completion time T_d(S) of every candidate donor (replicas still in
    attention); tokens_h[d][e]: tokens helper h dispatched to expert e of donor d; budget: B_h.  The donor
    with the latest completion is chosen; its experts that hold tokens of h are taken in descending
    tokens-per-byte order while they fit, stopping at the first that does not."""
    import itertools
    ranked_donors = sorted(donors_T.items(), key=lambda kv: (-kv[1], kv[0]))      # latest completion first, ties: lowest rank
    if not ranked_donors:
        return None
    donor = ranked_donors[0][0]
    held = tokens_h.get(donor, {})
    density_order = sorted((e for e in held if held[e] > 0), key=lambda e: (-held[e] / bytes_per_expert[e], e))
    # running byte total over the density-ordered experts; the selection is the longest prefix within the budget
    running = list(itertools.accumulate(bytes_per_expert[e] for e in density_order))
    n_fit = sum(1 for _ in itertools.takewhile(lambda total: total <= budget, running))
    if n_fit == 0:
        return None
    chosen = density_order[:n_fit]
    return FetchPlan(helper, donor, chosen, {e: held[e] for e in chosen}, running[n_fit - 1])


def overlap_fraction(T_h: float, s_h: float, F_trans: float) -> float:
    """alpha_h: the part of the reassigned kernel that extends past the helper's own completion."""
    if F_trans <= 0:
        return 0.0
    return max(0.0, s_h + F_trans - T_h) / F_trans


def admit(A_d: float, D_d: float, N_d: float, T_h: float, N_trans: float, s_h: float, F) -> Tuple[bool, float, float]:
    """Eqs. 5-6.  Returns (accepted, T_d', T_h') for moving N_trans unstarted expert tokens from the donor to a
    helper whose reassigned kernel would start s_h after the decision (0 <= s_h <= T_h)."""
    assert 0 <= N_trans <= N_d and 0 <= s_h <= T_h
    T_d = donor_completion(A_d, D_d, N_d, F)
    T_d2 = donor_completion(A_d, D_d, N_d - N_trans, F)
    T_h2 = T_h + overlap_fraction(T_h, s_h, F(N_trans)) * F(N_trans)
    return max(T_d2, T_h2) <= max(T_d, T_h), T_d2, T_h2


@dataclasses.dataclass
class Rank:
    A: float        # remaining attention time (0 for a helper)
    D: float        # dispatch latency
    N: float        # received expert tokens not yet started
    T_extra: float = 0.0     # completion-time increase from work taken over as a helper

    def T(self, F) -> float:
        return self.A + self.D + F(self.N) + self.T_extra


def apply_updates(ranks: List[Rank], proposals: Sequence[Tuple[int, int, float, float]], F):
    """Sequential updates on the joint plan.  Each proposal is (helper, donor, N_trans, s_h); it is applied
    only if Eq. 6 holds against the plan as it stands, including earlier commitments.  Returns the list of
    accepted proposals and the history of max_r T_r after every decision."""
    history = [max(r.T(F) for r in ranks)]
    accepted = []
    for h, d, n_trans, s_h in proposals:
        if h == d:
            history.append(history[-1])
            continue
        n_trans = min(n_trans, ranks[d].N)
        T_h = ranks[h].T(F)
        s = min(max(s_h, 0.0), T_h)
        ok, T_d2, T_h2 = admit(ranks[d].A, ranks[d].D + ranks[d].T_extra, ranks[d].N, T_h, n_trans, s, F)
        if ok and n_trans > 0:
            ranks[d].N -= n_trans
            ranks[h].T_extra += T_h2 - T_h
            accepted.append((h, d, n_trans, s))
        history.append(max(r.T(F) for r in ranks))
    return accepted, history
