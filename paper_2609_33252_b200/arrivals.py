"""Arrival harness: models attention-replica imbalance on one GPU.

Each replica's routed tokens are one chunk.  The host releases chunk r at time t0 + a_r by
calling ``ffn_submit_chunk`` on replica stream r (the stand-in for the per-replica completion
signal of Section 3.2), then flushes and joins.  Only host timing and pointer passing live here.
"""
from __future__ import annotations

import time
from typing import List, Optional, Sequence

from . import binding as cep


def run_with_arrivals(layer, out, chunks, arrival_s: Sequence[float], n_local_pairs: Optional[Sequence[int]] = None,
                      replica_streams: Optional[List] = None):
    """One layer call with host-released chunks.

    chunks: list of (token_offset, x, x_scale, ids, w); arrival_s[c] = release time of chunk c in
    seconds after the start.  Returns (completion_seconds, n_invocations): the host time from the
    start until the join stream has drained.
    """
    import torch
    order = sorted(range(len(chunks)), key=lambda c: (arrival_s[c], c))
    n_tok = sum(c[1].shape[0] for c in chunks)
    main = torch.cuda.current_stream()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    cep.ffn_begin(layer.plan, out, n_tok, len(chunks))
    for c in order:
        target = t0 + arrival_s[c]
        while time.perf_counter() < target:
            pass
        off, x, xs, ids, w = chunks[c]
        cep.ffn_submit_chunk(layer.plan, c, off, x.shape[0], x, xs, ids, w,
                             -1 if n_local_pairs is None else n_local_pairs[c],
                             None if replica_streams is None else replica_streams[c])
    cep.ffn_flush(layer.plan)
    cep.combine(layer.plan, main)
    main.synchronize()
    dt = time.perf_counter() - t0
    return dt, cep.ffn_num_invocations(layer.plan)
