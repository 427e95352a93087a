"""Byte and flop accounting for the decode path (integer bookkeeping only; no arithmetic of the method).

The algorithmic bytes of one decode launch are what the method has to move once: the shared states,
every DISTINCT record some live chain refers to (a shared ancestor counts once), the queries, the
outputs and the ancestry rows.  The un-deduplicated figure (every chain reads all its records) is the
traffic the on-chip caches see instead.
"""
from __future__ import annotations

from typing import Sequence

import numpy as np


def chain_table(parents: Sequence, widths: Sequence[int]) -> np.ndarray:
    """Beam index at every call on the lineage of each live beam: int64 [W_last, T], oldest first.
    parents[t] (t >= 1) maps beams of call t to beams of call t-1; parents[0] is ignored."""
    T = len(widths)
    rows = np.empty((widths[-1], T), dtype=np.int64)
    cur = np.arange(widths[-1], dtype=np.int64)
    for t in range(T - 1, -1, -1):
        rows[:, t] = cur
        if t > 0:
            cur = np.asarray(parents[t], dtype=np.int64)[cur]
    return rows


def distinct_records(parents: Sequence, widths: Sequence[int]) -> list[int]:
    """Number of distinct records referenced at each call level by the live beams of the last call."""
    rows = chain_table(parents, widths)
    return [int(np.unique(rows[:, t]).size) for t in range(len(widths))]


def record_bytes(dk: int, dv: int, elem_bytes: int) -> int:
    return (dk + dv) * elem_bytes + 8          # k, v and fp32 alpha, beta


def decode_bytes(*, R: int, H: int, dk: int, dv: int, W: int, depth: int, elem_bytes: int, out_bytes: int,
                 distinct_per_request: Sequence[int]) -> dict:
    """Algorithmic and un-deduplicated bytes of ONE decode launch over R requests of one layer.
    distinct_per_request[r] = number of distinct record slots request r's live chains touch."""
    rec = record_bytes(dk, dv, elem_bytes)
    fixed = R * H * dv * dk * 4 + R * W * H * (dk * elem_bytes + dv * out_bytes) + R * W * depth * 4
    alg = fixed + sum(distinct_per_request) * H * rec
    gathered = fixed + R * W * depth * H * rec
    return {"algorithmic": int(alg), "undeduplicated": int(gathered),
            "units": R * W * H, "flops_contraction": 2 * R * W * H * dv * dk,
            "flops_fold": 6 * R * W * H * depth * max(dk, dv)}


def append_bytes(*, R: int, H: int, dk: int, dv: int, W: int, elem_bytes: int) -> int:
    """Read + write of one append launch."""
    return 2 * R * W * H * record_bytes(dk, dv, elem_bytes)


def persistent_bytes(*, R: int, H: int, dk: int, dv: int, W: int, T: int, rec_bytes: int, layers: int = 1) -> dict:
    """Resident recurrent-state bytes after T decode calls: one fp32 state per (request, head) plus one
    record per (request, beam, head, call); and what a per-beam full fp32 state would need instead."""
    s0 = R * H * dv * dk * 4 * layers
    recs = R * W * H * T * rec_bytes * layers
    return {"s0": s0, "records": recs, "total": s0 + recs, "fullstate": R * W * H * dv * dk * 4 * layers,
            "writes": recs, "fullstate_writes": R * W * H * dv * dk * 4 * T * layers}
