"""Row sharding of a sampling batch over N ranks (one process per GPU).

Rows of the logits matrix are independent (section 6.1 of the paper), so the batch is cut
into contiguous blocks of ceil(B / N) rows; the last block is padded with copies of the
final row so that every rank runs the same shape (the paper's batch padding, section 6.2)
and the padded outputs are dropped after the gather.  Each rank passes ``row_base`` = the
global index of its first row, which keeps every draw identical to the unsharded call.
There is no data-path collective; only the tiny result gather (token id + logprob per row).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import numpy as np


@dataclass(frozen=True)
class Shard:
    rank: int
    lo: int          # first global row of this rank
    hi: int          # one past its last real row (lo == hi: the rank holds only padding)
    rows: int        # rows the rank actually runs (real + padding), equal on every rank


def plan(B: int, world: int) -> List[Shard]:
    if B < 0 or world < 1:
        raise ValueError("bad B or world size")
    per = -(-B // world) if B else 0
    out = []
    for r in range(world):
        lo = min(B, r * per)
        hi = min(B, lo + per)
        out.append(Shard(r, lo, hi, per))
    return out


def shard_workload(w, shard: Shard):
    """The rows of ``w`` this rank runs: its real rows followed by padding copies of the last
    row of the batch.  ``row_base`` is the global id of the shard's first row."""
    if shard.rows == 0:
        return w.rows(0, 0)
    if shard.hi > shard.lo:
        part = w.rows(shard.lo, shard.hi)
    else:
        part = w.rows(w.B - 1, w.B)
        part.row_base = w.row_base + shard.lo
    pad = shard.rows - max(shard.hi - shard.lo, 0) if shard.hi > shard.lo else shard.rows - 1
    if pad > 0:
        part = _pad_rows(part, pad)
    return part


def _pad_rows(w, pad: int):
    import copy
    out = copy.copy(w)

    def rep(a):
        return None if a is None else np.concatenate([a, np.repeat(a[-1:], pad, axis=0)])
    out.logits = rep(w.logits)
    for name in ("temperature", "top_k", "top_p", "min_p", "repetition_penalty", "presence_penalty",
                 "frequency_penalty", "seeds"):
        setattr(out, name, rep(getattr(w, name)))
    if w.history_ids is not None:
        o = w.history_offsets.astype(np.int64)
        last = w.history_ids[o[-2]:o[-1]]
        out.history_ids = np.concatenate([w.history_ids] + [last] * pad)
        out.history_offsets = np.concatenate([o, o[-1] + (np.arange(1, pad + 1) * last.size)]).astype(np.int32)
    out.B = w.B + pad
    return out


def unpad(values: np.ndarray, shard: Shard) -> np.ndarray:
    """Drops the padded outputs of one rank."""
    return values[: max(shard.hi - shard.lo, 0)]
